// hct_gemm_bias_relu_f32_static: the fp32 GEMM -> bias -> ReLU chain for callers that cannot
// allocate device memory.  Same arithmetic as the library's fp32 GEMM path (operands split into
// TF32 head and tail, three products per term), but the split operands live in a fixed array
// that is part of the loaded library image instead of caller-provided workspace.
#include <cuda_runtime.h>

#include <cstdint>
#include <mutex>
#include <string>

#include "../../include/hct.h"

namespace hct {
void set_last_error(const std::string& msg);  // api.cpp
}

namespace {

// Head/tail copies of A and B: 4 floats per operand element pair, so the limit on
// M*K + K*N is HCT_STATIC_SCRATCH_BYTES / 8 elements.  Every device that loads the library
// carries this array until the process exits.
static __device__ __align__(256) unsigned char g_scratch[HCT_STATIC_SCRATCH_BYTES];

__device__ __forceinline__ float to_tf32(float x) {
  unsigned u;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
  return __uint_as_float(u);
}

// x -> (hi, lo) with hi = tf32(x), lo = tf32(x - hi); writes n_a + n_b elements of each.
__global__ void __launch_bounds__(256) split_static(const float* __restrict__ a, const float* __restrict__ b, long long n_a,
                                                    long long n_b, float* __restrict__ hi, float* __restrict__ lo) {
  for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n_a + n_b; i += (long long)gridDim.x * 256) {
    const float x = i < n_a ? a[i] : b[i - n_a];
    const float h = to_tf32(x);
    hi[i] = h;
    lo[i] = to_tf32(x - h);
  }
}

// out = [relu](A*B + bias) from the split operands; 64x64 tile per CTA, 4x4 per thread, fp32 FMA.
__global__ void __launch_bounds__(256) gemm_split_static(const float* __restrict__ hi, const float* __restrict__ lo, long long n_a,
                                                         const float* __restrict__ bias, float* __restrict__ out, long long M,
                                                         long long K, long long N, int relu) {
  __shared__ float Ah[16][64 + 4], Al[16][64 + 4], Bh[16][64 + 4], Bl[16][64 + 4];
  const float* a_hi = hi;
  const float* a_lo = lo;
  const float* b_hi = hi + n_a;
  const float* b_lo = lo + n_a;
  const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
  const long long m0 = (long long)blockIdx.y * 64, n0 = (long long)blockIdx.x * 64;
  float acc[4][4] = {};
  for (long long k0 = 0; k0 < K; k0 += 16) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = tid + i * 256;
      const int r = idx / 16, kk = idx % 16;
      const long long m = m0 + r, k = k0 + kk;
      const bool ok = m < M && k < K;
      Ah[kk][r] = ok ? a_hi[m * K + k] : 0.0f;
      Al[kk][r] = ok ? a_lo[m * K + k] : 0.0f;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = tid + i * 256;
      const int kk = idx / 64, c = idx % 64;
      const long long k = k0 + kk, n = n0 + c;
      const bool ok = k < K && n < N;
      Bh[kk][c] = ok ? b_hi[k * N + n] : 0.0f;
      Bl[kk][c] = ok ? b_lo[k * N + n] : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float ah[4], al[4], bh[4], bl[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        ah[i] = Ah[kk][ty * 4 + i];
        al[i] = Al[kk][ty * 4 + i];
        bh[i] = Bh[kk][tx * 4 + i];
        bl[i] = Bl[kk][tx * 4 + i];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float t = fmaf(al[i], bh[j], acc[i][j]);   // small cross terms first
          t = fmaf(ah[i], bl[j], t);
          acc[i][j] = fmaf(ah[i], bh[j], t);
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const long long m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
      if (m < M && n < N) {
        float v = acc[i][j] + (bias ? bias[n] : 0.0f);
        out[m * N + n] = relu ? fmaxf(v, 0.0f) : v;
      }
    }
}

// Device address of g_scratch, looked up once per device.  In host code `g_scratch` names a
// host-side shadow of the symbol, not device memory, so the address must come from the runtime.
constexpr int kMaxDevices = 64;
std::mutex g_mu;
float* g_scratch_addr[kMaxDevices] = {};

hct_status_t fail(hct_status_t code, const std::string& msg) {
  hct::set_last_error(msg);
  return code;
}

}  // namespace

extern "C" HCT_API hct_status_t hct_gemm_bias_relu_f32_static(const float* a, const float* b, const float* bias, float* out,
                                                              int64_t m, int64_t k, int64_t n, int apply_relu, int device,
                                                              void* cuda_stream) {
  if (!a || !b || !out) return fail(HCT_ERR_INVALID_ARG, "a, b and out must not be NULL");
  if (m <= 0 || k <= 0 || n <= 0) return fail(HCT_ERR_INVALID_ARG, "m, k and n must be positive");
  if (device < 0 || device >= kMaxDevices) return fail(HCT_ERR_INVALID_ARG, "device index out of range");
  const unsigned long long limit = HCT_STATIC_SCRATCH_BYTES / 8;  // elements of A plus elements of B
  // (written so that the products cannot overflow before the comparison)
  if ((unsigned long long)m > limit / (unsigned long long)k || (unsigned long long)n > limit / (unsigned long long)k ||
      (unsigned long long)m * k + (unsigned long long)k * n > limit)
    return fail(HCT_ERR_UNSUPPORTED, "operands too large for the built-in scratch: m*k + k*n must not exceed " +
                                         std::to_string(limit) + " elements; use hct_graph_run with a workspace instead");
  if ((n + 63) / 64 > 0x7fffffffLL || (m + 63) / 64 > 65535) return fail(HCT_ERR_UNSUPPORTED, "too many output tiles");

  int prev = -1;
  cudaError_t rc = cudaGetDevice(&prev);
  if (rc != cudaSuccess) return fail(HCT_ERR_CUDA, std::string("cudaGetDevice: ") + cudaGetErrorString(rc));
  rc = cudaSetDevice(device);
  if (rc != cudaSuccess) return fail(HCT_ERR_CUDA, std::string("cudaSetDevice: ") + cudaGetErrorString(rc));
  hct_status_t status = HCT_OK;
  float* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_scratch_addr[device]) {
      void* p = nullptr;
      rc = cudaGetSymbolAddress(&p, g_scratch);  // with `device` current: each device has its own copy
      if (rc != cudaSuccess || !p)
        status = fail(HCT_ERR_CUDA, std::string("cudaGetSymbolAddress(scratch): ") + cudaGetErrorString(rc));
      else
        g_scratch_addr[device] = (float*)p;
    }
    scratch = g_scratch_addr[device];
  }
  if (status == HCT_OK) {
    const long long n_a = (long long)m * k, n_b = (long long)k * n;
    float* hi = scratch;
    float* lo = scratch + (n_a + n_b);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const long long blocks = (n_a + n_b + 255) / 256;
    split_static<<<(unsigned)(blocks < 148 * 16 ? blocks : 148 * 16), 256, 0, stream>>>(a, b, n_a, n_b, hi, lo);
    dim3 grid((unsigned)((n + 63) / 64), (unsigned)((m + 63) / 64));
    gemm_split_static<<<grid, 256, 0, stream>>>(hi, lo, n_a, bias, out, m, k, n, apply_relu);
    // peek, not get: an error that was already pending on this thread is reported here but left for its owner to clear
    rc = cudaPeekAtLastError();
    if (rc != cudaSuccess) status = fail(HCT_ERR_CUDA, std::string("kernel launch (or an earlier pending error): ") + cudaGetErrorString(rc));
  }
  cudaSetDevice(prev);
  return status;
}
