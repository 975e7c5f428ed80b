// Splits fp32 operands into TF32 head and tail for error-compensated tensor-core products:
// hi = tf32(x), lo = tf32(x - hi), so that x = hi + lo up to 2^-22 |x| and
// a*b ~ a_lo*b_hi + a_hi*b_lo + a_hi*b_hi with every factor exactly representable in TF32.
// A[M,K] keeps its layout; B[K,N] is written transposed ([N,K]) so that both tensor-core
// operands are K-major.
// With HCT_SPLIT_A = 0 only B is handled: A's head and tail were written by the kernel that produced A.
// Defined by the generator: HCT_M, HCT_N, HCT_K (K a multiple of 4), HCT_SPLIT_A, HctParams, HCT_KERNEL_NAME.
// Pointer slots: 0 = A, 1 = B, 2 = A_hi, 3 = A_lo, 4 = Bt_hi, 5 = Bt_lo, 6 = HCT_ZERO_VEC4 16-byte vectors to
// clear (accumulation tiles and arrival counters of a GEMM that splits its contraction; 0: none).
#ifndef HCT_ZERO_VEC4
#define HCT_ZERO_VEC4 0LL
#endif
#define HCT_A_BLOCKS (HCT_SPLIT_A ? (HCT_M * HCT_K / 4 + 1023) / 1024 : 0LL)          // 256 threads x 4 vectors
#define HCT_BT_K ((HCT_K + 31) / 32)
#define HCT_BT_N ((HCT_N + 31) / 32)
extern "C" __global__ void __launch_bounds__(256) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  __shared__ float tile[32][33];
  for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < HCT_ZERO_VEC4; i += (long long)gridDim.x * 256)
    ((float4*)hct_p.ptr[6])[i] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  for (long long blk = blockIdx.x; blk < HCT_A_BLOCKS + HCT_BT_K * HCT_BT_N; blk += gridDim.x) {
    if (blk < HCT_A_BLOCKS) {
      const long long nva = HCT_M * HCT_K / 4;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const long long j = blk * 1024 + u * 256 + threadIdx.x;
        if (j < nva) {
          const float4 x = __ldg((const float4*)hct_p.ptr[0] + j);
          float4 hi, lo;
          hi.x = hct_to_tf32(x.x); lo.x = hct_to_tf32(x.x - hi.x);
          hi.y = hct_to_tf32(x.y); lo.y = hct_to_tf32(x.y - hi.y);
          hi.z = hct_to_tf32(x.z); lo.z = hct_to_tf32(x.z - hi.z);
          hi.w = hct_to_tf32(x.w); lo.w = hct_to_tf32(x.w - hi.w);
          ((float4*)hct_p.ptr[2])[j] = hi;
          ((float4*)hct_p.ptr[3])[j] = lo;
        }
      }
    } else {
      const long long t = blk - HCT_A_BLOCKS;
      const long long k0 = (t / HCT_BT_N) * 32, n0 = (t % HCT_BT_N) * 32;
      const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
      const float* __restrict__ B = (const float*)hct_p.ptr[1];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const long long k = k0 + ty + 8 * i, n = n0 + tx;
        tile[ty + 8 * i][tx] = (k < HCT_K && n < HCT_N) ? __ldg(B + k * HCT_N + n) : 0.0f;
      }
      __syncthreads();
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const long long n = n0 + ty + 8 * i, k = k0 + tx;
        if (n < HCT_N && k < HCT_K) {
          const float x = tile[tx][ty + 8 * i];
          const float hi = hct_to_tf32(x);
          ((float*)hct_p.ptr[4])[n * HCT_K + k] = hi;
          ((float*)hct_p.ptr[5])[n * HCT_K + k] = hct_to_tf32(x - hi);
        }
      }
      __syncthreads();
    }
  }
}
