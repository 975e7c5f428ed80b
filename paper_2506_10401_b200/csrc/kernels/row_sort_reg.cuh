// Row-wise sort in registers (logic-intensive operator class): one CTA sorts one row of HCT_C values, padded to
// HCT_NP = 16 * HCT_T slots (a power of two; pads sort to the end), with a bitonic network whose
// compare-exchange steps run where the two partners already are:
//   - thread t holds slots 16 t .. 16 t + 15 in registers; a step with distance j < 16 pairs two of its own
//     registers (one minimum and one maximum per pair);
//   - 16 <= j < 512: the partner slot is the same register of lane ^ (j / 16): one shuffle, then the thread
//     keeps the minimum or the maximum of every pair (which one is the same for all of its 16 slots);
//   - j >= 512: the partner is the same register of thread t ^ (j / 16) in another warp: the threads exchange
//     their 16 values through shared memory (16-byte accesses, chunks permuted so that a quarter warp
//     covers all banks), two block barriers per step; a 4096-slot row has six such steps.
// Values are only moved, never changed (minimum and maximum of a pair return both of its values; inputs are
// expected to be free of NaN, which no ordering places).  The sorted row leaves through the same
// shared-memory buffer so that the stores (and the elementwise consumers applied there) are coalesced.
// Defined by the generator: HCT_R, HCT_C, HCT_NP, HCT_KOUT, HCT_DESC, HCT_T (= HCT_NP / 16, a multiple of 32),
// HCT_TA, HCT_PA, HctParams, hct_epilogue(), HCT_KERNEL_NAME.

// slot of 16-byte chunk c (0..3) of thread t's 16 values
__device__ __forceinline__ int hct_sort_chunk(int t, int c) { return t * 4 + (c ^ ((t >> 1) & 3)); }

__host__ __device__ constexpr int hct_sort_log2(int n) { return n <= 1 ? 0 : 1 + hct_sort_log2(n >> 1); }

extern "C" __global__ void __launch_bounds__(HCT_T) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  __shared__ float4 buf[HCT_NP / 4];
  const HCT_TA* __restrict__ X = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const int t = threadIdx.x;
  const float pad = HCT_DESC ? -HCT_INF : HCT_INF;
  const bool desc = HCT_DESC != 0;
  for (long long row = blockIdx.x; row < HCT_R; row += gridDim.x) {
    float r[16];
    const HCT_TA* xr = X + row * HCT_C;
    if (sizeof(HCT_TA) == 4 && HCT_C % 4 == 0) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int e = t * 16 + c * 4;
        float4 v = make_float4(pad, pad, pad, pad);
        if (e < HCT_C) v = __ldg((const float4*)(const void*)xr + (e >> 2));
        r[4 * c] = v.x; r[4 * c + 1] = v.y; r[4 * c + 2] = v.z; r[4 * c + 3] = v.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < 16; ++i) r[i] = t * 16 + i < HCT_C ? hct_ld1(xr + t * 16 + i) : pad;
    }
#pragma unroll
    for (int lk = 1; lk <= hct_sort_log2(HCT_NP); ++lk) {
      const int k = 1 << lk;
      // Phase k merges sorted runs of k / 2 slots into sorted runs of k.  Its first step pairs slot e with its
      // mirror image e ^ (k - 1) inside the run of k, the following steps pair e with e ^ j for j = k / 4 .. 1; in
      // every step the slot with the smaller index receives the value that sorts first, so the order of a pair
      // never depends on where it lies (steps inside a thread are one minimum and one maximum per pair).
#pragma unroll
      for (int lj = lk - 1; lj >= 0; --lj) {
        const int j = 1 << lj;
        const bool mirror = lj == lk - 1;
        const int x = mirror ? k - 1 : j;              // slot e meets slot e ^ x
        if (x >= 16) {
          const int px = x >> 4;                       // thread t meets thread t ^ px, register i meets i ^ (x & 15)
          const bool first = ((t >> (lj - 4)) & 1) == 0;   // this thread holds the smaller index of every pair
          float o[16];
          if (px >= 32) {
#pragma unroll
            for (int c = 0; c < 4; ++c) buf[hct_sort_chunk(t, c)] = make_float4(r[4 * c], r[4 * c + 1], r[4 * c + 2], r[4 * c + 3]);
            __syncthreads();
            const int pt = t ^ px;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const float4 v = buf[hct_sort_chunk(pt, mirror ? 3 - c : c)];
              if (mirror) { o[4 * c] = v.w; o[4 * c + 1] = v.z; o[4 * c + 2] = v.y; o[4 * c + 3] = v.x; }
              else { o[4 * c] = v.x; o[4 * c + 1] = v.y; o[4 * c + 2] = v.z; o[4 * c + 3] = v.w; }
            }
            __syncthreads();
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) o[i] = __shfl_xor_sync(0xffffffffu, r[mirror ? 15 - i : i], px);
          }
          // keep the value that sorts first if this thread holds the smaller index, else the other one (minimum and
          // maximum order -0 below +0, so the two partners never keep the same one of two equal values)
          const bool keep_small = first != desc;
#pragma unroll
          for (int i = 0; i < 16; ++i) r[i] = keep_small ? fminf(r[i], o[i]) : fmaxf(r[i], o[i]);
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int q = i ^ x;
            if (q < i) continue;
            const float a = r[i], b = r[q];
            r[i] = desc ? fmaxf(a, b) : fminf(a, b);
            r[q] = desc ? fminf(a, b) : fmaxf(a, b);
          }
        }
      }
    }
    // the first HCT_KOUT slots, through shared memory, to coalesced stores
#pragma unroll
    for (int c = 0; c < 4; ++c) buf[hct_sort_chunk(t, c)] = make_float4(r[4 * c], r[4 * c + 1], r[4 * c + 2], r[4 * c + 3]);
    __syncthreads();
    const float* flat = (const float*)buf;
    for (int i = t; i < HCT_KOUT; i += HCT_T) {
      const int owner = i >> 4, c = (i >> 2) & 3;
      hct_epilogue(hct_p, flat[hct_sort_chunk(owner, c) * 4 + (i & 3)], row * HCT_KOUT + i, row, i);
    }
    __syncthreads();
  }
}
