// Row-wise sort (logic-intensive operator class): one CTA sorts one row of HCT_C values with a bitonic
// network in shared memory and stores the first HCT_KOUT of them (all of them for a sort, the k
// largest for a top-k of large k), with the elementwise consumers of the result applied at the store.
// The row is padded to HCT_NP, a power of two >= 8, with values that sort to the end (+inf ascending,
// -inf descending).  A compare-exchange step pairs element i with i ^ j and orders the pair
// ascending or descending by bit `k` of i.  Steps are grouped so that a block barrier is needed only
// between groups:
//   - steps with j <= 4 stay inside blocks of 8 consecutive elements: a thread loads its block into
//     registers, runs the three steps (all steps of the phases k <= 8) and writes the block back;
//   - steps with j >= 8 are taken two at a time (j and j / 2) on quadruples i, i + j/2, i + j, i + 3j/2,
//     which one thread loads once; a phase with an odd number of such steps ends with a single one.
// Values are only moved, never changed.
// Defined by the generator: HCT_R, HCT_C, HCT_NP, HCT_KOUT, HCT_DESC, HCT_T (threads), HCT_TA, HCT_PA,
// HctParams, hct_epilogue(), HCT_KERNEL_NAME.
#define HCT_CSWAP(a, b, up)                 \
  {                                         \
    const float x_ = (a), y_ = (b);         \
    const bool s_ = (x_ > y_) == (up);      \
    (a) = s_ ? y_ : x_;                     \
    (b) = s_ ? x_ : y_;                     \
  }

// steps j = 4, 2, 1 of one phase on a block of 8 registers, all pairs ordered the same way
__device__ __forceinline__ void hct_sort_tail8(float (&r)[8], bool up) {
#pragma unroll
  for (int j = 4; j > 0; j >>= 1)
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const int i = ((p & ~(j - 1)) << 1) | (p & (j - 1));
      HCT_CSWAP(r[i], r[i | j], up);
    }
}

// block t of 8 consecutive slots as two 16-byte accesses (no bank conflicts, unlike eight 4-byte ones at a stride of 8)
__device__ __forceinline__ void hct_sort_load8(const float* key, int t, float (&r)[8]) {
  const float4 lo = ((const float4*)key)[2 * t], hi = ((const float4*)key)[2 * t + 1];
  r[0] = lo.x; r[1] = lo.y; r[2] = lo.z; r[3] = lo.w; r[4] = hi.x; r[5] = hi.y; r[6] = hi.z; r[7] = hi.w;
}
__device__ __forceinline__ void hct_sort_store8(float* key, int t, const float (&r)[8]) {
  ((float4*)key)[2 * t] = make_float4(r[0], r[1], r[2], r[3]);
  ((float4*)key)[2 * t + 1] = make_float4(r[4], r[5], r[6], r[7]);
}

extern "C" __global__ void __launch_bounds__(HCT_T) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  __shared__ __align__(16) float key[HCT_NP];
  const HCT_TA* __restrict__ X = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const int tid = threadIdx.x;
  const float pad = HCT_DESC ? -HCT_INF : HCT_INF;
  const bool desc = HCT_DESC != 0;
  for (long long row = blockIdx.x; row < HCT_R; row += gridDim.x) {
    for (int i = tid; i < HCT_NP; i += HCT_T) key[i] = i < HCT_C ? hct_ld1(X + row * HCT_C + i) : pad;
    __syncthreads();
    // phases k = 2, 4, 8: entirely inside blocks of 8
    for (int t = tid; t < HCT_NP / 8; t += HCT_T) {
      float r[8];
      hct_sort_load8(key, t, r);
#pragma unroll
      for (int k = 2; k <= 8; k <<= 1)
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1)
#pragma unroll
          for (int p = 0; p < 4; ++p) {
            const int i = ((p & ~(j - 1)) << 1) | (p & (j - 1));
            const bool up = (((8 * t + i) & k) == 0) != desc;
            HCT_CSWAP(r[i], r[i | j], up);
          }
      hct_sort_store8(key, t, r);
    }
    __syncthreads();
    for (int k = 16; k <= HCT_NP; k <<= 1) {
      int j = k >> 1;
      // pairs of steps (j, j / 2) with j / 2 >= 8
      for (; j >= 16; j >>= 2) {
        const int h = j >> 1;
        for (int q = tid; q < HCT_NP / 4; q += HCT_T) {
          const int i0 = ((q & ~(h - 1)) << 2) | (q & (h - 1));
          const bool up = ((i0 & k) == 0) != desc;
          float a = key[i0], b = key[i0 + h], c = key[i0 + j], d = key[i0 + j + h];
          HCT_CSWAP(a, c, up);
          HCT_CSWAP(b, d, up);
          HCT_CSWAP(a, b, up);
          HCT_CSWAP(c, d, up);
          key[i0] = a; key[i0 + h] = b; key[i0 + j] = c; key[i0 + j + h] = d;
        }
        __syncthreads();
      }
      if (j == 8) {   // a single step left before the register tail
        for (int t = tid; t < HCT_NP / 2; t += HCT_T) {
          const int i = ((t & ~7) << 1) | (t & 7);
          const bool up = ((i & k) == 0) != desc;
          float a = key[i], b = key[i | 8];
          HCT_CSWAP(a, b, up);
          key[i] = a; key[i | 8] = b;
        }
        __syncthreads();
      }
      for (int t = tid; t < HCT_NP / 8; t += HCT_T) {
        float r[8];
        hct_sort_load8(key, t, r);
        hct_sort_tail8(r, (((8 * t) & k) == 0) != desc);
        hct_sort_store8(key, t, r);
      }
      __syncthreads();
    }
    for (int i = tid; i < HCT_KOUT; i += HCT_T) hct_epilogue(hct_p, key[i], row * HCT_KOUT + i, row, i);
    __syncthreads();
  }
}
