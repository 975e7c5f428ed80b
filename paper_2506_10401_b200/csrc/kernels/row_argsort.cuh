// Row-wise argsort / top-k indices (logic-intensive operator class): one CTA orders one row and stores
// the COLUMNS of the first HCT_KOUT values in that order, as fp32 values, with the elementwise
// consumers of the result applied at the store.
// Every element becomes one 64-bit key: high word = its value mapped to an unsigned integer of the same
// order (-0 first made +0, so the two compare equal; complemented for a descending order), low word =
// its column.  Sorting the keys as plain unsigned integers therefore orders by value and, among equal
// values, by column, in both directions; the network need not be stable.  Padding keys are all ones.
// The bitonic network is the one of the value sort: steps at distance <= 4 in registers on blocks of 8
// consecutive slots, steps at larger distances two at a time on quadruples, a block barrier between groups.
// Defined by the generator: HCT_R, HCT_C, HCT_NP, HCT_KOUT, HCT_DESC, HCT_T (threads), HCT_TA, HCT_PA,
// HctParams, hct_epilogue(), HCT_KERNEL_NAME.
#define HCT_KSWAP(a, b, up)                 \
  {                                         \
    const hct_u64 x_ = (a), y_ = (b);       \
    const bool s_ = (x_ > y_) == (up);      \
    (a) = s_ ? y_ : x_;                     \
    (b) = s_ ? x_ : y_;                     \
  }

__device__ __forceinline__ hct_u64 hct_sort_key(float v, int col) {
  hct_u32 u = __float_as_uint(v + 0.0f);                   // -0 + 0 = +0
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);          // unsigned order = numeric order
  if (HCT_DESC) u = ~u;
  return ((hct_u64)u << 32) | (hct_u32)col;
}
__device__ __forceinline__ void hct_key_load8(const hct_u64* key, int t, hct_u64 (&r)[8]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const ulonglong2 p = ((const ulonglong2*)key)[4 * t + i];
    r[2 * i] = p.x; r[2 * i + 1] = p.y;
  }
}
__device__ __forceinline__ void hct_key_store8(hct_u64* key, int t, const hct_u64 (&r)[8]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) ((ulonglong2*)key)[4 * t + i] = make_ulonglong2(r[2 * i], r[2 * i + 1]);
}

extern "C" __global__ void __launch_bounds__(HCT_T) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  extern __shared__ __align__(16) unsigned char hct_sort_smem[];
  hct_u64* key = (hct_u64*)hct_sort_smem;
  const HCT_TA* __restrict__ X = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const int tid = threadIdx.x;
  for (long long row = blockIdx.x; row < HCT_R; row += gridDim.x) {
    for (int i = tid; i < HCT_NP; i += HCT_T) key[i] = i < HCT_C ? hct_sort_key(hct_ld1(X + row * HCT_C + i), i) : ~0ull;
    __syncthreads();
    // phases k = 2, 4, 8: entirely inside blocks of 8
    for (int t = tid; t < HCT_NP / 8; t += HCT_T) {
      hct_u64 r[8];
      hct_key_load8(key, t, r);
#pragma unroll
      for (int k = 2; k <= 8; k <<= 1)
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1)
#pragma unroll
          for (int p = 0; p < 4; ++p) {
            const int i = ((p & ~(j - 1)) << 1) | (p & (j - 1));
            const bool up = ((8 * t + i) & k) == 0;
            HCT_KSWAP(r[i], r[i | j], up);
          }
      hct_key_store8(key, t, r);
    }
    __syncthreads();
    for (int k = 16; k <= HCT_NP; k <<= 1) {
      int j = k >> 1;
      for (; j >= 16; j >>= 2) {   // pairs of steps (j, j / 2) with j / 2 >= 8
        const int h = j >> 1;
        for (int q = tid; q < HCT_NP / 4; q += HCT_T) {
          const int i0 = ((q & ~(h - 1)) << 2) | (q & (h - 1));
          const bool up = (i0 & k) == 0;
          hct_u64 a = key[i0], b = key[i0 + h], c = key[i0 + j], d = key[i0 + j + h];
          HCT_KSWAP(a, c, up);
          HCT_KSWAP(b, d, up);
          HCT_KSWAP(a, b, up);
          HCT_KSWAP(c, d, up);
          key[i0] = a; key[i0 + h] = b; key[i0 + j] = c; key[i0 + j + h] = d;
        }
        __syncthreads();
      }
      if (j == 8) {   // a single step left before the register tail
        for (int t = tid; t < HCT_NP / 2; t += HCT_T) {
          const int i = ((t & ~7) << 1) | (t & 7);
          const bool up = (i & k) == 0;
          hct_u64 a = key[i], b = key[i | 8];
          HCT_KSWAP(a, b, up);
          key[i] = a; key[i | 8] = b;
        }
        __syncthreads();
      }
      for (int t = tid; t < HCT_NP / 8; t += HCT_T) {
        hct_u64 r[8];
        hct_key_load8(key, t, r);
        const bool up = ((8 * t) & k) == 0;
#pragma unroll
        for (int jj = 4; jj > 0; jj >>= 1)
#pragma unroll
          for (int p = 0; p < 4; ++p) {
            const int i = ((p & ~(jj - 1)) << 1) | (p & (jj - 1));
            HCT_KSWAP(r[i], r[i | jj], up);
          }
        hct_key_store8(key, t, r);
      }
      __syncthreads();
    }
    for (int i = tid; i < HCT_KOUT; i += HCT_T) hct_epilogue(hct_p, (float)(hct_u32)(key[i] & 0xffffffffull), row * HCT_KOUT + i, row, i);
    __syncthreads();
  }
}
