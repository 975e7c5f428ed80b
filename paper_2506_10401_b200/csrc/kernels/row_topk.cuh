// Row-wise top-k for small k by radix selection: one CTA per row.
// The row is held in shared memory as 32-bit keys whose unsigned order is the order of the fp32
// values (sign bit flipped for non-negative values, all bits for negative ones).  Four passes over
// the row, one per key byte from the top, build a 256-bin histogram of the keys that still match
// the bytes fixed so far and pick the bin that contains the k-th largest key; after the last pass
// the k-th largest key is known exactly, together with how many keys equal to it belong to the
// result.  Keys above it are then collected (in any order), the remaining places take the k-th key
// itself, and a bitonic network over the HCT_KP >= k collected keys puts them in descending order.
// Values are only moved; the elementwise consumers of the result are applied at the store.
//
// For k <= 64 a shortcut comes first.  Every thread keeps the largest of its own keys; the k-th
// largest of these per-thread maxima, found by 32 rounds of bisection with a counting barrier, is a
// lower bound of the k-th largest key of the row (k different elements reach it).  The keys that
// reach the bound, usually little more than k of them, are collected and sorted by a 128-slot bitonic
// network.  When more than 128 keys reach the bound (many equal values, or a row whose large values
// all sit with one thread) the row takes the radix selection instead.
// Defined by the generator: HCT_R, HCT_C, HCT_K, HCT_KP (power of two >= HCT_K, <= 2 * HCT_T), HCT_T (threads,
// 256), HCT_TA, HCT_PA, HctParams, hct_epilogue(), HCT_KERNEL_NAME.
__device__ __forceinline__ unsigned hct_key_of(float f) {
  const unsigned u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float hct_value_of(unsigned k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

extern "C" __global__ void __launch_bounds__(HCT_T) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  __shared__ unsigned key[HCT_C];
  __shared__ unsigned hist[256];
  __shared__ unsigned sel[HCT_KP];
  __shared__ unsigned pick_bin, pick_need, n_above;
#if HCT_K <= 64
  __shared__ unsigned few[128];
#endif
  const HCT_TA* __restrict__ X = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const int tid = threadIdx.x;
  for (long long row = blockIdx.x; row < HCT_R; row += gridDim.x) {
    unsigned mymax = 0u;
    for (int i = tid; i < HCT_C; i += HCT_T) {
      const unsigned u = hct_key_of(hct_ld1(X + row * HCT_C + i));
      key[i] = u;
      mymax = u > mymax ? u : mymax;
    }
#if HCT_K <= 64
    {
      unsigned low = 0u;   // becomes the HCT_K-th largest per-thread maximum (at least HCT_K threads hold an element)
#pragma unroll 1
      for (int bit = 31; bit >= 0; --bit) {
        const unsigned cand = low | (1u << bit);
        if (__syncthreads_count(mymax >= cand) >= HCT_K) low = cand;
      }
      if (tid == 0) n_above = 0u;
      __syncthreads();
      for (int i = tid; i < HCT_C; i += HCT_T) {
        const unsigned u = key[i];
        if (u >= low) {
          const unsigned pos = atomicAdd(&n_above, 1u);
          if (pos < 128u) few[pos] = u;
        }
      }
      __syncthreads();
      const unsigned cnt = n_above;     // >= HCT_K; the same for every thread
      if (cnt <= 128u) {
        for (int i = (int)cnt + tid; i < 128; i += HCT_T) few[i] = 0u;   // 0 sorts last
        __syncthreads();
        for (int k = 2; k <= 128; k <<= 1) {
          for (int j = k >> 1; j > 0; j >>= 1) {
            if (tid < 64) {
              const int i = ((tid & ~(j - 1)) << 1) | (tid & (j - 1));
              const int l = i | j;
              const unsigned a = few[i], b = few[l];
              if ((a < b) == ((i & k) == 0)) {
                few[i] = b;
                few[l] = a;
              }
            }
            __syncthreads();
          }
        }
        for (int i = tid; i < HCT_K; i += HCT_T) hct_epilogue(hct_p, hct_value_of(few[i]), row * HCT_K + i, row, i);
        __syncthreads();
        continue;
      }
    }
#endif
    unsigned prefix = 0u, mask = 0u, need = HCT_K;
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8) {
      hist[tid] = 0u;   // HCT_T == 256 bins
      __syncthreads();
      for (int i = tid; i < HCT_C; i += HCT_T) {
        const unsigned u = key[i];
        if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & 255u], 1u);
      }
      __syncthreads();
      // bin `tid` holds the sought key when fewer than `need` matching keys lie in the bins above it
      // and at least `need` in those bins together with it; exactly one bin qualifies
      unsigned above = 0u;
      for (int b = tid + 1; b < 256; ++b) above += hist[b];
      const unsigned mine = hist[tid];
      if (above < need && above + mine >= need) {
        pick_bin = (unsigned)tid;
        pick_need = need - above;
      }
      __syncthreads();
      prefix |= pick_bin << shift;
      mask |= 255u << shift;
      need = pick_need;
    }
    // prefix is the k-th largest key; `need` of the keys equal to it belong to the result
    if (tid == 0) n_above = 0u;
    __syncthreads();
    for (int i = tid; i < HCT_C; i += HCT_T) {
      const unsigned u = key[i];
      if (u > prefix) sel[atomicAdd(&n_above, 1u)] = u;   // HCT_K - need of them: always fewer than HCT_K
    }
    __syncthreads();
    for (int i = (int)n_above + tid; i < HCT_KP; i += HCT_T) sel[i] = i < HCT_K ? prefix : 0u;   // 0 sorts last
    __syncthreads();
    for (int k = 2; k <= HCT_KP; k <<= 1) {
      for (int j = k >> 1; j > 0; j >>= 1) {
        for (int t = tid; t < HCT_KP / 2; t += HCT_T) {
          const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
          const int l = i | j;
          const unsigned a = sel[i], b = sel[l];
          const bool down = (i & k) == 0;     // descending overall
          if ((a < b) == down) {
            sel[i] = b;
            sel[l] = a;
          }
        }
        __syncthreads();
      }
    }
    for (int i = tid; i < HCT_K; i += HCT_T) hct_epilogue(hct_p, hct_value_of(sel[i]), row * HCT_K + i, row, i);
    __syncthreads();
  }
}
