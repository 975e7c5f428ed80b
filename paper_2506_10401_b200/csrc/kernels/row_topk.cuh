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
// largest of these per-thread maxima, found by the first warp in 32 rounds of bisection over the key bits, is a
// lower bound of the k-th largest key of the row (k different elements reach it).  The keys that
// reach the bound, usually little more than k of them, are collected and sorted by one warp in a 64- or
// 128-slot bitonic network (warp barriers only).  When more than 128 keys reach the bound (many equal values, or a row whose large values
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

static_assert(HCT_T == 256, "one thread per histogram bin");
static_assert(HCT_KP <= 2 * HCT_T && HCT_K <= HCT_KP, "the selected keys are sorted by one pass of the block");
template <typename T> struct hct_topk_is_f32 { static const bool value = false; };
template <> struct hct_topk_is_f32<float> { static const bool value = true; };

extern "C" __global__ void __launch_bounds__(HCT_T) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  __shared__ __align__(16) unsigned key[HCT_C];
  __shared__ unsigned hist[256];
  __shared__ unsigned sel[HCT_KP];
  __shared__ unsigned pick_bin, pick_need, n_above;
#if HCT_K <= 64
  __shared__ unsigned few[128];
  __shared__ unsigned tmax[HCT_T];
  __shared__ unsigned bound;
#endif
  const HCT_TA* __restrict__ X = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const int tid = threadIdx.x;
  for (long long row = blockIdx.x; row < HCT_R; row += gridDim.x) {
    unsigned mymax = 0u;
    if (hct_topk_is_f32<HCT_TA>::value && HCT_C % 4 == 0) {
      const float4* __restrict__ x4 = (const float4*)((const float*)X + row * HCT_C);
      for (int i = tid; i < HCT_C / 4; i += HCT_T) {
        const float4 v = __ldg(x4 + i);
        const uint4 u = make_uint4(hct_key_of(v.x), hct_key_of(v.y), hct_key_of(v.z), hct_key_of(v.w));
        ((uint4*)key)[i] = u;
        const unsigned a = u.x > u.y ? u.x : u.y, b = u.z > u.w ? u.z : u.w;
        const unsigned c = a > b ? a : b;
        mymax = c > mymax ? c : mymax;
      }
    } else {
      for (int i = tid; i < HCT_C; i += HCT_T) {
        const unsigned u = hct_key_of(hct_ld1(X + row * HCT_C + i));
        key[i] = u;
        mymax = u > mymax ? u : mymax;
      }
    }
#if HCT_K <= 64
    {
      // The first warp finds the HCT_K-th largest per-thread maximum (at least HCT_K threads hold an element)
      // by bisection over the key bits, eight maxima per lane.
      tmax[tid] = mymax;
      __syncthreads();
      if (tid < 32) {
        unsigned m[HCT_T / 32];
#pragma unroll
        for (int q = 0; q < HCT_T / 32; ++q) m[q] = tmax[tid + 32 * q];
        unsigned low = 0u;
#pragma unroll 1
        for (int bit = 31; bit >= 0; --bit) {
          const unsigned cand = low | (1u << bit);
          int c = 0;
#pragma unroll
          for (int q = 0; q < HCT_T / 32; ++q) c += m[q] >= cand ? 1 : 0;
          if (__reduce_add_sync(0xffffffffu, c) >= HCT_K) low = cand;
        }
        if (tid == 0) {
          bound = low;
          n_above = 0u;
        }
      }
      __syncthreads();
      const unsigned low = bound;
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
        if (tid < 32) {                 // one warp sorts the collected keys, largest first; 0 sorts last
          const int np = cnt <= 64u ? 64 : 128;
          for (int i = (int)cnt + tid; i < np; i += 32) few[i] = 0u;
          __syncwarp();
          for (int k = 2; k <= np; k <<= 1) {
            for (int j = k >> 1; j > 0; j >>= 1) {
              for (int t = tid; t < np / 2; t += 32) {
                const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
                const int l = i | j;
                const unsigned a = few[i], b = few[l];
                if ((a < b) == ((i & k) == 0)) {
                  few[i] = b;
                  few[l] = a;
                }
              }
              __syncwarp();
            }
          }
        }
        __syncthreads();
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
