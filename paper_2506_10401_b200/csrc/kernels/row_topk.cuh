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

// Radix selection over the keys of one row in shared memory, then a bitonic network over the selected keys and the
// stores (whole CTA; ends with a block barrier).
struct HctTopkShared {
  unsigned hist[256];
  unsigned sel[HCT_KP];
  unsigned pick_bin, pick_need, n_above;
};
__device__ __forceinline__ void hct_topk_radix(const HctParams& hct_p, const unsigned* key, HctTopkShared& sh, long long row, int tid) {
  unsigned* hist = sh.hist;
  unsigned* sel = sh.sel;
  unsigned& pick_bin = sh.pick_bin;
  unsigned& pick_need = sh.pick_need;
  unsigned& n_above = sh.n_above;
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

#ifndef HCT_TOPK_REG
#define HCT_TOPK_REG 0
#endif
#if HCT_TOPK_REG
// Register form (fp32 rows of up to 8192 values, a multiple of 4, k <= 64).  A thread keeps its HCT_E keys in
// registers from load to collection; the next row's loads are issued before the current row is worked on.
// Bound: every warp takes the r-th largest of its 32 per-thread maxima, r = ceil(k / warps), by r - 1 rounds of
// "find the maximum, drop one holder of it" on the warp-reduction unit; the smallest of the warps' results has
// at least k different elements at or above it, so it is a lower bound of the k-th largest key.  All warps
// work on it at the same time and one block barrier publishes it.  The keys that reach the bound (a few more
// than k) are collected in shared memory and ranked by the whole CTA (two threads per key count the keys that
// sort before it; a key whose count is below k is stored at that place), so no warp works alone while the
// others wait; collection buffers alternate between rows.  More than 128 such keys (many equal values, large values crowded into few threads): the keys are
// written to shared memory and the row takes the radix selection.
#define HCT_E ((HCT_C + HCT_T - 1) / HCT_T / 4 * 4 + (((HCT_C + HCT_T - 1) / HCT_T) % 4 ? 4 : 0))   // keys per thread, whole 16-byte vectors
#define HCT_NW (HCT_T / 32)
#define HCT_RTH ((HCT_K + HCT_NW - 1) / HCT_NW)

extern "C" __global__ void __launch_bounds__(HCT_T, 4) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  __shared__ __align__(16) unsigned key[HCT_C];
  __shared__ HctTopkShared sh;
  __shared__ unsigned few[2][128];
  __shared__ unsigned cnt_s[2];
  __shared__ unsigned wbound[2][HCT_NW];
  const float* __restrict__ X = (const float*)hct_p.ptr[HCT_PA];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float4 nxt[HCT_E / 4];
  auto load_row = [&](long long row) {
    const float4* __restrict__ x4 = (const float4*)(X + row * HCT_C);
#pragma unroll
    for (int q = 0; q < HCT_E / 4; ++q) {
      const int i = q * HCT_T + tid;
      nxt[q] = i < HCT_C / 4 ? __ldg(x4 + i) : make_float4(-HCT_INF, -HCT_INF, -HCT_INF, -HCT_INF);
    }
  };
  if ((long long)blockIdx.x < HCT_R) load_row(blockIdx.x);
  if (tid < 2) cnt_s[tid] = 0u;
  __syncthreads();
  int par = 0;
  for (long long row = blockIdx.x; row < HCT_R; row += gridDim.x, par ^= 1) {
    unsigned kr[HCT_E];
    unsigned mymax = 0u;
#pragma unroll
    for (int q = 0; q < HCT_E / 4; ++q) {
      const bool live = q * HCT_T + tid < HCT_C / 4;      // slots past the row hold key 0, which no bound admits before a real key
      kr[4 * q] = live ? hct_key_of(nxt[q].x) : 0u; kr[4 * q + 1] = live ? hct_key_of(nxt[q].y) : 0u;
      kr[4 * q + 2] = live ? hct_key_of(nxt[q].z) : 0u; kr[4 * q + 3] = live ? hct_key_of(nxt[q].w) : 0u;
#pragma unroll
      for (int j = 0; j < 4; ++j) mymax = kr[4 * q + j] > mymax ? kr[4 * q + j] : mymax;
    }
    if (row + gridDim.x < HCT_R) load_row(row + gridDim.x);
    // r-th largest per-thread maximum of this warp
    unsigned m = mymax, wr = 0u;
#pragma unroll
    for (int it = 0; it < HCT_RTH; ++it) {
      wr = __reduce_max_sync(0xffffffffu, m);
      const unsigned holders = __ballot_sync(0xffffffffu, m == wr);
      if (lane == __ffs(holders) - 1) m = 0u;
    }
    if (lane == 0) wbound[par][warp] = wr;
    __syncthreads();
    if (tid == 0) cnt_s[par ^ 1] = 0u;   // the previous row's count: every thread has read it, and it is next added to two barriers from here
    unsigned low = wbound[par][0];
#pragma unroll
    for (int w = 1; w < HCT_NW; ++w) low = wbound[par][w] < low ? wbound[par][w] : low;
#pragma unroll
    for (int e = 0; e < HCT_E; ++e)
      if (kr[e] >= low && kr[e] != 0u) {
        const unsigned pos = atomicAdd(&cnt_s[par], 1u);
        if (pos < 128u) few[par][pos] = kr[e];
      }
    __syncthreads();
    const unsigned cnt = cnt_s[par];     // >= HCT_K when the row has that many values; the same for every thread
    if (cnt <= 128u) {
      // Ranking by the whole CTA: two threads per collected key count, each over half of the keys, how many
      // sort before it (larger, or equal with a smaller index); the key's place in the result is that count.
      const int i = tid >> 1, h = tid & 1;
      const unsigned mykey = (unsigned)i < cnt ? few[par][i] : 0u;
      const int half = ((int)cnt + 1) >> 1;
      const int j0 = h * half, j1 = j0 + half < (int)cnt ? j0 + half : (int)cnt;
      int rank = 0;
#pragma unroll 4
      for (int j = j0; j < j1; ++j) {
        const unsigned o = few[par][j];
        rank += (o > mykey || (o == mykey && j < i)) ? 1 : 0;
      }
      rank += __shfl_xor_sync(0xffffffffu, rank, 1);
      if (h == 0 && (unsigned)i < cnt && rank < HCT_K) hct_epilogue(hct_p, hct_value_of(mykey), row * HCT_K + rank, row, rank);
      continue;
    }
    // crowded row: keys to shared memory, radix selection by the whole CTA
#pragma unroll
    for (int q = 0; q < HCT_E / 4; ++q)
      if (q * HCT_T + tid < HCT_C / 4) ((uint4*)key)[q * HCT_T + tid] = make_uint4(kr[4 * q], kr[4 * q + 1], kr[4 * q + 2], kr[4 * q + 3]);
    __syncthreads();
    hct_topk_radix(hct_p, key, sh, row, tid);
  }
}
#else
extern "C" __global__ void __launch_bounds__(HCT_T) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  __shared__ __align__(16) unsigned key[HCT_C];
  __shared__ HctTopkShared sh;
  unsigned& n_above = sh.n_above;
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
    hct_topk_radix(hct_p, key, sh, row, tid);
  }
}
#endif
