// Skeleton of the fused row kernel.  The generator defines, before this text:
//   HCT_T   threads that share one row (power of two)      HCT_G  rows handled side by side per CTA
//   HCT_V   elements per vector access (1, 2 or 4)         HCT_NV vectors per thread
//   HCT_R   rows                                           HCT_C  columns
//   HCT_NPTR number of pointer arguments
// and, after it, the kernel body built from HCT_ROW_BEGIN / HCT_ROW_END.
//
// A row lives in registers from its load to its store: thread t of the row's HCT_T threads owns
// the vectors t, t + HCT_T, t + 2 HCT_T, ... so that every access is coalesced.  Row reductions are
// a shuffle butterfly inside each warp followed, when the row spans several warps, by one
// exchange through shared memory guarded by a named barrier private to the row.
#define HCT_E (HCT_V * HCT_NV)
#define HCT_FULL_VECS ((HCT_C % (HCT_T * HCT_V * HCT_NV)) == 0)

struct HctParams { void* ptr[HCT_NPTR]; };

// column of element e of this thread
#define HCT_COL(e) ((((e) / HCT_V) * HCT_T + hct_t) * HCT_V + ((e) % HCT_V))
// whether element e exists (always true when the row fills every vector)
#define HCT_HAS(e) (HCT_FULL_VECS || HCT_COL(e) < HCT_C)

#if HCT_T > 32
#define HCT_RED_DECL __shared__ float hct_red_smem[HCT_G][2][32];
#else
#define HCT_RED_DECL
#endif

struct HctRowCtx {
  int t;         // thread index within the row
  int g;         // row slot within the CTA
  unsigned par;  // which of the two exchange buffers the next reduction uses
};

template <bool IS_MAX>
__device__ __forceinline__ float hct_row_reduce(float v, HctRowCtx& cx, float (*red)[2][32]) {
#pragma unroll
  for (int o = (HCT_T < 32 ? HCT_T : 32) / 2; o > 0; o >>= 1) {
    float u = __shfl_xor_sync(0xffffffffu, v, o);
    v = IS_MAX ? fmaxf(v, u) : v + u;
  }
#if HCT_T > 32
  float* slot = red[cx.g][cx.par];
  cx.par ^= 1u;
  if ((cx.t & 31) == 0) slot[cx.t >> 5] = v;
  asm volatile("bar.sync %0, %1;" ::"r"(cx.g + 1), "n"(HCT_T) : "memory");
  v = slot[0];
#pragma unroll
  for (int w = 1; w < HCT_T / 32; ++w) v = IS_MAX ? fmaxf(v, slot[w]) : v + slot[w];
#endif
  return v;
}
#if HCT_T > 32
#define HCT_RSUM(v) hct_row_reduce<false>(v, hct_cx, hct_red_smem)
#define HCT_RMAX(v) hct_row_reduce<true>(v, hct_cx, hct_red_smem)
#else
#define HCT_RSUM(v) hct_row_reduce<false>(v, hct_cx, nullptr)
#define HCT_RMAX(v) hct_row_reduce<true>(v, hct_cx, nullptr)
#endif

// Load / store one thread's share of a full-width row.
template <typename T>
__device__ __forceinline__ void hct_load_row(const T* base, long long row, int hct_t, float* v, bool keep) {
  const T* p = base + row * (long long)HCT_C;
#pragma unroll
  for (int k = 0; k < HCT_NV; ++k) {
    int col = (k * HCT_T + hct_t) * HCT_V;
    if (HCT_FULL_VECS || col < HCT_C) {
      if (keep) hct_vecio<HCT_V>::ld_keep(p + col, v + k * HCT_V);
      else hct_vecio<HCT_V>::ld_stream(p + col, v + k * HCT_V);
    } else {
#pragma unroll
      for (int i = 0; i < HCT_V; ++i) v[k * HCT_V + i] = 0.0f;
    }
  }
}
template <typename T>
__device__ __forceinline__ void hct_store_row(T* base, long long row, int hct_t, const float* v) {
  T* p = base + row * (long long)HCT_C;
#pragma unroll
  for (int k = 0; k < HCT_NV; ++k) {
    int col = (k * HCT_T + hct_t) * HCT_V;
    if (HCT_FULL_VECS || col < HCT_C) hct_vecio<HCT_V>::st(p + col, v + k * HCT_V);
  }
}

#define HCT_ROW_KERNEL_BEGIN(name)                                                            \
  extern "C" __global__ void __launch_bounds__(HCT_T * HCT_G) name(const HctParams hct_p) {   \
    HCT_RED_DECL                                                                              \
    HctRowCtx hct_cx;                                                                         \
    hct_cx.t = threadIdx.x % HCT_T;                                                           \
    hct_cx.g = threadIdx.x / HCT_T;                                                           \
    hct_cx.par = 0;                                                                           \
    const int hct_t = hct_cx.t;

#define HCT_ROW_LOOP_BEGIN                                                                    \
    for (long long hct_base = (long long)blockIdx.x * HCT_G; hct_base < HCT_R;                \
         hct_base += (long long)gridDim.x * HCT_G) {                                          \
      const bool hct_live = hct_base + hct_cx.g < HCT_R;                                      \
      const long long hct_row = hct_live ? hct_base + hct_cx.g : HCT_R - 1;

#define HCT_ROW_LOOP_END }
#define HCT_ROW_KERNEL_END }
