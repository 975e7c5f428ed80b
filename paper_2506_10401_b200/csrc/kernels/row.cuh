// Skeleton of the fused row kernel.  The generator defines, before this text:
//   HCT_T   threads that share one row (power of two)      HCT_G  rows handled side by side per CTA
//   HCT_V   elements per vector access (1, 2 or 4)         HCT_NV vectors per thread
//   HCT_R   rows                                           HCT_C  columns
//   HCT_B   consecutive rows each row group carries at once (their reductions travel together,
//           so the latency of a block reduction is paid once per HCT_B rows)
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
#define HCT_RED_DECL __shared__ float hct_red_smem[HCT_G][2][HCT_B][32]; __shared__ float hct_sm_smem[HCT_G][2][HCT_B][3][32];
#else
#define HCT_RED_DECL
#endif

struct HctRowCtx {
  int t;         // thread index within the row
  int g;         // row slot within the CTA
  unsigned par;  // which of the two exchange buffers the next reduction uses
};

template <bool IS_MAX>
__device__ __forceinline__ void hct_row_reduce(float (&v)[HCT_B], HctRowCtx& cx, float (*red)[2][HCT_B][32]) {
#pragma unroll
  for (int o = (HCT_T < 32 ? HCT_T : 32) / 2; o > 0; o >>= 1) {
#pragma unroll
    for (int b = 0; b < HCT_B; ++b) {
      float u = __shfl_xor_sync(0xffffffffu, v[b], o);
      v[b] = IS_MAX ? fmaxf(v[b], u) : v[b] + u;
    }
  }
#if HCT_T > 32
  // one partial per warp and row goes through shared memory; every warp then folds the HCT_T/32
  // partials with a second, shorter butterfly, so all threads end with the same values
  float (*slot)[32] = red[cx.g][cx.par];
  cx.par ^= 1u;
  if ((cx.t & 31) == 0) {
#pragma unroll
    for (int b = 0; b < HCT_B; ++b) slot[b][cx.t >> 5] = v[b];
  }
  asm volatile("bar.sync %0, %1;" ::"r"(cx.g + 1), "n"(HCT_T) : "memory");
#pragma unroll
  for (int b = 0; b < HCT_B; ++b) v[b] = slot[b][cx.t & (HCT_T / 32 - 1)];
#pragma unroll
  for (int o = HCT_T / 64; o > 0; o >>= 1) {
#pragma unroll
    for (int b = 0; b < HCT_B; ++b) {
      float u = __shfl_xor_sync(0xffffffffu, v[b], o);
      v[b] = IS_MAX ? fmaxf(v[b], u) : v[b] + u;
    }
  }
#endif
}
// Reduction over the lanes of one warp that share a row (no barrier): all of them end with the result.
template <bool IS_MAX>
__device__ __forceinline__ void hct_warp_reduce(float (&v)[HCT_B]) {
#pragma unroll
  for (int o = (HCT_T < 32 ? HCT_T : 32) / 2; o > 0; o >>= 1) {
#pragma unroll
    for (int b = 0; b < HCT_B; ++b) {
      float u = __shfl_xor_sync(0xffffffffu, v[b], o);
      v[b] = IS_MAX ? fmaxf(v[b], u) : v[b] + u;
    }
  }
}

// Softmax statistics of a row in ONE exchange between its warps.  Every warp has taken its terms
// t = 2^((x - m) log2 e) relative to its OWN maximum m (reference 0 when the warp saw no finite
// value); on entry m, s, q hold the warp's maximum, sum of terms and (WITH_Q) sum of squared terms.
// The warps' triples meet in shared memory and are folded with weights 2^((m_warp - m_row) log2 e).
// On exit m is the row maximum, s and q the row's sums relative to it, and f the weight of the calling
// thread's own terms: term * f / s is the softmax value.
template <bool WITH_Q>
__device__ __forceinline__ void hct_softmax_combine(float (&m)[HCT_B], float (&s)[HCT_B], float (&q)[HCT_B], float (&f)[HCT_B], HctRowCtx& cx,
                                                    float (*red)[2][HCT_B][3][32]) {
#if HCT_T > 32
  float (*slot)[3][32] = red[cx.g][cx.par];
  cx.par ^= 1u;
  if ((cx.t & 31) == 0) {
#pragma unroll
    for (int b = 0; b < HCT_B; ++b) {
      slot[b][0][cx.t >> 5] = m[b];
      slot[b][1][cx.t >> 5] = s[b];
      if (WITH_Q) slot[b][2][cx.t >> 5] = q[b];
    }
  }
  asm volatile("bar.sync %0, %1;" ::"r"(cx.g + 1), "n"(HCT_T) : "memory");
  const int j = cx.t & (HCT_T / 32 - 1);
#pragma unroll
  for (int b = 0; b < HCT_B; ++b) {
    const float mj = slot[b][0][j];
    float sj = slot[b][1][j], qj = WITH_Q ? slot[b][2][j] : 0.0f;
    float mr = mj;
#pragma unroll
    for (int o = HCT_T / 64; o > 0; o >>= 1) mr = fmaxf(mr, __shfl_xor_sync(0xffffffffu, mr, o));
    const float ref = mr == -HCT_INF ? 0.0f : mr;
    const float fj = hct_exp2_fast(((mj == -HCT_INF ? 0.0f : mj) - ref) * HCT_LOG2E);
    sj *= fj;
    qj *= fj * fj;
#pragma unroll
    for (int o = HCT_T / 64; o > 0; o >>= 1) {
      sj += __shfl_xor_sync(0xffffffffu, sj, o);
      if (WITH_Q) qj += __shfl_xor_sync(0xffffffffu, qj, o);
    }
    f[b] = hct_exp2_fast(((m[b] == -HCT_INF ? 0.0f : m[b]) - ref) * HCT_LOG2E);
    m[b] = mr;
    s[b] = sj;
    q[b] = qj;
  }
#else
  (void)cx; (void)red; (void)m; (void)s; (void)q;
#pragma unroll
  for (int b = 0; b < HCT_B; ++b) f[b] = 1.0f;
#endif
}
// Arg-reduction over a row: on entry v / ix hold each thread's best value and its column (the first
// one among equals); on exit every thread holds the row's best value and the smallest column that has it.
template <bool IS_MAX>
__device__ __forceinline__ void hct_row_argreduce(float (&v)[HCT_B], int (&ix)[HCT_B], HctRowCtx& cx, float (*red)[2][HCT_B][3][32]) {
  auto fold = [](float& a, int& ia, float b, int ib) {
    const bool take = IS_MAX ? (b > a || (b == a && ib < ia)) : (b < a || (b == a && ib < ia));
    if (take) { a = b; ia = ib; }
  };
#pragma unroll
  for (int o = (HCT_T < 32 ? HCT_T : 32) / 2; o > 0; o >>= 1) {
#pragma unroll
    for (int b = 0; b < HCT_B; ++b) {
      const float u = __shfl_xor_sync(0xffffffffu, v[b], o);
      const int iu = __shfl_xor_sync(0xffffffffu, ix[b], o);
      fold(v[b], ix[b], u, iu);
    }
  }
#if HCT_T > 32
  float (*slot)[3][32] = red[cx.g][cx.par];
  cx.par ^= 1u;
  if ((cx.t & 31) == 0) {
#pragma unroll
    for (int b = 0; b < HCT_B; ++b) {
      slot[b][0][cx.t >> 5] = v[b];
      slot[b][1][cx.t >> 5] = __int_as_float(ix[b]);
    }
  }
  asm volatile("bar.sync %0, %1;" ::"r"(cx.g + 1), "n"(HCT_T) : "memory");
  const int j = cx.t & (HCT_T / 32 - 1);
#pragma unroll
  for (int b = 0; b < HCT_B; ++b) {
    v[b] = slot[b][0][j];
    ix[b] = __float_as_int(slot[b][1][j]);
#pragma unroll
    for (int o = HCT_T / 64; o > 0; o >>= 1) {
      const float u = __shfl_xor_sync(0xffffffffu, v[b], o);
      const int iu = __shfl_xor_sync(0xffffffffu, ix[b], o);
      fold(v[b], ix[b], u, iu);
    }
  }
#else
  (void)cx; (void)red;
#endif
}

#if HCT_T > 32
#define HCT_SM_SMEM hct_sm_smem
#else
#define HCT_SM_SMEM nullptr
#endif

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

// Store of a value that only fp32 tensor-core GEMMs read as their first operand: its TF32 head and tail.
__device__ __forceinline__ void hct_store_row_split(float* hi_base, float* lo_base, long long row, int hct_t, const float* v) {
  float* ph = hi_base + row * (long long)HCT_C;
  float* pl = lo_base + row * (long long)HCT_C;
#pragma unroll
  for (int k = 0; k < HCT_NV; ++k) {
    int col = (k * HCT_T + hct_t) * HCT_V;
    if (HCT_FULL_VECS || col < HCT_C) {
      float h[HCT_V], l[HCT_V];
#pragma unroll
      for (int i = 0; i < HCT_V; ++i) {
        h[i] = hct_to_tf32(v[k * HCT_V + i]);
        l[i] = hct_to_tf32(v[k * HCT_V + i] - h[i]);
      }
      hct_vecio<HCT_V>::st(ph + col, h);
      hct_vecio<HCT_V>::st(pl + col, l);
    }
  }
}

// ---- staged variant: full-width inputs are prefetched into a shared-memory ring by bulk
// asynchronous copies (one per row and input, completion counted on an mbarrier), HCT_NSTG rows
// ahead of the row being computed, so that loads stay in flight during the arithmetic and the
// reductions of earlier rows.  The generator defines HCT_STAGED, HCT_NSTG, HCT_STAGE_BYTES
// (bytes of all staged inputs of one row), HCT_RING_OFF (bytes of resident row vectors placed
// before the ring) and HCT_STATUS_SLOT.
#ifdef HCT_STAGED
__device__ __forceinline__ hct_u32 hct_smem_u32(const void* p) { return (hct_u32)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void hct_bulk_load(hct_u32 dst, const void* src, hct_u32 bytes, hct_u32 bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src), "r"(bytes),
               "r"(bar)
               : "memory");
}
__device__ __forceinline__ bool hct_row_mbar_try(hct_u32 bar, hct_u32 parity) {
  hct_u32 ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: on expiry the status word is set and a CTA-wide flag makes later waits return at once.
__device__ __forceinline__ void hct_row_mbar_wait(hct_u32 bar, hct_u32 parity, volatile int* failed, unsigned int* status) {
  if (hct_row_mbar_try(bar, parity)) return;
  for (unsigned it = 0; it < (1u << 24); ++it) {
    if (hct_row_mbar_try(bar, parity)) return;
    if (*failed) return;
    if (it > 64) __nanosleep(20);
  }
  *failed = 1;
  if (status) { atomicCAS(status, 0u, 1u); status[1] = 100u; }
}
// one thread's share of a staged row: the same vectors it would have loaded from global memory
template <typename T>
__device__ __forceinline__ void hct_read_staged(const unsigned char* slot, int hct_t, float* v);
template <>
__device__ __forceinline__ void hct_read_staged<float>(const unsigned char* slot, int hct_t, float* v) {
#pragma unroll
  for (int k = 0; k < HCT_NV; ++k) {
    const int col = (k * HCT_T + hct_t) * HCT_V;
    if (HCT_FULL_VECS || col < HCT_C) {
      const float4 t = *(const float4*)(slot + (size_t)col * 4);
      v[4 * k] = t.x; v[4 * k + 1] = t.y; v[4 * k + 2] = t.z; v[4 * k + 3] = t.w;
    } else {
      v[4 * k] = v[4 * k + 1] = v[4 * k + 2] = v[4 * k + 3] = 0.0f;
    }
  }
}
template <>
__device__ __forceinline__ void hct_read_staged<hct_bf16_t>(const unsigned char* slot, int hct_t, float* v) {
#pragma unroll
  for (int k = 0; k < HCT_NV; ++k) {
    const int col = (k * HCT_T + hct_t) * HCT_V;
    if (HCT_FULL_VECS || col < HCT_C) {
      const uint2 t = *(const uint2*)(slot + (size_t)col * 2);
      v[4 * k] = __uint_as_float(t.x << 16); v[4 * k + 1] = __uint_as_float(t.x & 0xffff0000u);
      v[4 * k + 2] = __uint_as_float(t.y << 16); v[4 * k + 3] = __uint_as_float(t.y & 0xffff0000u);
    } else {
      v[4 * k] = v[4 * k + 1] = v[4 * k + 2] = v[4 * k + 3] = 0.0f;
    }
  }
}

#define HCT_STAGED_KERNEL_BEGIN(name)                                                          \
  extern "C" __global__ void __launch_bounds__(HCT_T * HCT_G, HCT_MINB) name(const HctParams hct_p) {    \
    HCT_RED_DECL                                                                               \
    extern __shared__ __align__(128) unsigned char hct_ring[];                                 \
    __shared__ unsigned long long hct_full[HCT_G][HCT_NSTG];                                   \
    __shared__ int hct_failed;                                                                 \
    HctRowCtx hct_cx;                                                                          \
    hct_cx.t = threadIdx.x % HCT_T;                                                            \
    hct_cx.g = threadIdx.x / HCT_T;                                                            \
    hct_cx.par = 0;                                                                            \
    const int hct_t = hct_cx.t;                                                                \
    unsigned int* hct_status = (unsigned int*)hct_p.ptr[HCT_STATUS_SLOT];                      \
    unsigned char* hct_my_ring = hct_ring + HCT_RING_OFF + (size_t)hct_cx.g * HCT_NSTG * (HCT_STAGE_BYTES * HCT_B);      \
    hct_pdl_launch_dependents();                                                               \
    if (threadIdx.x == 0) hct_failed = 0;                                                      \
    if (hct_t == 0) {                                                                          \
      for (int s_ = 0; s_ < HCT_NSTG; ++s_) {                                                  \
        hct_u32 b_ = hct_smem_u32(&hct_full[hct_cx.g][s_]);                                    \
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(b_) : "memory");           \
      }                                                                                        \
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");                       \
    }                                                                                          \
    hct_pdl_wait();                                                                            \
    __syncthreads();

// issue the copies of the HCT_B rows starting at `r_` (those that exist) into ring slot `s_`;
// called by thread 0 of the row group.  Consecutive rows are contiguous in memory: one copy per input.
#define HCT_STAGED_ISSUE_BEGIN(r_, s_)                                                         \
  if ((r_) < HCT_R) {                                                                          \
    const long long hct_ir = (r_);                                                             \
    const hct_u32 hct_in = (hct_u32)(HCT_R - hct_ir < HCT_B ? HCT_R - hct_ir : HCT_B);          \
    const hct_u32 hct_ib = hct_smem_u32(&hct_full[hct_cx.g][(s_)]);                            \
    const hct_u32 hct_id = hct_smem_u32(hct_my_ring + (size_t)(s_) * (HCT_STAGE_BYTES * HCT_B)); \
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(hct_ib), "r"(hct_in * (hct_u32)HCT_STAGE_BYTES) : "memory");
#define HCT_STAGED_ISSUE_ONE(ptr, off, bytes_per_row) \
    hct_bulk_load(hct_id + (off) * HCT_B, (const unsigned char*)(ptr) + hct_ir * (long long)(bytes_per_row), hct_in * (hct_u32)(bytes_per_row), hct_ib);
#define HCT_STAGED_ISSUE_END }

#if HCT_T > 32
#define HCT_GROUP_SYNC asm volatile("bar.sync %0, %1;" ::"r"(hct_cx.g + 1), "n"(HCT_T) : "memory")
#else
#define HCT_GROUP_SYNC __syncwarp()
#endif
#endif  // HCT_STAGED

#define HCT_ROW_KERNEL_BEGIN(name)                                                            \
  extern "C" __global__ void __launch_bounds__(HCT_T * HCT_G) name(const HctParams hct_p) {   \
    HCT_RED_DECL                                                                              \
    HctRowCtx hct_cx;                                                                         \
    hct_cx.t = threadIdx.x % HCT_T;                                                           \
    hct_cx.g = threadIdx.x / HCT_T;                                                           \
    hct_cx.par = 0;                                                                           \
    const int hct_t = hct_cx.t;                                                               \
    hct_pdl_launch_dependents();                                                              \
    hct_pdl_wait();

#define HCT_ROW_LOOP_BEGIN                                                                    \
    for (long long hct_base = (long long)blockIdx.x * (HCT_G * HCT_B); hct_base < HCT_R;      \
         hct_base += (long long)gridDim.x * (HCT_G * HCT_B)) {                                \
      const long long hct_row0 = hct_base + (long long)hct_cx.g * HCT_B;                      \
      const bool hct_live = hct_row0 < HCT_R;

// row b of this group's batch: clamped for loads, exact for stores (guarded by HCT_LIVEB)
#define HCT_ROWB(b) (hct_row0 + (b) < HCT_R ? hct_row0 + (b) : HCT_R - 1)
#define HCT_LIVEB(b) (hct_row0 + (b) < HCT_R)

#define HCT_ROW_LOOP_END }
#define HCT_ROW_KERNEL_END }
