// Layout pre-pass for the tensor-core convolution: activations NCHW -> NHWC and weights
// KCRS -> RSKC (both bf16), so that channels, the contraction axis, are contiguous for TMA.
// With HCT_PREP_X = 0 only the weights are rearranged (the convolution then reads NCHW itself): that
// variant uses no shared memory and few CTAs, so that the convolution kernel, launched as a programmatic
// dependent and needing a whole SM's shared memory per CTA, becomes resident beside it at once and
// fills its pixel pipeline while the weights are being rearranged.
// Defined by the generator: HCT_NB_IMG, HCT_C, HCT_HW (H*W), HCT_KO, HCT_RS (R*S), HCT_PREP_X, HCT_GROUPS, HCT_CWP (grouped only),
// HctParams, HCT_KERNEL_NAME.
// Pointer slots: 0 = X (NCHW), 1 = Wt (KCRS), 2 = X as NHWC, 3 = Wt as RSKC, 4 = HCT_ZERO_WORDS 32-bit words
// to clear (the arrival counters of a convolution that splits the contraction of its last round; 0: none).
#ifndef HCT_ZERO_WORDS
#define HCT_ZERO_WORDS 0
#endif
#define HCT_XT_C ((HCT_C + 63) / 64)
#define HCT_XT_P ((HCT_HW + 63) / 64)
#define HCT_X_BLOCKS (HCT_PREP_X ? (long long)HCT_NB_IMG * HCT_XT_C * HCT_XT_P : 0LL)
// Grouped convolution (HCT_GROUPS > 1, filters [KO, C / groups, R, S]): per filter the copy holds HCT_CWP channels
// (a multiple of 64) starting at the first channel of the first group that the filter's block of 128 filters
// spans; channels of other groups (and past C) are written as zeros, so the convolution kernel contracts a dense
// window of input channels and the zeros cancel what does not belong to the filter's group.
#ifndef HCT_GROUPS
#define HCT_GROUPS 1
#endif
#if HCT_GROUPS > 1
#define HCT_WC HCT_CWP
#else
#define HCT_WC HCT_C
#endif
#define HCT_W_ELEMS ((long long)HCT_KO * HCT_WC * HCT_RS)
// element i of the copy, laid out [tap][filter][channel of the window]
__device__ __forceinline__ hct_bf16_t hct_w_elem(const hct_bf16_t* __restrict__ Wt, long long i) {
  const int j = (int)(i % HCT_WC);
  const int k = (int)((i / HCT_WC) % HCT_KO);
  const int rs = (int)(i / ((long long)HCT_WC * HCT_KO));
#if HCT_GROUPS > 1
  const int cpg = HCT_C / HCT_GROUPS, kpg = HCT_KO / HCT_GROUPS;
  const int c = ((k / 128) * 128 / kpg) * cpg + j, g = k / kpg;
  if (c >= HCT_C || c / cpg != g) return (hct_bf16_t)0;
  return Wt[((long long)k * cpg + (c - g * cpg)) * HCT_RS + rs];
#else
  return Wt[((long long)k * HCT_C + j) * HCT_RS + rs];
#endif
}
#if !HCT_PREP_X
// one thread per 16-byte piece of the RSKC copy: 8 consecutive channels of one (tap, filter)
extern "C" __global__ void __launch_bounds__(256) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  const hct_bf16_t* __restrict__ Wt = (const hct_bf16_t*)hct_p.ptr[1];
  hct_bf16_t* __restrict__ Wo = (hct_bf16_t*)hct_p.ptr[3];
  if (blockIdx.x == 0)
    for (int i = threadIdx.x; i < HCT_ZERO_WORDS; i += 256) ((unsigned*)hct_p.ptr[4])[i] = 0u;
#if HCT_GROUPS > 1
  for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < HCT_W_ELEMS; i += (long long)gridDim.x * 256) Wo[i] = hct_w_elem(Wt, i);
  return;
#endif
  for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < HCT_W_ELEMS / 8; i += (long long)gridDim.x * 256) {
    const int c = (int)(i % (HCT_C / 8)) * 8;
    const int k = (int)((i / (HCT_C / 8)) % HCT_KO);
    const int rs = (int)(i / ((long long)(HCT_C / 8) * HCT_KO));
    const hct_bf16_t* src = Wt + ((long long)k * HCT_C + c) * HCT_RS + rs;
    hct_u32 w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) w[j] = (hct_u32)__ldg(src + (2 * j) * HCT_RS) | ((hct_u32)__ldg(src + (2 * j + 1) * HCT_RS) << 16);
    *(uint4*)(Wo + i * 8) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}
#else
#define HCT_W_BLOCKS ((HCT_W_ELEMS + 255) / 256)
extern "C" __global__ void __launch_bounds__(256) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  __shared__ hct_bf16_t tile[64][66];
  const hct_bf16_t* __restrict__ X = (const hct_bf16_t*)hct_p.ptr[0];
  const hct_bf16_t* __restrict__ Wt = (const hct_bf16_t*)hct_p.ptr[1];
  hct_bf16_t* __restrict__ Xo = (hct_bf16_t*)hct_p.ptr[2];
  hct_bf16_t* __restrict__ Wo = (hct_bf16_t*)hct_p.ptr[3];
  for (long long blk = blockIdx.x; blk < HCT_X_BLOCKS + HCT_W_BLOCKS; blk += gridDim.x) {
    if (blk < HCT_X_BLOCKS) {
      // 64 channels x 64 pixels per tile: 16-byte reads along pixels, 16-byte writes along channels
      const long long n = blk / (HCT_XT_C * HCT_XT_P);
      const int rem = (int)(blk % (HCT_XT_C * HCT_XT_P));
      const int c0 = (rem / HCT_XT_P) * 64, p0 = (rem % HCT_XT_P) * 64;
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int id = threadIdx.x + 256 * u;       // 512 chunks of 8 pixels
        const int c = c0 + (id >> 3), p = p0 + (id & 7) * 8;
        __align__(16) hct_bf16_t v[8];
        if (c < HCT_C && p + 7 < HCT_HW && HCT_HW % 8 == 0) {
          *(uint4*)v = __ldg((const uint4*)(X + (n * HCT_C + c) * HCT_HW + p));
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j) v[j] = (c < HCT_C && p + j < HCT_HW) ? X[(n * HCT_C + c) * HCT_HW + p + j] : (hct_bf16_t)0;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) tile[id >> 3][(id & 7) * 8 + j] = v[j];
      }
      __syncthreads();
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int id = threadIdx.x + 256 * u;       // 512 chunks of 8 channels
        const int p = p0 + (id >> 3), cc = (id & 7) * 8;
        if (p < HCT_HW) {
          __align__(16) hct_bf16_t v[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) v[j] = tile[cc + j][id >> 3];
          hct_bf16_t* dst = Xo + (n * HCT_HW + p) * HCT_C + c0 + cc;
          if (c0 + cc + 7 < HCT_C) {
            *(uint4*)dst = *(const uint4*)v;       // HCT_C is a multiple of 8: 16-byte aligned
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (c0 + cc + j < HCT_C) dst[j] = v[j];
          }
        }
      }
      __syncthreads();
    } else {
      const long long i = (blk - HCT_X_BLOCKS) * 256 + threadIdx.x;   // index into RSKC
      if (i < HCT_W_ELEMS) Wo[i] = hct_w_elem(Wt, i);
    }
  }
}
#endif
