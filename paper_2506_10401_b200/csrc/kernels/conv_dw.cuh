// Depthwise convolution (groups == input channels): filter k reads only input channel k / HCT_MULT, so
// the operator moves one plane in and HCT_MULT planes out per channel and is bound by memory traffic.
// One thread owns HCT_P vertically adjacent output pixels of one plane; consecutive threads own
// consecutive columns, so every load and store of a warp touches consecutive addresses.  The thread
// walks the input rows its outputs need once, top to bottom, and feeds each loaded pixel to every
// (output, filter row) pair that uses it; the pairing is resolved at compile time by full unrolling.
// Pixels outside the image contribute zero.  Accumulation is in fp32, taps in row-major order.
//
// With stride 1, no dilation and rows that are whole 16-byte vectors (HCT_VEC) a thread owns a block of
// 8 columns x HCT_P rows instead: per input row one 16-byte (bf16) load plus the few halo columns, per
// output row one vector store through the generated run epilogue, so that about nine of every
// thirteen instructions are the multiply-adds themselves.
//
// Defined by the generator: HCT_VEC, HCT_PAIR, HCT_CTA (threads per block), HCT_NB, HCT_C, HCT_MULT, HCT_H, HCT_W, HCT_FR, HCT_FS, HCT_STRIDE, HCT_PAD, HCT_DIL,
// HCT_HO, HCT_WO, HCT_P, HCT_TA, HCT_TB, HCT_PA, HCT_PB, HctParams, hct_epilogue(), HCT_KERNEL_NAME.
#define HCT_KO (HCT_C * HCT_MULT)
#define HCT_HB ((HCT_HO + HCT_P - 1) / HCT_P)                                  // blocks of HCT_P output rows per plane
#define HCT_NROWS ((HCT_P - 1) * HCT_STRIDE + (HCT_FR - 1) * HCT_DIL + 1)      // input rows under one block

#if HCT_VEC
#define HCT_WB (HCT_WO / 8)                 // 8-column blocks per output row
#define HCT_XW (8 + HCT_FS - 1)             // input columns under one block
#endif

#if HCT_VEC && HCT_PAIR
// Two planes per thread (filters k and k + 1 at the same block of pixels): every multiply-add is one packed
// fma.rn.f32x2 whose low half belongs to filter k and whose high half to filter k + 1, so pixel, weight and
// accumulator pairs are formed where the values are produced and nothing has to be shuffled between halves.
// Each half is an ordinary round-to-nearest fused multiply-add: results equal those of the one-plane form.
// (pair helpers hct_pk, hct_upk, hct_fma2: common.cuh)
extern "C" __global__ void __launch_bounds__(HCT_CTA) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  const HCT_TA* __restrict__ X = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const HCT_TB* __restrict__ Wt = (const HCT_TB*)hct_p.ptr[HCT_PB];
  const unsigned units = (unsigned)HCT_NB * (HCT_KO / 2) * HCT_HB * HCT_WB;   // below 2^31 (checked by the generator)
  for (unsigned u = blockIdx.x * (unsigned)HCT_CTA + threadIdx.x; u < units; u += gridDim.x * (unsigned)HCT_CTA) {
    const int w0 = (int)(u % HCT_WB) * 8;
    unsigned t = u / HCT_WB;
    const int h0 = (int)(t % HCT_HB) * HCT_P;
    const unsigned pp = t / HCT_HB;                      // n * (HCT_KO / 2) + k / 2
    const unsigned k = (pp % (HCT_KO / 2)) * 2, n = pp / (HCT_KO / 2);
    const unsigned plane = n * HCT_KO + k;
    const HCT_TA* __restrict__ xp0 = X + ((long long)n * HCT_C + k / HCT_MULT) * ((long long)HCT_H * HCT_W);
    const HCT_TA* __restrict__ xp1 = X + ((long long)n * HCT_C + (k + 1) / HCT_MULT) * ((long long)HCT_H * HCT_W);
    unsigned long long wt[HCT_FR * HCT_FS];
#pragma unroll
    for (int i = 0; i < HCT_FR * HCT_FS; ++i)
      wt[i] = hct_pk(hct_ld1(Wt + (long long)k * (HCT_FR * HCT_FS) + i), hct_ld1(Wt + (long long)(k + 1) * (HCT_FR * HCT_FS) + i));
    unsigned long long acc[HCT_P][8];
#pragma unroll
    for (int p = 0; p < HCT_P; ++p)
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[p][c] = 0ull;
#pragma unroll
    for (int j = 0; j < HCT_NROWS; ++j) {
      const int ih = h0 - HCT_PAD + j;
      const bool row_ok = ih >= 0 && ih < HCT_H;
      const HCT_TA* __restrict__ xr0 = xp0 + (long long)ih * HCT_W;    // dereferenced only where row_ok
      const HCT_TA* __restrict__ xr1 = xp1 + (long long)ih * HCT_W;
      unsigned long long xw[HCT_XW];                                   // xw[i] = x[ih][w0 - HCT_PAD + i] of both planes
      {
        float v0[32], v1[32];
        hct_ld_run32<HCT_TA>(xr0 + w0, v0, row_ok ? 8 : 0, true);
        hct_ld_run32<HCT_TA>(xr1 + w0, v1, row_ok ? 8 : 0, true);
#pragma unroll
        for (int c = 0; c < 8; ++c) xw[HCT_PAD + c] = hct_pk(v0[c], v1[c]);
      }
#pragma unroll
      for (int i = 0; i < HCT_PAD; ++i) {
        const bool ok = row_ok && w0 - HCT_PAD + i >= 0;
        xw[i] = hct_pk(ok ? hct_ld1(xr0 + w0 - HCT_PAD + i) : 0.0f, ok ? hct_ld1(xr1 + w0 - HCT_PAD + i) : 0.0f);
      }
#pragma unroll
      for (int i = HCT_PAD + 8; i < HCT_XW; ++i) {
        const bool ok = row_ok && w0 - HCT_PAD + i < HCT_W;
        xw[i] = hct_pk(ok ? hct_ld1(xr0 + w0 - HCT_PAD + i) : 0.0f, ok ? hct_ld1(xr1 + w0 - HCT_PAD + i) : 0.0f);
      }
#pragma unroll
      for (int p = 0; p < HCT_P; ++p)
#pragma unroll
        for (int r = 0; r < HCT_FR; ++r)
          if (p + r == j) {
#pragma unroll
            for (int s = 0; s < HCT_FS; ++s)
#pragma unroll
              for (int c = 0; c < 8; ++c) acc[p][c] = hct_fma2(xw[c + s], wt[r * HCT_FS + s], acc[p][c]);
          }
    }
#pragma unroll
    for (int p = 0; p < HCT_P; ++p) {
      if (h0 + p < HCT_HO) {
        float a0[32], a1[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) a0[c] = a1[c] = 0.0f;
#pragma unroll
        for (int c = 0; c < 8; ++c) hct_upk(acc[p][c], a0[c], a1[c]);
        hct_epilogue_run(hct_p, a0, (long long)plane, (h0 + p) * HCT_WO + w0, 8);
        hct_epilogue_run(hct_p, a1, (long long)plane + 1, (h0 + p) * HCT_WO + w0, 8);
      }
    }
  }
}
#elif HCT_VEC
extern "C" __global__ void __launch_bounds__(HCT_CTA) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  const HCT_TA* __restrict__ X = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const HCT_TB* __restrict__ Wt = (const HCT_TB*)hct_p.ptr[HCT_PB];
  const unsigned units = (unsigned)HCT_NB * HCT_KO * HCT_HB * HCT_WB;   // below 2^31 (checked by the generator)
  for (unsigned u = blockIdx.x * (unsigned)HCT_CTA + threadIdx.x; u < units; u += gridDim.x * (unsigned)HCT_CTA) {
    const int w0 = (int)(u % HCT_WB) * 8;
    unsigned t = u / HCT_WB;
    const int h0 = (int)(t % HCT_HB) * HCT_P;
    const unsigned plane = t / HCT_HB;                   // n * HCT_KO + k
    const unsigned k = plane % HCT_KO, n = plane / HCT_KO;
    const HCT_TA* __restrict__ xp = X + ((long long)n * HCT_C + k / HCT_MULT) * ((long long)HCT_H * HCT_W);
    float wt[HCT_FR * HCT_FS];
#pragma unroll
    for (int i = 0; i < HCT_FR * HCT_FS; ++i) wt[i] = hct_ld1(Wt + (long long)k * (HCT_FR * HCT_FS) + i);
    float acc[HCT_P][8];
#pragma unroll
    for (int p = 0; p < HCT_P; ++p)
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[p][c] = 0.0f;
#pragma unroll
    for (int j = 0; j < HCT_NROWS; ++j) {
      const int ih = h0 - HCT_PAD + j;
      const bool row_ok = ih >= 0 && ih < HCT_H;
      const HCT_TA* __restrict__ xr = xp + (long long)ih * HCT_W;     // dereferenced only where row_ok
      float xw[HCT_XW];                                               // xw[i] = x[ih][w0 - HCT_PAD + i]
      {
        float v[32];
        // columns w0 .. w0+7 lie inside the image (HCT_WO <= HCT_W) and start a 16-byte vector
        hct_ld_run32<HCT_TA>(xr + w0, v, row_ok ? 8 : 0, true);
#pragma unroll
        for (int c = 0; c < 8; ++c) xw[HCT_PAD + c] = v[c];
      }
#pragma unroll
      for (int i = 0; i < HCT_PAD; ++i) xw[i] = (row_ok && w0 - HCT_PAD + i >= 0) ? hct_ld1(xr + w0 - HCT_PAD + i) : 0.0f;
#pragma unroll
      for (int i = HCT_PAD + 8; i < HCT_XW; ++i) xw[i] = (row_ok && w0 - HCT_PAD + i < HCT_W) ? hct_ld1(xr + w0 - HCT_PAD + i) : 0.0f;
#pragma unroll
      for (int p = 0; p < HCT_P; ++p)
#pragma unroll
        for (int r = 0; r < HCT_FR; ++r)
          if (p + r == j) {
#pragma unroll
            for (int s = 0; s < HCT_FS; ++s)
#pragma unroll
              for (int c = 0; c < 8; ++c) acc[p][c] = fmaf(xw[c + s], wt[r * HCT_FS + s], acc[p][c]);
          }
    }
#pragma unroll
    for (int p = 0; p < HCT_P; ++p) {
      if (h0 + p < HCT_HO) {
        float a[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) a[c] = c < 8 ? acc[p][c] : 0.0f;
        hct_epilogue_run(hct_p, a, (long long)plane, (h0 + p) * HCT_WO + w0, 8);
      }
    }
  }
}
#else
extern "C" __global__ void __launch_bounds__(HCT_CTA) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  const HCT_TA* __restrict__ X = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const HCT_TB* __restrict__ Wt = (const HCT_TB*)hct_p.ptr[HCT_PB];
  const long long units = (long long)HCT_NB * HCT_KO * HCT_HB * HCT_WO;
  for (long long u = (long long)blockIdx.x * HCT_CTA + threadIdx.x; u < units; u += (long long)gridDim.x * HCT_CTA) {
    const int w = (int)(u % HCT_WO);
    long long t = u / HCT_WO;
    const int hb = (int)(t % HCT_HB);
    t /= HCT_HB;
    const int k = (int)(t % HCT_KO);
    const long long n = t / HCT_KO;
    const HCT_TA* __restrict__ xp = X + (n * HCT_C + k / HCT_MULT) * ((long long)HCT_H * HCT_W);
    float wt[HCT_FR * HCT_FS];
#pragma unroll
    for (int i = 0; i < HCT_FR * HCT_FS; ++i) wt[i] = hct_ld1(Wt + (long long)k * (HCT_FR * HCT_FS) + i);
    float acc[HCT_P];
#pragma unroll
    for (int p = 0; p < HCT_P; ++p) acc[p] = 0.0f;
    const int ih0 = hb * HCT_P * HCT_STRIDE - HCT_PAD, iw0 = w * HCT_STRIDE - HCT_PAD;
#pragma unroll
    for (int j = 0; j < HCT_NROWS; ++j) {
      const int ih = ih0 + j;
      const bool row_ok = ih >= 0 && ih < HCT_H;
      float xv[HCT_FS];
#pragma unroll
      for (int s = 0; s < HCT_FS; ++s) {
        const int iw = iw0 + s * HCT_DIL;
        xv[s] = (row_ok && iw >= 0 && iw < HCT_W) ? hct_ld1(xp + (long long)ih * HCT_W + iw) : 0.0f;
      }
#pragma unroll
      for (int p = 0; p < HCT_P; ++p)
#pragma unroll
        for (int r = 0; r < HCT_FR; ++r)
          if (p * HCT_STRIDE + r * HCT_DIL == j) {
#pragma unroll
            for (int s = 0; s < HCT_FS; ++s) acc[p] = fmaf(xv[s], wt[r * HCT_FS + s], acc[p]);
          }
    }
#pragma unroll
    for (int p = 0; p < HCT_P; ++p) {
      const int h = hb * HCT_P + p;
      if (h < HCT_HO) hct_epilogue(hct_p, acc[p], ((n * HCT_KO + k) * HCT_HO + h) * HCT_WO + w, n * HCT_KO + k, k);
    }
  }
}
#endif
