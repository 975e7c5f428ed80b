// Depthwise convolution (groups == input channels): filter k reads only input channel k / HCT_MULT, so
// the operator moves one plane in and HCT_MULT planes out per channel and is bound by memory traffic.
// One thread owns HCT_P vertically adjacent output pixels of one plane; consecutive threads own
// consecutive columns, so every load and store of a warp touches consecutive addresses.  The thread
// walks the input rows its outputs need once, top to bottom, and feeds each loaded pixel to every
// (output, filter row) pair that uses it; the pairing is resolved at compile time by full unrolling.
// Pixels outside the image contribute zero.  Accumulation is in fp32, taps in row-major order.
//
// Defined by the generator: HCT_NB, HCT_C, HCT_MULT, HCT_H, HCT_W, HCT_FR, HCT_FS, HCT_STRIDE, HCT_PAD, HCT_DIL,
// HCT_HO, HCT_WO, HCT_P, HCT_TA, HCT_TB, HCT_PA, HCT_PB, HctParams, hct_epilogue(), HCT_KERNEL_NAME.
#define HCT_KO (HCT_C * HCT_MULT)
#define HCT_HB ((HCT_HO + HCT_P - 1) / HCT_P)                                  // blocks of HCT_P output rows per plane
#define HCT_NROWS ((HCT_P - 1) * HCT_STRIDE + (HCT_FR - 1) * HCT_DIL + 1)      // input rows under one block

extern "C" __global__ void __launch_bounds__(256) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  const HCT_TA* __restrict__ X = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const HCT_TB* __restrict__ Wt = (const HCT_TB*)hct_p.ptr[HCT_PB];
  const long long units = (long long)HCT_NB * HCT_KO * HCT_HB * HCT_WO;
  for (long long u = (long long)blockIdx.x * 256 + threadIdx.x; u < units; u += (long long)gridDim.x * 256) {
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
