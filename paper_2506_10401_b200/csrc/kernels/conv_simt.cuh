// Direct convolution, one thread per output element, for shapes the tensor-core kernel does not take.
// HCT_CI is the number of input channels one filter sums over (all of them divided by HCT_GROUPS).
// Defined by the generator: HCT_NB, HCT_CI, HCT_H, HCT_W, HCT_KO, HCT_FR, HCT_FS, HCT_STRIDE, HCT_PAD, HCT_DIL, HCT_GROUPS,
// HCT_HO, HCT_WO, HCT_TA, HCT_TB, HCT_PA, HCT_PB, HctParams, hct_epilogue(), HCT_KERNEL_NAME.
extern "C" __global__ void __launch_bounds__(256) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  const HCT_TA* __restrict__ X = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const HCT_TB* __restrict__ Wt = (const HCT_TB*)hct_p.ptr[HCT_PB];
  const long long total = (long long)HCT_NB * HCT_KO * HCT_HO * HCT_WO;
  for (long long idx = (long long)blockIdx.x * 256 + threadIdx.x; idx < total; idx += (long long)gridDim.x * 256) {
    int w = (int)(idx % HCT_WO);
    int h = (int)((idx / HCT_WO) % HCT_HO);
    int k = (int)((idx / ((long long)HCT_WO * HCT_HO)) % HCT_KO);
    long long n = idx / ((long long)HCT_WO * HCT_HO * HCT_KO);
    float acc = 0.0f;
    const int c0 = k / (HCT_KO / HCT_GROUPS) * HCT_CI;   // first input channel of this filter's group
    for (int c = 0; c < HCT_CI; ++c)
      for (int r = 0; r < HCT_FR; ++r) {
        int ih = h * HCT_STRIDE - HCT_PAD + r * HCT_DIL;
        if (ih < 0 || ih >= HCT_H) continue;
        for (int s = 0; s < HCT_FS; ++s) {
          int iw = w * HCT_STRIDE - HCT_PAD + s * HCT_DIL;
          if (iw < 0 || iw >= HCT_W) continue;
          acc = fmaf(hct_ld1(X + ((n * (HCT_CI * HCT_GROUPS) + c0 + c) * HCT_H + ih) * HCT_W + iw),
                     hct_ld1(Wt + (((long long)k * HCT_CI + c) * HCT_FR + r) * HCT_FS + s), acc);
        }
      }
    hct_epilogue(hct_p, acc, idx, n * HCT_KO + k, k);
  }
}
