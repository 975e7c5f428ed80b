// Reshape: the elements of a dense row-major tensor, in the same order, under the 2-D shape
// [HCT_ROWS, HCT_COLS]; a flat copy whose stores go through the generated epilogue, so the elementwise
// consumers of the reshaped value (which see the new rows and columns) cost no further pass.
// Defined by the generator: HCT_ROWS, HCT_COLS, HCT_TA (element type of the source), HCT_PA (its pointer
// slot), HctParams, hct_epilogue(), HCT_KERNEL_NAME.
extern "C" __global__ void __launch_bounds__(256) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  const HCT_TA* __restrict__ X = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const long long total = (long long)HCT_ROWS * HCT_COLS;
  for (long long off = (long long)blockIdx.x * 256 + threadIdx.x; off < total; off += (long long)gridDim.x * 256) {
    const long long r = off / HCT_COLS;
    hct_epilogue(hct_p, hct_ld1(X + off), off, r, (int)(off - r * HCT_COLS));
  }
}
