// Layout transform y = permute(x, axes) for tensors of up to four axes (leading axes of extent 1 are
// added below four): output axis d is input axis HCT_P<d>, so y[o0,o1,o2,o3] = x[i] with i[HCT_P<d>] = o<d>.
// The elementwise consumers of y are applied at the store.
// Two cases.  When the innermost axis stays innermost, rows of that axis are copied whole: consecutive
// threads take consecutive elements on both sides.  Otherwise the input's innermost axis I and the
// axis J that becomes the output's innermost one span a plane that is transposed through 64 x 64
// shared-memory tiles (reads run along I, writes along J, both coalesced; the tile has 65 columns so
// that the transposed reads miss each other's banks); the two remaining axes are a batch.
// Defined by the generator: HCT_S0..3 (input extents), HCT_P0..3 (the permutation), HCT_TA (input element
// type), HCT_PA (its pointer slot), HctParams, hct_epilogue(), HCT_KERNEL_NAME.
#define HCT_NEL ((long long)HCT_S0 * HCT_S1 * HCT_S2 * HCT_S3)
__device__ __forceinline__ long long hct_perm_in_stride(int axis) {
  return axis == 3 ? 1LL : axis == 2 ? (long long)HCT_S3 : axis == 1 ? (long long)HCT_S3 * HCT_S2 : (long long)HCT_S3 * HCT_S2 * HCT_S1;
}
__device__ __forceinline__ long long hct_perm_extent(int axis) {
  return axis == 3 ? HCT_S3 : axis == 2 ? HCT_S2 : axis == 1 ? HCT_S1 : HCT_S0;
}
// output extents and strides
#define HCT_O0 hct_perm_extent(HCT_P0)
#define HCT_O1 hct_perm_extent(HCT_P1)
#define HCT_O2 hct_perm_extent(HCT_P2)
#define HCT_O3 hct_perm_extent(HCT_P3)

extern "C" __global__ void __launch_bounds__(256) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  const HCT_TA* __restrict__ X = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const long long o3 = HCT_O3, o2 = HCT_O2, o1 = HCT_O1;
#if HCT_P3 == 3
  // innermost axis unchanged: element `off` of the output comes from the same position along axis 3
  for (long long off = (long long)blockIdx.x * 256 + threadIdx.x; off < HCT_NEL; off += (long long)gridDim.x * 256) {
    const long long c3 = off % o3, r3 = off / o3;
    const long long c2 = r3 % o2, r2 = r3 / o2;
    const long long c1 = r2 % o1, c0 = r2 / o1;
    const long long src = c0 * hct_perm_in_stride(HCT_P0) + c1 * hct_perm_in_stride(HCT_P1) + c2 * hct_perm_in_stride(HCT_P2) + c3;
    hct_epilogue(hct_p, hct_ld1(X + src), off, r3, (int)c3);
  }
#else
  // plane (I = input axis 3, J = input axis HCT_P3); the output position of axis 3 is HCT_Q3
  __shared__ float tile[64][65];
  constexpr int Q3 = HCT_P0 == 3 ? 0 : HCT_P1 == 3 ? 1 : 2;          // output axis that holds input axis 3
  // the two output axes other than Q3 and 3 form the batch
  constexpr int B0 = Q3 == 0 ? 1 : 0, B1 = Q3 == 2 ? 1 : 2;
  const long long ext_o[4] = {HCT_O0, o1, o2, o3};
  const long long str_o[4] = {o1 * o2 * o3, o2 * o3, o3, 1};
  const int perm[4] = {HCT_P0, HCT_P1, HCT_P2, HCT_P3};
  const long long EI = HCT_S3, EJ = o3;                                 // extents of the plane's two axes
  const long long TI = (EI + 63) / 64, TJ = (EJ + 63) / 64, NB = ext_o[B0] * ext_o[B1];
  const long long sJ_in = hct_perm_in_stride(HCT_P3), sI_out = str_o[Q3];
  const int tid = threadIdx.x;
  for (long long t = blockIdx.x; t < NB * TI * TJ; t += gridDim.x) {
    const long long b = t / (TI * TJ), tt = t % (TI * TJ);
    const long long i0 = (tt % TI) * 64, j0 = (tt / TI) * 64;
    const long long b0 = b / ext_o[B1], b1 = b % ext_o[B1];
    const long long in_base = b0 * hct_perm_in_stride(perm[B0]) + b1 * hct_perm_in_stride(perm[B1]);
    const long long out_base = b0 * str_o[B0] + b1 * str_o[B1];
    {
      const int ii = tid & 63, jq = tid >> 6;     // 64 consecutive input elements along I, 4 values of J per pass
#pragma unroll
      for (int p = 0; p < 16; ++p) {
        const int jj = jq + 4 * p;
        float v = 0.0f;
        if (i0 + ii < EI && j0 + jj < EJ) v = hct_ld1(X + in_base + (j0 + jj) * sJ_in + (i0 + ii));
        tile[jj][ii] = v;
      }
    }
    __syncthreads();
    {
      const int jj = tid & 63, iq = tid >> 6;     // 64 consecutive output elements along J, 4 values of I per pass
#pragma unroll
      for (int p = 0; p < 16; ++p) {
        const int ii = iq + 4 * p;
        if (i0 + ii < EI && j0 + jj < EJ) {
          const long long off = out_base + (i0 + ii) * sI_out + (j0 + jj);
          hct_epilogue(hct_p, tile[jj][ii], off, off / o3, (int)(j0 + jj));
        }
      }
    }
    __syncthreads();
  }
#endif
}
