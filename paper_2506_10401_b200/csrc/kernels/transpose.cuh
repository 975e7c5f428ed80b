// Layout transform y[j,i] = x[i,j] of a row-major [HCT_R, HCT_C] tensor, with the elementwise
// consumers of y applied at the store.  A CTA moves 64 x 64 tiles through shared memory: reads run
// along the input's rows (16-byte loads when the rows allow it), writes along the output's rows, both
// coalesced; the tile is padded to 65 columns so that the transposed reads miss each other's banks.
// Defined by the generator: HCT_R, HCT_C, HCT_TA (input element type), HCT_PA (its pointer slot),
// HctParams, hct_epilogue(), HCT_KERNEL_NAME.
#define HCT_TR ((HCT_R + 63) / 64)
#define HCT_TC ((HCT_C + 63) / 64)
template <typename T> struct hct_is_f32 { static const bool value = false; };
template <> struct hct_is_f32<float> { static const bool value = true; };
extern "C" __global__ void __launch_bounds__(256) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  __shared__ float tile[64][65];
  const HCT_TA* __restrict__ X = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const int tid = threadIdx.x;
  for (long long t = blockIdx.x; t < HCT_TR * HCT_TC; t += gridDim.x) {
    const long long r0 = (t / HCT_TC) * 64, c0 = (t % HCT_TC) * 64;
    {
      const int tx = tid & 15, ty = tid >> 4;   // 16 groups of 4 columns, 16 rows per pass
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const long long r = r0 + ty + 16 * i, c = c0 + tx * 4;
        float v[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        if (r < HCT_R) {
          if (hct_is_f32<HCT_TA>::value && HCT_C % 4 == 0 && c + 3 < HCT_C) {
            const float4 q = __ldg((const float4*)((const float*)X + r * HCT_C + c));
            v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
          } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (c + j < HCT_C) v[j] = hct_ld1(X + r * HCT_C + c + j);
          }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) tile[ty + 16 * i][tx * 4 + j] = v[j];
      }
    }
    __syncthreads();
    {
      const int rr = tid & 63, cq = tid >> 6;   // 64 consecutive output columns, 4 output rows per pass
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int cc = cq + 4 * i;
        const long long orow = c0 + cc, ocol = r0 + rr;   // output is [HCT_C, HCT_R]
        if (orow < HCT_C && ocol < HCT_R) hct_epilogue(hct_p, tile[rr][cc], orow * HCT_R + ocol, orow, (int)ocol);
      }
    }
    __syncthreads();
  }
}
