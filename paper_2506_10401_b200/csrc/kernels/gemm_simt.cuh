// fp32 FMA GEMM for shapes the tensor-core kernels do not take (tiny or unaligned extents).
// Defined by the generator: HCT_M, HCT_N, HCT_K, HCT_TA, HCT_TB (operand element types),
// HCT_PA, HCT_PB (pointer slots), HctParams, hct_epilogue(), HCT_KERNEL_NAME.
extern "C" __global__ void __launch_bounds__(256) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  __shared__ float As[16][64 + 4];
  __shared__ float Bs[16][64 + 4];
  const HCT_TA* __restrict__ A = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const HCT_TB* __restrict__ B = (const HCT_TB*)hct_p.ptr[HCT_PB];
  const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
  const long long m0 = (long long)blockIdx.y * 64, n0 = (long long)blockIdx.x * 64;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
  for (long long k0 = 0; k0 < HCT_K; k0 += 16) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int idx = tid + i * 256;
      int r = idx / 16, kk = idx % 16;
      long long m = m0 + r, k = k0 + kk;
      As[kk][r] = (m < HCT_M && k < HCT_K) ? hct_ld1(A + m * HCT_K + k) : 0.0f;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int idx = tid + i * 256;
      int kk = idx / 64, c = idx % 64;
      long long k = k0 + kk, n = n0 + c;
      Bs[kk][c] = (k < HCT_K && n < HCT_N) ? hct_ld1(B + k * HCT_N + n) : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      long long m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
      if (m < HCT_M && n < HCT_N) hct_epilogue(hct_p, acc[i][j], m * HCT_N + n, m, (int)n);
    }
}
