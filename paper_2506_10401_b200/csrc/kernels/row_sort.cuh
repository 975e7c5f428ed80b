// Row-wise sort (logic-intensive operator class): one CTA sorts one row of HCT_C values with a bitonic
// network in shared memory and stores the first HCT_KOUT of them (all of them for a sort, the k
// largest for a top-k), with the elementwise consumers of the result applied at the store.
// The row is padded to HCT_NP, a power of two, with values that sort to the end (+inf ascending,
// -inf descending).  Every compare-exchange step pairs element i with i ^ j and orders the pair
// ascending or descending by bit `k` of i; HCT_NP / 2 pairs per step are spread over the threads, with
// a block barrier between steps.  Values are only moved, never changed.
// Defined by the generator: HCT_R, HCT_C, HCT_NP, HCT_KOUT, HCT_DESC, HCT_T (threads), HCT_TA, HCT_PA,
// HctParams, hct_epilogue(), HCT_KERNEL_NAME.
extern "C" __global__ void __launch_bounds__(HCT_T) HCT_KERNEL_NAME(const HctParams hct_p) {
  hct_pdl_launch_dependents();
  hct_pdl_wait();
  __shared__ float key[HCT_NP];
  const HCT_TA* __restrict__ X = (const HCT_TA*)hct_p.ptr[HCT_PA];
  const int tid = threadIdx.x;
  const float pad = HCT_DESC ? -HCT_INF : HCT_INF;
  for (long long row = blockIdx.x; row < HCT_R; row += gridDim.x) {
    for (int i = tid; i < HCT_NP; i += HCT_T) key[i] = i < HCT_C ? hct_ld1(X + row * HCT_C + i) : pad;
    __syncthreads();
    for (int k = 2; k <= HCT_NP; k <<= 1) {
      for (int j = k >> 1; j > 0; j >>= 1) {
        for (int t = tid; t < HCT_NP / 2; t += HCT_T) {
          // the t-th pair of this step: insert a zero at bit position log2(j)
          const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
          const int l = i | j;
          const float a = key[i], b = key[l];
          const bool up = ((i & k) == 0) != (HCT_DESC != 0);   // ascending run (descending when the whole sort is)
          if ((a > b) == up) {
            key[i] = b;
            key[l] = a;
          }
        }
        __syncthreads();
      }
    }
    for (int i = tid; i < HCT_KOUT; i += HCT_T) hct_epilogue(hct_p, key[i], row * HCT_KOUT + i, row, i);
    __syncthreads();
  }
}
