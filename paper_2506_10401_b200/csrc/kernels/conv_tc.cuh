// Persistent tensor-core conv2d (zero padding, any stride and dilation the tensor map can traverse)
// as an implicit GEMM with fused epilogue.
//
// GEMM view: rows (M = 128) = output channels, columns (N <= 256) = the pixels of HCT_TH full output
// rows of one image, contraction over (filter tap, input channel).  For every tap (r,s) and block
// of 64 input channels the producer warp loads the tap's [128 x 64] weight slice (A operand) and,
// with one 4-D TMA box from the NHWC copy of the input, the pixels shifted by the tap (B operand;
// coordinates outside the image read zeros, which is the padding; the channel coordinate is the
// innermost one and a multiple of 64, so every copy starts 16-byte aligned; with a stride the box
// is traversed in steps of HCT_STRIDE pixels and rows, so it still delivers HCT_WO pixels per row).  The MMA warp
// accumulates into one of two tensor-memory accumulators; four epilogue warps (one output channel
// per thread, 32 consecutive pixels per step, contiguous in NCHW) apply the generated epilogue.
//
// Work is split into tiles of HCT_TH output rows; when the last round over the SMs would be
// nearly empty, its tiles are cut into HCT_TH2-row pieces so that all SMs finish together.
//
// Defined by the generator: HCT_NB_IMG, HCT_C, HCT_H, HCT_W, HCT_KO, HCT_FR, HCT_FS, HCT_PAD, HCT_STRIDE, HCT_DIL, HCT_PHASED, HCT_HO, HCT_WO,
// HCT_TH, HCT_TH2, HCT_SPLIT (pieces per cut tile, HCT_TH2 * HCT_SPLIT >= HCT_TH), HCT_STAGES,
// HCT_STATUS_SLOT, HCT_KERNEL_NAME, HctParams, hct_epilogue_run().
//
// HCT_PHASED (stride > 1 dividing the image's height and width; used where a row times the stride
// exceeds the 256 elements a box may span): the NHWC copy is viewed as
// [n][h / stride][w / stride][w mod stride][c] through one tensor map per row phase h mod stride, so the
// pixels a tap needs are a dense box of that view (coordinate = tap offset divided by the stride,
// phase = its remainder).  Both forms deliver the same pixels at the same measured speed.
// Maps: [0] weights, [1 + phase] whole tiles, [1 + stride + phase] one-row pieces.
#define HCT_BM 128
#define HCT_A_BYTES (HCT_BM * 128)                       // weights: 128 channels x 64 inputs, bf16
#define HCT_B_BYTES 32768                                // pixels: up to 256 x 64 inputs
#define HCT_STAGE_BYTES (HCT_A_BYTES + HCT_B_BYTES)
// Grouped convolution (HCT_GROUPS > 1): a block of 128 filters reads only the input channels of the groups it
// spans.  The weight copy holds, per filter, HCT_CBW blocks of 64 channels starting at the first channel of the
// block's first group (HCT_C_LO), zero wherever a channel is not of the filter's own group.
#if HCT_GROUPS > 1
#define HCT_CB HCT_CBW
#define HCT_C_LO(mbk) ((((mbk) * HCT_BM) / (HCT_KO / HCT_GROUPS)) * (HCT_C / HCT_GROUPS))
#else
#define HCT_CB ((HCT_C + 63) / 64)
#define HCT_C_LO(mbk) 0
#endif
#define HCT_KB (HCT_FR * HCT_FS * HCT_CB)
#define HCT_HT ((HCT_HO + HCT_TH - 1) / HCT_TH)
#define HCT_MBK ((HCT_KO + HCT_BM - 1) / HCT_BM)
#define HCT_FULL_TILES ((long long)HCT_NB_IMG * HCT_HT * HCT_MBK)

#if HCT_PHASED
__device__ __forceinline__ void hct_tma_load_5d(hct_u32 dst, const HctTensorMap* map, int c0, int c1, int c2, int c3, int c4, hct_u32 bar) {
  asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];" ::"r"(dst),
               "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar)
               : "memory");
}
// floor(a / HCT_STRIDE) and the non-negative remainder, for offsets that may be negative (padding)
__device__ __forceinline__ int hct_floordiv(int a) { return (a >= 0 ? a : a - (HCT_STRIDE - 1)) / HCT_STRIDE; }
#endif

struct HctConvTile { int n, h0, th, mbk; bool cut; };

// Tile t of the schedule.  Tiles below `t1` are whole; the rest are pieces of the remaining whole tiles.
__device__ __forceinline__ HctConvTile hct_conv_tile(long long t, long long t1) {
  HctConvTile r;
  long long whole = t;
  int sub = 0;
  r.cut = t >= t1;
  if (r.cut) {
    whole = t1 + (t - t1) / HCT_SPLIT;
    sub = (int)((t - t1) % HCT_SPLIT);
  }
  r.mbk = (int)(whole % HCT_MBK); whole /= HCT_MBK;
  r.h0 = (int)(whole % HCT_HT) * HCT_TH + sub * HCT_TH2;
  r.n = (int)(whole / HCT_HT);
  int th = r.cut ? HCT_TH2 : HCT_TH;
  if (r.cut && sub * HCT_TH2 + th > HCT_TH) th = HCT_TH - sub * HCT_TH2;
  if (r.h0 + th > HCT_HO) th = HCT_HO - r.h0;
  r.th = th > 0 ? th : 0;   // 0: nothing to do (identically for every warp role)
  return r;
}

extern "C" __global__ void __launch_bounds__(192, 1) HCT_KERNEL_NAME(const __grid_constant__ HctParams hct_p) {
  extern __shared__ unsigned char hct_smem_raw[];
  __shared__ unsigned long long bars[2 * HCT_STAGES + 4];
  __shared__ hct_u32 tmem_holder;
  __shared__ int failed;
  const hct_u32 smem_base = (hct_smem_addr(hct_smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned int* status = (unsigned int*)hct_p.ptr[HCT_STATUS_SLOT];
  const hct_u32 full0 = hct_smem_addr(&bars[0]), empty0 = hct_smem_addr(&bars[HCT_STAGES]);
  const hct_u32 tfull0 = hct_smem_addr(&bars[2 * HCT_STAGES]), tempty0 = hct_smem_addr(&bars[2 * HCT_STAGES + 2]);

  // schedule: whole tiles for as many full rounds over the grid as there are, the rest cut in pieces
  long long t1 = HCT_FULL_TILES, n_tiles = HCT_FULL_TILES;
  {
    const long long rest = HCT_FULL_TILES % gridDim.x;
    if (HCT_SPLIT > 1 && rest > 0 && rest * HCT_SPLIT <= (long long)gridDim.x) {
      t1 = HCT_FULL_TILES - rest;
      n_tiles = t1 + rest * HCT_SPLIT;
    }
  }

  hct_pdl_launch_dependents();
  if (threadIdx.x == 0) {
    failed = 0;
    for (int s = 0; s < HCT_STAGES; ++s) {
      hct_mbar_init(full0 + 8 * s, 1);
      hct_mbar_init(empty0 + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      hct_mbar_init(tfull0 + 8 * a, 1);
      hct_mbar_init(tempty0 + 8 * a, 128);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    hct_prefetch_tmap(&hct_p.tmap[0]);
#if HCT_PHASED
    for (int i = 1; i < 1 + 2 * HCT_STRIDE; ++i) hct_prefetch_tmap(&hct_p.tmap[i]);
#else
    hct_prefetch_tmap(&hct_p.tmap[1]);
    hct_prefetch_tmap(&hct_p.tmap[2]);
#endif
  }
  if (warp == 1) hct_tmem_alloc(hct_smem_addr(&tmem_holder), 512);
  hct_tc_fence_before();
  __syncthreads();
  hct_tc_fence_after();
  const hct_u32 tmem_base = *(volatile hct_u32*)&tmem_holder;
  hct_pdl_wait();   // barriers, tensor memory and descriptors are ready; now the predecessor's data may be read

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      hct_u32 phase = 0;
      for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const HctConvTile t = hct_conv_tile(tile, t1);
        if (t.th == 0) continue;
        // whole tiles use the HCT_TH-row box, pieces the HCT_TH2-row box
#if !HCT_PHASED
        const HctTensorMap* xmap = t.cut ? &hct_p.tmap[2] : &hct_p.tmap[1];
#endif
        const hct_u32 bytes = HCT_A_BYTES + (hct_u32)(t.cut ? HCT_TH2 : HCT_TH) * HCT_WO * 128u;
        for (int kb = 0; kb < HCT_KB; ++kb) {
          const int tap = kb / HCT_CB, cb = kb % HCT_CB;
          const int r = tap / HCT_FS, s = tap % HCT_FS;
          hct_mbar_wait(empty0 + 8 * stage, phase ^ 1u, &failed, status, 1);
          const hct_u32 full = full0 + 8 * stage;
          hct_mbar_expect_tx(full, bytes);
          const hct_u32 dst = smem_base + stage * HCT_STAGE_BYTES;
          hct_tma_load_2d(dst, &hct_p.tmap[0], cb * 64, tap * HCT_KO + t.mbk * HCT_BM, full);
#if HCT_PHASED
          {
            const int a = s * HCT_DIL - HCT_PAD, b = r * HCT_DIL - HCT_PAD;
            const int wq = hct_floordiv(a), hq = hct_floordiv(b);
            const int pw = a - wq * HCT_STRIDE, ph = b - hq * HCT_STRIDE;
            hct_tma_load_5d(dst + HCT_A_BYTES, &hct_p.tmap[1 + (t.cut ? HCT_STRIDE : 0) + ph], HCT_C_LO(t.mbk) + cb * 64, pw, wq, t.h0 + hq, t.n, full);
          }
#else
          hct_tma_load_4d(dst + HCT_A_BYTES, xmap, HCT_C_LO(t.mbk) + cb * 64, s * HCT_DIL - HCT_PAD, t.h0 * HCT_STRIDE + r * HCT_DIL - HCT_PAD, t.n, full);
#endif
          if (++stage == HCT_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int stage = 0, acc = 0;
      hct_u32 phase = 0, acc_phase = 0;
      for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const HctConvTile t = hct_conv_tile(tile, t1);
        if (t.th == 0) continue;
        // bf16 x bf16 -> fp32, both operands K-major, M = 128, N = pixels of this tile rounded up to 16
        const hct_u32 n_mma = (hct_u32)((t.th * HCT_WO + 15) & ~15);
        const hct_u32 idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((n_mma >> 3) << 17) | ((hct_u32)(HCT_BM >> 4) << 24);
        hct_mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, &failed, status, 2);
        hct_tc_fence_after();
        const hct_u32 d_tmem = tmem_base + acc * 256;
        for (int kb = 0; kb < HCT_KB; ++kb) {
          hct_mbar_wait(full0 + 8 * stage, phase, &failed, status, 3);
          hct_tc_fence_after();
          const hct_u32 a_addr = smem_base + stage * HCT_STAGE_BYTES, b_addr = a_addr + HCT_A_BYTES;
          const hct_u64 a_desc0 = hct_smem_desc(a_addr, 16, 1024), b_desc0 = hct_smem_desc(b_addr, 16, 1024);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) hct_mma_f16(d_tmem, a_desc0 + kk * 2, b_desc0 + kk * 2, idesc, (kb | kk) != 0);
          hct_mma_commit(empty0 + 8 * stage);
          if (++stage == HCT_STAGES) { stage = 0; phase ^= 1u; }
        }
        hct_mma_commit(tfull0 + 8 * acc);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    const int q = warp & 3;
    int acc = 0;
    hct_u32 acc_phase = 0;
    for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
      const HctConvTile t = hct_conv_tile(tile, t1);
      if (t.th == 0) continue;
      hct_mbar_wait(tfull0 + 8 * acc, acc_phase, &failed, status, 4);
      hct_tc_fence_after();
      const int k = t.mbk * HCT_BM + q * 32 + lane;      // output channel of this thread's TMEM lane
      const int npix = t.th * HCT_WO;                    // contiguous in the (n,k) plane from h0*WO on
      const int chunks = (npix + 31) / 32;
#pragma unroll 1
      for (int c = 0; c < chunks; ++c) {
        float v[32];
        hct_tmem_ld32(tmem_base + ((hct_u32)(q * 32) << 16) + acc * 256 + c * 32, v);
        const int ncols = npix - c * 32 < 32 ? npix - c * 32 : 32;
        if (k < HCT_KO) hct_epilogue_run(hct_p, v, (long long)t.n * HCT_KO + k, t.h0 * HCT_WO + c * 32, ncols);
      }
      hct_tc_fence_before();
      hct_mbar_arrive(tempty0 + 8 * acc);
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
  }
  hct_tc_fence_before();
  __syncthreads();
  if (warp == 1) hct_tmem_dealloc(tmem_base, 512);
}
