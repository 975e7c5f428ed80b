// Persistent tensor-core conv2d (stride 1, zero padding), variant that loads every input pixel
// once per filter ROW instead of once per tap.
//
// GEMM view as in conv_tc: rows (M = 128) = output channels, columns = pixels, contraction over
// (tap, input channel).  The pixel operand of filter row r and a 64-channel block is one 4-D TMA
// box of HCT_TH input rows x HCT_PITCH columns starting PAD columns left of the image (columns and
// rows outside the image read zeros: the padding), kept in shared memory as HCT_TH*HCT_PITCH rows
// of 128 bytes.  The taps s = 0..S-1 of that filter row read the SAME buffer through descriptors
// that start s rows (s*128 bytes) later: output column j = hh*HCT_PITCH + w then multiplies input
// pixel (hh, w + s).  Columns w >= WO of each pitch are computed and dropped.  Weights (one
// [128 x 64] slice per tap) and pixels travel in separate rings because a pixel buffer outlives
// S weight slices.  HCT_PITCH is a multiple of 32 so that the epilogue's 32-column steps never
// straddle an output row.
//
// Defined by the generator: HCT_NB_IMG, HCT_C, HCT_H, HCT_W, HCT_KO, HCT_FR, HCT_FS, HCT_PAD, HCT_HO, HCT_WO,
// HCT_PITCH, HCT_TH, HCT_TH2 (= 1), HCT_SPLIT, HCT_NA, HCT_NBUF, HCT_STATUS_SLOT,
// HCT_KERNEL_NAME, HctParams, hct_epilogue_run().
#define HCT_BM 128
#define HCT_A_BYTES (HCT_BM * 128)                       // weights: 128 channels x 64 inputs, bf16
#define HCT_B_BYTES 33792                                // pixels: 256 rows of 128 bytes + room for the shifted reads
#define HCT_RING_B_OFF (HCT_NA * HCT_A_BYTES)
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
#define HCT_RB (HCT_FR * HCT_CB)                          // pixel buffers per tile
#define HCT_HT ((HCT_HO + HCT_TH - 1) / HCT_TH)
#define HCT_MBK ((HCT_KO + HCT_BM - 1) / HCT_BM)
#define HCT_FULL_TILES ((long long)HCT_NB_IMG * HCT_HT * HCT_MBK)

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
  __shared__ unsigned long long bars[2 * HCT_NA + 2 * HCT_NBUF + 4];
  __shared__ hct_u32 tmem_holder;
  __shared__ int failed;
  const hct_u32 smem_base = (hct_smem_addr(hct_smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned int* status = (unsigned int*)hct_p.ptr[HCT_STATUS_SLOT];
  const hct_u32 afull0 = hct_smem_addr(&bars[0]), aempty0 = hct_smem_addr(&bars[HCT_NA]);
  const hct_u32 bfull0 = hct_smem_addr(&bars[2 * HCT_NA]), bempty0 = hct_smem_addr(&bars[2 * HCT_NA + HCT_NBUF]);
  const hct_u32 tfull0 = hct_smem_addr(&bars[2 * HCT_NA + 2 * HCT_NBUF]), tempty0 = tfull0 + 16;

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
    for (int s = 0; s < HCT_NA; ++s) {
      hct_mbar_init(afull0 + 8 * s, 1);
      hct_mbar_init(aempty0 + 8 * s, 1);
    }
    for (int s = 0; s < HCT_NBUF; ++s) {
      hct_mbar_init(bfull0 + 8 * s, 1);
      hct_mbar_init(bempty0 + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      hct_mbar_init(tfull0 + 8 * a, 1);
      hct_mbar_init(tempty0 + 8 * a, 128);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    hct_prefetch_tmap(&hct_p.tmap[0]);
    hct_prefetch_tmap(&hct_p.tmap[1]);
    hct_prefetch_tmap(&hct_p.tmap[2]);
  }
  if (warp == 1) hct_tmem_alloc(hct_smem_addr(&tmem_holder), 512);
  hct_tc_fence_before();
  __syncthreads();
  hct_tc_fence_after();
  const hct_u32 tmem_base = *(volatile hct_u32*)&tmem_holder;
  hct_pdl_wait();   // barriers, tensor memory and descriptors are ready; now the predecessor's data may be read

  if (warp == 0) {
    if (lane == 0) {
      int sa = 0, sb = 0;
      hct_u32 pa = 0, pb = 0;
      for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const HctConvTile t = hct_conv_tile(tile, t1);
        if (t.th == 0) continue;
        // whole tiles use the HCT_TH-row box, pieces the one-row box
        const HctTensorMap* xmap = t.cut ? &hct_p.tmap[2] : &hct_p.tmap[1];
        const hct_u32 bbytes = (hct_u32)(t.cut ? HCT_TH2 : HCT_TH) * HCT_PITCH * 128u;
        for (int rb = 0; rb < HCT_RB; ++rb) {
          const int r = rb / HCT_CB, cb = rb % HCT_CB;
          hct_mbar_wait(bempty0 + 8 * sb, pb ^ 1u, &failed, status, 1);
          hct_mbar_expect_tx(bfull0 + 8 * sb, bbytes);
          hct_tma_load_4d(smem_base + HCT_RING_B_OFF + sb * HCT_B_BYTES, xmap, HCT_C_LO(t.mbk) + cb * 64, -HCT_PAD, t.h0 + r - HCT_PAD, t.n, bfull0 + 8 * sb);
          if (++sb == HCT_NBUF) { sb = 0; pb ^= 1u; }
          for (int s = 0; s < HCT_FS; ++s) {
            hct_mbar_wait(aempty0 + 8 * sa, pa ^ 1u, &failed, status, 5);
            hct_mbar_expect_tx(afull0 + 8 * sa, HCT_A_BYTES);
            hct_tma_load_2d(smem_base + sa * HCT_A_BYTES, &hct_p.tmap[0], cb * 64, (r * HCT_FS + s) * HCT_KO + t.mbk * HCT_BM, afull0 + 8 * sa);
            if (++sa == HCT_NA) { sa = 0; pa ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int sa = 0, sb = 0, acc = 0;
      hct_u32 pa = 0, pb = 0, acc_phase = 0;
      for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const HctConvTile t = hct_conv_tile(tile, t1);
        if (t.th == 0) continue;
        // bf16 x bf16 -> fp32, both operands K-major, M = 128, N = rows of this tile times the pitch
        const hct_u32 n_mma = (hct_u32)(t.th * HCT_PITCH);
        const hct_u32 idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((n_mma >> 3) << 17) | ((hct_u32)(HCT_BM >> 4) << 24);
        hct_mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, &failed, status, 2);
        hct_tc_fence_after();
        const hct_u32 d_tmem = tmem_base + acc * 256;
        for (int rb = 0; rb < HCT_RB; ++rb) {
          hct_mbar_wait(bfull0 + 8 * sb, pb, &failed, status, 3);
          const hct_u32 b_addr = smem_base + HCT_RING_B_OFF + sb * HCT_B_BYTES;
          for (int s = 0; s < HCT_FS; ++s) {
            hct_mbar_wait(afull0 + 8 * sa, pa, &failed, status, 6);
            hct_tc_fence_after();
            const hct_u32 a_addr = smem_base + sa * HCT_A_BYTES;
            // tap s reads the pixel buffer s rows (s * 128 bytes) further on.  The 128-byte swizzle is a
            // function of the absolute shared-memory address (measured: results are exact with the
            // descriptor's base-offset field left at zero), so a start that is not a multiple of 8 rows
            // needs nothing else.  Descriptors differ only in the start-address field (16-byte units).
            const hct_u64 a_desc0 = hct_smem_desc(a_addr, 16, 1024), b_desc0 = hct_smem_desc(b_addr + s * 128, 16, 1024);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) hct_mma_f16(d_tmem, a_desc0 + kk * 2, b_desc0 + kk * 2, idesc, (rb | s | kk) != 0);
            hct_mma_commit(aempty0 + 8 * sa);
            if (++sa == HCT_NA) { sa = 0; pa ^= 1u; }
          }
          hct_mma_commit(bempty0 + 8 * sb);
          if (++sb == HCT_NBUF) { sb = 0; pb ^= 1u; }
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
      const int chunks = t.th * (HCT_PITCH / 32);
#pragma unroll 1
      for (int c = 0; c < chunks; ++c) {
        const int hh = c / (HCT_PITCH / 32), part = c % (HCT_PITCH / 32);
        const int ncols = HCT_WO - part * 32 < 32 ? HCT_WO - part * 32 : 32;   // columns past WO are padding
        if (ncols <= 0) continue;
        float v[32];
        hct_tmem_ld32(tmem_base + ((hct_u32)(q * 32) << 16) + acc * 256 + c * 32, v);
        if (k < HCT_KO) hct_epilogue_run(hct_p, v, (long long)t.n * HCT_KO + k, (t.h0 + hh) * HCT_WO + part * 32, ncols);
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
