// Persistent tensor-core conv2d (stride 1, zero padding) as an implicit GEMM with fused epilogue.
//
// GEMM view: rows = output pixels of one image, columns = output channels, contraction over
// (filter tap, input channel).  A tile of HCT_TH output rows x HCT_TW output columns (at most 128
// pixels) is one accumulator of 128 x HCT_BN in tensor memory.  For every filter tap (r,s) and
// block of 64 input channels the producer warp loads, with one 4-D TMA box from the NHWC copy of
// the input, the pixels shifted by the tap (coordinates outside the image read zeros, which is
// the padding) and the tap's [HCT_BN x 64] weight slice; the MMA warp multiplies them into the
// accumulator; four epilogue warps apply the generated epilogue and write NCHW.
//
// Defined by the generator: HCT_NB_IMG, HCT_C, HCT_H, HCT_W, HCT_KO, HCT_FR, HCT_FS, HCT_PAD, HCT_HO, HCT_WO,
// HCT_TW, HCT_TH, HCT_BN, HCT_STAGES, HCT_STATUS_SLOT, HCT_KERNEL_NAME, HctParams, hct_epilogue_conv().
#define HCT_BM 128
#define HCT_A_BYTES (HCT_BM * 128)
#define HCT_A_BOX_BYTES (HCT_TW * HCT_TH * 128)
#define HCT_B_BYTES (HCT_BN * 128)
#define HCT_STAGE_BYTES (HCT_A_BYTES + HCT_B_BYTES)
#define HCT_CB ((HCT_C + 63) / 64)
#define HCT_KB (HCT_FR * HCT_FS * HCT_CB)
#define HCT_HT ((HCT_HO + HCT_TH - 1) / HCT_TH)
#define HCT_WT ((HCT_WO + HCT_TW - 1) / HCT_TW)
#define HCT_NBK ((HCT_KO + HCT_BN - 1) / HCT_BN)
#define HCT_TILES ((long long)HCT_NB_IMG * HCT_HT * HCT_WT * HCT_NBK)
#define HCT_TMEM_COLS (2 * HCT_BN < 32 ? 32 : 2 * HCT_BN)

struct HctConvTile { int n, h0, w0, nbk; };
__device__ __forceinline__ HctConvTile hct_conv_tile(long long t) {
  HctConvTile r;
  r.nbk = (int)(t % HCT_NBK); t /= HCT_NBK;
  r.w0 = (int)(t % HCT_WT) * HCT_TW; t /= HCT_WT;
  r.h0 = (int)(t % HCT_HT) * HCT_TH; t /= HCT_HT;
  r.n = (int)t;
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
    hct_prefetch_tmap(&hct_p.tmap[1]);
  }
  if (warp == 1) hct_tmem_alloc(hct_smem_addr(&tmem_holder), HCT_TMEM_COLS);
  hct_tc_fence_before();
  __syncthreads();
  hct_tc_fence_after();
  const hct_u32 tmem_base = *(volatile hct_u32*)&tmem_holder;

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      hct_u32 phase = 0;
      for (long long tile = blockIdx.x; tile < HCT_TILES; tile += gridDim.x) {
        const HctConvTile t = hct_conv_tile(tile);
        for (int kb = 0; kb < HCT_KB; ++kb) {
          const int tap = kb / HCT_CB, cb = kb % HCT_CB;
          const int r = tap / HCT_FS, s = tap % HCT_FS;
          hct_mbar_wait(empty0 + 8 * stage, phase ^ 1u, &failed, status, 1);
          const hct_u32 full = full0 + 8 * stage;
          hct_mbar_expect_tx(full, HCT_A_BOX_BYTES + HCT_B_BYTES);
          const hct_u32 dst = smem_base + stage * HCT_STAGE_BYTES;
          // input pixels of this tap: channel coordinate is a multiple of 64 (16-byte aligned start);
          // w and h may start outside the image and then read the zero padding
          hct_tma_load_4d(dst, &hct_p.tmap[0], cb * 64, t.w0 + s - HCT_PAD, t.h0 + r - HCT_PAD, t.n, full);
          hct_tma_load_2d(dst + HCT_A_BYTES, &hct_p.tmap[1], cb * 64, tap * HCT_KO + t.nbk * HCT_BN, full);
          if (++stage == HCT_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // bf16 x bf16 -> fp32, both operands K-major, M = 128, N = HCT_BN
      const hct_u32 idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((hct_u32)(HCT_BN >> 3) << 17) | ((hct_u32)(HCT_BM >> 4) << 24);
      int stage = 0, acc = 0;
      hct_u32 phase = 0, acc_phase = 0;
      for (long long tile = blockIdx.x; tile < HCT_TILES; tile += gridDim.x) {
        hct_mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, &failed, status, 2);
        hct_tc_fence_after();
        const hct_u32 d_tmem = tmem_base + acc * HCT_BN;
        for (int kb = 0; kb < HCT_KB; ++kb) {
          hct_mbar_wait(full0 + 8 * stage, phase, &failed, status, 3);
          hct_tc_fence_after();
          const hct_u32 a_addr = smem_base + stage * HCT_STAGE_BYTES, b_addr = a_addr + HCT_A_BYTES;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const hct_u64 adesc = hct_smem_desc(a_addr + kk * 32, 16, 1024);
            const hct_u64 bdesc = hct_smem_desc(b_addr + kk * 32, 16, 1024);
            hct_mma_f16(d_tmem, adesc, bdesc, idesc, (kb | kk) != 0);
          }
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
    const int p = q * 32 + lane;              // pixel of the tile held by this thread's TMEM lane
    const int hh = p / HCT_TW, ww = p % HCT_TW;
    for (long long tile = blockIdx.x; tile < HCT_TILES; tile += gridDim.x) {
      const HctConvTile t = hct_conv_tile(tile);
      hct_mbar_wait(tfull0 + 8 * acc, acc_phase, &failed, status, 4);
      hct_tc_fence_after();
      const int h = t.h0 + hh, w = t.w0 + ww;
      const bool live = p < HCT_TW * HCT_TH && h < HCT_HO && w < HCT_WO;
#pragma unroll 1
      for (int c = 0; c < HCT_BN / 32; ++c) {
        float v[32];
        hct_tmem_ld32(tmem_base + ((hct_u32)(q * 32) << 16) + acc * HCT_BN + c * 32, v);
        const int k0 = t.nbk * HCT_BN + c * 32;
        const int nk = HCT_KO - k0 < 32 ? HCT_KO - k0 : 32;
        if (live && nk > 0) hct_epilogue_conv(hct_p, v, t.n, h, w, k0, nk);
      }
      hct_tc_fence_before();
      hct_mbar_arrive(tempty0 + 8 * acc);
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
  }
  hct_tc_fence_before();
  __syncthreads();
  if (warp == 1) hct_tmem_dealloc(tmem_base, HCT_TMEM_COLS);
}
