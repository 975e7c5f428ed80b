// Persistent tensor-core pointwise (1x1, stride 1, no padding) conv2d with fused epilogue.
//
// Per image a 1x1 convolution on NCHW data is the product Y_n[KO, HW] = W[KO, C] * X_n[C, HW]: the
// weights [KO, C, 1, 1] already are a K-major A operand and the image, pixels contiguous, is an
// N-major B operand, so neither takes a layout pass.  One CTA per SM walks over tiles of 128 output
// channels x 256 pixels of one image (channel blocks fastest, so the CTAs that share pixels run
// together and find them in L2).  Warp 0 loads a stage per block of 64 input channels (one weight box,
// four pixel boxes of 64 pixels x 64 channels; channels past C and pixels past HW read zeros), warp 1
// issues tcgen05.mma into one of two accumulators in tensor memory, HCT_EPW epilogue warps (8 or 16: two or
// four per lane quarter, 128 or 64 pixels each) drain the other; a tile has little MMA work, so the step time is
// set by the epilogue.  A single bf16 result leaves through shared memory and TMA stores of 32 channels x 64
// pixels; anything else is stored by the generated epilogue itself.
//
// Defined by the generator: HCT_NB_IMG, HCT_C, HCT_KO, HCT_HW, HCT_STAGES, HCT_EPW, HCT_TMA_STORE, HCT_STATUS_SLOT,
// HCT_KERNEL_NAME, HctParams, hct_epilogue_run() or (HCT_TMA_STORE) hct_epilogue_vals().
// Maps: [0] weights {C, KO}, [1] pixels {HW, C, image}, [2] (HCT_TMA_STORE) result {HW, KO, image}.
#define HCT_BM 128
#define HCT_BN 256
#define HCT_A_BYTES (HCT_BM * 128)
#define HCT_B_BYTES (HCT_BN * 128)
#define HCT_BBOX_BYTES 8192
#define HCT_STAGE_BYTES (HCT_A_BYTES + HCT_B_BYTES)
#define HCT_KB ((HCT_C + 63) / 64)
#define HCT_MBK ((HCT_KO + HCT_BM - 1) / HCT_BM)
#define HCT_NBK ((HCT_HW + HCT_BN - 1) / HCT_BN)
#define HCT_TILES ((long long)HCT_NB_IMG * HCT_NBK * HCT_MBK)
#define HCT_RING_O_OFF (HCT_STAGES * HCT_STAGE_BYTES)
#define HCT_CPW (8 / (HCT_EPW / 4))                     // chunks of 32 pixels per epilogue warp and tile

__device__ __forceinline__ void hct_tma_load_3d(hct_u32 dst, const HctTensorMap* map, int c0, int c1, int c2, hct_u32 bar) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
               "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
               : "memory");
}

struct HctPwTile { int n, nb, mbk; };
__device__ __forceinline__ HctPwTile hct_pw_tile(long long t) {
  HctPwTile r;
  r.mbk = (int)(t % HCT_MBK); t /= HCT_MBK;
  r.nb = (int)(t % HCT_NBK);
  r.n = (int)(t / HCT_NBK);
  return r;
}

extern "C" __global__ void __launch_bounds__(64 + 32 * HCT_EPW, 1) HCT_KERNEL_NAME(const __grid_constant__ HctParams hct_p) {
  extern __shared__ unsigned char hct_smem_raw[];
  __shared__ unsigned long long bars[2 * HCT_STAGES + 4];
  __shared__ hct_u32 tmem_holder;
  __shared__ int failed;
  const hct_u32 smem_base = (hct_smem_addr(hct_smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned int* status = (unsigned int*)hct_p.ptr[HCT_STATUS_SLOT];
  const hct_u32 full0 = hct_smem_addr(&bars[0]), empty0 = hct_smem_addr(&bars[HCT_STAGES]);
  const hct_u32 tfull0 = hct_smem_addr(&bars[2 * HCT_STAGES]), tempty0 = hct_smem_addr(&bars[2 * HCT_STAGES + 2]);

  hct_pdl_launch_dependents();
  if (threadIdx.x == 0) {
    failed = 0;
    for (int s = 0; s < HCT_STAGES; ++s) {
      hct_mbar_init(full0 + 8 * s, 1);
      hct_mbar_init(empty0 + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      hct_mbar_init(tfull0 + 8 * a, 1);
      hct_mbar_init(tempty0 + 8 * a, 32 * HCT_EPW);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    hct_prefetch_tmap(&hct_p.tmap[0]);
    hct_prefetch_tmap(&hct_p.tmap[1]);
#if HCT_TMA_STORE
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
      for (long long tile = blockIdx.x; tile < HCT_TILES; tile += gridDim.x) {
        const HctPwTile t = hct_pw_tile(tile);
        for (int kb = 0; kb < HCT_KB; ++kb) {
          hct_mbar_wait(empty0 + 8 * stage, phase ^ 1u, &failed, status, 1);
          const hct_u32 full = full0 + 8 * stage;
          hct_mbar_expect_tx(full, HCT_STAGE_BYTES);
          hct_u32 dst = smem_base + stage * HCT_STAGE_BYTES;
          hct_tma_load_2d(dst, &hct_p.tmap[0], kb * 64, t.mbk * HCT_BM, full);
          dst += HCT_A_BYTES;
#pragma unroll
          for (int j = 0; j < 4; ++j) hct_tma_load_3d(dst + j * HCT_BBOX_BYTES, &hct_p.tmap[1], t.nb * HCT_BN + j * 64, kb * 64, t.n, full);
          if (++stage == HCT_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // bf16 x bf16 -> fp32, A K-major, B N-major, M = 128, N = 256
      const hct_u32 idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((hct_u32)(HCT_BN >> 3) << 17) | ((hct_u32)(HCT_BM >> 4) << 24);
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
          const hct_u64 a_desc0 = hct_smem_desc(a_addr, 16, 1024), b_desc0 = hct_smem_desc(b_addr, HCT_BBOX_BYTES, 1024);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) hct_mma_f16(d_tmem, a_desc0 + kk * 2, b_desc0 + kk * (2048 >> 4), idesc, (kb | kk) != 0);
          hct_mma_commit(empty0 + 8 * stage);
          if (++stage == HCT_STAGES) { stage = 0; phase ^= 1u; }
        }
        hct_mma_commit(tfull0 + 8 * acc);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    // ---- epilogue: one output channel per thread; the warps of a lane quarter share the tile's pixels
    const int q = warp & 3, part = (warp - 2) >> 2;
    int acc = 0;
    hct_u32 acc_phase = 0;
    for (long long tile = blockIdx.x; tile < HCT_TILES; tile += gridDim.x) {
      const HctPwTile t = hct_pw_tile(tile);
      hct_mbar_wait(tfull0 + 8 * acc, acc_phase, &failed, status, 4);
      hct_tc_fence_after();
      const int k = t.mbk * HCT_BM + q * 32 + lane;
      const bool live = t.mbk * HCT_BM + q * 32 < HCT_KO;   // this warp's 32 channels exist (warp-uniform)
#if HCT_TMA_STORE
      // 32 channels x 64 pixels (two chunks) leave through shared memory and one TMA store; pixels past HW and
      // channels past KO are clipped by the copy.  Row = channel (128 bytes), 128-byte swizzle: 16-byte piece p of
      // row i sits at piece p ^ (i & 7), which also keeps the writes of neighbouring lanes in different banks.
      // Rows of 128 bytes matter: the copy engine spends its time per row, and with 64-byte rows the stores of a
      // tile took longer than everything else in it.  One slot per warp, rewritten once the store issued from
      // it (a tile ago) has read it.
      const hct_u32 o_slot = smem_base + HCT_RING_O_OFF + (hct_u32)((warp - 2) * 4096);
#pragma unroll 1
      for (int cp = 0; cp < HCT_CPW / 2; ++cp) {
        const int c0 = part * HCT_CPW + cp * 2;
        const int pix0 = t.nb * HCT_BN + c0 * 32;
        if (HCT_HW - pix0 <= 0 || !live) break;
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          const int ncols = HCT_HW - (pix0 + cc * 32) < 32 ? HCT_HW - (pix0 + cc * 32) : 32;
          if (ncols <= 0) break;
          float v[32], o[32];
          hct_tmem_ld32(tmem_base + ((hct_u32)(q * 32) << 16) + acc * HCT_BN + (c0 + cc) * 32, v);
          if (k < HCT_KO) {
            hct_epilogue_vals(hct_p, v, (long long)t.n * HCT_KO + k, pix0 + cc * 32, ncols, o);
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = 0.0f;
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const hct_u32 dst = o_slot + (hct_u32)lane * 128u + (((hct_u32)(cc * 4 + j) ^ ((hct_u32)lane & 7u)) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(hct_pack_bf16x2(o[8 * j], o[8 * j + 1])),
                         "r"(hct_pack_bf16x2(o[8 * j + 2], o[8 * j + 3])), "r"(hct_pack_bf16x2(o[8 * j + 4], o[8 * j + 5])),
                         "r"(hct_pack_bf16x2(o[8 * j + 6], o[8 * j + 7]))
                         : "memory");
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];" ::"l"(&hct_p.tmap[2]), "r"(pix0),
                       "r"(t.mbk * HCT_BM + q * 32), "r"(t.n), "r"(o_slot)
                       : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
#else
#pragma unroll 1
      for (int c = part * HCT_CPW; c < (part + 1) * HCT_CPW; ++c) {
        const int pix0 = t.nb * HCT_BN + c * 32;
        const int ncols = HCT_HW - pix0 < 32 ? HCT_HW - pix0 : 32;
        if (ncols <= 0 || !live) break;
        float v[32];
        hct_tmem_ld32(tmem_base + ((hct_u32)(q * 32) << 16) + acc * HCT_BN + c * 32, v);
        if (k < HCT_KO) hct_epilogue_run(hct_p, v, (long long)t.n * HCT_KO + k, pix0, ncols);
      }
#endif
      hct_tc_fence_before();
      hct_mbar_arrive(tempty0 + 8 * acc);
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
#if HCT_TMA_STORE
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all stores done before the CTA ends
#endif
  }
  hct_tc_fence_before();
  __syncthreads();
  if (warp == 1) hct_tmem_dealloc(tmem_base, 512);
}
