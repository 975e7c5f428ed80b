// Persistent tensor-core GEMM on CTA pairs (bf16 operands, fp32 accumulation, fused epilogue):
// D[M,N] = epilogue(A[M,K] * B[K,N]).
//
// Two CTAs of a cluster (two SMs) share 256 x 256 output tiles.  Each CTA loads ITS half of both
// operands per 64-deep k step -- 128 rows of A and 128 columns of B, 32 KB -- and one thread of the
// even CTA issues tcgen05.mma.cta_group::2 (M = 256, N = 256), which reads A from each CTA's own
// shared memory and B from both; every CTA ends up with its 128 rows x 256 columns of the
// accumulator in its own tensor memory.  Against one CTA working a 128 x 256 tile alone this halves
// the B bytes each SM stages and reads per unit of tensor work, which is what bounds that kernel
// (96 KB through shared memory per 512 tensor cycles); six 32 KB stages fit instead of four 48 KB ones.
//
// Hand-offs.  full[s] lives in the even CTA: its producer announces the bytes of BOTH CTAs' loads,
// and both CTAs' TMA copies count on it.  empty[s] and tfull[a] exist in both CTAs and are completed
// by two tcgen05.commit (one per CTA) from the issuing thread.  tempty[a] lives in the even CTA and
// counts the epilogue threads of both.  Every CTA issues its own loads.  All waits are bounded.
//
// The fp32 variant (HCT_TF32X3) works on 256 x 256 tiles per pair from the head/tail operands its
// split pre-pass wrote (B transposed to [N,K]): three TF32 products per k step, at most 128 elements
// of K accumulated in tensor memory and those chunks summed in registers, exactly as in the
// single-CTA kernel; each CTA stages 128 rows of A and 128 rows of B^T (64 KB per 32-deep stage), and
// eight epilogue warps share the running sums (128 columns each).
//
// Defined by the generator: HCT_M, HCT_N, HCT_K, HCT_STAGES, HCT_TF32X3 (0/1), HCT_STATUS_SLOT,
// HCT_KERNEL_NAME, HctParams, hct_epilogue_run().
#if HCT_TF32X3
#define HCT_BK 32
#define HCT_BNP 256                             // tile columns per pair
#define HCT_A_BYTES 16384                       // 128 rows x 32 k, fp32 (head; the tail follows)
#define HCT_B_BYTES 16384                       // 128 rows of B^T x 32 k, fp32
#define HCT_EPI_WARPS 8                         // two warps per lane quarter: 128 columns of the running sum each
#define HCT_STAGE_BYTES (2 * HCT_A_BYTES + 2 * HCT_B_BYTES)
#define HCT_KBC 4                               // k blocks accumulated in tensor memory before the chunk is drained
#else
#define HCT_BK 64
#define HCT_BNP 256
#define HCT_EPI_WARPS 4
#define HCT_A_BYTES 16384                       // 128 rows x 64 k, bf16
#define HCT_B_BYTES 16384                       // 64 k x 128 columns, bf16 (two 64-column boxes)
#define HCT_STAGE_BYTES (HCT_A_BYTES + HCT_B_BYTES)
#define HCT_KBC HCT_KB
#endif
#define HCT_KB ((HCT_K + HCT_BK - 1) / HCT_BK)
#define HCT_NCH ((HCT_KB + HCT_KBC - 1) / HCT_KBC)
#define HCT_MB ((HCT_M + 255) / 256)
#define HCT_NB ((HCT_N + HCT_BNP - 1) / HCT_BNP)
#define HCT_TILES ((long long)HCT_MB * HCT_NB)
#define HCT_TMEM_COLS (2 * HCT_BNP)

extern "C" __global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(64 + 32 * HCT_EPI_WARPS, 1) HCT_KERNEL_NAME(const __grid_constant__ HctParams hct_p) {
  extern __shared__ unsigned char hct_smem_raw[];
  __shared__ unsigned long long bars[2 * HCT_STAGES + 4];
  __shared__ hct_u32 tmem_holder;
  __shared__ int failed;
  const hct_u32 smem_base = (hct_smem_addr(hct_smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const hct_u32 rank = hct_cluster_ctarank();
  unsigned int* status = (unsigned int*)hct_p.ptr[HCT_STATUS_SLOT];
  const hct_u32 full0 = hct_smem_addr(&bars[0]), empty0 = hct_smem_addr(&bars[HCT_STAGES]);
  const hct_u32 tfull0 = hct_smem_addr(&bars[2 * HCT_STAGES]), tempty0 = hct_smem_addr(&bars[2 * HCT_STAGES + 2]);
  const long long pair = blockIdx.x / 2, n_pairs = gridDim.x / 2;

  hct_pdl_launch_dependents();
  if (threadIdx.x == 0) {
    failed = 0;
    for (int s = 0; s < HCT_STAGES; ++s) {
      hct_mbar_init(full0 + 8 * s, 1);
      hct_mbar_init(empty0 + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      hct_mbar_init(tfull0 + 8 * a, 1);
      hct_mbar_init(tempty0 + 8 * a, 64 * HCT_EPI_WARPS);   // the epilogue threads of both CTAs
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    hct_prefetch_tmap(&hct_p.tmap[0]);
    hct_prefetch_tmap(&hct_p.tmap[1]);
#if HCT_TF32X3
    hct_prefetch_tmap(&hct_p.tmap[2]);
    hct_prefetch_tmap(&hct_p.tmap[3]);
#endif
  }
  if (warp == 1) hct_tmem_alloc_pair(hct_smem_addr(&tmem_holder), HCT_TMEM_COLS);
  hct_tc_fence_before();
  __syncthreads();
  hct_cluster_sync();   // the other CTA's barriers exist before anything is signalled across
  hct_tc_fence_after();
  const hct_u32 tmem_base = *(volatile hct_u32*)&tmem_holder;
  hct_pdl_wait();

  if (warp == 0) {
    // ---------------- TMA producer (both CTAs, each for its own half)
    if (lane == 0) {
      int stage = 0;
      hct_u32 phase = 0;
      for (long long tile = pair; tile < HCT_TILES; tile += n_pairs) {
        const int nb = (int)(tile % HCT_NB), mb = (int)(tile / HCT_NB);
        for (int kb = 0; kb < HCT_KB; ++kb) {
          hct_mbar_wait(empty0 + 8 * stage, phase ^ 1u, &failed, status, 1);
          const hct_u32 full_even = hct_mapa(full0 + 8 * stage, 0);
          if (rank == 0) hct_mbar_expect_tx(full0 + 8 * stage, 2 * HCT_STAGE_BYTES);
          hct_u32 dst = smem_base + stage * HCT_STAGE_BYTES;
#if HCT_TF32X3
          hct_tma_load_2d_pair(dst, &hct_p.tmap[0], kb * HCT_BK, mb * 256 + (int)rank * 128, full_even);                     // A head
          hct_tma_load_2d_pair(dst + HCT_A_BYTES, &hct_p.tmap[1], kb * HCT_BK, mb * 256 + (int)rank * 128, full_even);       // A tail
          dst += 2 * HCT_A_BYTES;
          hct_tma_load_2d_pair(dst, &hct_p.tmap[2], kb * HCT_BK, nb * HCT_BNP + (int)rank * 128, full_even);                  // B^T head
          hct_tma_load_2d_pair(dst + HCT_B_BYTES, &hct_p.tmap[3], kb * HCT_BK, nb * HCT_BNP + (int)rank * 128, full_even);    // B^T tail
#else
          hct_tma_load_2d_pair(dst, &hct_p.tmap[0], kb * 64, mb * 256 + (int)rank * 128, full_even);
          dst += HCT_A_BYTES;
          for (int j = 0; j < 2; ++j)
            hct_tma_load_2d_pair(dst + j * 8192, &hct_p.tmap[1], nb * 256 + (int)rank * 128 + j * 64, kb * 64, full_even);
#endif
          if (++stage == HCT_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (even CTA only)
    if (lane == 0 && rank == 0) {
#if HCT_TF32X3
      // fp32 accumulate, tf32 operands, both K-major, M = 256 over the pair, N = 128
      const hct_u32 idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((hct_u32)(HCT_BNP >> 3) << 17) | ((hct_u32)(256 >> 4) << 24);
#else
      // fp32 accumulate, bf16 operands, A K-major, B N-major, M = 256 over the pair, N = 256
      const hct_u32 idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((hct_u32)(HCT_BNP >> 3) << 17) | ((hct_u32)(256 >> 4) << 24);
#endif
      int stage = 0, acc = 0;
      hct_u32 phase = 0, acc_phase = 0;
      for (long long tile = pair; tile < HCT_TILES; tile += n_pairs) {
       for (int ch = 0; ch < HCT_NCH; ++ch) {
        hct_mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, &failed, status, 2);
        hct_tc_fence_after();
        const hct_u32 d_tmem = tmem_base + acc * HCT_BNP;
        const int kb0 = ch * HCT_KBC, kb1 = kb0 + HCT_KBC < HCT_KB ? kb0 + HCT_KBC : HCT_KB;
        for (int kb = kb0; kb < kb1; ++kb) {
          hct_mbar_wait(full0 + 8 * stage, phase, &failed, status, 3);
          hct_tc_fence_after();
          const hct_u32 a_addr = smem_base + stage * HCT_STAGE_BYTES;
#if HCT_TF32X3
          const hct_u32 b_addr = a_addr + 2 * HCT_A_BYTES;
          const hct_u64 a_desc0 = hct_smem_desc(a_addr, 16, 1024), b_desc0 = hct_smem_desc(b_addr, 16, 1024);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const hct_u64 a_hi = a_desc0 + kk * 2, a_lo = a_desc0 + (HCT_A_BYTES >> 4) + kk * 2;
            const hct_u64 b_hi = b_desc0 + kk * 2, b_lo = b_desc0 + (HCT_B_BYTES >> 4) + kk * 2;
            // small cross terms first, then the leading product
            hct_mma_tf32_pair(d_tmem, a_lo, b_hi, idesc, (kb > kb0) || (kk != 0));
            hct_mma_tf32_pair(d_tmem, a_hi, b_lo, idesc, 1);
            hct_mma_tf32_pair(d_tmem, a_hi, b_hi, idesc, 1);
          }
#else
          const hct_u32 b_addr = a_addr + HCT_A_BYTES;
          const hct_u64 a_desc0 = hct_smem_desc(a_addr, 16, 1024), b_desc0 = hct_smem_desc(b_addr, 8192, 1024);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) hct_mma_f16_pair(d_tmem, a_desc0 + kk * 2, b_desc0 + kk * (2048 >> 4), idesc, (kb > kb0) || (kk != 0));
#endif
          hct_mma_commit_pair(hct_mapa(empty0 + 8 * stage, 0));   // frees the stage in both CTAs
          hct_mma_commit_pair(hct_mapa(empty0 + 8 * stage, 1));
          if (++stage == HCT_STAGES) { stage = 0; phase ^= 1u; }
        }
        hct_mma_commit_pair(hct_mapa(tfull0 + 8 * acc, 0));       // both halves of this chunk's accumulator are complete
        hct_mma_commit_pair(hct_mapa(tfull0 + 8 * acc, 1));
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
       }
      }
    }
  } else {
    // ---------------- epilogue (both CTAs): warp w may only touch TMEM lanes 32 (w mod 4) .. +31
    const int q = warp & 3;
    int acc = 0;
    hct_u32 acc_phase = 0;
    for (long long tile = pair; tile < HCT_TILES; tile += n_pairs) {
      const int nb = (int)(tile % HCT_NB), mb = (int)(tile / HCT_NB);
      const long long row = (long long)mb * 256 + rank * 128 + q * 32 + lane;
#if !HCT_TF32X3
      hct_mbar_wait(tfull0 + 8 * acc, acc_phase, &failed, status, 4);
      hct_tc_fence_after();
#pragma unroll 1
      for (int c = 0; c < HCT_BNP / 32; ++c) {
        float v[32];
        hct_tmem_ld32(tmem_base + ((hct_u32)(q * 32) << 16) + acc * HCT_BNP + c * 32, v);
        const long long col0 = (long long)nb * HCT_BNP + c * 32;
        const int ncols = (int)(HCT_N - col0 < 32 ? HCT_N - col0 : 32);
        if (row < HCT_M && ncols > 0) hct_epilogue_run(hct_p, v, row, (int)col0, ncols);
      }
      hct_tc_fence_before();
      hct_mbar_arrive_cluster(hct_mapa(tempty0 + 8 * acc, 0));
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
#else
      // this warp's share of the columns: HCT_BNP / (HCT_EPI_WARPS / 4) starting at c0 chunks of 32
      constexpr int NCW = HCT_BNP / 32 / (HCT_EPI_WARPS / 4);
      const int c0 = ((warp - 2) >> 2) * NCW;
      float sum[NCW * 32];
#pragma unroll
      for (int j = 0; j < NCW * 32; ++j) sum[j] = 0.0f;
#pragma unroll 1
      for (int ch = 0; ch < HCT_NCH; ++ch) {
        hct_mbar_wait(tfull0 + 8 * acc, acc_phase, &failed, status, 4);
        hct_tc_fence_after();
#pragma unroll
        for (int c = 0; c < NCW; ++c) {
          float v[32];
          hct_tmem_ld32(tmem_base + ((hct_u32)(q * 32) << 16) + acc * HCT_BNP + (c0 + c) * 32, v);
#pragma unroll
          for (int j = 0; j < 32; ++j) sum[c * 32 + j] += v[j];
        }
        hct_tc_fence_before();
        hct_mbar_arrive_cluster(hct_mapa(tempty0 + 8 * acc, 0));
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
#pragma unroll
      for (int c = 0; c < NCW; ++c) {
        const long long col0 = (long long)nb * HCT_BNP + (c0 + c) * 32;
        const int ncols = (int)(HCT_N - col0 < 32 ? HCT_N - col0 : 32);
        if (row < HCT_M && ncols > 0) hct_epilogue_run(hct_p, *(float(*)[32])(sum + c * 32), row, (int)col0, ncols);
      }
#endif
    }
  }
  hct_tc_fence_before();
  __syncthreads();
  hct_cluster_sync();   // neither CTA leaves (or frees tensor memory) while the other may still signal it
  if (warp == 1) hct_tmem_dealloc_pair(tmem_base, HCT_TMEM_COLS);
}
