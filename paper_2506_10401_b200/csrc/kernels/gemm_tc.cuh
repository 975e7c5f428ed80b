// Persistent tensor-core GEMM with fused epilogue:  D[M,N] = epilogue(A[M,K] * B[K,N]).
//
// One CTA per SM walks over 128 x HCT_BN output tiles.  Warp 0 feeds a ring of shared-memory
// stages with TMA tile loads (A is K-major; bf16 B is row-major [K,N], i.e. N-major; the TF32
// variant reads B already transposed to [N,K] by its split pre-pass), warp 1 issues
// tcgen05.mma from those stages into one of two accumulators in tensor memory, warps 2..5 drain
// the other accumulator (tcgen05.ld), apply the generated epilogue and store, so the epilogue of
// tile i overlaps the main loop of tile i+1.  All hand-offs are mbarriers with bounded waits.
//
// Defined by the generator: HCT_M, HCT_N, HCT_K, HCT_BN, HCT_STAGES, HCT_TF32X3 (0/1),
// HCT_NPTR, HCT_STATUS_SLOT, HCT_KERNEL_NAME, HctParams, hct_epilogue_run().
#define HCT_BM 128
#if HCT_TF32X3
#define HCT_BK 32                                  // 32 fp32 = one 128-byte swizzle row
#define HCT_ELT 4
#define HCT_UMMA_K 8
#else
#define HCT_BK 64                                  // 64 bf16 = one 128-byte swizzle row
#define HCT_ELT 2
#define HCT_UMMA_K 16
#endif
#define HCT_NBOX (128 / HCT_ELT)                   // B elements along N per 128-byte row
#define HCT_A_BYTES (HCT_BM * 128)
#define HCT_B_BYTES (HCT_BN * 128)
#define HCT_BBOX_BYTES (HCT_NBOX * HCT_BK * HCT_ELT)  // one [BK x NBOX] box of B
#if HCT_TF32X3
#define HCT_STAGE_BYTES (2 * HCT_A_BYTES + 2 * HCT_B_BYTES)   // hi and lo parts of both operands
#else
#define HCT_STAGE_BYTES (HCT_A_BYTES + HCT_B_BYTES)
#endif
#define HCT_KB ((HCT_K + HCT_BK - 1) / HCT_BK)
// The tensor core adds into its fp32 accumulator with truncation, which biases long sums by about
// 1e-8 per accumulated element.  The TF32 variant therefore accumulates at most HCT_KBC k-blocks
// (128 elements of K) in tensor memory and sums those partial results in registers, rounding to
// nearest; the bf16 variant, judged at 2e-2, accumulates the whole K extent in tensor memory.
#if HCT_TF32X3
#define HCT_KBC 4
#else
#define HCT_KBC HCT_KB
#endif
#define HCT_NCH ((HCT_KB + HCT_KBC - 1) / HCT_KBC)
// Split of the contraction (TF32 variant, problems with far fewer tiles than SMs): a work item is one of
// HCT_KSPLIT parts of a tile's K extent, HCT_CPP chunks each (the generator picks HCT_KSPLIT so that no part is
// empty).  Every part adds its partial tile into an fp32 accumulation tile in scratch (vector atomics, cleared
// by the split pre-pass) and counts its arrival; the last part to arrive reads the sums back and runs the epilogue.
// The order of the additions is the order of arrival, so the last bits of a result may differ between runs.
#ifndef HCT_KSPLIT
#define HCT_KSPLIT 1
#endif
#define HCT_CPP ((HCT_NCH + HCT_KSPLIT - 1) / HCT_KSPLIT)
#define HCT_ITEMS (HCT_TILES * HCT_KSPLIT)
#define HCT_NCH_IS_ONE (!HCT_TF32X3)
#define HCT_MB ((HCT_M + HCT_BM - 1) / HCT_BM)
#define HCT_NB ((HCT_N + HCT_BN - 1) / HCT_BN)
#define HCT_TILES ((long long)HCT_MB * HCT_NB)
#define HCT_TMEM_COLS (2 * HCT_BN < 32 ? 32 : 2 * HCT_BN)
// A TF32 instruction covers 8 elements of K and takes about as long at 128 columns as at 256, so wide
// tiles halve the instruction count.  Their running sums (one register per column) are then shared by
// two epilogue warps per lane quarter, 128 columns each.
#if HCT_TF32X3 && HCT_BN > 128
#define HCT_EPI_WARPS 8
#else
#define HCT_EPI_WARPS 4
#endif

extern "C" __global__ void __launch_bounds__(64 + 32 * HCT_EPI_WARPS, 1) HCT_KERNEL_NAME(const __grid_constant__ HctParams hct_p) {
  extern __shared__ unsigned char hct_smem_raw[];
  __shared__ unsigned long long bars[2 * HCT_STAGES + 4];
  __shared__ hct_u32 tmem_holder;
  __shared__ int failed;
#if HCT_KSPLIT > 1
  __shared__ int ks_last;
#endif
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
      hct_mbar_init(tempty0 + 8 * a, 32 * HCT_EPI_WARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    hct_prefetch_tmap(&hct_p.tmap[0]);
    hct_prefetch_tmap(&hct_p.tmap[1]);
#if HCT_TF32X3
    hct_prefetch_tmap(&hct_p.tmap[2]);
    hct_prefetch_tmap(&hct_p.tmap[3]);
#endif
  }
  if (warp == 1) hct_tmem_alloc(hct_smem_addr(&tmem_holder), HCT_TMEM_COLS);
  hct_tc_fence_before();
  __syncthreads();
  hct_tc_fence_after();
  const hct_u32 tmem_base = *(volatile hct_u32*)&tmem_holder;
  hct_pdl_wait();   // barriers, tensor memory and descriptors are ready; now the predecessor's data may be read

  if (warp == 0) {
    // ---------------- TMA producer
    if (lane == 0) {
      int stage = 0;
      hct_u32 phase = 0;
      for (long long item = blockIdx.x; item < HCT_ITEMS; item += gridDim.x) {
        const long long tile = item / HCT_KSPLIT;
        const int part = (int)(item % HCT_KSPLIT);
        const int nb = (int)(tile % HCT_NB), mb = (int)(tile / HCT_NB);
        const int kb_lo = part * HCT_CPP * HCT_KBC, kb_hi = kb_lo + HCT_CPP * HCT_KBC < HCT_KB ? kb_lo + HCT_CPP * HCT_KBC : HCT_KB;
        for (int kb = kb_lo; kb < kb_hi; ++kb) {
          hct_mbar_wait(empty0 + 8 * stage, phase ^ 1u, &failed, status, 1);
#if defined(HCT_FAULT_NEVER_ARRIVE) && HCT_FAULT_NEVER_ARRIVE
          // failure-path test build: nothing ever completes the stage's barrier
          if (++stage == HCT_STAGES) { stage = 0; phase ^= 1u; }
          continue;
#endif
          const hct_u32 full = full0 + 8 * stage;
          hct_mbar_expect_tx(full, HCT_STAGE_BYTES);
          hct_u32 dst = smem_base + stage * HCT_STAGE_BYTES;
#if HCT_TF32X3
          hct_tma_load_2d(dst, &hct_p.tmap[0], kb * HCT_BK, mb * HCT_BM, full);                    // A hi
          hct_tma_load_2d(dst + HCT_A_BYTES, &hct_p.tmap[1], kb * HCT_BK, mb * HCT_BM, full);      // A lo
          dst += 2 * HCT_A_BYTES;
          hct_tma_load_2d(dst, &hct_p.tmap[2], kb * HCT_BK, nb * HCT_BN, full);                    // B^T hi
          hct_tma_load_2d(dst + HCT_B_BYTES, &hct_p.tmap[3], kb * HCT_BK, nb * HCT_BN, full);      // B^T lo
#else
          hct_tma_load_2d(dst, &hct_p.tmap[0], kb * HCT_BK, mb * HCT_BM, full);
          dst += HCT_A_BYTES;
          for (int j = 0; j < HCT_BN / HCT_NBOX; ++j)
            hct_tma_load_2d(dst + j * HCT_BBOX_BYTES, &hct_p.tmap[1], nb * HCT_BN + j * HCT_NBOX, kb * HCT_BK, full);
#endif
          if (++stage == HCT_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    if (lane == 0) {
      // instruction descriptor: fp32 accumulate, A K-major, B N-major (bf16) or K-major (TF32), M = 128, N = HCT_BN
#if HCT_TF32X3
      const hct_u32 idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((hct_u32)(HCT_BN >> 3) << 17) | ((hct_u32)(HCT_BM >> 4) << 24);
#else
      const hct_u32 idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((hct_u32)(HCT_BN >> 3) << 17) | ((hct_u32)(HCT_BM >> 4) << 24);
#endif
      int stage = 0, acc = 0;
      hct_u32 phase = 0, acc_phase = 0;
      for (long long item = blockIdx.x; item < HCT_ITEMS; item += gridDim.x) {
       const int ch_lo = (int)(item % HCT_KSPLIT) * HCT_CPP, ch_hi = ch_lo + HCT_CPP < HCT_NCH ? ch_lo + HCT_CPP : HCT_NCH;
       for (int ch = ch_lo; ch < ch_hi; ++ch) {
        hct_mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, &failed, status, 2);
        hct_tc_fence_after();
        const hct_u32 d_tmem = tmem_base + acc * HCT_BN;
        const int kb0 = ch * HCT_KBC, kb1 = kb0 + HCT_KBC < HCT_KB ? kb0 + HCT_KBC : HCT_KB;
        for (int kb = kb0; kb < kb1; ++kb) {
          hct_mbar_wait(full0 + 8 * stage, phase, &failed, status, 3);
          hct_tc_fence_after();
          const hct_u32 a_addr = smem_base + stage * HCT_STAGE_BYTES;
#if HCT_TF32X3
          const hct_u32 b_addr = a_addr + 2 * HCT_A_BYTES;
          const hct_u64 a_desc0 = hct_smem_desc(a_addr, 16, 1024), b_desc0 = hct_smem_desc(b_addr, 16, 1024);
#pragma unroll
          for (int kk = 0; kk < HCT_BK / HCT_UMMA_K; ++kk) {
            // both operands K-major: one MMA step is 32 bytes further along the swizzled rows
            // descriptors differ from the stage's first one only in the start-address field (16-byte units)
            const hct_u64 a_hi = a_desc0 + kk * 2, a_lo = a_desc0 + (HCT_A_BYTES >> 4) + kk * 2;
            const hct_u64 b_hi = b_desc0 + kk * 2, b_lo = b_desc0 + (HCT_B_BYTES >> 4) + kk * 2;
            // small cross terms first, then the leading product
            hct_mma_tf32(d_tmem, a_lo, b_hi, idesc, (kb > kb0) || (kk != 0));
            hct_mma_tf32(d_tmem, a_hi, b_lo, idesc, 1);
            hct_mma_tf32(d_tmem, a_hi, b_hi, idesc, 1);
          }
#else
          const hct_u32 b_addr = a_addr + HCT_A_BYTES;
          // descriptors differ from the stage's first one only in the start-address field (16-byte units)
          const hct_u64 a_desc0 = hct_smem_desc(a_addr, 16, 1024), b_desc0 = hct_smem_desc(b_addr, HCT_BBOX_BYTES, 1024);
#pragma unroll
          for (int kk = 0; kk < HCT_BK / HCT_UMMA_K; ++kk) {
            hct_mma_f16(d_tmem, a_desc0 + kk * 2, b_desc0 + kk * (2048 >> 4), idesc, (kb > kb0) || (kk != 0));
          }
#endif
          hct_mma_commit(empty0 + 8 * stage);   // frees the stage once these MMAs have read it
          if (++stage == HCT_STAGES) { stage = 0; phase ^= 1u; }
        }
        hct_mma_commit(tfull0 + 8 * acc);       // this chunk's accumulator is complete
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
       }
      }
    }
  } else {
    // ---------------- epilogue: warp w may only touch TMEM lanes 32 (w mod 4) .. +31
    const int q = warp & 3;
    int acc = 0;
    hct_u32 acc_phase = 0;
    for (long long item = blockIdx.x; item < HCT_ITEMS; item += gridDim.x) {
      const long long tile = item / HCT_KSPLIT;
      const int nb = (int)(tile % HCT_NB), mb = (int)(tile / HCT_NB);
      const long long row = (long long)mb * HCT_BM + q * 32 + lane;
#if HCT_NCH_IS_ONE
      hct_mbar_wait(tfull0 + 8 * acc, acc_phase, &failed, status, 4);
      hct_tc_fence_after();
#pragma unroll 1
      for (int c = 0; c < HCT_BN / 32; ++c) {
        float v[32];
        hct_tmem_ld32(tmem_base + ((hct_u32)(q * 32) << 16) + acc * HCT_BN + c * 32, v);
        const long long col0 = (long long)nb * HCT_BN + c * 32;
        const int ncols = (int)(HCT_N - col0 < 32 ? HCT_N - col0 : 32);
        if (row < HCT_M && ncols > 0) hct_epilogue_run(hct_p, v, row, (int)col0, ncols);
      }
      hct_tc_fence_before();
      hct_mbar_arrive(tempty0 + 8 * acc);
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
#else
      // this warp's share of the columns: NCW chunks of 32 starting at chunk c0
      constexpr int NCW = HCT_BN / 32 / (HCT_EPI_WARPS / 4);
      const int c0 = ((warp - 2) >> 2) * NCW;
      float sum[NCW * 32];
#pragma unroll
      for (int j = 0; j < NCW * 32; ++j) sum[j] = 0.0f;
      const int ch_lo = (int)(item % HCT_KSPLIT) * HCT_CPP, ch_hi = ch_lo + HCT_CPP < HCT_NCH ? ch_lo + HCT_CPP : HCT_NCH;
#pragma unroll 1
      for (int ch = ch_lo; ch < ch_hi; ++ch) {
        hct_mbar_wait(tfull0 + 8 * acc, acc_phase, &failed, status, 4);
        hct_tc_fence_after();
#pragma unroll
        for (int c = 0; c < NCW; ++c) {
          float v[32];
          hct_tmem_ld32(tmem_base + ((hct_u32)(q * 32) << 16) + acc * HCT_BN + (c0 + c) * 32, v);
#pragma unroll
          for (int j = 0; j < 32; ++j) sum[c * 32 + j] += v[j];
        }
        hct_tc_fence_before();
        hct_mbar_arrive(tempty0 + 8 * acc);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
#if HCT_KSPLIT > 1
      {
        // accumulation tile: 16-byte vector j of chunk c of row r at ((tile * chunks + c) * 8 + j) * 128 + r, so that a
        // warp's access is 512 contiguous bytes; arrival counters follow the tiles
        float4* accbuf = (float4*)hct_p.ptr[HCT_KS_SLOT];
        unsigned* ctr = (unsigned*)(accbuf + HCT_TILES * (HCT_BN / 32) * 8 * HCT_BM);
        float4* mine = accbuf + (tile * (HCT_BN / 32) + c0) * 8 * HCT_BM + q * 32 + lane;
#pragma unroll
        for (int c = 0; c < NCW; ++c)
#pragma unroll
          for (int j = 0; j < 8; ++j)
            atomicAdd(mine + (c * 8 + j) * HCT_BM, make_float4(sum[c * 32 + 4 * j], sum[c * 32 + 4 * j + 1], sum[c * 32 + 4 * j + 2], sum[c * 32 + 4 * j + 3]));
        // the epilogue warps' additions are ordered before the count by the barrier and one thread's fence
        asm volatile("bar.sync 1, %0;" ::"n"(32 * HCT_EPI_WARPS) : "memory");
        if (warp == 2 && lane == 0) {
          __threadfence();
          ks_last = atomicAdd(ctr + tile, 1u) == (unsigned)(HCT_KSPLIT - 1) ? 1 : 0;
          __threadfence();
        }
        asm volatile("bar.sync 1, %0;" ::"n"(32 * HCT_EPI_WARPS) : "memory");
        const bool last = *(volatile int*)&ks_last != 0;
        if (last) {
#pragma unroll
          for (int c = 0; c < NCW; ++c)
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const float4 a = __ldcg(mine + (c * 8 + j) * HCT_BM);
              sum[c * 32 + 4 * j] = a.x; sum[c * 32 + 4 * j + 1] = a.y; sum[c * 32 + 4 * j + 2] = a.z; sum[c * 32 + 4 * j + 3] = a.w;
            }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(32 * HCT_EPI_WARPS) : "memory");   // ks_last may be written again
        if (!last) continue;
      }
#endif
#pragma unroll
      for (int c = 0; c < NCW; ++c) {
        const long long col0 = (long long)nb * HCT_BN + (c0 + c) * 32;
        const int ncols = (int)(HCT_N - col0 < 32 ? HCT_N - col0 : 32);
        if (row < HCT_M && ncols > 0) hct_epilogue_run(hct_p, *(float(*)[32])(sum + c * 32), row, (int)col0, ncols);
      }
#endif
    }
  }
  hct_tc_fence_before();
  __syncthreads();
  if (warp == 1) hct_tmem_dealloc(tmem_base, HCT_TMEM_COLS);
}
