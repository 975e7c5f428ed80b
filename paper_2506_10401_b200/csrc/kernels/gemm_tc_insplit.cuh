// Persistent tensor-core GEMM on fp32 operands that splits them into TF32 head and tail INSIDE the
// kernel: D[M,N] = epilogue(A[M,K] * B[K,N]) in one launch, with no pre-pass and no scratch memory.
// For small problems, where a separate split pass and its launch would cost as much as the product.
//
// Pipeline per 32-deep k step:
//   warp 0     TMA: the raw fp32 tiles A[128 x 32] (128-byte swizzle) and B[32 x HCT_BN] (as [32 k x
//              32 n] boxes, no swizzle) into a ring of raw stages;
//   warps 6-13 split: hi = tf32(x), lo = tf32(x - hi).  A keeps its layout, so its head and tail are
//              written at the offsets they were read from; B is transposed on the way ([n][k], one
//              128-byte row per column, 128-byte swizzle): four 4-byte reads down a raw column, one
//              16-byte write per part.  The results fill a ring of operand stages;
//   warp 1     three TF32 MMAs per 8-deep step (tail x head, head x tail, head x head) into one of two
//              accumulators; at most 128 elements of K accumulate in tensor memory;
//   warps 2-5  add the chunks in registers (round to nearest), apply the generated epilogue, store.
// All hand-offs are mbarriers with bounded waits.
//
// Defined by the generator: HCT_M, HCT_N, HCT_K, HCT_BN (64 or 128), HCT_RSTAGES, HCT_STAGES,
// HCT_STATUS_SLOT, HCT_KERNEL_NAME, HctParams, hct_epilogue_run().
#define HCT_BM 128
#define HCT_BK 32
#define HCT_NS 256                                   // splitter threads
#define HCT_RA_BYTES (HCT_BM * 128)                  // raw A: 128 rows x 32 fp32
#define HCT_RB_BYTES (HCT_BN * 128)                  // raw B: HCT_BN / 32 boxes of [32 k][32 n] fp32
#define HCT_RSTAGE_BYTES (HCT_RA_BYTES + HCT_RB_BYTES)
#define HCT_A_BYTES (HCT_BM * 128)
#define HCT_B_BYTES (HCT_BN * 128)
#define HCT_STAGE_BYTES (2 * HCT_A_BYTES + 2 * HCT_B_BYTES)   // head and tail of both operands
#define HCT_OP_OFF (HCT_RSTAGES * HCT_RSTAGE_BYTES)
#define HCT_KB ((HCT_K + HCT_BK - 1) / HCT_BK)
#define HCT_KBC 4
#define HCT_NCH ((HCT_KB + HCT_KBC - 1) / HCT_KBC)
#define HCT_MB ((HCT_M + HCT_BM - 1) / HCT_BM)
#define HCT_NB ((HCT_N + HCT_BN - 1) / HCT_BN)
#define HCT_TILES ((long long)HCT_MB * HCT_NB)
#define HCT_TMEM_COLS (2 * HCT_BN)


extern "C" __global__ void __launch_bounds__(192 + HCT_NS, 1) HCT_KERNEL_NAME(const __grid_constant__ HctParams hct_p) {
  extern __shared__ unsigned char hct_smem_raw[];
  __shared__ unsigned long long bars[2 * HCT_RSTAGES + 2 * HCT_STAGES + 4];
  __shared__ hct_u32 tmem_holder;
  __shared__ int failed;
  const hct_u32 smem_base = (hct_smem_addr(hct_smem_raw) + 1023u) & ~1023u;
  unsigned char* smem_gen = hct_smem_raw + (smem_base - hct_smem_addr(hct_smem_raw));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned int* status = (unsigned int*)hct_p.ptr[HCT_STATUS_SLOT];
  const hct_u32 rfull0 = hct_smem_addr(&bars[0]), rempty0 = rfull0 + 8 * HCT_RSTAGES;
  const hct_u32 full0 = rempty0 + 8 * HCT_RSTAGES, empty0 = full0 + 8 * HCT_STAGES;
  const hct_u32 tfull0 = empty0 + 8 * HCT_STAGES, tempty0 = tfull0 + 16;

  hct_pdl_launch_dependents();
  if (threadIdx.x == 0) {
    failed = 0;
    for (int s = 0; s < HCT_RSTAGES; ++s) {
      hct_mbar_init(rfull0 + 8 * s, 1);
      hct_mbar_init(rempty0 + 8 * s, HCT_NS / 32);   // one lane of every splitter warp
    }
    for (int s = 0; s < HCT_STAGES; ++s) {
      hct_mbar_init(full0 + 8 * s, HCT_NS);          // every splitter thread
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
  hct_pdl_wait();

  if (warp == 0) {
    // ---------------- TMA producer of raw tiles
    if (lane == 0) {
      int rs = 0;
      hct_u32 rphase = 0;
      for (long long tile = blockIdx.x; tile < HCT_TILES; tile += gridDim.x) {
        const int nb = (int)(tile % HCT_NB), mb = (int)(tile / HCT_NB);
        for (int kb = 0; kb < HCT_KB; ++kb) {
          hct_mbar_wait(rempty0 + 8 * rs, rphase ^ 1u, &failed, status, 1);
          const hct_u32 full = rfull0 + 8 * rs;
          hct_mbar_expect_tx(full, HCT_RSTAGE_BYTES);
          const hct_u32 dst = smem_base + rs * HCT_RSTAGE_BYTES;
          hct_tma_load_2d(dst, &hct_p.tmap[0], kb * HCT_BK, mb * HCT_BM, full);
          for (int j = 0; j < HCT_BN / 32; ++j)
            hct_tma_load_2d(dst + HCT_RA_BYTES + j * 4096, &hct_p.tmap[1], nb * HCT_BN + j * 32, kb * HCT_BK, full);
          if (++rs == HCT_RSTAGES) { rs = 0; rphase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    if (lane == 0) {
      const hct_u32 idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((hct_u32)(HCT_BN >> 3) << 17) | ((hct_u32)(HCT_BM >> 4) << 24);
      int stage = 0, acc = 0;
      hct_u32 phase = 0, acc_phase = 0;
      for (long long tile = blockIdx.x; tile < HCT_TILES; tile += gridDim.x) {
       for (int ch = 0; ch < HCT_NCH; ++ch) {
        hct_mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, &failed, status, 2);
        hct_tc_fence_after();
        const hct_u32 d_tmem = tmem_base + acc * HCT_BN;
        const int kb0 = ch * HCT_KBC, kb1 = kb0 + HCT_KBC < HCT_KB ? kb0 + HCT_KBC : HCT_KB;
        for (int kb = kb0; kb < kb1; ++kb) {
          hct_mbar_wait(full0 + 8 * stage, phase, &failed, status, 3);
          hct_tc_fence_after();
          const hct_u32 a_addr = smem_base + HCT_OP_OFF + stage * HCT_STAGE_BYTES, b_addr = a_addr + 2 * HCT_A_BYTES;
          const hct_u64 a_desc0 = hct_smem_desc(a_addr, 16, 1024), b_desc0 = hct_smem_desc(b_addr, 16, 1024);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const hct_u64 a_hi = a_desc0 + kk * 2, a_lo = a_desc0 + (HCT_A_BYTES >> 4) + kk * 2;
            const hct_u64 b_hi = b_desc0 + kk * 2, b_lo = b_desc0 + (HCT_B_BYTES >> 4) + kk * 2;
            // small cross terms first, then the leading product
            hct_mma_tf32(d_tmem, a_lo, b_hi, idesc, (kb > kb0) || (kk != 0));
            hct_mma_tf32(d_tmem, a_hi, b_lo, idesc, 1);
            hct_mma_tf32(d_tmem, a_hi, b_hi, idesc, 1);
          }
          hct_mma_commit(empty0 + 8 * stage);
          if (++stage == HCT_STAGES) { stage = 0; phase ^= 1u; }
        }
        hct_mma_commit(tfull0 + 8 * acc);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
       }
      }
    }
  } else if (warp < 6) {
    // ---------------- epilogue: warp w may only touch TMEM lanes 32 (w mod 4) .. +31
    const int q = warp & 3;
    int acc = 0;
    hct_u32 acc_phase = 0;
    for (long long tile = blockIdx.x; tile < HCT_TILES; tile += gridDim.x) {
      const int nb = (int)(tile % HCT_NB), mb = (int)(tile / HCT_NB);
      const long long row = (long long)mb * HCT_BM + q * 32 + lane;
      float sum[HCT_BN];
#pragma unroll
      for (int j = 0; j < HCT_BN; ++j) sum[j] = 0.0f;
#pragma unroll 1
      for (int ch = 0; ch < HCT_NCH; ++ch) {
        hct_mbar_wait(tfull0 + 8 * acc, acc_phase, &failed, status, 4);
        hct_tc_fence_after();
#pragma unroll
        for (int c = 0; c < HCT_BN / 32; ++c) {
          float v[32];
          hct_tmem_ld32(tmem_base + ((hct_u32)(q * 32) << 16) + acc * HCT_BN + c * 32, v);
#pragma unroll
          for (int j = 0; j < 32; ++j) sum[c * 32 + j] += v[j];
        }
        hct_tc_fence_before();
        hct_mbar_arrive(tempty0 + 8 * acc);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
#pragma unroll
      for (int c = 0; c < HCT_BN / 32; ++c) {
        const long long col0 = (long long)nb * HCT_BN + c * 32;
        const int ncols = (int)(HCT_N - col0 < 32 ? HCT_N - col0 : 32);
        if (row < HCT_M && ncols > 0) hct_epilogue_run(hct_p, *(float(*)[32])(sum + c * 32), row, (int)col0, ncols);
      }
    }
  } else {
    // ---------------- splitters: raw fp32 tiles -> TF32 head and tail operands
    const int st = threadIdx.x - 192;   // 0 .. HCT_NS-1
    int rs = 0, stage = 0;
    hct_u32 rphase = 0, phase = 0;
    for (long long tile = blockIdx.x; tile < HCT_TILES; tile += gridDim.x) {
      for (int kb = 0; kb < HCT_KB; ++kb) {
        hct_mbar_wait(empty0 + 8 * stage, phase ^ 1u, &failed, status, 5);
        hct_mbar_wait(rfull0 + 8 * rs, rphase, &failed, status, 6);
        const unsigned char* raw = smem_gen + rs * HCT_RSTAGE_BYTES;
        unsigned char* op = smem_gen + HCT_OP_OFF + stage * HCT_STAGE_BYTES;
        // all reads of the raw stage first (they are independent), then the arithmetic and the writes
        // A: same layout in and out, one 16-byte piece at a time
        float4 xa[HCT_RA_BYTES / 16 / HCT_NS];
#pragma unroll
        for (int u = 0; u < HCT_RA_BYTES / 16 / HCT_NS; ++u) xa[u] = *(const float4*)(raw + (st + u * HCT_NS) * 16);
        // B: item = (column n, group of 4 k); a warp covers 32 consecutive columns of one group, so its
        // 4-byte reads run along raw rows and its 16-byte writes land in 8 different swizzle slots per phase
        float xb[HCT_BN * 8 / HCT_NS][4];
#pragma unroll
        for (int u = 0; u < HCT_BN * 8 / HCT_NS; ++u) {
          const int i = st + u * HCT_NS, n = i % HCT_BN, kc = i / HCT_BN;
          const float* src = (const float*)(raw + HCT_RA_BYTES + (n >> 5) * 4096) + (kc * 4) * 32 + (n & 31);
#pragma unroll
          for (int j = 0; j < 4; ++j) xb[u][j] = src[32 * j];
        }
        __syncwarp();
        if (lane == 0) hct_mbar_arrive(rempty0 + 8 * rs);    // the raw stage is in registers: refill it
        if (++rs == HCT_RSTAGES) { rs = 0; rphase ^= 1u; }
#pragma unroll
        for (int u = 0; u < HCT_RA_BYTES / 16 / HCT_NS; ++u) {
          const float4 x = xa[u];
          float4 hi, lo;
          hi.x = hct_to_tf32(x.x); lo.x = hct_to_tf32(x.x - hi.x);
          hi.y = hct_to_tf32(x.y); lo.y = hct_to_tf32(x.y - hi.y);
          hi.z = hct_to_tf32(x.z); lo.z = hct_to_tf32(x.z - hi.z);
          hi.w = hct_to_tf32(x.w); lo.w = hct_to_tf32(x.w - hi.w);
          *(float4*)(op + (st + u * HCT_NS) * 16) = hi;
          *(float4*)(op + HCT_A_BYTES + (st + u * HCT_NS) * 16) = lo;
        }
#pragma unroll
        for (int u = 0; u < HCT_BN * 8 / HCT_NS; ++u) {
          const int i = st + u * HCT_NS, n = i % HCT_BN, kc = i / HCT_BN;
          float4 hi, lo;
          hi.x = hct_to_tf32(xb[u][0]); lo.x = hct_to_tf32(xb[u][0] - hi.x);
          hi.y = hct_to_tf32(xb[u][1]); lo.y = hct_to_tf32(xb[u][1] - hi.y);
          hi.z = hct_to_tf32(xb[u][2]); lo.z = hct_to_tf32(xb[u][2] - hi.z);
          hi.w = hct_to_tf32(xb[u][3]); lo.w = hct_to_tf32(xb[u][3] - hi.w);
          unsigned char* dst = op + 2 * HCT_A_BYTES + n * 128 + ((kc ^ (n & 7)) << 4);
          *(float4*)dst = hi;
          *(float4*)(dst + HCT_B_BYTES) = lo;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> tensor-core reads
        hct_mbar_arrive(full0 + 8 * stage);
        if (++stage == HCT_STAGES) { stage = 0; phase ^= 1u; }
      }
    }
  }
  hct_tc_fence_before();
  __syncthreads();
  if (warp == 1) hct_tmem_dealloc(tmem_base, HCT_TMEM_COLS);
}
