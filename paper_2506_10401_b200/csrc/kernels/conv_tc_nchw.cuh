// Persistent tensor-core conv2d (stride 1, zero padding) that reads the activations straight from
// their NCHW buffer: no layout pre-pass over the input (only the small weight tensor is rearranged
// by a preceding kernel).
//
// GEMM view as in conv_tc_halo: rows (M = 128) = output channels, columns = the pixels of HCT_TH
// output rows at a pitch of HCT_PITCH columns, contraction over (input-channel block, tap).  The
// tensor core wants the contraction axis (channels) contiguous, NCHW has the pixels contiguous,
// and a filter tap is a shift by whole pixels, which shared-memory descriptors can express only
// when a pixel is a whole 128-byte row.  So the pixel operand is re-laid inside the kernel:
//   1. a producer thread copies, per input row and block of 64 channels, a [64 channels x
//      HCT_PITCH pixels] box of the NCHW tensor into a small staging ring (TMA, starting at
//      column 0, so always 16-byte aligned; columns and rows outside the image read zeros);
//   2. eight warps transpose each staged box into the channel-contiguous operand buffer (one
//      128-byte row per pixel, 128-byte swizzle), shifted right by the padding so that position
//      0 of every row is the left zero border;
//   3. the operand buffer of a tile holds HCT_TH + HCT_FR - 1 input rows; tap (r,s) reads it
//      through a descriptor that starts r * HCT_PITCH + s rows later, so every input pixel is
//      fetched from global memory once per tile and serves all HCT_FR * HCT_FS taps.
// Weights ([128 x 64] slice per tap and channel block) stream through their own ring.
// Columns w >= HCT_WO of each pitch are computed and dropped.
//
// Warps: 0 weight producer, 1 MMA issue, 2-5 epilogue, 6 pixel producer, 7-14 transposers.
// When the activations are a graph input (HCT_X_IS_INPUT) only the weight producer and the epilogue
// wait for the preceding kernel (programmatic dependent launch) and the pixel pipeline fills meanwhile.
//
// Flat tiling (HCT_FLAT).  An MMA instruction of this shape takes about the same time whatever its
// width, so what counts is the number of K loops on the busiest CTA.  With tiles of whole output
// rows at a pitch that is a multiple of 32, part of every MMA works on padding columns, and a tile
// count just above a multiple of the grid costs one more K loop.  In flat mode the positions of an
// image are numbered row after row at a pitch of HCT_P = W + 2 * pad (the padded row, no rounding),
// a tile is 256 consecutive positions of one image wherever they start, and the operand buffer holds
// the window of padded input positions under it: tap (r,s) still starts r * HCT_P + s rows later.
// The HCT_P - HCT_WO positions at the end of every row are computed and dropped; the epilogue closes
// the gap they leave, so that the values of a 32-column chunk form one contiguous run of the NCHW
// plane, stages the run in shared memory, and the warp stores it channel by channel (64 contiguous
// bytes per instruction; the run may start at any element, so no vector or TMA store).
//
// Defined by the generator: HCT_NB_IMG, HCT_C, HCT_H, HCT_W, HCT_KO, HCT_FR, HCT_FS, HCT_PAD, HCT_HO, HCT_WO,
// HCT_PITCH, HCT_TH, HCT_TH2 (= 1), HCT_SPLIT, HCT_NA, HCT_NBUF, HCT_NSTG, HCT_X_IS_INPUT, HCT_TMA_STORE, HCT_STATUS_SLOT,
// HCT_KERNEL_NAME, HctParams, hct_epilogue_run() or (HCT_TMA_STORE) hct_epilogue_vals().
#define HCT_BM 128
#define HCT_A_BYTES (HCT_BM * 128)                       // weights: 128 channels x 64 inputs, bf16
#if HCT_FLAT
#define HCT_WIN (256 + (HCT_FR - 1) * HCT_P + HCT_FS - 1)     // padded input positions under a tile of 256 output positions
#define HCT_B_BYTES ((HCT_WIN * 128 + 1023) / 1024 * 1024)
#define HCT_TPI ((HCT_HO * HCT_P + 255) / 256)                // tiles per image
#else
#define HCT_ROWS_MAX (HCT_TH + HCT_FR - 1)               // input rows under a whole tile
#define HCT_B_BYTES (HCT_ROWS_MAX * HCT_PITCH * 128 + 1024)   // operand buffer + room for the shifted reads
#endif
#define HCT_S_BYTES (HCT_PITCH * 128)                    // staging box: 64 channels x pitch pixels
#define HCT_RING_B_OFF (HCT_NA * HCT_A_BYTES)
#define HCT_RING_S_OFF (HCT_RING_B_OFF + HCT_NBUF * HCT_B_BYTES)
#define HCT_RING_O_OFF (HCT_RING_S_OFF + HCT_NSTG * HCT_S_BYTES)   // output staging: 4 warps x 2 slots x 2 KB
#define HCT_CB ((HCT_C + 63) / 64)
#define HCT_HT ((HCT_HO + HCT_TH - 1) / HCT_TH)
#define HCT_MBK ((HCT_KO + HCT_BM - 1) / HCT_BM)
#if HCT_FLAT
#define HCT_FULL_TILES ((long long)HCT_NB_IMG * HCT_TPI * HCT_MBK)
#else
#define HCT_FULL_TILES ((long long)HCT_NB_IMG * HCT_HT * HCT_MBK)
#endif
#define HCT_NT 256                                       // transposer threads
#if HCT_FLAT
#define HCT_EPI2 4                                       // extra epilogue warps (15-18): every lane quarter is drained by two warps
#else
#define HCT_EPI2 0
#endif
#define HCT_NBAR (2 * HCT_NA + 2 * HCT_NBUF + 2 * HCT_NSTG + 4)

#ifndef HCT_KSPLIT
#define HCT_KSPLIT 0
#endif
#if HCT_KSPLIT && HCT_FLAT
#error "the split of the contraction is built for whole-row tiles only"
#endif
#define HCT_KP (HCT_CB * HCT_FR)                         // parts of a contraction split by (channel block, filter row)

// A work item: output rows h0 .. h0 + th - 1 of image n (filters of block mbk), contracted over channel blocks
// cb_lo .. cb_hi - 1 and filter rows r_lo .. r_hi - 1 (a whole tile: all of them).  `ks`: the item is one part of
// a split contraction, piece number q; its partial sums go to scratch and the last part to arrive finishes the row.
struct HctConvTile { int n, h0, th, mbk; bool cut; int o0, lo, nrows; int cb_lo, cb_hi, r_lo, r_hi; bool ks; int q; };

// Tile t of the schedule.  Tiles below `t1` are whole; the rest are pieces of the remaining whole tiles.
__device__ __forceinline__ HctConvTile hct_conv_tile(long long t, long long t1, int ksplit) {
  HctConvTile r;
  r.cb_lo = 0; r.cb_hi = HCT_CB; r.r_lo = 0; r.r_hi = HCT_FR; r.ks = false; r.q = 0;
#if HCT_FLAT
  // tile = 256 consecutive positions of one image; `lo` .. `lo + nrows - 1` are the padded input rows its window meets
  (void)t1; (void)ksplit;
  long long w_ = t;
  r.mbk = (int)(w_ % HCT_MBK); w_ /= HCT_MBK;
  r.o0 = (int)(w_ % HCT_TPI) * 256;
  r.n = (int)(w_ / HCT_TPI);
  r.lo = r.o0 / HCT_P;
  int hi = (r.o0 + HCT_WIN - 1) / HCT_P;
  if (hi > HCT_H + 2 * HCT_PAD - 1) hi = HCT_H + 2 * HCT_PAD - 1;
  r.nrows = hi - r.lo + 1;
  r.h0 = 0; r.th = 1; r.cut = false;
  return r;
#endif
  long long whole = t;
  int sub = 0;
  r.cut = t >= t1;
  if (r.cut && ksplit) {
    // one output row, one (channel block, filter row) part of its contraction
    const long long q = t - t1;
    whole = t1 + q / (HCT_SPLIT * HCT_KP);
    const int rem = (int)(q % (HCT_SPLIT * HCT_KP));
    sub = rem / HCT_KP;
    const int part = rem % HCT_KP;
    r.cb_lo = part / HCT_FR; r.cb_hi = r.cb_lo + 1;
    r.r_lo = part % HCT_FR; r.r_hi = r.r_lo + 1;
    r.ks = true; r.q = (int)q;
  } else if (r.cut) {
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

#if HCT_FLAT
// Epilogue of one 32-column chunk of a flat tile (columns 32 c .. 32 c + 31 of the accumulator at `taddr`), by one
// warp whose lanes own output channels q * 32 + lane.  Positions oc .. oc + 31 of the image hold n1 valid ones up
// to the end of output row `hrow`, then `skip` dropped ones (the padding columns of that row), then valid ones of
// the next row: the gap is closed, the run staged in `o_slot` (2 KB of shared memory), and stored channel by channel.
__device__ __forceinline__ void hct_flat_chunk(const HctParams& hct_p, const HctConvTile& t, hct_u32 taddr, int c, int q, int lane, hct_u32 o_slot) {
  const int oc = t.o0 + c * 32;
  if (oc >= HCT_HO * HCT_P) return;
  const int hrow = oc / HCT_P, a = oc - hrow * HCT_P;
  const int n1 = a < HCT_WO ? (HCT_WO - a < 32 ? HCT_WO - a : 32) : 0;
  const int jend = HCT_P - a < 32 ? HCT_P - a : 32;
  const int skip = jend - n1;
  const int run = n1 + (hrow + 1 < HCT_HO ? 32 - jend : 0);
  if (run == 0) return;
  const int idx0 = hrow * HCT_WO + (a < HCT_WO ? a : HCT_WO);     // index of the run's first element in its plane
  const int k = t.mbk * HCT_BM + q * 32 + lane;                    // output channel of this thread's TMEM lane
  float v[32], w[32];
  hct_tmem_ld32(taddr + c * 32, v);
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    float x = v[j];
#pragma unroll
    for (int g = 1; g <= HCT_P - HCT_WO; ++g)
      if (j + g < 32) x = (skip == g && j >= n1) ? v[j + g < 32 ? j + g : 31] : x;
    w[j] = x;
  }
  float o[32];
  if (k < HCT_KO) {
    hct_epilogue_vals(hct_p, w, (long long)t.n * HCT_KO + k, idx0, run, o);
  } else {
#pragma unroll
    for (int j = 0; j < 32; ++j) o[j] = 0.0f;
  }
  // rows of 64 bytes (one channel each), 16-byte piece j of row i at piece j ^ ((i >> 1) & 3)
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const hct_u32 dst = o_slot + (hct_u32)lane * 64u + (((hct_u32)j ^ (((hct_u32)lane >> 1) & 3u)) << 4);
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(hct_pack_bf16x2(o[8 * j], o[8 * j + 1])),
                 "r"(hct_pack_bf16x2(o[8 * j + 2], o[8 * j + 3])), "r"(hct_pack_bf16x2(o[8 * j + 4], o[8 * j + 5])),
                 "r"(hct_pack_bf16x2(o[8 * j + 6], o[8 * j + 7]))
                 : "memory");
  }
  __syncwarp();
  const int kbase = t.mbk * HCT_BM + q * 32;
  hct_bf16_t* ybase = (hct_bf16_t*)hct_p.ptr[HCT_OUT_SLOT] + ((long long)t.n * HCT_KO + kbase) * (long long)(HCT_HO * HCT_WO) + idx0;
#if HCT_P % 2 == 0 && HCT_WO % 2 == 0
  // every run starts at an even element and has an even length: two elements per lane, two channels per instruction
  {
    const int pp = lane & 15, ro = lane >> 4;
    if (2 * pp < run) {
#pragma unroll 8
      for (int i = 0; i < 16; ++i) {
        const int ch = 2 * i + ro;
        if (kbase + ch < HCT_KO) {
          hct_u32 e_;
          asm volatile("ld.shared.b32 %0, [%1];" : "=r"(e_) : "r"(o_slot + (hct_u32)ch * 64u + ((((hct_u32)pp >> 2) ^ (((hct_u32)ch >> 1) & 3u)) << 4) + ((hct_u32)pp & 3u) * 4u) : "memory");
          *(hct_u32*)(ybase + (long long)ch * (HCT_HO * HCT_WO) + 2 * pp) = e_;
        }
      }
    }
  }
#else
  if (lane < run) {   // lane = element of the run
    const hct_u32 src0 = o_slot + ((hct_u32)lane & 7u) * 2u;
#pragma unroll 8
    for (int i = 0; i < 32; ++i) {
      if (kbase + i < HCT_KO) {
        unsigned short e_;
        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(e_) : "r"(src0 + (hct_u32)i * 64u + ((((hct_u32)lane >> 3) ^ (((hct_u32)i >> 1) & 3u)) << 4)) : "memory");
        ybase[(long long)i * (HCT_HO * HCT_WO) + lane] = e_;
      }
    }
  }
#endif
  __syncwarp();
}
#endif

extern "C" __global__ void __launch_bounds__(224 + HCT_NT + 32 * HCT_EPI2, 1) HCT_KERNEL_NAME(const __grid_constant__ HctParams hct_p) {
  extern __shared__ unsigned char hct_smem_raw[];
  __shared__ unsigned long long bars[HCT_NBAR];
  __shared__ hct_u32 tmem_holder;
  __shared__ int failed;
#if HCT_KSPLIT
  __shared__ int ks_last;
#endif
  const hct_u32 smem_base = (hct_smem_addr(hct_smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned int* status = (unsigned int*)hct_p.ptr[HCT_STATUS_SLOT];
  const hct_u32 afull0 = hct_smem_addr(&bars[0]), aempty0 = afull0 + 8 * HCT_NA;
  const hct_u32 bfull0 = aempty0 + 8 * HCT_NA, bempty0 = bfull0 + 8 * HCT_NBUF;
  const hct_u32 sfull0 = bempty0 + 8 * HCT_NBUF, sempty0 = sfull0 + 8 * HCT_NSTG;
  const hct_u32 tfull0 = sempty0 + 8 * HCT_NSTG, tempty0 = tfull0 + 16;

  // schedule: whole tiles for as many full rounds over the grid as there are, the rest cut in pieces
  // A short last round is spread over the grid by output row; with HCT_KSPLIT also by part of the
  // contraction, when the pieces fit the grid and the scratch slices (a piece then costs a few MMA
  // instructions instead of a whole K loop, but its partial sums travel through scratch).
  long long t1 = HCT_FULL_TILES, n_tiles = HCT_FULL_TILES;
  int ksplit = 0;
  {
    const long long rest = HCT_FULL_TILES % gridDim.x;
#if HCT_KSPLIT
    const long long pieces = rest * HCT_SPLIT * HCT_KP;
    if (rest > 0 && HCT_KP > 1 && pieces <= (long long)gridDim.x && pieces <= HCT_KS_MAX) {
      t1 = HCT_FULL_TILES - rest;
      n_tiles = t1 + pieces;
      ksplit = 1;
    } else
#endif
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
      hct_mbar_init(bfull0 + 8 * s, HCT_NT);   // every transposer thread
      hct_mbar_init(bempty0 + 8 * s, 1);
    }
    for (int s = 0; s < HCT_NSTG; ++s) {
      hct_mbar_init(sfull0 + 8 * s, 1);
      hct_mbar_init(sempty0 + 8 * s, HCT_NT / 32);    // one lane of every transposer warp
    }
    for (int a = 0; a < 2; ++a) {
      hct_mbar_init(tfull0 + 8 * a, 1);
      hct_mbar_init(tempty0 + 8 * a, 128 + 32 * HCT_EPI2);
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

  if (warp == 0) {
    // ---- weights: one [128 x 64] slice per (channel block, tap), in the order the MMA warp consumes them
    if (lane == 0) {
      hct_pdl_wait();   // the rearranged weights are written by the preceding kernel
      int sa = 0;
      hct_u32 pa = 0;
      for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const HctConvTile t = hct_conv_tile(tile, t1, ksplit);
        if (t.th == 0) continue;
        for (int cb = t.cb_lo; cb < t.cb_hi; ++cb)
          for (int tap = t.r_lo * HCT_FS; tap < t.r_hi * HCT_FS; ++tap) {
            hct_mbar_wait(aempty0 + 8 * sa, pa ^ 1u, &failed, status, 5);
            hct_mbar_expect_tx(afull0 + 8 * sa, HCT_A_BYTES);
            hct_tma_load_2d(smem_base + sa * HCT_A_BYTES, &hct_p.tmap[0], cb * 64, tap * HCT_KO + t.mbk * HCT_BM, afull0 + 8 * sa);
            if (++sa == HCT_NA) { sa = 0; pa ^= 1u; }
          }
      }
    }
  } else if (warp == 1) {
    // ---- MMA issue
    if (lane == 0) {
      int sa = 0, sb = 0, acc = 0;
      hct_u32 pa = 0, pb = 0, acc_phase = 0;
      for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const HctConvTile t = hct_conv_tile(tile, t1, ksplit);
        if (t.th == 0) continue;
        // bf16 x bf16 -> fp32, both operands K-major, M = 128, N = rows of this tile times the pitch
#if HCT_FLAT
        const hct_u32 n_mma = 256u;
#else
        const hct_u32 n_mma = (hct_u32)(t.th * HCT_PITCH);
#endif
        const hct_u32 idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((n_mma >> 3) << 17) | ((hct_u32)(HCT_BM >> 4) << 24);
        hct_mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, &failed, status, 2);
        hct_tc_fence_after();
        const hct_u32 d_tmem = tmem_base + acc * 256;
        for (int cb = t.cb_lo; cb < t.cb_hi; ++cb) {
          hct_mbar_wait(bfull0 + 8 * sb, pb, &failed, status, 3);
          hct_tc_fence_after();
          const hct_u32 b_addr = smem_base + HCT_RING_B_OFF + sb * HCT_B_BYTES;
          for (int r = t.r_lo; r < t.r_hi; ++r)
            for (int s = 0; s < HCT_FS; ++s) {
              hct_mbar_wait(afull0 + 8 * sa, pa, &failed, status, 6);
              hct_tc_fence_after();
              // tap (r,s) reads the operand buffer r * pitch + s pixel rows (128 bytes each) further on; the
              // 128-byte swizzle follows the absolute shared-memory address, so only the start field changes
              const hct_u64 a_desc0 = hct_smem_desc(smem_base + sa * HCT_A_BYTES, 16, 1024);
#if HCT_FLAT
              const hct_u64 b_desc0 = hct_smem_desc(b_addr + (r * HCT_P + s) * 128, 16, 1024);
#else
              const hct_u64 b_desc0 = hct_smem_desc(b_addr + ((r - t.r_lo) * HCT_PITCH + s) * 128, 16, 1024);   // the buffer starts at input row h0 - pad + r_lo
#endif
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) hct_mma_f16(d_tmem, a_desc0 + kk * 2, b_desc0 + kk * 2, idesc, ((cb - t.cb_lo) | (r - t.r_lo) | s | kk) != 0);
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
  } else if (warp < 6 || warp >= 15) {
    // ---- epilogue: one output channel per thread, 32 consecutive pixels per step
    const int q = warp & 3;
    int acc = 0;
    hct_u32 acc_phase = 0;
#if HCT_TMA_STORE
    unsigned ostep = 0;
#endif
    hct_pdl_wait();   // epilogue operands may come from earlier kernels of the graph
    for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
      const HctConvTile t = hct_conv_tile(tile, t1, ksplit);
      if (t.th == 0) continue;
      hct_mbar_wait(tfull0 + 8 * acc, acc_phase, &failed, status, 4);
      hct_tc_fence_after();
      const int k = t.mbk * HCT_BM + q * 32 + lane;      // output channel of this thread's TMEM lane
#if HCT_FLAT
      // chunks of this lane quarter are shared by its two epilogue warps; on the CTA's last tile, whose epilogue
      // nothing overlaps, the two transposer warps of the quarter (idle by then) take a share as well
      const bool last_tile = tile + gridDim.x >= n_tiles;
      const int part = warp >= 15 ? 1 : 0;
#pragma unroll 1
      for (int c = part; c < 8; c += last_tile ? 4 : 2)
        hct_flat_chunk(hct_p, t, tmem_base + ((hct_u32)(q * 32) << 16) + acc * 256, c, q, lane, smem_base + HCT_RING_O_OFF + (hct_u32)((q * 2 + part) * 2048));
#else
      // values of one 32-column chunk (row h0 + hh, columns part * 32 ..) -> elementwise consumers -> store
      auto finish = [&](float (&v)[32], int hh, int part, int ncols) {
#if HCT_TMA_STORE
        // The 32 channels x 32 pixels of this warp leave through shared memory and one TMA store (columns
        // past WO and channels past KO are clipped by the copy).  Row = channel (64 bytes), 64-byte swizzle:
        // 16-byte piece j of row i sits at piece j ^ ((i >> 1) & 3), which also keeps the writes of
        // neighbouring lanes in different banks.  Two slots per warp: a slot is rewritten only after the
        // store issued from it two steps ago has read it.
        float o[32];
        if (k < HCT_KO) {
          hct_epilogue_vals(hct_p, v, (long long)t.n * HCT_KO + k, (t.h0 + hh) * HCT_WO + part * 32, ncols, o);
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) o[j] = 0.0f;
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        __syncwarp();
        const hct_u32 o_slot = smem_base + HCT_RING_O_OFF + (hct_u32)((q * 2 + (ostep & 1)) * 2048);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const hct_u32 dst = o_slot + (hct_u32)lane * 64u + (((hct_u32)j ^ (((hct_u32)lane >> 1) & 3u)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(hct_pack_bf16x2(o[8 * j], o[8 * j + 1])),
                       "r"(hct_pack_bf16x2(o[8 * j + 2], o[8 * j + 3])), "r"(hct_pack_bf16x2(o[8 * j + 4], o[8 * j + 5])),
                       "r"(hct_pack_bf16x2(o[8 * j + 6], o[8 * j + 7]))
                       : "memory");
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4}], [%5];" ::"l"(&hct_p.tmap[2]),
                       "r"(part * 32), "r"(t.h0 + hh), "r"(t.mbk * HCT_BM + q * 32), "r"(t.n), "r"(o_slot)
                       : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        ++ostep;
#else
        if (k < HCT_KO) hct_epilogue_run(hct_p, v, (long long)t.n * HCT_KO + k, (t.h0 + hh) * HCT_WO + part * 32, ncols);
#endif
      };
#if HCT_KSPLIT
      if (t.ks) {
        // Part of a split contraction (one output row).  The partial sums go to this piece's scratch slice
        // (128 channels x pitch fp32); a counter per row tells the last part to arrive, whose CTA adds the
        // slices in part order (so the result does not depend on the order of arrival) and finishes the row.
        unsigned* ctr = (unsigned*)hct_p.ptr[HCT_KS_SLOT];
        float* slices = (float*)(ctr + HCT_KS_CTRS);
        const int m = q * 32 + lane;
#pragma unroll 1
        for (int part = 0; part < HCT_PITCH / 32; ++part) {
          if (HCT_WO - part * 32 <= 0) continue;
          float v[32];
          hct_tmem_ld32(tmem_base + ((hct_u32)(q * 32) << 16) + acc * 256 + part * 32, v);
          // slice layout [chunk][group of 4 columns][channel][4]: a warp's 16-byte accesses are 512 contiguous bytes
          float4* dst = (float4*)(slices + (long long)t.q * (HCT_BM * HCT_PITCH)) + (part * 8) * HCT_BM + m;
#pragma unroll
          for (int j = 0; j < 8; ++j) __stcg(dst + j * HCT_BM, make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]));
        }
        hct_tc_fence_before();
        hct_mbar_arrive(tempty0 + 8 * acc);
        // the four warps' stores are ordered before the counter update by the barrier and one thread's fence
        // (fences are cumulative); the last part's reads follow the update in the same way
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (warp == 2 && lane == 0) {
          __threadfence();
          ks_last = atomicAdd(ctr + t.q / HCT_KP, 1u) == (unsigned)(HCT_KP - 1) ? 1 : 0;
          __threadfence();
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (*(volatile int*)&ks_last) {
          const int q0 = t.q - t.q % HCT_KP;
#pragma unroll 1
          for (int part = 0; part < HCT_PITCH / 32; ++part) {
            const int ncols = HCT_WO - part * 32 < 32 ? HCT_WO - part * 32 : 32;
            if (ncols <= 0) continue;
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = 0.0f;
#pragma unroll 1
            for (int pp = 0; pp < HCT_KP; ++pp) {
              const float4* src = (const float4*)(slices + (long long)(q0 + pp) * (HCT_BM * HCT_PITCH)) + (part * 8) * HCT_BM + m;
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const float4 a = __ldcg(src + j * HCT_BM);
                v[4 * j] += a.x; v[4 * j + 1] += a.y; v[4 * j + 2] += a.z; v[4 * j + 3] += a.w;
              }
            }
            finish(v, 0, part, ncols);
          }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");   // ks_last may be written again
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
        continue;
      }
#endif
      const int chunks = t.th * (HCT_PITCH / 32);
#pragma unroll 1
      for (int c = 0; c < chunks; ++c) {
        const int hh = c / (HCT_PITCH / 32), part = c % (HCT_PITCH / 32);
        const int ncols = HCT_WO - part * 32 < 32 ? HCT_WO - part * 32 : 32;   // columns past WO are padding
        if (ncols <= 0) continue;
        float v[32];
        hct_tmem_ld32(tmem_base + ((hct_u32)(q * 32) << 16) + acc * 256 + c * 32, v);
        finish(v, hh, part, ncols);
      }
#endif   // HCT_FLAT
      hct_tc_fence_before();
      hct_mbar_arrive(tempty0 + 8 * acc);
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
#if HCT_TMA_STORE
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all stores done before the CTA ends
#endif
  } else if (warp == 6) {
    // ---- pixels: one staged box per (channel block, input row)
    if (lane == 0) {
#if !HCT_X_IS_INPUT
      hct_pdl_wait();   // the activations are an earlier kernel's result
#endif
      int ss = 0;
      hct_u32 ps = 0;
      for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const HctConvTile t = hct_conv_tile(tile, t1, ksplit);
        if (t.th == 0) continue;
#if HCT_FLAT
        const int nrows = t.nrows, row0 = t.lo - HCT_PAD;
#else
        const int nrows = t.th + (t.r_hi - t.r_lo) - 1, row0 = t.h0 - HCT_PAD + t.r_lo;
#endif
        for (int cb = t.cb_lo; cb < t.cb_hi; ++cb)
          for (int rr = 0; rr < nrows; ++rr) {
            hct_mbar_wait(sempty0 + 8 * ss, ps ^ 1u, &failed, status, 7);
            hct_mbar_expect_tx(sfull0 + 8 * ss, HCT_S_BYTES);
            hct_tma_load_4d(smem_base + HCT_RING_S_OFF + ss * HCT_S_BYTES, &hct_p.tmap[1], 0, row0 + rr, cb * 64, t.n, sfull0 + 8 * ss);
            if (++ss == HCT_NSTG) { ss = 0; ps ^= 1u; }
          }
      }
    }
  } else {
    // ---- transposers: staged [channel][pixel] box -> operand rows [pixel][channel], shifted by the padding
    const int tt = threadIdx.x - 224;    // 0 .. HCT_NT-1
    const unsigned char* smem_gen = hct_smem_raw + (smem_base - hct_smem_addr(hct_smem_raw));   // generic view of smem_base
#if !HCT_FLAT
    // the left border (positions below the padding) is never written again: zero it once in every buffer
    for (int i = tt; i < HCT_NBUF * HCT_ROWS_MAX * HCT_PAD * 8; i += HCT_NT) {
      const int unit = i & 7, rest = i >> 3;
      const int pos = rest % (HCT_PAD > 0 ? HCT_PAD : 1), rowi = rest / (HCT_PAD > 0 ? HCT_PAD : 1);
      const int buf = rowi / HCT_ROWS_MAX, rr = rowi % HCT_ROWS_MAX;
      *(uint4*)(smem_gen + HCT_RING_B_OFF + buf * HCT_B_BYTES + (rr * HCT_PITCH + pos) * 128 + unit * 16) = make_uint4(0u, 0u, 0u, 0u);
    }
#endif
    int ss = 0, sb = 0;
    hct_u32 ps = 0, pb = 0;
    for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
      const HctConvTile t = hct_conv_tile(tile, t1, ksplit);
      if (t.th == 0) continue;
#if HCT_FLAT
      const int nrows = t.nrows;
#else
      const int nrows = t.th + (t.r_hi - t.r_lo) - 1;
#endif
      for (int cb = t.cb_lo; cb < t.cb_hi; ++cb) {
        hct_mbar_wait(bempty0 + 8 * sb, pb ^ 1u, &failed, status, 1);
        unsigned char* b_gen = (unsigned char*)smem_gen + HCT_RING_B_OFF + sb * HCT_B_BYTES;
        for (int rr = 0; rr < nrows; ++rr) {
          hct_mbar_wait(sfull0 + 8 * ss, ps, &failed, status, 8);
          const unsigned char* s_gen = smem_gen + HCT_RING_S_OFF + ss * HCT_S_BYTES;
#if HCT_FLAT
          // position of this padded row's first column in the window (may lie before it); the columns left of
          // the image are zero, the ones right of it arrive as zeros in the staged box
          const int rowbase = (t.lo + rr) * HCT_P - t.o0;
          if (tt < 8 * HCT_PAD) {
            const int q0 = rowbase + (tt >> 3);
            if (q0 >= 0 && q0 < HCT_WIN) *(uint4*)(b_gen + (hct_u32)q0 * 128u + (((hct_u32)(tt & 7) ^ ((hct_u32)q0 & 7u)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
          }
#endif
          // work item = (pair of neighbouring pixels, group of 8 channels): eight 4-byte reads along the staged
          // channel rows give both pixels; each pixel's 8 channels leave as one 16-byte write into its row.
          // A warp shares the channel group and covers 32 consecutive pairs; half of every 8 lanes writes its
          // odd pixel first, so that the 8 rows of a write phase differ in (row mod 8) and miss each other's banks.
#pragma unroll
          for (int i0 = 0; i0 < HCT_PITCH * 4; i0 += HCT_NT) {
            const int it = i0 + tt;
            if (HCT_PITCH * 4 % HCT_NT != 0 && it >= HCT_PITCH * 4) break;
            const int m = it % (HCT_PITCH / 2), u = it / (HCT_PITCH / 2);
#if HCT_FLAT
            if (rowbase + 2 * m + HCT_PAD + 1 < 0 || rowbase + 2 * m + HCT_PAD >= HCT_WIN || 2 * m + HCT_PAD >= HCT_P) continue;
#endif
            const hct_u32* src = (const hct_u32*)(s_gen + ((u * 8) * HCT_PITCH + 2 * m) * 2);
            hct_u32 e[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) e[j] = src[j * (HCT_PITCH / 2)];
            uint4 lo, hi;   // lo: pixel 2m, hi: pixel 2m + 1
            lo.x = __byte_perm(e[0], e[1], 0x5410); hi.x = __byte_perm(e[0], e[1], 0x7632);
            lo.y = __byte_perm(e[2], e[3], 0x5410); hi.y = __byte_perm(e[2], e[3], 0x7632);
            lo.z = __byte_perm(e[4], e[5], 0x5410); hi.z = __byte_perm(e[4], e[5], 0x7632);
            lo.w = __byte_perm(e[6], e[7], 0x5410); hi.w = __byte_perm(e[6], e[7], 0x7632);
            const bool odd_first = (m & 4) != 0;
            const int pos_a = 2 * m + HCT_PAD + (odd_first ? 1 : 0), pos_b = 2 * m + HCT_PAD + (odd_first ? 0 : 1);
#if HCT_FLAT
            const int qa_ = rowbase + pos_a, qb_ = rowbase + pos_b;
            const hct_u32 qa = (hct_u32)qa_, qb = (hct_u32)qb_;
            if (pos_a < HCT_P && qa_ >= 0 && qa_ < HCT_WIN) *(uint4*)(b_gen + qa * 128u + (((hct_u32)u ^ (qa & 7u)) << 4)) = odd_first ? hi : lo;
            if (pos_b < HCT_P && qb_ >= 0 && qb_ < HCT_WIN) *(uint4*)(b_gen + qb * 128u + (((hct_u32)u ^ (qb & 7u)) << 4)) = odd_first ? lo : hi;
#else
            const hct_u32 qa = (hct_u32)(rr * HCT_PITCH + pos_a), qb = (hct_u32)(rr * HCT_PITCH + pos_b);
            if (pos_a < HCT_PITCH) *(uint4*)(b_gen + qa * 128u + (((hct_u32)u ^ (qa & 7u)) << 4)) = odd_first ? hi : lo;
            if (pos_b < HCT_PITCH) *(uint4*)(b_gen + qb * 128u + (((hct_u32)u ^ (qb & 7u)) << 4)) = odd_first ? lo : hi;
#endif
          }
          __syncwarp();
          if (lane == 0) hct_mbar_arrive(sempty0 + 8 * ss);
          if (++ss == HCT_NSTG) { ss = 0; ps ^= 1u; }
        }
        // make the generic-proxy writes visible to the tensor core's (async-proxy) reads
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        hct_mbar_arrive(bfull0 + 8 * sb);
        if (++sb == HCT_NBUF) { sb = 0; pb ^= 1u; }
      }
    }
#if HCT_FLAT
    // Nothing is left to transpose: take a share of the last tile's epilogue (chunks 2 and 6, or 3 and 7, of this
    // warp's lane quarter), staged in the idle pixel ring.  The tile's accumulator and the phase of its barrier
    // follow from how many tiles this CTA has worked on.
    if ((long long)blockIdx.x < n_tiles) {
      const long long ntl = (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x;
      const HctConvTile t = hct_conv_tile(blockIdx.x + (ntl - 1) * gridDim.x, t1, ksplit);
      const int acc_l = (int)((ntl - 1) & 1);
      const hct_u32 phase_l = (hct_u32)(((ntl - 1) >> 1) & 1);
      const int q = warp & 3, part = 2 + ((warp - 7) >> 2);
      hct_mbar_wait(tfull0 + 8 * acc_l, phase_l, &failed, status, 9);
      hct_tc_fence_after();
#pragma unroll 1
      for (int c = part; c < 8; c += 4)
        hct_flat_chunk(hct_p, t, tmem_base + ((hct_u32)(q * 32) << 16) + acc_l * 256, c, q, lane, smem_base + HCT_RING_S_OFF + (hct_u32)((q * 2 + part - 2) * 2048));
    }
#endif
  }
  hct_tc_fence_before();
  __syncthreads();
  if (warp == 1) hct_tmem_dealloc(tmem_base, 512);
}
