// Building blocks for the tensor-core kernels: mbarriers with bounded waits, TMA tile loads,
// tcgen05 (5th-generation tensor core) issue, commit, and tensor-memory access.
struct alignas(64) HctTensorMap { unsigned long long opaque[16]; };

__device__ __forceinline__ hct_u32 hct_smem_addr(const void* p) { return (hct_u32)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void hct_mbar_init(hct_u32 bar, hct_u32 count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void hct_mbar_expect_tx(hct_u32 bar, hct_u32 bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void hct_mbar_arrive(hct_u32 bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool hct_mbar_try(hct_u32 bar, hct_u32 parity) {
  hct_u32 ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  When the limit is reached the kernel records where it gave up in the status word,
// raises a CTA-wide flag that makes every later wait return at once, and carries on: all loops
// have fixed trip counts, so the CTA still reaches its end and releases what it holds.
#ifndef HCT_WAIT_LIMIT
#define HCT_WAIT_LIMIT (1u << 24)
#endif
__device__ __forceinline__ void hct_mbar_wait(hct_u32 bar, hct_u32 parity, volatile int* failed, unsigned int* status, unsigned where) {
  if (hct_mbar_try(bar, parity)) return;
  for (unsigned it = 0; it < HCT_WAIT_LIMIT; ++it) {
    if (hct_mbar_try(bar, parity)) return;
    if (*failed) return;
    if (it > 64) __nanosleep(20);
  }
  *failed = 1;
  if (status) {
    atomicCAS(status, 0u, 1u);
    status[1] = where;
  }
}

__device__ __forceinline__ void hct_tma_load_2d(hct_u32 dst, const HctTensorMap* map, int c0, int c1, hct_u32 bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"(map), "r"(c0), "r"(c1), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void hct_tma_load_4d(hct_u32 dst, const HctTensorMap* map, int c0, int c1, int c2, int c3, hct_u32 bar) {
  asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst),
               "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void hct_prefetch_tmap(const HctTensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// ---- tensor memory
__device__ __forceinline__ void hct_tmem_alloc(hct_u32 holder_smem, hct_u32 ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void hct_tmem_dealloc(hct_u32 taddr, hct_u32 ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void hct_tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void hct_tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]; issued by one thread for the whole CTA
__device__ __forceinline__ void hct_mma_f16(hct_u32 d_tmem, hct_u64 adesc, hct_u64 bdesc, hct_u32 idesc, hct_u32 accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void hct_mma_tf32(hct_u32 d_tmem, hct_u64 adesc, hct_u64 bdesc, hct_u32 idesc, hct_u32 accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Makes `bar` complete once every MMA issued so far by this thread has finished.
__device__ __forceinline__ void hct_mma_commit(hct_u32 bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i of the warp receives row (lane base + i)
__device__ __forceinline__ void hct_tmem_ld32(hct_u32 taddr, float* v) {
  hct_u32 r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory operand descriptor, 128-byte swizzle.  lbo/sbo in bytes.
__device__ __forceinline__ hct_u64 hct_smem_desc(hct_u32 addr, hct_u32 lbo, hct_u32 sbo) {
  return (hct_u64)((addr & 0x3ffffu) >> 4) | ((hct_u64)(lbo >> 4) << 16) | ((hct_u64)(sbo >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// ---- CTA pairs (cta_group::2): two CTAs of a cluster share one MMA of 256 rows; the even CTA issues it
__device__ __forceinline__ hct_u32 hct_cluster_ctarank() {
  hct_u32 r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of this CTA's shared-memory location `addr` as seen in CTA `rank` of the cluster
__device__ __forceinline__ hct_u32 hct_mapa(hct_u32 addr, hct_u32 rank) {
  hct_u32 r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void hct_mbar_arrive_cluster(hct_u32 cluster_bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// TMA tile load into this CTA's shared memory whose completion is counted on a barrier of either CTA of the pair
__device__ __forceinline__ void hct_tma_load_2d_pair(hct_u32 dst, const HctTensorMap* map, int c0, int c1, hct_u32 cluster_bar) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"(map), "r"(c0), "r"(c1), "r"(cluster_bar)
               : "memory");
}
__device__ __forceinline__ void hct_mma_f16_pair(hct_u32 d_tmem, hct_u64 adesc, hct_u64 bdesc, hct_u32 idesc, hct_u32 accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void hct_mma_tf32_pair(hct_u32 d_tmem, hct_u64 adesc, hct_u64 bdesc, hct_u32 idesc, hct_u32 accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// completes `cluster_bar` (a barrier of either CTA) once every MMA issued so far by this thread has finished
__device__ __forceinline__ void hct_mma_commit_pair(hct_u32 cluster_bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void hct_tmem_alloc_pair(hct_u32 holder_smem, hct_u32 ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void hct_tmem_dealloc_pair(hct_u32 taddr, hct_u32 ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void hct_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// ---- contiguous runs of up to 32 epilogue elements (16-byte accesses when the run is a whole number of vectors)
template <typename T>
__device__ __forceinline__ void hct_ld_run32(const T* p, float* v, int n, bool vec_ok);
template <>
__device__ __forceinline__ void hct_ld_run32<float>(const float* p, float* v, int n, bool vec_ok) {
  if ((n & 3) == 0 && vec_ok) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float4 t = 4 * i < n ? __ldg((const float4*)p + i) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
      v[4 * i] = t.x; v[4 * i + 1] = t.y; v[4 * i + 2] = t.z; v[4 * i + 3] = t.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = i < n ? __ldg(p + i) : 0.0f;
  }
}
template <>
__device__ __forceinline__ void hct_ld_run32<hct_bf16_t>(const hct_bf16_t* p, float* v, int n, bool vec_ok) {
  if ((n & 7) == 0 && vec_ok) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint4 t = 8 * i < n ? __ldg((const uint4*)p + i) : make_uint4(0u, 0u, 0u, 0u);
      v[8 * i] = __uint_as_float(t.x << 16); v[8 * i + 1] = __uint_as_float(t.x & 0xffff0000u);
      v[8 * i + 2] = __uint_as_float(t.y << 16); v[8 * i + 3] = __uint_as_float(t.y & 0xffff0000u);
      v[8 * i + 4] = __uint_as_float(t.z << 16); v[8 * i + 5] = __uint_as_float(t.z & 0xffff0000u);
      v[8 * i + 6] = __uint_as_float(t.w << 16); v[8 * i + 7] = __uint_as_float(t.w & 0xffff0000u);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = i < n ? hct_bf16_to_f32(__ldg(p + i)) : 0.0f;
  }
}
template <typename T>
__device__ __forceinline__ void hct_st_run32(T* p, const float* v, int n, bool vec_ok);
template <>
__device__ __forceinline__ void hct_st_run32<float>(float* p, const float* v, int n, bool vec_ok) {
  if ((n & 3) == 0 && vec_ok) {
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (4 * i < n) ((float4*)p)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i)
      if (i < n) p[i] = v[i];
  }
}
template <>
__device__ __forceinline__ void hct_st_run32<hct_bf16_t>(hct_bf16_t* p, const float* v, int n, bool vec_ok) {
  if ((n & 7) == 0 && vec_ok) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (8 * i < n) ((uint4*)p)[i] = make_uint4(hct_pack_bf16x2(v[8 * i], v[8 * i + 1]), hct_pack_bf16x2(v[8 * i + 2], v[8 * i + 3]),
                                  hct_pack_bf16x2(v[8 * i + 4], v[8 * i + 5]), hct_pack_bf16x2(v[8 * i + 6], v[8 * i + 7]));
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i)
      if (i < n) p[i] = hct_f32_to_bf16(v[i]);
  }
}
