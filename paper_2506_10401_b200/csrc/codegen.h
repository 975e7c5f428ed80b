// Kernel generators: turn a planned group into specialised CUDA source for sm_100a.
#pragma once
#include <string>
#include <vector>

#include "graph.h"
#include "plan.h"

namespace hct {

struct BufRef {
  enum Kind { NodeBuf, Scratch } kind = NodeBuf;
  int node = -1;          // NodeBuf: graph input, graph output or workspace slot of this node
  bool ws_copy = false;   // NodeBuf: the fp32 workspace copy rather than the output buffer
  int64_t scratch_off = 0;  // Scratch: byte offset inside the kernel-private part of the workspace
};

// One tensor map the runtime must encode before launch (TMA-fed kernels only).
struct TmaDesc {
  BufRef buf;
  int elem_bytes = 2;             // 2: bf16, 4: fp32/tf32
  int rank = 2;
  uint64_t dims[5] = {1, 1, 1, 1, 1};     // innermost first
  uint64_t strides[5] = {0, 0, 0, 0, 0};  // bytes, for dims[1..]; strides[0] unused
  uint32_t box[5] = {1, 1, 1, 1, 1};       // elements traversed; ceil(box / estride) of them are loaded
  uint32_t estride[5] = {1, 1, 1, 1, 1};   // traversal stride per dimension (estride[0] must stay 1)
  uint64_t base_offset = 0;                // bytes added to the buffer's address (a multiple of 16)
  int swizzle = 3;                // 0 none, 1 32B, 2 64B, 3 128B
};

struct KernelSpec {
  std::string name;    // entry point
  std::string source;  // full translation unit
  std::string desc;    // one-line description for the plan text
  unsigned grid[3] = {1, 1, 1};
  unsigned block[3] = {1, 1, 1};
  unsigned smem_bytes = 0;       // dynamic shared memory
  bool persistent = false;       // grid[0] is scaled to SM count x occupancy at load time
  unsigned cluster = 1;          // CTAs per cluster (compiled into the kernel); the grid is kept a multiple of it
  unsigned max_grid = 0;         // upper bound for a persistent grid (number of work items)
  std::vector<BufRef> ptrs;      // pointer arguments in order (params.ptr[i])
  std::vector<TmaDesc> tmaps;    // tensor maps in order (params.tmap[i])
  bool wants_status = false;     // last pointer argument is the device status word
};

struct Tunables {
  int row_nv = 4;        // vectors per thread in row kernels
  int row_cta = 256;     // threads per CTA in row kernels
  int row_batch = 1;               // rows a row group of a staged kernel with reductions carries at once
  int row_cta_batched = 512;       // threads per CTA when rows are batched (twice the registers per thread)
  int row_cta_elementwise = 512;   // threads per CTA of a staged row kernel without reductions
  int row_cta_staged = 1024;       // threads per CTA of a staged row kernel (one CTA per SM)
  int row_min_blocks = 1;          // CTAs per SM the compiler must leave registers for (staged kernels of <= 512 threads)
  bool row_no_small_ctas = false;  // run reduction chains as one large CTA per SM even when several small ones fit
  int row_cta_small = 256;         // threads per CTA in the several-small-CTAs shape
  int row_ring_bytes_small = 48 * 1024;  // ring of one small CTA
  bool row_no_reg_rowvec = false;  // keep row vectors of reduction-free chains in shared memory instead of registers
  bool row_no_softmax_ln_fusion = false;  // layer norm after softmax: take the variance with its own reduction
  bool row_no_packed = false;      // row kernels: one-value arithmetic everywhere (no .f32x2 pairs, no multiply-add folding, special-function reciprocal in sigmoid)
  bool row_no_stage = false;       // load rows straight from global memory instead of through the shared-memory ring
  int row_ring_bytes = 200 * 1024; // shared memory a staged row kernel may spend on resident row vectors plus its prefetch ring
  int gemm_insplit = 0;            // fp32 GEMM splits its operands inside the kernel (one launch, no scratch) when 1; otherwise a split pre-pass runs first
  bool gemm_no_ksplit = false;     // fp32 GEMM with few tiles: never split the contraction over idle SMs
  int gemm_pair = 0;               // bf16 GEMM on CTA pairs (256x256 tiles): 0 by rule (enough tiles for every pair), 1 always, 2 never
  int gemm_bn = 0;                 // output-tile width of the tensor-core GEMMs (0: by rule; else 32..256, clamped to what the kernel takes)
  bool conv_no_halo = false;       // load conv pixels once per tap even when the shared-row schedule applies
  bool conv_no_tma_store = false;  // NCHW-reading convolution: store the output with plain vector stores instead of TMA
  int dw_p = 0;                    // depthwise conv: output rows per thread (0: rule; 1, 2, 4 or 8)
  int dw_pair = 0;                 // depthwise conv: 1 = two filters per thread on packed multiply-adds (needs an even number of filters)
  int dw_cta = 0;                  // depthwise conv: threads per block (0: rule; else a multiple of 32, up to 1024)
  int conv_nstg = 0;               // NCHW-reading conv: slots of the pixel staging ring (0: rule)
  int conv_nbuf = 0;               // NCHW-reading conv: operand buffers (0: rule)
  int conv_flat = 0;               // NCHW-reading conv: tiles of 256 consecutive positions instead of whole rows (0: rule, 1: always, 2: never)
  bool sort_no_reg = false;        // row_sort: the shared-memory network for every row length (no register / shuffle kernel)
  bool topk_no_reg = false;        // row_topk for small k: keys in shared memory and a bound found by one warp's bisection (the earlier form)
  bool topk_no_select = false;     // row_topk: full bitonic sort of the row even for small k
  bool conv_phase = false;         // strided convolutions: a stride-phase view wherever one exists, not only for rows too wide for a strided box
  bool conv_ksplit = false;        // NCHW-reading conv: a short last round is cut by output row and by part of the contraction (partial sums meet in scratch); measured slower than the cut by rows alone, so on request only
  bool conv_no_direct = false;     // always take the NHWC pre-pass, even when the convolution could read NCHW itself
  int conv_pw_warps = 0;           // 1x1 convolution as a per-image GEMM: epilogue warps (0: by rule; 8 or 16)
  bool conv_no_pointwise = false;  // 1x1 convolutions take the general schedules instead of the per-image GEMM
  bool simt_only = false;
  // Failure-path testing: the GEMM producer never issues its loads, so the consumer's bounded wait runs out
  // (the kernel then reports through the status word and ends normally).  wait_limit shortens the bound.
  bool fault_never_arrive = false;
  unsigned wait_limit = 0;  // 0: kernel default  // keep contractions on the fp32 FMA kernels (for debugging tensor-core paths)
  static Tunables from_env();
  // Sets one knob by its schedule name; false when the name is unknown or the value is not an integer.
  bool set(const std::string& key, const std::string& value);
  // Applies "knob=integer;knob=integer" on top of *this; throws Error(HCT_ERR_INVALID_ARG) on an unknown knob or bad value.
  void apply_text(const std::string& text);
};

// Extra workspace a group's kernels need beyond the planner's intermediates is appended to
// `scratch_bytes` (byte offsets in BufRef::Scratch are relative to the start of that region).
void gen_row_kernel(const Graph& g, const Plan& p, int group, const Tunables& t, std::vector<KernelSpec>* out);
void gen_contraction_kernels(const Graph& g, const Plan& p, int group, const Tunables& t, size_t* scratch_bytes,
                             std::vector<KernelSpec>* out);

// Source text of a named kernel skeleton (embedded at build time).
const char* skeleton_source(const char* name);

}  // namespace hct
