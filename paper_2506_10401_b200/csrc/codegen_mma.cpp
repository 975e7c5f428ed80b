// Generators for contraction groups (gemm / conv2d plus fused epilogue).
#include <sstream>

#include "../../include/hct.h"
#include "codegen.h"

namespace hct {

std::string float_lit(double v);
const char* ctype(DType d);

namespace {

struct EpiGen {
  const Graph& g;
  const Plan& p;
  const Group& grp;
  int gi;
  std::vector<BufRef> ptrs;
  int64_t conv_ko = 0, conv_hw = 0;   // output channels and pixels per plane of a convolution group (for channels-last stores)

  // A graph output declared nhwc: element (n, k, pixel) of the [N,K,H,W] value goes to ((n * HW + pixel) * K + k).
  bool nhwc_store(const Store& st) const { return st.to_output && g.nodes[st.node].out_nhwc; }

  int ptr_index(int node, bool ws_copy) {
    for (size_t i = 0; i < ptrs.size(); ++i)
      if (ptrs[i].kind == BufRef::NodeBuf && ptrs[i].node == node && ptrs[i].ws_copy == ws_copy) return (int)i;
    BufRef b;
    b.node = node;
    b.ws_copy = ws_copy;
    ptrs.push_back(b);
    return (int)ptrs.size() - 1;
  }
  DType buf_dtype(int node) const { return g.nodes[node].dtype; }   // inputs: as declared; computed values: fp32, or bf16 after a cast
  bool is_ws(int node) const { return g.nodes[node].cls != OpClass::Input && p.ws_offset[node] >= 0; }

  // Scalar epilogue: value `acc` of element at linear offset `off`, per-row index `ri`
  // (GEMM row, or n*K+k for NCHW), per-column index `ci` (GEMM column, or channel k).
  std::string scalar_fn() {
    std::ostringstream f;
    f << "__device__ __forceinline__ void hct_epilogue(const HctParams& hct_p, float acc, long long off, long long ri, int ci) {\n";
    int anchor = grp.nodes[0];
    f << "  const float e" << anchor << " = acc;\n";
    auto ref = [&](const Operand& a) -> std::string {
      if (a.is_literal()) return float_lit(a.literal);
      if (p.group_of[a.node] == gi) return "e" + std::to_string(a.node);
      int k = find_ext(grp, a.node);
      const ExtOperand& e = grp.ext[k];
      int pi = ptr_index(e.node, is_ws(e.node));
      std::string ptr = std::string("((const ") + ctype(buf_dtype(e.node)) + "*)hct_p.ptr[" + std::to_string(pi) + "])";
      switch (e.bcast) {
        case Bcast::Full: return "hct_ld1(" + ptr + " + off)";
        case Bcast::RowVec: return "hct_ld1(" + ptr + " + ci)";
        case Bcast::Scalar: return "hct_ld1(" + ptr + ")";
        case Bcast::RowIdx: return grp.kind == GroupKind::Conv ? "hct_ld1(" + ptr + " + ci)" : "hct_ld1(" + ptr + " + ri)";
      }
      return "";
    };
    for (size_t i = 1; i < grp.nodes.size(); ++i) {
      const Node& nd = g.nodes[grp.nodes[i]];
      std::vector<std::string> av;
      for (auto& a : nd.args) av.push_back(ref(a));
      f << "  const float e" << grp.nodes[i] << " = " << elementwise_call(nd, av, "off") << ";  // " << nd.name << "\n";
    }
    for (auto& s : grp.stores) {
      int pi = ptr_index(s.node, !s.to_output);
      if (nhwc_store(s)) {
        if (conv_ko <= 0) throw Error(HCT_ERR_UNSUPPORTED, "an nhwc output must be produced by a convolution kernel");
        f << "  hct_st1((" << ctype(s.dtype) << "*)hct_p.ptr[" << pi << "] + ((ri / " << conv_ko << "LL) * " << conv_hw << "LL + off % " << conv_hw
          << "LL) * " << conv_ko << "LL + ci, e" << s.node << ");\n";
        continue;
      }
      f << "  hct_st1((" << ctype(s.dtype) << "*)hct_p.ptr[" << pi << "] + off, e" << s.node << ");\n";
    }
    f << "}\n";
    return f.str();
  }

  // Run epilogue for the tensor-core GEMM: one thread owns 32 consecutive columns of one row.
  // `ncols` of them exist; vector access is legal when N is a multiple of the vector length.
  // `N` is the distance between consecutive rows; every run starts at a multiple of `vec_unit`
  // elements plus a multiple of 32; `rowidx` is the index expression of per-row operands.
  // With `vals_only` (one store only) the function is named hct_epilogue_vals and hands the 32 values to
  // be stored back in `out` instead of writing them: the caller stores them its own way.
  std::string run_fn(int64_t N, int64_t vec_unit = -1, const std::string& rowidx = "row", bool vals_only = false) {
    if (vec_unit < 0) vec_unit = N;
    std::ostringstream f;
    if (vals_only)
      f << "__device__ __forceinline__ void hct_epilogue_vals(const HctParams& hct_p, float (&acc)[32], long long row, int col0, int ncols, "
           "float (&out)[32]) {\n";
    else
      f << "__device__ __forceinline__ void hct_epilogue_run(const HctParams& hct_p, float (&acc)[32], long long row, int col0, int ncols) {\n";
    int anchor = grp.nodes[0];
    std::ostringstream loads;
    auto vec_ok = [&](DType d) { return (N % (d == BF16 ? 8 : 4) == 0 && vec_unit % (d == BF16 ? 8 : 4) == 0) ? "true" : "false"; };
    // Runs whose start is not a whole 16-byte vector but still a multiple of 2 or 4 elements use accesses of
    // that width (helpers of run_partial.cuh, emitted in front of the function when needed): 0 = not applicable.
    bool need_partial = false;
    auto part_w = [&](DType d) -> int {
      const int64_t full = d == BF16 ? 8 : 4;
      if (N % full == 0 && vec_unit % full == 0) return 0;
      for (int64_t w = full / 2; w >= 2; w /= 2)
        if (N % w == 0 && vec_unit % w == 0) { need_partial = true; return (int)w; }
      return 0;
    };
    auto ld_call = [&](DType d, const std::string& ptr_expr, const std::string& dst) {
      const int w = part_w(d);
      if (w) return std::string("hct_ld_run32w<") + std::to_string(w) + ">(" + ptr_expr + ", " + dst + ", ncols);\n";
      return std::string("hct_ld_run32<") + ctype(d) + ">(" + ptr_expr + ", " + dst + ", ncols, " + vec_ok(d) + ");\n";
    };
    auto ref = [&](const Operand& a) -> std::string {
      if (a.is_literal()) return float_lit(a.literal);
      if (p.group_of[a.node] == gi) return a.node == anchor ? "acc[j]" : "e" + std::to_string(a.node);
      int k = find_ext(grp, a.node);
      const ExtOperand& e = grp.ext[k];
      if (e.bcast == Bcast::Full || e.bcast == Bcast::RowVec) return "x" + std::to_string(k) + "[j]";
      return "c" + std::to_string(k);
    };
    for (size_t k = 0; k < grp.ext.size(); ++k) {
      const ExtOperand& e = grp.ext[k];
      int pi = ptr_index(e.node, is_ws(e.node));
      DType d = buf_dtype(e.node);
      std::string ptr = std::string("((const ") + ctype(d) + "*)hct_p.ptr[" + std::to_string(pi) + "])";
      switch (e.bcast) {
        case Bcast::Full:
          loads << "  float x" << k << "[32]; " << ld_call(d, ptr + " + row * " + std::to_string(N) + "LL + col0", "x" + std::to_string(k));
          break;
        case Bcast::RowVec:
          loads << "  float x" << k << "[32]; " << ld_call(d, ptr + " + col0", "x" + std::to_string(k));
          break;
        case Bcast::Scalar: loads << "  const float c" << k << " = hct_ld1(" << ptr << ");\n"; break;
        case Bcast::RowIdx: loads << "  const float c" << k << " = hct_ld1(" << ptr << " + " << rowidx << ");\n"; break;
      }
    }
    f << loads.str();
    if (!vals_only)
      for (auto& st : grp.stores) {
        if (p.partial_cols[st.node] > 0 && !st.to_output)
          f << "  float ps" << st.node << " = 0.0f;\n";   // row sum of this 32-column chunk
        else
          f << "  float o" << st.node << "_" << (st.to_output ? 1 : 0) << "[32];\n";
      }
    f << "  _Pragma(\"unroll\") for (int j = 0; j < 32; ++j) {\n";
    for (size_t i = 1; i < grp.nodes.size(); ++i) {
      const Node& nd = g.nodes[grp.nodes[i]];
      std::vector<std::string> av;
      for (auto& a : nd.args) av.push_back(ref(a));
      f << "    const float e" << grp.nodes[i] << " = " << elementwise_call(nd, av, "row * " + std::to_string(N) + "LL + col0 + j") << ";  // "
        << nd.name << "\n";
    }
    for (auto& st : grp.stores) {
      std::string val = st.node == anchor ? "acc[j]" : "e" + std::to_string(st.node);
      // A cast_bf16 stored as bf16: the store rounds (to nearest even, once), so the node's own rounding and the
      // widening back to fp32 are skipped for the stored copy.
      const Node& sn = g.nodes[st.node];
      if (st.dtype == BF16 && sn.op == "cast_bf16" && st.node != anchor && !sn.args[0].is_literal() && p.group_of[sn.args[0].node] == gi)
        val = sn.args[0].node == anchor ? "acc[j]" : "e" + std::to_string(sn.args[0].node);
      if (!vals_only && p.partial_cols[st.node] > 0 && !st.to_output)
        f << "    if (j < ncols) ps" << st.node << " += " << val << ";\n";
      else
        f << "    " << (vals_only ? std::string("out") : "o" + std::to_string(st.node) + "_" + (st.to_output ? "1" : "0")) << "[j] = " << val << ";\n";
    }
    f << "  }\n";
    if (vals_only) {
      f << "}\n";
      return (need_partial ? std::string(skeleton_source("run_partial")) + "\n" : std::string()) + f.str();
    }
    for (auto& st : grp.stores) {
      int pi = ptr_index(st.node, !st.to_output);
      if (p.partial_cols[st.node] > 0 && !st.to_output) {   // one value per row and chunk; every chunk starts at a multiple of 32 columns
        f << "  ((float*)hct_p.ptr[" << pi << "])[row * " << p.partial_cols[st.node] << "LL + (col0 >> 5)] = ps" << st.node << ";\n";
        continue;
      }
      if (nhwc_store(st)) {   // consecutive lanes hold consecutive channels: every store of a warp covers 32 neighbouring elements
        if (conv_ko <= 0 || N != conv_hw) throw Error(HCT_ERR_UNSUPPORTED, "an nhwc output must be produced by a convolution kernel");
        f << "  {\n    " << ctype(st.dtype) << "* q = (" << ctype(st.dtype) << "*)hct_p.ptr[" << pi << "] + ((row / " << conv_ko << "LL) * " << N
          << "LL + col0) * " << conv_ko << "LL + row % " << conv_ko << "LL;\n    _Pragma(\"unroll\") for (int j = 0; j < 32; ++j) if (j < ncols) hct_st1(q + j * "
          << conv_ko << "LL, o" << st.node << "_1[j]);\n  }\n";
        continue;
      }
      const int w = part_w(st.dtype);
      if (w)
        f << "  hct_st_run32w<" << w << ">((" << ctype(st.dtype) << "*)hct_p.ptr[" << pi << "] + row * " << N << "LL + col0, o" << st.node << "_"
          << (st.to_output ? 1 : 0) << ", ncols);\n";
      else
        f << "  hct_st_run32<" << ctype(st.dtype) << ">((" << ctype(st.dtype) << "*)hct_p.ptr[" << pi << "] + row * " << N << "LL + col0, o"
          << st.node << "_" << (st.to_output ? 1 : 0) << ", ncols, " << vec_ok(st.dtype) << ");\n";
    }
    f << "}\n";
    return (need_partial ? std::string(skeleton_source("run_partial")) + "\n" : std::string()) + f.str();
  }

  // Epilogue of the tensor-core convolution: one thread owns one output pixel (n,h,w) and 32
  // consecutive output channels k0..k0+31, `nk` of which exist.  NCHW: channel j lies j planes further.
  std::string conv_fn(int64_t KO, int64_t HO, int64_t WO) {
    std::ostringstream f;
    f << "__device__ __forceinline__ void hct_epilogue_conv(const HctParams& hct_p, float (&acc)[32], int n, int h, int w, int k0, int nk) {\n";
    f << "  const long long plane = " << HO * WO << "LL;\n";
    f << "  const long long off0 = (((long long)n * " << KO << "LL + k0) * " << HO << "LL + h) * " << WO << "LL + w;\n";
    int anchor = grp.nodes[0];
    auto ref = [&](const Operand& a) -> std::string {
      if (a.is_literal()) return float_lit(a.literal);
      if (p.group_of[a.node] == gi) return a.node == anchor ? "acc[j]" : "e" + std::to_string(a.node);
      int k = find_ext(grp, a.node);
      const ExtOperand& e = grp.ext[k];
      if (e.bcast == Bcast::Scalar) return "c" + std::to_string(k);
      return "x" + std::to_string(k) + "[j]";
    };
    for (size_t k = 0; k < grp.ext.size(); ++k) {
      const ExtOperand& e = grp.ext[k];
      int pi = ptr_index(e.node, is_ws(e.node));
      DType d = buf_dtype(e.node);
      std::string ptr = std::string("((const ") + ctype(d) + "*)hct_p.ptr[" + std::to_string(pi) + "])";
      switch (e.bcast) {
        case Bcast::RowIdx:  // per-channel operand [K,1,1]
          f << "  float x" << k << "[32]; hct_ld_run32<" << ctype(d) << ">(" << ptr << " + k0, x" << k << ", nk, true);\n";
          break;
        case Bcast::Full:
          f << "  float x" << k << "[32];\n  _Pragma(\"unroll\") for (int j = 0; j < 32; ++j) x" << k << "[j] = j < nk ? hct_ld1(" << ptr
            << " + off0 + j * plane) : 0.0f;\n";
          break;
        case Bcast::Scalar: f << "  const float c" << k << " = hct_ld1(" << ptr << ");\n"; break;
        case Bcast::RowVec: throw Error(HCT_ERR_UNSUPPORTED, "row-vector operand in a convolution epilogue");
      }
    }
    f << "  _Pragma(\"unroll\") for (int j = 0; j < 32; ++j) {\n";
    for (size_t i = 1; i < grp.nodes.size(); ++i) {
      const Node& nd = g.nodes[grp.nodes[i]];
      std::vector<std::string> av;
      for (auto& a : nd.args) av.push_back(ref(a));
      f << "    const float e" << grp.nodes[i] << " = " << elementwise_call(nd, av, "off0 + j * plane") << ";  // " << nd.name << "\n";
    }
    for (auto& st : grp.stores) {
      int pi = ptr_index(st.node, !st.to_output);
      f << "    if (j < nk) hct_st1((" << ctype(st.dtype) << "*)hct_p.ptr[" << pi << "] + off0 + j * plane, "
        << (st.node == anchor ? "acc[j]" : "e" + std::to_string(st.node)) << ");\n";
    }
    f << "  }\n}\n";
    return f.str();
  }
};

}  // namespace

void gen_contraction_kernels(const Graph& g, const Plan& p, int gi, const Tunables& tun, size_t* scratch_bytes,
                             std::vector<KernelSpec>* out) {
  (void)scratch_bytes;
  const Group& grp = p.groups[gi];
  const Node& anchor = g.nodes[grp.nodes[0]];
  const Node& a = g.nodes[anchor.args[0].node];
  const Node& b = g.nodes[anchor.args[anchor.args.size() > 1 ? 1 : 0].node];   // transpose and sort have one operand
  EpiGen eg{g, p, grp, gi, {}};
  bool nhwc_out = false;   // some graph output of this group is declared channels-last
  for (auto& st : grp.stores) nhwc_out = nhwc_out || eg.nhwc_store(st);
  if (grp.kind == GroupKind::Conv) {
    eg.conv_ko = anchor.shape[1];
    eg.conv_hw = anchor.shape[2] * anchor.shape[3];
  } else if (nhwc_out) {
    throw Error(HCT_ERR_UNSUPPORTED, "an nhwc output must be produced by a convolution kernel");
  }

  // ---- reshape: flat copy through the generated epilogue
  if (grp.kind == GroupKind::Reshape) {
    const int src = anchor.args[0].node;
    const int pa = eg.ptr_index(src, g.nodes[src].cls != OpClass::Input && p.ws_offset[src] >= 0);
    const DType ta = eg.buf_dtype(src);
    std::string epi = eg.scalar_fn();
    KernelSpec k;
    k.name = "hct_reshape_g" + std::to_string(gi);
    std::ostringstream st;
    st << "#define HCT_ROWS " << anchor.shape[0] << "LL\n#define HCT_COLS " << anchor.shape[1] << "LL\n#define HCT_TA " << ctype(ta)
       << "\n#define HCT_PA " << pa << "\n#define HCT_KERNEL_NAME " << k.name << "\n"
       << skeleton_source("common") << "\nstruct HctParams { void* ptr[" << eg.ptrs.size() << "]; };\n" << epi << skeleton_source("reshape");
    k.source = st.str();
    k.ptrs = eg.ptrs;
    k.grid[0] = (unsigned)std::max<int64_t>(1, std::min<int64_t>((anchor.numel() + 255) / 256, 148 * 64));
    k.block[0] = 256;
    k.desc = "reshape: flat copy, consumers fused at the store";
    out->push_back(k);
    return;
  }

  // ---- row sort / top-k: bitonic network in shared memory, one CTA per row, consumers applied at the store
  if (grp.kind == GroupKind::Sort) {
    const int src = anchor.args[0].node;
    const int64_t R = a.shape[0], C = a.shape[1], KOUT = anchor.shape[1];
    int64_t NP = 8;
    while (NP < C) NP *= 2;
    const int64_t T = std::max<int64_t>(32, std::min<int64_t>(512, NP / 8));   // a thread owns blocks of 8 slots
    const int pa = eg.ptr_index(src, g.nodes[src].cls != OpClass::Input && p.ws_offset[src] >= 0);
    const DType ta = eg.buf_dtype(src);
    std::string epi = eg.scalar_fn();
    if (anchor.sort_indices) {
      // columns instead of values: 64-bit (value, column) keys through the same network, 8 bytes of shared memory per slot
      KernelSpec k;
      k.name = "hct_row_argsort_g" + std::to_string(gi);
      std::ostringstream st;
      st << "#define HCT_R " << R << "LL\n#define HCT_C " << C << "\n#define HCT_NP " << NP << "\n#define HCT_KOUT " << KOUT
         << "\n#define HCT_DESC " << (anchor.descending ? 1 : 0) << "\n#define HCT_T " << T << "\n#define HCT_TA " << ctype(ta)
         << "\n#define HCT_PA " << pa << "\n#define HCT_KERNEL_NAME " << k.name << "\n"
         << skeleton_source("common") << "\nstruct HctParams { void* ptr[" << eg.ptrs.size() << "]; };\n" << epi << skeleton_source("row_argsort");
      k.source = st.str();
      k.ptrs = eg.ptrs;
      k.smem_bytes = (unsigned)(8 * NP);
      const int64_t per_sm = std::max<int64_t>(1, std::min<int64_t>(2048 / T, std::min<int64_t>(16, (200 * 1024) / (8 * NP))));
      k.grid[0] = (unsigned)std::max<int64_t>(1, std::min<int64_t>(R, 148 * per_sm));
      k.block[0] = (unsigned)T;
      k.desc = std::string(anchor.sort_k ? "row top-k indices" : "row argsort") + ": bitonic network over " + std::to_string(NP) +
               " 64-bit (value, column) keys in shared memory, one CTA per row";
      out->push_back(k);
      return;
    }
    if (anchor.sort_k > 0 && anchor.sort_k <= 256 && C >= 2 && !tun.topk_no_select) {
      // small k: radix selection of the k-th largest key, then a sort of the k selected values only
      int64_t KP = 2;
      while (KP < KOUT) KP *= 2;
      // fp32 rows of up to 8192 values in whole 16-byte vectors, k <= 64: keys stay in registers (see row_topk.cuh)
      const bool topk_reg = KOUT <= 64 && ta == F32 && C % 4 == 0 && C <= 8192 && !tun.topk_no_reg;
      KernelSpec k;
      k.name = "hct_row_topk_g" + std::to_string(gi);
      std::ostringstream st;
      st << "#define HCT_R " << R << "LL\n#define HCT_C " << C << "\n#define HCT_K " << KOUT << "\n#define HCT_KP " << KP
         << "\n#define HCT_T 256\n#define HCT_TA " << ctype(ta) << "\n#define HCT_PA " << pa << "\n#define HCT_TOPK_REG " << (topk_reg ? 1 : 0)
         << "\n#define HCT_KERNEL_NAME " << k.name << "\n"
         << skeleton_source("common") << "\nstruct HctParams { void* ptr[" << eg.ptrs.size() << "]; };\n" << epi << skeleton_source("row_topk");
      k.source = st.str();
      k.ptrs = eg.ptrs;
      const int64_t per_sm = std::max<int64_t>(1, std::min<int64_t>(8, (200 * 1024) / (4 * C + 4 * KP + 1280)));
      k.grid[0] = (unsigned)std::max<int64_t>(1, std::min<int64_t>(R, 148 * per_sm));
      k.block[0] = 256;
      k.desc = std::string("row top-k: ") + (KOUT <= 64 ? "bound from per-thread maxima and a 128-slot bitonic network, else " : "") +
               "radix selection of the k-th largest key in shared memory, one CTA per row, then a bitonic network over " + std::to_string(KP) +
               " selected keys";
      out->push_back(k);
      return;
    }
    if (NP >= 512 && NP <= 16384 && !tun.sort_no_reg) {
      // rows of 512 to 16384 slots: 16 slots per thread in registers, partners met by shuffles, and by shared-memory
      // exchanges only across warps (row_sort_reg.cuh)
      const int64_t TR = NP / 16;
      KernelSpec k;
      k.name = "hct_row_sort_g" + std::to_string(gi);
      std::ostringstream st;
      st << "#define HCT_R " << R << "LL\n#define HCT_C " << C << "\n#define HCT_NP " << NP << "\n#define HCT_KOUT " << KOUT
         << "\n#define HCT_DESC " << (anchor.descending ? 1 : 0) << "\n#define HCT_T " << TR << "\n#define HCT_TA " << ctype(ta)
         << "\n#define HCT_PA " << pa << "\n#define HCT_KERNEL_NAME " << k.name << "\n"
         << skeleton_source("common") << "\nstruct HctParams { void* ptr[" << eg.ptrs.size() << "]; };\n" << epi << skeleton_source("row_sort_reg");
      k.source = st.str();
      k.ptrs = eg.ptrs;
      const int64_t per_sm = std::max<int64_t>(1, std::min<int64_t>(2048 / TR, 16));
      k.grid[0] = (unsigned)std::max<int64_t>(1, std::min<int64_t>(R, 148 * per_sm));
      k.block[0] = (unsigned)TR;
      k.desc = std::string(anchor.sort_k ? "row top-k" : "row sort") + ": bitonic network over " + std::to_string(NP) +
               " slots, 16 per thread in registers, shuffles within a warp, shared-memory exchanges across warps, one CTA per row";
      out->push_back(k);
      return;
    }
    KernelSpec k;
    k.name = "hct_row_sort_g" + std::to_string(gi);
    std::ostringstream src_text;
    src_text << "#define HCT_R " << R << "LL\n#define HCT_C " << C << "\n#define HCT_NP " << NP << "\n#define HCT_KOUT " << KOUT
             << "\n#define HCT_DESC " << (anchor.descending ? 1 : 0) << "\n#define HCT_T " << T << "\n#define HCT_TA " << ctype(ta)
             << "\n#define HCT_PA " << pa << "\n#define HCT_KERNEL_NAME " << k.name << "\n"
             << skeleton_source("common") << "\nstruct HctParams { void* ptr[" << eg.ptrs.size() << "]; };\n" << epi << skeleton_source("row_sort");
    k.source = src_text.str();
    k.ptrs = eg.ptrs;
    // resident CTAs per SM: limited by threads (2048) and by shared memory (4 * NP bytes each)
    const int64_t per_sm = std::max<int64_t>(1, std::min<int64_t>(2048 / T, std::min<int64_t>(16, (200 * 1024) / (4 * NP))));
    k.grid[0] = (unsigned)std::max<int64_t>(1, std::min<int64_t>(R, 148 * per_sm));
    k.block[0] = (unsigned)T;
    k.desc = std::string(anchor.sort_k ? "row top-k" : "row sort") + ": bitonic network over " + std::to_string(NP) + " shared-memory slots, one CTA per row";
    out->push_back(k);
    return;
  }

  // ---- layout transform: permutation of up to four axes, consumers applied at the store
  if (grp.kind == GroupKind::Permute) {
    const int src = anchor.args[0].node;
    const int pa = eg.ptr_index(src, g.nodes[src].cls != OpClass::Input && p.ws_offset[src] >= 0);
    const DType ta = eg.buf_dtype(src);
    std::string epi = eg.scalar_fn();
    int64_t S[4] = {1, 1, 1, 1};
    for (size_t d = 0; d < a.shape.size(); ++d) S[4 - a.shape.size() + d] = a.shape[d];
    KernelSpec k;
    k.name = "hct_permute_g" + std::to_string(gi);
    std::ostringstream st;
    for (int d = 0; d < 4; ++d) st << "#define HCT_S" << d << " " << S[d] << "LL\n#define HCT_P" << d << " " << anchor.perm[d] << "\n";
    st << "#define HCT_TA " << ctype(ta) << "\n#define HCT_PA " << pa << "\n#define HCT_KERNEL_NAME " << k.name << "\n"
       << skeleton_source("common") << "\nstruct HctParams { void* ptr[" << eg.ptrs.size() << "]; };\n" << epi << skeleton_source("permute");
    k.source = st.str();
    k.ptrs = eg.ptrs;
    const bool inner_kept = anchor.perm[3] == 3;
    const int64_t work = inner_kept ? (anchor.numel() + 255) / 256
                                    : (anchor.numel() / std::max<int64_t>(1, S[3] * S[anchor.perm[3]])) * ((S[3] + 63) / 64) * ((S[anchor.perm[3]] + 63) / 64);
    k.grid[0] = (unsigned)std::max<int64_t>(1, std::min<int64_t>(work, 148 * (inner_kept ? 32 : 8)));
    k.block[0] = 256;
    k.desc = inner_kept ? "permute: rows of the innermost axis copied whole, consumers fused at the store"
                        : "permute: the plane of the old and the new innermost axis transposed through 64x64 shared-memory tiles, consumers fused at the store";
    out->push_back(k);
    return;
  }

  // ---- layout transform: tiled transposition through shared memory, consumers applied at the store
  if (grp.kind == GroupKind::Transpose) {
    const int src = anchor.args[0].node;
    const int64_t R = a.shape[0], C = a.shape[1];
    const int pa = eg.ptr_index(src, g.nodes[src].cls != OpClass::Input && p.ws_offset[src] >= 0);
    const DType ta = eg.buf_dtype(src);
    std::string epi = eg.scalar_fn();
    KernelSpec k;
    k.name = "hct_transpose_g" + std::to_string(gi);
    std::ostringstream src_text;
    src_text << "#define HCT_R " << R << "LL\n#define HCT_C " << C << "LL\n#define HCT_TA " << ctype(ta) << "\n#define HCT_PA " << pa
             << "\n#define HCT_KERNEL_NAME " << k.name << "\n"
             << skeleton_source("common") << "\nstruct HctParams { void* ptr[" << eg.ptrs.size() << "]; };\n" << epi << skeleton_source("transpose");
    k.source = src_text.str();
    k.ptrs = eg.ptrs;
    const int64_t tiles = ((R + 63) / 64) * ((C + 63) / 64);
    k.grid[0] = (unsigned)std::max<int64_t>(1, std::min<int64_t>(tiles, 148 * 8));
    k.block[0] = 256;
    k.desc = "transpose through 64x64 shared-memory tiles, consumers fused at the store";
    out->push_back(k);
    return;
  }

  // ---- tensor-core GEMM: bf16 operands straight from their buffers
  if (grp.kind == GroupKind::Gemm && !tun.simt_only) {
    int64_t M = a.shape[0], K = a.shape[1], N = b.shape[1];
    DType da = a.dtype, db = b.dtype;
    // CTA pairs on 256 x 256 tiles when every pair of SMs gets at least one tile
    const int64_t pair_tiles = ((M + 255) / 256) * ((N + 255) / 256);
    const bool use_pair = tun.gemm_pair == 1 || (tun.gemm_pair == 0 && pair_tiles >= 74 && !tun.fault_never_arrive && tun.gemm_bn == 0);
    if (da == BF16 && db == BF16 && K % 8 == 0 && N % 8 == 0 && M <= 0x7fffffff && N <= 0x7fffffff && K <= 0x7fffffff && use_pair) {
      const int stages = 6;
      std::string epi = eg.run_fn(N);
      KernelSpec k;
      k.name = "hct_gemm_tc2_bf16_g" + std::to_string(gi);
      std::ostringstream src;
      src << "#define HCT_M " << M << "LL\n#define HCT_N " << N << "LL\n#define HCT_K " << K << "LL\n#define HCT_STAGES " << stages
          << "\n#define HCT_TF32X3 0"
          << (tun.wait_limit ? "\n#define HCT_WAIT_LIMIT " + std::to_string(tun.wait_limit) + "u" : std::string())
          << "\n#define HCT_STATUS_SLOT " << eg.ptrs.size() << "\n#define HCT_KERNEL_NAME " << k.name << "\n";
      src << skeleton_source("common") << "\n" << skeleton_source("tc_common") << "\nstruct HctParams { HctTensorMap tmap[2]; void* ptr["
          << eg.ptrs.size() + 1 << "]; };\n" << epi << skeleton_source("gemm_tc2");
      k.source = src.str();
      k.ptrs = eg.ptrs;
      k.wants_status = true;
      TmaDesc ta, tb;
      ta.buf.node = anchor.args[0].node;
      ta.buf.ws_copy = a.cls != OpClass::Input && p.ws_offset[anchor.args[0].node] >= 0;
      ta.elem_bytes = 2;
      ta.rank = 2;
      ta.dims[0] = (uint64_t)K; ta.dims[1] = (uint64_t)M;
      ta.strides[1] = (uint64_t)K * 2;
      ta.box[0] = 64; ta.box[1] = 128;
      tb.buf.node = anchor.args[1].node;
      tb.buf.ws_copy = b.cls != OpClass::Input && p.ws_offset[anchor.args[1].node] >= 0;
      tb.elem_bytes = 2;
      tb.rank = 2;
      tb.dims[0] = (uint64_t)N; tb.dims[1] = (uint64_t)K;
      tb.strides[1] = (uint64_t)N * 2;
      tb.box[0] = 64; tb.box[1] = 64;
      k.tmaps = {ta, tb};
      k.block[0] = 192;
      k.smem_bytes = (unsigned)(stages * 32768 + 1024);
      k.persistent = true;
      k.cluster = 2;
      k.max_grid = (unsigned)std::min<int64_t>(2 * pair_tiles, 0x7ffffffe);
      k.grid[0] = k.max_grid;
      k.desc = "gemm tcgen05 bf16 on CTA pairs, 256x256x64 per pair, " + std::to_string(stages) + " stages";
      out->push_back(k);
      return;
    }
    if (da == BF16 && db == BF16 && K % 8 == 0 && N % 8 == 0 && M <= 0x7fffffff && N <= 0x7fffffff && K <= 0x7fffffff) {
      const int bn_max = N > 128 ? 256 : N > 64 ? 128 : 64;
      int BN = bn_max;
      // few tiles leave SMs idle: halve the tile width while that at least doubles the busy SMs
      while (BN > 64 && ((M + 127) / 128) * ((N + BN - 1) / BN) * 2 <= 148) BN /= 2;
      if (tun.gemm_bn >= 64) BN = std::min(bn_max, tun.gemm_bn >= 256 ? 256 : tun.gemm_bn >= 128 ? 128 : 64);
      int stages = BN == 256 ? 4 : 6;
      std::string epi = eg.run_fn(N);
      KernelSpec k;
      k.name = "hct_gemm_tc_bf16_g" + std::to_string(gi);
      std::ostringstream src;
      src << "#define HCT_M " << M << "LL\n#define HCT_N " << N << "LL\n#define HCT_K " << K << "LL\n#define HCT_BN " << BN
          << "\n#define HCT_STAGES " << stages << "\n#define HCT_TF32X3 0\n#define HCT_FAULT_NEVER_ARRIVE " << (tun.fault_never_arrive ? 1 : 0)
          << (tun.wait_limit ? "\n#define HCT_WAIT_LIMIT " + std::to_string(tun.wait_limit) + "u" : std::string())
          << "\n#define HCT_STATUS_SLOT " << eg.ptrs.size()
          << "\n#define HCT_KERNEL_NAME " << k.name << "\n";
      src << skeleton_source("common") << "\n" << skeleton_source("tc_common") << "\nstruct HctParams { HctTensorMap tmap[2]; void* ptr["
          << eg.ptrs.size() + 1 << "]; };\n" << epi << skeleton_source("gemm_tc");
      k.source = src.str();
      k.ptrs = eg.ptrs;
      k.wants_status = true;
      TmaDesc ta, tb;
      ta.buf.node = anchor.args[0].node;
      ta.buf.ws_copy = a.cls != OpClass::Input && p.ws_offset[anchor.args[0].node] >= 0;
      ta.elem_bytes = 2;
      ta.rank = 2;
      ta.dims[0] = (uint64_t)K; ta.dims[1] = (uint64_t)M;
      ta.strides[1] = (uint64_t)K * 2;
      ta.box[0] = 64; ta.box[1] = 128;
      tb.buf.node = anchor.args[1].node;
      tb.buf.ws_copy = b.cls != OpClass::Input && p.ws_offset[anchor.args[1].node] >= 0;
      tb.elem_bytes = 2;
      tb.rank = 2;
      tb.dims[0] = (uint64_t)N; tb.dims[1] = (uint64_t)K;
      tb.strides[1] = (uint64_t)N * 2;
      tb.box[0] = 64; tb.box[1] = 64;
      k.tmaps = {ta, tb};
      int64_t tiles = ((M + 127) / 128) * ((N + BN - 1) / BN);
      k.block[0] = 192;
      k.smem_bytes = (unsigned)(stages * (128 * 128 + BN * 128) + 1024);
      k.persistent = true;
      k.max_grid = (unsigned)std::min<int64_t>(tiles, 0x7fffffff);
      k.grid[0] = k.max_grid;
      std::ostringstream d;
      d << "gemm tcgen05 bf16 128x" << BN << "x64, " << stages << " stages";
      k.desc = d.str();
      out->push_back(k);
      return;
    }
  }

  // ---- tensor-core GEMM on fp32 operands: split pre-pass, then three TF32 products per k step
  if (grp.kind == GroupKind::Gemm && !tun.simt_only) {
    int64_t M = a.shape[0], K = a.shape[1], N = b.shape[1];
    DType da = a.dtype, db = b.dtype;
    // On request (schedule knob or tuning): one launch that splits the operands inside the kernel, with no
    // pre-pass and no scratch.  Not the default: measured, it only ties the two-launch path on 256^3
    // (16 us both) and loses on larger problems (4096x1024x1024: 115 us against 63 us), the split warps
    // being the slowest stage of its pipeline.
    const bool a_presplit = p.split_store[anchor.args[0].node] != 0;   // A arrives as TF32 head and tail written by its producer
    const bool insplit = da == F32 && db == F32 && K % 4 == 0 && N % 4 == 0 && tun.gemm_pair != 1 && tun.gemm_insplit == 1 && !a_presplit;
    if (insplit && M <= 0x7fffffff && N <= 0x7fffffff && K <= 0x7fffffff) {
      const int BN = 64;   // 448 threads share the register file: a 128-column running sum per epilogue thread would spill
      const int rstages = 3, stages = 3;
      std::string epi = eg.run_fn(N);
      KernelSpec k;
      k.name = "hct_gemm_tc_tf32x3_insplit_g" + std::to_string(gi);
      std::ostringstream src;
      src << "#define HCT_M " << M << "LL\n#define HCT_N " << N << "LL\n#define HCT_K " << K << "LL\n#define HCT_BN " << BN
          << "\n#define HCT_RSTAGES " << rstages << "\n#define HCT_STAGES " << stages << "\n#define HCT_STATUS_SLOT " << eg.ptrs.size()
          << "\n#define HCT_KERNEL_NAME " << k.name << "\n";
      src << skeleton_source("common") << "\n" << skeleton_source("tc_common") << "\nstruct HctParams { HctTensorMap tmap[2]; void* ptr["
          << eg.ptrs.size() + 1 << "]; };\n" << epi << skeleton_source("gemm_tc_insplit");
      k.source = src.str();
      k.ptrs = eg.ptrs;
      k.wants_status = true;
      auto operand_ref = [&](int node) {
        BufRef r;
        r.node = node;
        r.ws_copy = g.nodes[node].cls != OpClass::Input && p.ws_offset[node] >= 0;
        return r;
      };
      TmaDesc ta, tb;
      ta.buf = operand_ref(anchor.args[0].node);
      ta.elem_bytes = 4;
      ta.rank = 2;
      ta.dims[0] = (uint64_t)K; ta.dims[1] = (uint64_t)M;
      ta.strides[1] = (uint64_t)K * 4;
      ta.box[0] = 32; ta.box[1] = 128;
      tb.buf = operand_ref(anchor.args[1].node);
      tb.elem_bytes = 4;
      tb.rank = 2;
      tb.dims[0] = (uint64_t)N; tb.dims[1] = (uint64_t)K;
      tb.strides[1] = (uint64_t)N * 4;
      tb.box[0] = 32; tb.box[1] = 32;
      tb.swizzle = 0;
      k.tmaps = {ta, tb};
      int64_t tiles = ((M + 127) / 128) * ((N + BN - 1) / BN);
      k.block[0] = 448;
      k.smem_bytes = (unsigned)(rstages * (16384 + BN * 128) + stages * (2 * 16384 + 2 * BN * 128) + 1024);
      k.persistent = true;
      k.max_grid = (unsigned)std::min<int64_t>(tiles, 0x7fffffff);
      k.grid[0] = k.max_grid;
      std::ostringstream d;
      d << "gemm tcgen05 tf32x3 128x" << BN << "x32, operands split in the kernel (" << rstages << " raw + " << stages << " operand stages)";
      k.desc = d.str();
      out->push_back(k);
      return;
    }
    if (da == F32 && db == F32 && K % 4 == 0 && M <= 0x7fffffff && N <= 0x7fffffff && K <= 0x7fffffff) {
      auto align256 = [](int64_t v) { return (v + 255) / 256 * 256; };
      const int64_t a_bytes = a_presplit ? 0 : align256(M * K * 4), b_bytes = align256(K * N * 4);
      const int64_t off_ahi = 0, off_alo = a_bytes, off_bhi = 2 * a_bytes, off_blo = 2 * a_bytes + b_bytes, off_acc = 2 * a_bytes + 2 * b_bytes;
      // Problems with far fewer 128 x 128 tiles than SMs split the contraction over the idle SMs (single-CTA kernel
      // only): an MMA instruction takes about 90 ns whatever its width, so the time of a small product is the
      // number of k steps of one tile, and narrower tiles do not shorten it.  ks parts of whole 128-element chunks,
      // none empty; partial tiles meet in an fp32 accumulation tile that the pre-pass clears.
      int ks = 1;
      const bool will_pair = tun.gemm_pair == 1 || (tun.gemm_pair == 0 && ((((M + 255) / 256) * ((N + 255) / 256) >= 56 && K >= 512) || ((M + 255) / 256) * ((N + 255) / 256) >= 512) && tun.gemm_bn == 0);
      {
        const int64_t tiles128 = ((M + 127) / 128) * ((N + 127) / 128), nch = ((K + 31) / 32 + 3) / 4;
        if (!will_pair && !tun.gemm_no_ksplit && tun.gemm_bn == 0 && N > 64 && tiles128 * 2 <= 148 && nch >= 8) {   // K >= 1024: measured 1024^3 chains 31.7 -> 29.9 us, 1024 x 4096 x 1024 95 -> 70 us; at K = 256 the clearing, the atomics and the read-back cost more than the shorter loop saves (13.5 -> 16.8 us)
          const int64_t want = std::min<int64_t>(148 / tiles128, nch);
          const int64_t cpp = (nch + want - 1) / want;
          ks = (int)((nch + cpp - 1) / cpp);
        }
      }
      const int64_t ks_tiles = ((M + 127) / 128) * ((N + 127) / 128);
      const int64_t acc_bytes = ks > 1 ? align256(ks_tiles * 128 * 128 * 4 + ks_tiles * 4) : 0;
      *scratch_bytes = std::max<size_t>(*scratch_bytes, (size_t)(2 * a_bytes + 2 * b_bytes + acc_bytes));
      auto scratch = [](int64_t off) {
        BufRef r;
        r.kind = BufRef::Scratch;
        r.scratch_off = off;
        return r;
      };
      auto node_buf = [&](int node) {
        BufRef r;
        r.node = node;
        r.ws_copy = g.nodes[node].cls != OpClass::Input && p.ws_offset[node] >= 0;
        return r;
      };
      {  // split pre-pass
        KernelSpec k;
        k.name = "hct_split_tf32_g" + std::to_string(gi);
        std::ostringstream src;
        src << "#define HCT_M " << M << "LL\n#define HCT_N " << N << "LL\n#define HCT_K " << K << "LL\n#define HCT_SPLIT_A " << (a_presplit ? 0 : 1)
            << "\n#define HCT_ZERO_VEC4 " << acc_bytes / 16 << "LL\n#define HCT_KERNEL_NAME " << k.name << "\n"
            << skeleton_source("common") << "\nstruct HctParams { void* ptr[7]; };\n" << skeleton_source("split_tf32");
        k.source = src.str();
        k.ptrs = {node_buf(anchor.args[0].node), node_buf(anchor.args[1].node), scratch(off_ahi), scratch(off_alo), scratch(off_bhi),
                  scratch(off_blo), scratch(off_acc)};
        int64_t blocks = (a_presplit ? 0 : (M * K / 4 + 1023) / 1024) + ((K + 31) / 32) * ((N + 31) / 32);
        k.grid[0] = (unsigned)std::max<int64_t>(1, std::min<int64_t>(blocks, 148 * 16));
        k.block[0] = 256;
        k.desc = a_presplit ? "tf32 head/tail split of the second gemm operand, transposed (the first arrives split)"
                            : "tf32 head/tail split of both gemm operands, B transposed";
        out->push_back(k);
      }
      // 256-column tiles (`gemm_bn=256`) halve the instruction count but were measured no faster than 128-column ones
      // (28 against 26 us on 1024 x 256 x 4096): with head and tail of both operands a k step moves 96 KB into shared
      // memory per 6 MFLOP, and the kernel runs at the rate L2 delivers them.  They are taken on request only.
      const int bn_max = N > 128 ? 256 : N > 64 ? 128 : N > 32 ? 64 : 32;
      int BN = std::min(bn_max, 128);
      while (ks == 1 && BN > 64 && ((M + 127) / 128) * ((N + BN - 1) / BN) * 2 <= 148) BN /= 2;
      if (tun.gemm_bn >= 32) BN = std::min(bn_max, tun.gemm_bn >= 256 ? 256 : tun.gemm_bn >= 128 ? 128 : tun.gemm_bn >= 64 ? 64 : 32);
      int stages = BN == 256 ? 2 : BN == 128 ? 3 : BN == 64 ? 4 : 5;
      std::string epi = eg.run_fn(N);
      // CTA pairs on 256 x 256 tiles when every pair of SMs gets at least one tile.  Measured on
      // 16384 x 4096 x 4096: 2.31 ms against 2.93 ms for 128 x 128 tiles on single CTAs (a TF32 MMA of
      // 128 columns does not fill the tensor pipe's issue interval; 256 columns per instruction do).
      const int64_t pair_tiles32 = ((M + 255) / 256) * ((N + 255) / 256);
      // (from 56 tiles on, and a contraction deep enough to amortise the pair's set-up: measured break-even)
      // (a shallow contraction still gains once there are several rounds of tiles: 16384 x 256 x 4096 measured 224 against 254 us)
      if (tun.gemm_pair == 1 || (tun.gemm_pair == 0 && ((pair_tiles32 >= 56 && K >= 512) || pair_tiles32 >= 512) && tun.gemm_bn == 0)) {
        const int pstages = 3;
        KernelSpec k;
        k.name = "hct_gemm_tc2_tf32x3_g" + std::to_string(gi);
        std::ostringstream src;
        src << "#define HCT_M " << M << "LL\n#define HCT_N " << N << "LL\n#define HCT_K " << K << "LL\n#define HCT_STAGES " << pstages
            << "\n#define HCT_TF32X3 1\n#define HCT_STATUS_SLOT " << eg.ptrs.size() << "\n#define HCT_KERNEL_NAME " << k.name << "\n";
        src << skeleton_source("common") << "\n" << skeleton_source("tc_common") << "\nstruct HctParams { HctTensorMap tmap[4]; void* ptr["
            << eg.ptrs.size() + 1 << "]; };\n" << epi << skeleton_source("gemm_tc2");
        k.source = src.str();
        k.ptrs = eg.ptrs;
        k.wants_status = true;
        for (int i = 0; i < 4; ++i) {
          TmaDesc t;
          t.buf = scratch(i == 0 ? off_ahi : i == 1 ? off_alo : i == 2 ? off_bhi : off_blo);
          if (a_presplit && i < 2) {
            t.buf = node_buf(anchor.args[0].node);
            t.base_offset = i == 0 ? 0 : (uint64_t)p.split_lo_offset[anchor.args[0].node];
          }
          t.elem_bytes = 4;
          t.rank = 2;
          t.dims[0] = (uint64_t)K; t.dims[1] = (uint64_t)(i < 2 ? M : N);   // B is transposed to [N,K]
          t.strides[1] = (uint64_t)K * 4;
          t.box[0] = 32; t.box[1] = 128;
          k.tmaps.push_back(t);
        }
        k.block[0] = 320;
        k.smem_bytes = (unsigned)(pstages * 65536 + 1024);
        k.persistent = true;
        k.cluster = 2;
        k.max_grid = (unsigned)std::min<int64_t>(2 * pair_tiles32, 0x7ffffffe);
        k.grid[0] = k.max_grid;
        k.desc = "gemm tcgen05 tf32x3 on CTA pairs, 256x256x32 per pair, " + std::to_string(pstages) + " stages";
        out->push_back(k);
        return;
      }
      KernelSpec k;
      k.name = "hct_gemm_tc_tf32x3_g" + std::to_string(gi);
      std::ostringstream src;
      src << "#define HCT_M " << M << "LL\n#define HCT_N " << N << "LL\n#define HCT_K " << K << "LL\n#define HCT_BN " << BN
          << "\n#define HCT_STAGES " << stages << "\n#define HCT_TF32X3 1\n#define HCT_KSPLIT " << ks << "\n#define HCT_KS_SLOT " << eg.ptrs.size()
          << "\n#define HCT_STATUS_SLOT " << eg.ptrs.size() + (ks > 1 ? 1 : 0)
          << "\n#define HCT_KERNEL_NAME " << k.name << "\n";
      src << skeleton_source("common") << "\n" << skeleton_source("tc_common") << "\nstruct HctParams { HctTensorMap tmap[4]; void* ptr["
          << eg.ptrs.size() + (ks > 1 ? 2 : 1) << "]; };\n" << epi << skeleton_source("gemm_tc");
      k.source = src.str();
      k.ptrs = eg.ptrs;
      if (ks > 1) k.ptrs.push_back(scratch(off_acc));
      k.wants_status = true;
      for (int i = 0; i < 4; ++i) {
        TmaDesc t;
        t.buf = scratch(i == 0 ? off_ahi : i == 1 ? off_alo : i == 2 ? off_bhi : off_blo);
        if (a_presplit && i < 2) {
          t.buf = node_buf(anchor.args[0].node);
          t.base_offset = i == 0 ? 0 : (uint64_t)p.split_lo_offset[anchor.args[0].node];
        }
        t.elem_bytes = 4;
        t.rank = 2;
        if (i < 2) {
          t.dims[0] = (uint64_t)K; t.dims[1] = (uint64_t)M;
          t.strides[1] = (uint64_t)K * 4;
          t.box[0] = 32; t.box[1] = 128;
        } else {  // B transposed to [N,K]
          t.dims[0] = (uint64_t)K; t.dims[1] = (uint64_t)N;
          t.strides[1] = (uint64_t)K * 4;
          t.box[0] = 32; t.box[1] = (uint32_t)BN;
        }
        k.tmaps.push_back(t);
      }
      int64_t tiles = ((M + 127) / 128) * ((N + BN - 1) / BN) * ks;
      k.block[0] = BN > 128 ? 320 : 192;   // wide tiles: eight epilogue warps
      k.smem_bytes = (unsigned)(stages * (2 * 128 * 128 + 2 * BN * 128) + 1024);
      k.persistent = true;
      k.max_grid = (unsigned)std::min<int64_t>(tiles, 0x7fffffff);
      k.grid[0] = k.max_grid;
      std::ostringstream d;
      d << "gemm tcgen05 tf32x3 128x" << BN << "x32, " << stages << " stages";
      if (ks > 1) d << ", contraction split " << ks << " ways over idle SMs";
      k.desc = d.str();
      out->push_back(k);
      return;
    }
  }

  // ---- tensor-core convolution: bf16 inputs; layout pre-pass, then implicit GEMM
  if (grp.kind == GroupKind::Conv && !tun.simt_only) {
    const auto& xs = a.shape;
    const auto& ws = b.shape;
    // weights must be a graph input (they take a layout pre-pass); the activations may be an earlier kernel's bf16 result
    bool in_bf16 = b.cls == OpClass::Input && a.dtype == BF16 && b.dtype == BF16;
    int64_t NB = xs[0], C = xs[1], H = xs[2], W = xs[3], KO = ws[0], FR = ws[2], FS = ws[3];
    int64_t HO = anchor.shape[2], WO = anchor.shape[3];
    // Stride and dilation other than 1 take the per-tap schedule: the pixel box of a tap is loaded with a
    // traversal stride (every ST-th pixel of every ST-th row), which the tensor map allows up to 8 and a box of 256.
    const int64_t ST = anchor.stride, DIL = anchor.dilation;
    const bool unit = ST == 1 && DIL == 1;
    // Rows too wide for one strided box (W' * stride > 256) with a stride that divides both image extents:
    // dense boxes of a stride-phase view.  Both forms were measured at the same speed; `conv_phase=1` prefers the view.
    const bool phased = ST > 1 && ST <= 8 && H % ST == 0 && W % ST == 0 && (WO * ST > 256 || tun.conv_phase);
    // Pointwise convolution on NCHW data: per image the product W[KO,C] * X_n[C,HW], both operands usable as they lie
    // in memory (weights K-major, pixels N-major): no layout pass at all.
    if (in_bf16 && anchor.groups == 1 && FR == 1 && FS == 1 && ST == 1 && anchor.pad == 0 && !a.nhwc && (H * W) % 8 == 0 && C % 8 == 0 &&
        NB <= 0x7fffffff && KO <= 0x7fffffff && H * W <= 0x7fffffff && !tun.conv_no_pointwise) {
      const int64_t HW = H * W;
      const bool tma_store = grp.stores.size() == 1 && grp.stores[0].dtype == BF16 && !tun.conv_no_tma_store && !nhwc_out;
      // Epilogue warps: with 64 filters or fewer only one or two lane quarters hold results, so four warps per quarter
      // (measured 14.3 against 18.4 us on 192 -> 32 channels at 32 x 56 x 56); with many filters and a deep
      // contraction two per quarter and a fourth stage are faster (22.0 against 27.8 us on 256 -> 256 channels).
      const int epw = tun.conv_pw_warps == 8 ? 8 : tun.conv_pw_warps == 16 ? 16 : KO <= 64 ? 16 : 8;
      const int stages = tma_store && epw == 16 ? 3 : 4;
      std::string epi = eg.run_fn(HW, 32, "(row % " + std::to_string(KO) + "LL)", tma_store);
      KernelSpec k;
      k.name = "hct_conv_pw_bf16_g" + std::to_string(gi);
      std::ostringstream src;
      src << "#define HCT_NB_IMG " << NB << "\n#define HCT_C " << C << "\n#define HCT_KO " << KO << "\n#define HCT_HW " << HW
          << "\n#define HCT_STAGES " << stages << "\n#define HCT_EPW " << epw << "\n#define HCT_TMA_STORE " << (tma_store ? 1 : 0) << "\n#define HCT_STATUS_SLOT " << eg.ptrs.size()
          << "\n#define HCT_KERNEL_NAME " << k.name << "\n";
      src << skeleton_source("common") << "\n" << skeleton_source("tc_common") << "\nstruct HctParams { HctTensorMap tmap[" << (tma_store ? 3 : 2)
          << "]; void* ptr[" << eg.ptrs.size() + 1 << "]; };\n" << epi << skeleton_source("conv_pw_tc");
      k.source = src.str();
      k.ptrs = eg.ptrs;
      k.wants_status = true;
      auto node_buf = [&](int node) {
        BufRef r;
        r.node = node;
        r.ws_copy = g.nodes[node].cls != OpClass::Input && p.ws_offset[node] >= 0;
        return r;
      };
      TmaDesc tw;   // weights [KO, C]
      tw.buf = node_buf(anchor.args[1].node);
      tw.elem_bytes = 2;
      tw.rank = 2;
      tw.dims[0] = (uint64_t)C; tw.dims[1] = (uint64_t)KO;
      tw.strides[1] = (uint64_t)C * 2;
      tw.box[0] = 64; tw.box[1] = 128;
      TmaDesc tx;   // pixels [image][C][HW]
      tx.buf = node_buf(anchor.args[0].node);
      tx.elem_bytes = 2;
      tx.rank = 3;
      tx.dims[0] = (uint64_t)HW; tx.dims[1] = (uint64_t)C; tx.dims[2] = (uint64_t)NB;
      tx.strides[1] = (uint64_t)HW * 2; tx.strides[2] = (uint64_t)C * HW * 2;
      tx.box[0] = 64; tx.box[1] = 64; tx.box[2] = 1;
      k.tmaps = {tw, tx};
      if (tma_store) {   // result [image][KO][HW]: 32 channels x 64 pixels, 128-byte swizzle
        TmaDesc ty;
        ty.buf.node = grp.stores[0].node;
        ty.buf.ws_copy = !grp.stores[0].to_output;
        ty.elem_bytes = 2;
        ty.rank = 3;
        ty.dims[0] = (uint64_t)HW; ty.dims[1] = (uint64_t)KO; ty.dims[2] = (uint64_t)NB;
        ty.strides[1] = (uint64_t)HW * 2; ty.strides[2] = (uint64_t)KO * HW * 2;
        ty.box[0] = 64; ty.box[1] = 32; ty.box[2] = 1;
        ty.swizzle = 3;
        k.tmaps.push_back(ty);
      }
      const int64_t tiles = NB * ((HW + 255) / 256) * ((KO + 127) / 128);
      k.block[0] = (unsigned)(64 + 32 * epw);
      k.smem_bytes = (unsigned)(stages * (128 * 128 + 32768) + (tma_store ? epw * 4096 : 0) + 1024);
      k.persistent = true;
      k.max_grid = (unsigned)std::min<int64_t>(tiles, 0x7fffffff);
      k.grid[0] = k.max_grid;
      k.desc = "conv2d 1x1 tcgen05 bf16 as a per-image GEMM on NCHW data (weights and pixels read in place), tile 128 channels x 256 pixels";
      out->push_back(k);
      return;
    }
    // Groups (other than depthwise, which has a kernel of its own): every block of 128 filters contracts the dense
    // window of input channels that its groups span, against weights that are zero outside each filter's own group.
    // The window must start on a 16-byte boundary of the channels-last pixel rows for every block.
    const int64_t G = anchor.groups, CPG = C / G, KPG = KO / G;
    int64_t cbw = 0;    // 64-channel blocks of the widest window
    bool grouped_ok = G > 1 && CPG > 1;
    if (grouped_ok)
      for (int64_t k0 = 0; k0 < KO; k0 += 128) {
        const int64_t g_lo = k0 / KPG, g_hi = (std::min<int64_t>(k0 + 127, KO - 1)) / KPG;
        if ((g_lo * CPG) % 8 != 0) grouped_ok = false;
        cbw = std::max<int64_t>(cbw, ((g_hi - g_lo + 1) * CPG + 63) / 64);
      }
    const int64_t CWP = cbw * 64;
    if (in_bf16 && (G == 1 || grouped_ok) && ST <= 8 && (WO * ST <= 256 || phased) && C % 8 == 0 && WO <= 256 && NB <= 0x7fffffff && FR * FS * KO <= 0x7fffffff && H <= 0x7fffff && W <= 0x7fffff) {
      // Three schedules.  (1) Rows whose byte length is a multiple of 16 and that fill most of a 32-column
      // pitch: the kernel reads NCHW itself and re-lays pixels in shared memory (conv_tc_nchw); only the
      // weights take a pre-pass.  Otherwise a pre-pass writes an NHWC copy and pixels are loaded
      // (2) once per filter row and shared by its taps (conv_tc_halo) or (3) once per tap (conv_tc).
      const int64_t pitch = (WO + FS - 1 + 31) / 32 * 32;
      const bool dense_pitch = pitch <= 256 && WO * 10 >= pitch * 7;
      const int th_pitch = (int)std::max<int64_t>(1, std::min<int64_t>(256 / std::max<int64_t>(pitch, 1), HO));
      // Slots of the pixel staging ring and operand buffers (a deeper ring was measured on 1x1 convolutions,
      // whose tiles have a single weight stage, and changed nothing: their limit is the epilogue's store rate).
      int n_stg = 3, n_buf = 2;
      if (tun.conv_nstg >= 2 && tun.conv_nstg <= 12) n_stg = tun.conv_nstg;
      if (tun.conv_nbuf >= 2 && tun.conv_nbuf <= 3) n_buf = tun.conv_nbuf;
      int n_a = 0;
      bool direct = false, flat = false;
      // Flat tiling of the NCHW-reading kernel: tiles of 256 consecutive positions at the pitch of the padded row.
      // An MMA takes about the same time whatever its width, so the schedule with fewer K loops on the busiest
      // CTA wins: whole-row tiles cost one more loop whenever their count is not a multiple of the grid.
      const int64_t flat_p = W + 2 * anchor.pad, flat_win = 256 + (FR - 1) * flat_p + FS - 1;
      const int64_t flat_tiles = NB * ((HO * flat_p + 255) / 256) * ((KO + 127) / 128);
      const int64_t flat_buf = (flat_win * 128 + 1023) / 1024 * 1024;
      // The epilogue of the NCHW-reading kernel hands its bf16 output to TMA stores (through 16 KB of
      // shared memory) when it stores a single bf16 tensor (output or intermediate) whose rows are 16-byte multiples.
      const bool tma_store = grp.stores.size() == 1 && grp.stores[0].dtype == BF16 && WO % 8 == 0 && !tun.conv_no_tma_store && !nhwc_out;
      const bool x_nhwc = a.nhwc;   // the activations already are channels-last: no layout pass, and no NCHW-reading schedule
      if (unit && dense_pitch && W % 8 == 0 && !tun.conv_no_direct && !x_nhwc && G == 1) {
        // shared memory: operand buffers of TH + FR - 1 rows, staging ring, output staging, and what is left for the weight ring
        const int64_t fixed = n_buf * ((th_pitch + FR - 1) * pitch * 128 + 1024) + n_stg * pitch * 128 + 1024 + (tma_store ? 16384 : 0);
        n_a = (int)std::min<int64_t>(6, (232448 - 512 - fixed) / 16384);
        direct = n_a >= 3;
        if (direct && grp.stores.size() == 1 && grp.stores[0].dtype == BF16 && WO >= 32 && FS - 1 <= 4 && flat_p <= pitch && tun.conv_flat != 2 && !nhwc_out) {
          const int64_t row_tiles = NB * ((HO + th_pitch - 1) / th_pitch) * ((KO + 127) / 128);
          const int64_t loops_row = row_tiles / 148 + (row_tiles % 148 ? 1 : 0), loops_flat = (flat_tiles + 147) / 148;
          const int64_t fixed_flat = n_buf * flat_buf + n_stg * pitch * 128 + 1024 + 16384;
          const int n_a_flat = (int)std::min<int64_t>(6, (232448 - 512 - fixed_flat) / 16384);
          (void)loops_row; (void)loops_flat;
          // measured slower than whole-row tiles on the benchmark convolution (37.9 against 35.8 us: its epilogue cannot use TMA
          // stores and its tiles need more input rows), so it is taken on request only
          if (n_a_flat >= 3 && tun.conv_flat == 1) {
            flat = true;
            n_a = n_a_flat;
            // what the weight ring leaves over goes to the pixel staging ring: a flat tile needs more input rows before its first MMA
            const int64_t left_over = 232448 - 512 - fixed_flat - (int64_t)n_a * 16384;
            if (tun.conv_nstg == 0) n_stg += (int)std::min<int64_t>(3, left_over / (pitch * 128));
          }
        }
      }
      const bool halo = unit && !direct && FS > 1 && dense_pitch && !tun.conv_no_halo;
      const int TH = (direct || halo) ? th_pitch : (int)std::max<int64_t>(1, std::min<int64_t>(256 / WO, std::min<int64_t>(HO, phased ? 256 : 256 / ST)));
      auto align256 = [](int64_t v) { return (v + 255) / 256 * 256; };
      const int64_t x_bytes = (direct || x_nhwc) ? 0 : align256(NB * C * H * W * 2), w_bytes = align256(KO * (G > 1 ? CWP : C) * FR * FS * 2);
      // On request (conv_ksplit=1; measured slower than the cut by rows alone, whose pieces overlap the other
      // CTAs' last tiles) a short last round of the NCHW-reading kernel is split by output row and by (channel
      // block, filter row) part of the contraction: 256 arrival counters (zeroed by the pre-pass) and one fp32 slice of
      // [128 channels][pitch] per piece follow the weight copy in scratch.
      const int ks_ctrs = 256, ks_max = 160;
      const bool ksplit = direct && !flat && tun.conv_ksplit && ((C + 63) / 64) * FR > 1;
      const int64_t ks_bytes = ksplit ? align256(ks_ctrs * 4 + (int64_t)ks_max * 128 * pitch * 4) : 0;
      *scratch_bytes = std::max<size_t>(*scratch_bytes, (size_t)(x_bytes + w_bytes + ks_bytes));
      auto scratch = [](int64_t off) {
        BufRef r;
        r.kind = BufRef::Scratch;
        r.scratch_off = off;
        return r;
      };
      auto node_buf = [&](int node) {
        BufRef r;
        r.node = node;
        r.ws_copy = g.nodes[node].cls != OpClass::Input && p.ws_offset[node] >= 0;
        return r;
      };
      {
        KernelSpec k;
        k.name = "hct_conv_prep_g" + std::to_string(gi);
        std::ostringstream src;
        src << "#define HCT_NB_IMG " << NB << "\n#define HCT_C " << C << "\n#define HCT_HW " << H * W << "\n#define HCT_KO " << KO
            << "\n#define HCT_RS " << FR * FS << "\n#define HCT_PREP_X " << ((direct || x_nhwc) ? 0 : 1) << "\n#define HCT_GROUPS " << G << "\n#define HCT_CWP " << CWP
            << "\n#define HCT_ZERO_WORDS " << (ksplit ? ks_ctrs : 0) << "\n#define HCT_KERNEL_NAME " << k.name << "\n"
            << skeleton_source("common") << "\nstruct HctParams { void* ptr[5]; };\n" << skeleton_source("conv_prep");
        k.source = src.str();
        k.ptrs = {node_buf(anchor.args[0].node), node_buf(anchor.args[1].node), scratch(0), scratch(x_bytes), scratch(x_bytes + w_bytes)};
        const bool w_only = direct || x_nhwc;
        const int64_t w_elems = KO * (G > 1 ? CWP : C) * FR * FS;
        int64_t blocks = w_only ? (w_elems / (G > 1 ? 1 : 8) + 255) / 256 : NB * ((C + 63) / 64) * ((H * W + 63) / 64) + (w_elems + 255) / 256;
        k.grid[0] = (unsigned)std::max<int64_t>(1, std::min<int64_t>(blocks, w_only ? 148 : 148 * 16));
        k.block[0] = 256;
        k.desc = w_only ? "conv weight pre-pass: KCRS->RSKC" : "conv layout pre-pass: NCHW->NHWC activations, KCRS->RSKC weights";
        if (G > 1) k.desc += " (per filter a window of " + std::to_string(CWP) + " channels, zero outside its group)";
        out->push_back(k);
      }
      int stages = 4;
      const bool use_tma_store = direct && tma_store && !flat;
      std::string epi = eg.run_fn(HO * WO, flat ? 1 : WO, "(row % " + std::to_string(KO) + "LL)", use_tma_store || flat);
      const int out_slot = flat ? eg.ptr_index(grp.stores[0].node, !grp.stores[0].to_output) : 0;
      KernelSpec k;
      k.name = "hct_conv_tc_bf16_g" + std::to_string(gi);
      std::ostringstream src;
      src << "#define HCT_NB_IMG " << NB << "\n#define HCT_C " << C << "\n#define HCT_H " << H << "\n#define HCT_W " << W
          << "\n#define HCT_GROUPS " << G << "\n#define HCT_CBW " << cbw
          << "\n#define HCT_KO " << KO << "\n#define HCT_FR " << FR << "\n#define HCT_FS " << FS << "\n#define HCT_PAD " << anchor.pad
          << "\n#define HCT_STRIDE " << ST << "\n#define HCT_DIL " << DIL << "\n#define HCT_PHASED " << (phased ? 1 : 0) << "\n#define HCT_HO " << HO << "\n#define HCT_WO " << WO << "\n#define HCT_TH " << TH << "\n#define HCT_TH2 1\n#define HCT_SPLIT "
          << (flat ? 1 : TH) << "\n#define HCT_PITCH " << pitch << "\n#define HCT_NA " << (direct ? n_a : 6) << "\n#define HCT_NBUF " << (direct ? n_buf : 3)
          << "\n#define HCT_FLAT " << (flat ? 1 : 0) << "\n#define HCT_P " << flat_p << "\n#define HCT_OUT_SLOT " << out_slot
          << "\n#define HCT_NSTG " << n_stg << "\n#define HCT_X_IS_INPUT " << (a.cls == OpClass::Input ? 1 : 0) << "\n#define HCT_TMA_STORE " << (use_tma_store ? 1 : 0) << "\n#define HCT_STAGES " << stages
          << "\n#define HCT_KSPLIT " << (ksplit ? 1 : 0) << "\n#define HCT_KS_SLOT " << eg.ptrs.size() << "\n#define HCT_KS_CTRS " << ks_ctrs << "\n#define HCT_KS_MAX " << ks_max
          << "\n#define HCT_STATUS_SLOT " << eg.ptrs.size() + (ksplit ? 1 : 0)
          << "\n#define HCT_KERNEL_NAME " << k.name << "\n";
      src << skeleton_source("common") << "\n" << skeleton_source("tc_common") << "\nstruct HctParams { HctTensorMap tmap[" << (phased ? 1 + 2 * ST : use_tma_store ? 3 : direct ? 2 : 3)
          << "]; void* ptr[" << eg.ptrs.size() + (ksplit ? 2 : 1) << "]; };\n" << epi << skeleton_source(direct ? "conv_tc_nchw" : halo ? "conv_tc_halo" : "conv_tc");
      k.source = src.str();
      k.ptrs = eg.ptrs;
      if (ksplit) k.ptrs.push_back(scratch(x_bytes + w_bytes));
      k.wants_status = true;
      TmaDesc tw;
      tw.buf = scratch(x_bytes);
      tw.elem_bytes = 2;
      tw.rank = 2;
      tw.dims[0] = (uint64_t)(G > 1 ? CWP : C); tw.dims[1] = (uint64_t)(FR * FS * KO);
      tw.strides[1] = (uint64_t)(G > 1 ? CWP : C) * 2;
      tw.box[0] = 64; tw.box[1] = 128;
      TmaDesc tx;
      tx.buf = x_nhwc ? node_buf(anchor.args[0].node) : scratch(0);
      tx.elem_bytes = 2;
      tx.rank = 4;
      tx.dims[0] = (uint64_t)C; tx.dims[1] = (uint64_t)W; tx.dims[2] = (uint64_t)H; tx.dims[3] = (uint64_t)NB;
      tx.strides[1] = (uint64_t)C * 2; tx.strides[2] = (uint64_t)W * C * 2; tx.strides[3] = (uint64_t)H * W * C * 2;
      tx.box[0] = 64; tx.box[1] = (uint32_t)(halo ? pitch : phased ? 1 : WO * ST); tx.box[2] = (uint32_t)(phased ? 1 : TH * ST); tx.box[3] = 1;
      tx.estride[1] = tx.estride[2] = (uint32_t)(phased ? 1 : ST);   // (with a phase view these two maps are replaced below)
      TmaDesc tx2 = tx;
      tx2.box[2] = (uint32_t)(phased ? 1 : ST);
      k.tmaps = {tw, tx, tx2};
      if (phased) {
        // view of the NHWC copy for row phase ph: [n][h / ST][w / ST][w mod ST][c], starting ph rows into each image
        k.tmaps = {tw};
        for (int piece = 0; piece < 2; ++piece)
          for (int64_t ph = 0; ph < ST; ++ph) {
            TmaDesc tp;
            tp.buf = x_nhwc ? node_buf(anchor.args[0].node) : scratch(0);
            tp.base_offset = (uint64_t)(ph * W * C * 2);
            tp.elem_bytes = 2;
            tp.rank = 5;
            tp.dims[0] = (uint64_t)C; tp.dims[1] = (uint64_t)ST; tp.dims[2] = (uint64_t)(W / ST); tp.dims[3] = (uint64_t)(H / ST); tp.dims[4] = (uint64_t)NB;
            tp.strides[1] = (uint64_t)C * 2; tp.strides[2] = (uint64_t)ST * C * 2; tp.strides[3] = (uint64_t)ST * W * C * 2;
            tp.strides[4] = (uint64_t)H * W * C * 2;
            tp.box[0] = 64; tp.box[1] = 1; tp.box[2] = (uint32_t)WO; tp.box[3] = (uint32_t)(piece ? 1 : TH); tp.box[4] = 1;
            k.tmaps.push_back(tp);
          }
      }
      if (direct) {  // NCHW input: [64 channels x pitch pixels] of one row, no swizzle (the kernel re-lays it)
        TmaDesc tn;
        tn.buf = node_buf(anchor.args[0].node);
        tn.elem_bytes = 2;
        tn.rank = 4;
        tn.dims[0] = (uint64_t)W; tn.dims[1] = (uint64_t)H; tn.dims[2] = (uint64_t)C; tn.dims[3] = (uint64_t)NB;
        tn.strides[1] = (uint64_t)W * 2; tn.strides[2] = (uint64_t)H * W * 2; tn.strides[3] = (uint64_t)C * H * W * 2;
        tn.box[0] = (uint32_t)pitch; tn.box[1] = 1; tn.box[2] = 64; tn.box[3] = 1;
        tn.swizzle = 0;
        k.tmaps = {tw, tn};
        if (use_tma_store) {  // NCHW output: [32 channels x 32 pixels] of one row, 64-byte swizzle
          TmaDesc ty;
          ty.buf.node = grp.stores[0].node;
          ty.buf.ws_copy = !grp.stores[0].to_output;
          ty.elem_bytes = 2;
          ty.rank = 4;
          ty.dims[0] = (uint64_t)WO; ty.dims[1] = (uint64_t)HO; ty.dims[2] = (uint64_t)KO; ty.dims[3] = (uint64_t)NB;
          ty.strides[1] = (uint64_t)WO * 2; ty.strides[2] = (uint64_t)HO * WO * 2; ty.strides[3] = (uint64_t)KO * HO * WO * 2;
          ty.box[0] = 32; ty.box[1] = 1; ty.box[2] = 32; ty.box[3] = 1;
          ty.swizzle = 2;
          k.tmaps.push_back(ty);
        }
      }
      int64_t tiles = flat ? flat_tiles : NB * ((HO + TH - 1) / TH) * ((KO + 127) / 128);
      k.block[0] = flat ? 608 : direct ? 480 : 192;
      k.smem_bytes = flat   ? (unsigned)(n_a * 16384 + n_buf * flat_buf + n_stg * pitch * 128 + 1024 + 16384)
                     : direct ? (unsigned)(n_a * 16384 + n_buf * ((TH + FR - 1) * pitch * 128 + 1024) + n_stg * pitch * 128 + 1024 +
                                         (use_tma_store ? 16384 : 0))
                     : halo ? (unsigned)(6 * 16384 + 3 * 33792 + 1024) : (unsigned)(stages * (128 * 128 + 32768) + 1024);
      k.persistent = true;
      k.max_grid = (unsigned)std::min<int64_t>(tiles, 0x7fffffff);
      k.grid[0] = k.max_grid;
      std::ostringstream d;
      d << "conv2d tcgen05 bf16 implicit GEMM, tile 128 channels x " << TH << " rows of " << WO << " pixels, ";
      if (G > 1) d << G << " groups as dense windows of " << CWP << " input channels per block of filters, ";
      if (flat)
        d << "NCHW read directly and re-laid in shared memory, flat tiles of 256 positions at pitch " << flat_p;
      else if (direct)
        d << "NCHW read directly and re-laid in shared memory, every pixel loaded once per tile (pitch " << pitch << ")";
      else if (halo)
        d << "pixels shared by the taps of a filter row (pitch " << pitch << ")" << (x_nhwc ? ", channels-last input read in place" : "");
      else
        d << stages << " stages" << (unit ? "" : phased ? ", dense pixel boxes of a stride-phase view" : ", strided pixel boxes")
          << (x_nhwc ? ", channels-last input read in place" : "");
      k.desc = d.str();
      out->push_back(k);
      return;
    }
  }

  if (grp.kind == GroupKind::Conv && a.nhwc)
    throw Error(HCT_ERR_UNSUPPORTED, "a channels-last (nhwc) input needs the tensor-core convolution: bf16 operands, channels a multiple of 8 (per group too), stride <= 8");
  for (auto& st : grp.stores)
    if (p.partial_cols[st.node] > 0)
      throw Error(HCT_ERR_UNSUPPORTED, "row sums folded into a GEMM epilogue need the tensor-core kernel (not available with simt_only)");
  if (grp.kind == GroupKind::Gemm && p.split_store[anchor.args[0].node])
    throw Error(HCT_ERR_UNSUPPORTED, "an operand stored as TF32 head and tail needs the tensor-core GEMM (not available with simt_only)");
  auto operand_buf = [&](int node) {
    return eg.ptr_index(node, g.nodes[node].cls != OpClass::Input && p.ws_offset[node] >= 0);
  };
  int pa = operand_buf(anchor.args[0].node);
  int pb = operand_buf(anchor.args[1].node);
  DType ta = eg.buf_dtype(anchor.args[0].node), tb = eg.buf_dtype(anchor.args[1].node);
  std::string epi = eg.scalar_fn();

  KernelSpec k;
  std::ostringstream src;
  if (grp.kind == GroupKind::Gemm) {
    int64_t M = a.shape[0], K = a.shape[1], N = b.shape[1];
    k.name = "hct_gemm_simt_g" + std::to_string(gi);
    src << "#define HCT_M " << M << "LL\n#define HCT_N " << N << "LL\n#define HCT_K " << K << "LL\n";
    src << "#define HCT_TA " << ctype(ta) << "\n#define HCT_TB " << ctype(tb) << "\n#define HCT_PA " << pa << "\n#define HCT_PB "
        << pb << "\n#define HCT_KERNEL_NAME " << k.name << "\n";
    src << skeleton_source("common") << "\nstruct HctParams { void* ptr[" << eg.ptrs.size() << "]; };\n" << epi
        << skeleton_source("gemm_simt");
    k.grid[0] = (unsigned)((N + 63) / 64);
    k.grid[1] = (unsigned)((M + 63) / 64);
    if ((M + 63) / 64 > 65535) throw Error(HCT_ERR_UNSUPPORTED, "gemm with more than 4M rows is not supported");
    k.block[0] = 256;
    k.desc = "gemm fp32-FMA 64x64x16";
  } else if (anchor.groups == a.shape[1] && b.shape[1] == 1 && b.shape[2] * b.shape[3] <= 49 && !tun.simt_only) {
    // depthwise: memory-bound, one thread per column of P vertically adjacent output pixels
    const auto& xs = a.shape;
    const auto& ws = b.shape;
    int P = 1;
    for (int cand : {4, 2})
      if (cand <= anchor.shape[2] && ((cand - 1) * anchor.stride + (ws[2] - 1) * anchor.dilation + 1) * ws[3] <= 160) { P = cand; break; }
    // Stride 1, no dilation, rows of whole 16-byte vectors, padding no wider than half the filter: blocks of 8 columns per thread
    const int64_t HOd = anchor.shape[2], WOd = anchor.shape[3];
    const bool vec = anchor.stride == 1 && anchor.dilation == 1 && xs[3] % 8 == 0 && WOd % 8 == 0 && 2 * anchor.pad <= ws[3] - 1 &&
                     ws[3] <= 7 && xs[0] * ws[0] * HOd * (WOd / 8) < 0x7fffffffLL;
    // Two filters per thread on packed multiply-adds (half the rows, so the accumulators need the same registers).
    // Measured slower than one filter per thread (24.5 against 22.6 us on 32 x 192 x 56 x 56: 128 registers instead
    // of 74 halve the resident warps, which costs more than the saved issue slots), so it is taken on request only.
    const bool pair = vec && ws[0] % 2 == 0 && tun.dw_pair == 1;
    if (vec) P = HOd >= 16 ? (pair ? 4 : 8) : HOd >= 4 ? 4 : HOd >= 2 ? 2 : 1;
    if (tun.dw_p == 1 || tun.dw_p == 2 || tun.dw_p == 4 || (tun.dw_p == 8 && vec)) P = tun.dw_p;
    const unsigned cta = (unsigned)std::min(1024, std::max(32, (tun.dw_cta > 0 ? tun.dw_cta : vec ? 128 : 256) / 32 * 32));
    const std::string epi_dw = vec ? eg.run_fn(HOd * WOd, WOd, "(row % " + std::to_string(ws[0]) + "LL)") : epi;
    k.name = "hct_conv_dw_g" + std::to_string(gi);
    src << "#define HCT_VEC " << (vec ? 1 : 0) << "\n#define HCT_PAIR " << (pair ? 1 : 0) << "\n#define HCT_CTA " << cta << "\n";
    src << "#define HCT_NB " << xs[0] << "\n#define HCT_C " << xs[1] << "\n#define HCT_MULT " << ws[0] / xs[1] << "\n#define HCT_H " << xs[2]
        << "\n#define HCT_W " << xs[3] << "\n#define HCT_FR " << ws[2] << "\n#define HCT_FS " << ws[3] << "\n#define HCT_STRIDE "
        << anchor.stride << "\n#define HCT_PAD " << anchor.pad << "\n#define HCT_DIL " << anchor.dilation << "\n#define HCT_HO "
        << anchor.shape[2] << "\n#define HCT_WO " << anchor.shape[3] << "\n#define HCT_P " << P << "\n";
    src << "#define HCT_TA " << ctype(ta) << "\n#define HCT_TB " << ctype(tb) << "\n#define HCT_PA " << pa << "\n#define HCT_PB "
        << pb << "\n#define HCT_KERNEL_NAME " << k.name << "\n";
    src << skeleton_source("common") << "\n" << (vec ? skeleton_source("tc_common") : std::string()) << "\nstruct HctParams { void* ptr["
        << eg.ptrs.size() << "]; };\n" << epi_dw << skeleton_source("conv_dw");
    int64_t units = xs[0] * (pair ? ws[0] / 2 : ws[0]) * ((anchor.shape[2] + P - 1) / P) * (vec ? WOd / 8 : WOd);
    k.grid[0] = (unsigned)std::max<int64_t>(1, std::min<int64_t>((units + cta - 1) / cta, 148 * 64));
    k.block[0] = cta;
    k.desc = "conv2d depthwise fp32-FMA, " + std::string(vec ? "8 columns x " : "") + std::to_string(P) + " output rows" +
             (pair ? " of two filters per thread (packed multiply-adds)" : " per thread");
  } else {
    const auto& xs = a.shape;
    const auto& ws = b.shape;
    k.name = "hct_conv_simt_g" + std::to_string(gi);
    src << "#define HCT_NB " << xs[0] << "\n#define HCT_CI " << ws[1] << "\n#define HCT_GROUPS " << anchor.groups << "\n#define HCT_H " << xs[2] << "\n#define HCT_W " << xs[3]
        << "\n#define HCT_KO " << ws[0] << "\n#define HCT_FR " << ws[2] << "\n#define HCT_FS " << ws[3] << "\n#define HCT_STRIDE "
        << anchor.stride << "\n#define HCT_PAD " << anchor.pad << "\n#define HCT_DIL " << anchor.dilation << "\n#define HCT_HO "
        << anchor.shape[2] << "\n#define HCT_WO " << anchor.shape[3] << "\n";
    src << "#define HCT_TA " << ctype(ta) << "\n#define HCT_TB " << ctype(tb) << "\n#define HCT_PA " << pa << "\n#define HCT_PB "
        << pb << "\n#define HCT_KERNEL_NAME " << k.name << "\n";
    src << skeleton_source("common") << "\nstruct HctParams { void* ptr[" << eg.ptrs.size() << "]; };\n" << epi
        << skeleton_source("conv_simt");
    int64_t total = anchor.numel();
    k.grid[0] = (unsigned)std::min<int64_t>((total + 255) / 256, 148 * 64);
    k.block[0] = 256;
    k.desc = "conv2d direct fp32-FMA";
  }
  k.source = src.str();
  k.ptrs = eg.ptrs;
  out->push_back(k);
}

}  // namespace hct
