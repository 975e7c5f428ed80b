// Generator for fused row kernels: elementwise, broadcast and row-reduction chains over one [R,C] space.
#include <cctype>
#include <cstdio>
#include <cstdlib>
#include <sstream>

#include "../../include/hct.h"
#include "codegen.h"

namespace hct {

namespace {
struct Knob {
  const char* key;    // schedule name; the environment variable is HCT_ + upper case
  int Tunables::*i;   // integer knob (with its lower bound), or
  int lo;
  bool Tunables::*b;  // boolean knob
};
const Knob kKnobs[] = {
    {"row_nv", &Tunables::row_nv, 1, nullptr},
    {"row_cta", &Tunables::row_cta, 32, nullptr},
    {"row_b", &Tunables::row_batch, 1, nullptr},
    {"row_cta_batched", &Tunables::row_cta_batched, 32, nullptr},
    {"row_cta_elementwise", &Tunables::row_cta_elementwise, 32, nullptr},
    {"row_cta_staged", &Tunables::row_cta_staged, 32, nullptr},
    {"row_minb", &Tunables::row_min_blocks, 1, nullptr},
    {"row_cta_small", &Tunables::row_cta_small, 32, nullptr},
    {"row_ring_bytes_small", &Tunables::row_ring_bytes_small, 1024, nullptr},
    {"row_ring_bytes", &Tunables::row_ring_bytes, 1024, nullptr},
    {"gemm_bn", &Tunables::gemm_bn, 0, nullptr},
    {"gemm_pair", &Tunables::gemm_pair, 0, nullptr},
    {"gemm_insplit", &Tunables::gemm_insplit, 0, nullptr},
    {"gemm_no_ksplit", nullptr, 0, &Tunables::gemm_no_ksplit},
    {"conv_nstg", &Tunables::conv_nstg, 0, nullptr},
    {"conv_nbuf", &Tunables::conv_nbuf, 0, nullptr},
    {"conv_flat", &Tunables::conv_flat, 0, nullptr},
    {"dw_p", &Tunables::dw_p, 0, nullptr},
    {"dw_cta", &Tunables::dw_cta, 0, nullptr},
    {"dw_pair", &Tunables::dw_pair, 0, nullptr},
    {"simt_only", nullptr, 0, &Tunables::simt_only},
    {"fault_never_arrive", nullptr, 0, &Tunables::fault_never_arrive},
    {"conv_no_halo", nullptr, 0, &Tunables::conv_no_halo},
    {"conv_no_tma_store", nullptr, 0, &Tunables::conv_no_tma_store},
    {"conv_no_direct", nullptr, 0, &Tunables::conv_no_direct},
    {"conv_ksplit", nullptr, 0, &Tunables::conv_ksplit},
    {"conv_no_pointwise", nullptr, 0, &Tunables::conv_no_pointwise},
    {"conv_pw_warps", &Tunables::conv_pw_warps, 0, nullptr},
    {"conv_phase", nullptr, 0, &Tunables::conv_phase},
    {"topk_no_select", nullptr, 0, &Tunables::topk_no_select},
    {"topk_no_reg", nullptr, 0, &Tunables::topk_no_reg},
    {"sort_no_reg", nullptr, 0, &Tunables::sort_no_reg},
    {"row_no_small_ctas", nullptr, 0, &Tunables::row_no_small_ctas},
    {"row_no_reg_rowvec", nullptr, 0, &Tunables::row_no_reg_rowvec},
    {"row_no_softmax_ln_fusion", nullptr, 0, &Tunables::row_no_softmax_ln_fusion},
    {"row_no_stage", nullptr, 0, &Tunables::row_no_stage},
    {"row_no_packed", nullptr, 0, &Tunables::row_no_packed},
};
}  // namespace

bool Tunables::set(const std::string& key, const std::string& value) {
  char* end = nullptr;
  long v = std::strtol(value.c_str(), &end, 10);
  if (value.empty() || *end != '\0') return false;
  if (key == "wait_limit") {
    wait_limit = (unsigned)std::max(1L, v);
    return true;
  }
  for (const Knob& k : kKnobs)
    if (key == k.key) {
      if (k.i)
        this->*(k.i) = (int)std::max<long>(k.lo, v);
      else
        this->*(k.b) = v != 0;
      return true;
    }
  return false;
}

void Tunables::apply_text(const std::string& text) {
  size_t pos = 0;
  while (pos < text.size()) {
    size_t semi = text.find(';', pos);
    if (semi == std::string::npos) semi = text.size();
    std::string item = text.substr(pos, semi - pos);
    pos = semi + 1;
    std::string packed;
    for (char c : item)
      if (c != ' ' && c != '\t' && c != '\n') packed += c;
    if (packed.empty()) continue;
    size_t eq = packed.find('=');
    if (eq == std::string::npos || !set(packed.substr(0, eq), packed.substr(eq + 1)))
      throw Error(HCT_ERR_INVALID_ARG, "schedule item '" + item + "' is not a known knob=integer");
  }
}

Tunables Tunables::from_env() {
  Tunables t;
  auto env_of = [](const char* key) {
    std::string name = "HCT_";
    for (const char* c = key; *c; ++c) name += (char)std::toupper((unsigned char)*c);
    return std::getenv(name.c_str());
  };
  for (const Knob& k : kKnobs)
    if (const char* s = env_of(k.key)) t.set(k.key, s);
  if (const char* s = env_of("wait_limit")) t.set("wait_limit", s);
  return t;
}

std::string float_lit(double v) {
  char buf[64];
  float f = (float)v;
  if (f != f) return "__int_as_float(0x7fc00000)";
  if (f == 1.0f / 0.0f) return "HCT_INF";
  if (f == -1.0f / 0.0f) return "(-HCT_INF)";
  std::snprintf(buf, sizeof buf, "%.9ef", (double)f);
  return buf;
}

const char* ctype(DType d) { return d == BF16 ? "hct_bf16_t" : "float"; }

namespace {

inline bool HCT_T_GT32(int T) { return T > 32; }
inline std::string strip_marker(std::string s) {
  size_t m = s.find("@REFILL@");
  if (m != std::string::npos) s.erase(m, 8);
  return s;
}  // rows that span several warps reduce through a barrier

struct RowGen {
  const Graph& g;
  const Plan& p;
  const Group& grp;
  int gi;
  std::ostringstream body;
  std::vector<BufRef> ptrs;

  int ptr_index(int node, bool ws_copy) {
    for (size_t i = 0; i < ptrs.size(); ++i)
      if (ptrs[i].node == node && ptrs[i].ws_copy == ws_copy) return (int)i;
    BufRef b;
    b.node = node;
    b.ws_copy = ws_copy;
    ptrs.push_back(b);
    return (int)ptrs.size() - 1;
  }

  // storage dtype of a buffer this group reads
  DType ext_dtype(int node) const { return g.nodes[node].dtype; }   // inputs: as declared; computed values: fp32, or bf16 after a cast
  bool ext_is_ws(int node) const { return g.nodes[node].cls != OpClass::Input && p.ws_offset[node] >= 0; }

  // expression for operand `a` inside loops over b (row of the batch) and, in full-width context, e
  std::string ref(const Operand& a, bool full_ctx) {
    if (a.is_literal()) return float_lit(a.literal);
    int n = a.node;
    if (p.group_of[n] == gi) {
      if (p.is_colv[n]) return "s" + std::to_string(n) + "[b]";
      return full_ctx ? "v" + std::to_string(n) + "[b][e]" : "v" + std::to_string(n) + "[b][0]";
    }
    int k = find_ext(grp, n);
    switch (grp.ext[k].bcast) {
      case Bcast::Full: return "x" + std::to_string(k) + "[b][e]";
      case Bcast::RowVec: return "x" + std::to_string(k) + "[e]";
      case Bcast::RowIdx: return "c" + std::to_string(k) + "[b]";
      default: return "c" + std::to_string(k);
    }
  }
};

}  // namespace

void gen_row_kernel(const Graph& g, const Plan& p, int gi, const Tunables& tun, std::vector<KernelSpec>* out) {
  const Group& grp = p.groups[gi];
  const int64_t R = grp.R, C = grp.C;
  if (C > (1 << 17)) throw Error(HCT_ERR_UNSUPPORTED, "rows longer than 131072 elements are not supported");
  for (auto& st : grp.stores)
    if (st.to_output && g.nodes[st.node].out_nhwc) throw Error(HCT_ERR_UNSUPPORTED, "an nhwc output must be produced by a convolution kernel");

  // vector width from alignment of every full-width buffer: rows start at multiples of C elements
  int V = (C % 4 == 0) ? 4 : (C % 2 == 0) ? 2 : 1;
  int64_t nvec = (C + V - 1) / V;
  int T = 8;
  while (T < 1024 && (nvec + T - 1) / T > tun.row_nv) T *= 2;
  int NV = (int)((nvec + T - 1) / T);
  if (NV * V > 128) throw Error(HCT_ERR_UNSUPPORTED, "row does not fit the register budget of one CTA");
  int cta = std::max(T, std::min(tun.row_cta, 1024));
  int G = std::max(1, cta / T);
  if (G > 15) G = 15;  // one named barrier per row slot
  if ((int64_t)G > R) G = (int)std::max<int64_t>(1, R);
  // whole warps only
  while ((G * T) % 32 != 0) ++G;

  // Staging through shared memory: every full-width external input whose rows are 16-byte multiples
  int64_t stage_bytes = 0;
  bool staged = T >= 32 && V == 4 && !tun.row_no_stage;
  for (auto& e : grp.ext)
    if (e.bcast == Bcast::Full) {
      int64_t rb = C * (g.nodes[e.node].cls == OpClass::Input && g.nodes[e.node].dtype == BF16 ? 2 : 4);
      if (rb % 16 != 0) staged = false;
      stage_bytes += rb;
    }
  if (stage_bytes == 0) staged = false;
  // A staged kernel runs one large CTA per SM: its row groups share the row-vector operands, which
  // are copied to shared memory once (as fp32) instead of being re-read through L1 for every row.
  int nstg = 0, B = 1;
  bool reg_rowvec = false;
  int64_t rowvec_bytes = 0;
  int n_rowvec = 0;
  if (staged) {
    for (auto& e : grp.ext)
      if (e.bcast == Bcast::RowVec) {
        rowvec_bytes += C * 4;
        ++n_rowvec;
      }
    if (rowvec_bytes > 80 * 1024) {
      rowvec_bytes = 0;  // too large to keep resident: read them through the cache instead
      n_rowvec = 0;
    }
    reg_rowvec = n_rowvec > 0 && n_rowvec * NV * V <= 64 && !tun.row_no_reg_rowvec;
    if (reg_rowvec) rowvec_bytes = 0;
    // Chains with reductions whose row vectors fit in registers (or that have none) run as several
    // small CTAs per SM, each with a short ring: measured best on the benchmark chain and the sweep.
    const bool small_ctas = grp.has_reduction && rowvec_bytes == 0 && !tun.row_no_small_ctas;
    if (grp.has_reduction && tun.row_batch > 1 && R >= 4096) B = tun.row_batch;
    // chains without reductions have short iterations and want a deep ring (few row groups per CTA);
    // chains with reductions want many rows in flight to cover the reductions' latency
    const int cta_threads = B > 1 ? tun.row_cta_batched : small_ctas ? tun.row_cta_small : grp.has_reduction ? tun.row_cta_staged : tun.row_cta_elementwise;
    int Gs = std::max(1, std::min<int>(cta_threads / T, 15));
    if ((int64_t)Gs > R) Gs = (int)std::max<int64_t>(1, R);
    while ((Gs * T) % 32 != 0) ++Gs;
    int64_t budget = (small_ctas ? (int64_t)tun.row_ring_bytes_small : (int64_t)tun.row_ring_bytes) - rowvec_bytes;
    while (Gs > 1 && budget / (Gs * B * stage_bytes) < 2) --Gs;
    if (budget / (Gs * B * stage_bytes) < 2) B = 1;
    nstg = (int)std::min<int64_t>(8, budget / (Gs * B * stage_bytes));
    if (nstg < 2 || (Gs * T) % 32 != 0)
      staged = false;
    else
      G = Gs;
  }
  // Row vectors of a chain with registers to spare stay in registers for the whole kernel (each thread
  // always meets the same columns); otherwise they are copied to shared memory once per CTA.
  if (!staged) reg_rowvec = false;
  const bool smem_rowvec = staged && n_rowvec > 0 && !reg_rowvec;

  RowGen rg{g, p, grp, gi, {}, {}};
  std::ostringstream& b = rg.body;
  std::string name = "hct_row_g" + std::to_string(gi);

  // ---- external operands
  const std::string FORB = "_Pragma(\"unroll\") for (int b = 0; b < HCT_B; ++b) ";
  const std::string FORE = "_Pragma(\"unroll\") for (int e = 0; e < HCT_E; ++e) ";
  // Packed arithmetic: neighbouring elements 2p and 2p + 1 of a thread (same vector) go through .f32x2
  // instructions, which halves the issue slots of multiply-adds.  Reductions that mask the ragged end of a row
  // (HCT_HAS) keep the one-value form unless every vector of the row is whole.
  const std::string FORP = "_Pragma(\"unroll\") for (int p_ = 0; p_ < HCT_E / 2; ++p_) ";
  const bool packed = V % 2 == 0 && !tun.row_no_packed;
  const bool packed_full = packed && C % ((int64_t)T * V * NV) == 0;
  auto half = [](std::string e, bool hi) {
    const std::string from = "[e]", to = hi ? "[2 * p_ + 1]" : "[2 * p_]";
    for (size_t at = e.find(from); at != std::string::npos; at = e.find(from, at + to.size())) e.replace(at, from.size(), to);
    return e;
  };
  auto pk = [&](const std::string& e) { return "hct_pk(" + half(e, false) + ", " + half(e, true) + ")"; };
  auto upk_into = [&](const std::string& value2, const std::string& arr) {
    return "hct_upk(" + value2 + ", " + arr + "[b][2 * p_], " + arr + "[b][2 * p_ + 1]);";
  };
  // uses of every node of this group (arguments anywhere in the graph); a product with a single use that is not
  // stored can be folded into the sum that consumes it
  std::vector<int> uses(g.nodes.size(), 0);
  for (auto& n : g.nodes)
    for (auto& a : n.args)
      if (!a.is_literal()) ++uses[a.node];
  auto stored = [&](int node) {
    for (auto& st : grp.stores)
      if (st.node == node) return true;
    return g.nodes[node].output_index >= 0;
  };
  auto foldable_mul = [&](const Operand& a) {
    return packed && !a.is_literal() && p.group_of[a.node] == gi && !p.is_colv[a.node] && g.nodes[a.node].cls == OpClass::Binary &&
           g.nodes[a.node].op == "mul" && uses[a.node] == 1 && !stored(a.node);
  };
  // Where the special-function unit would be busier than DRAM (16 results per clock and SM against the bytes the
  // chain moves per element, both at their measured rates), sigmoid takes its reciprocal on the multiply-add
  // pipe (three Newton steps); elsewhere the extra instructions would only cost issue slots.
  double xu_ops = 0, bytes_per_elem = 0;
  for (int ni : grp.nodes) {
    const Node& nd = g.nodes[ni];
    if (p.is_colv[ni]) continue;
    if (nd.op == "sigmoid" || nd.op == "gelu_tanh" || nd.op == "tanh" || nd.op == "div" || nd.op == "sin" || nd.op == "cos") xu_ops += 2;
    else if (nd.op == "exp" || nd.op == "log" || nd.op == "sqrt" || nd.op == "rsqrt" || nd.op == "reciprocal" || nd.op == "gelu_erf" || nd.cls == OpClass::RowSoftmax) xu_ops += 1;
  }
  for (auto& e : grp.ext)
    if (e.bcast == Bcast::Full) bytes_per_elem += (g.nodes[e.node].cls == OpClass::Input && g.nodes[e.node].dtype == BF16) ? 2 : 4;
  for (auto& st : grp.stores)
    if (!p.is_colv[st.node]) bytes_per_elem += st.dtype == BF16 ? 2 : 4;
  const bool xu_bound = xu_ops * 6.5 >= bytes_per_elem * 4.5;
  std::vector<char> folded(g.nodes.size(), 0);
  if (packed)
    for (int ni : grp.nodes) {
      const Node& nd = g.nodes[ni];
      if (nd.cls == OpClass::Binary && !p.is_colv[ni] && (nd.op == "add" || nd.op == "sub")) {
        if (foldable_mul(nd.args[0])) folded[nd.args[0].node] = 1;
        else if (foldable_mul(nd.args[1])) folded[nd.args[1].node] = 1;
      }
    }
  std::ostringstream pre, loads, issue, fill, hoisted;
  int64_t staged_off = 0, rowvec_off = 0;
  for (size_t k = 0; k < grp.ext.size(); ++k) {
    const ExtOperand& e = grp.ext[k];
    int pi = rg.ptr_index(e.node, rg.ext_is_ws(e.node));
    const char* ct = ctype(rg.ext_dtype(e.node));
    pre << "    const " << ct << "* __restrict__ q" << k << " = (const " << ct << "*)hct_p.ptr[" << pi << "];\n";
    switch (e.bcast) {
      case Bcast::Full:
        if (staged) {
          loads << "      float x" << k << "[HCT_B][HCT_E];\n      " << FORB << "hct_read_staged<" << ct << ">(hct_slot + " << staged_off
                << " * HCT_B + b * " << C * (rg.ext_dtype(e.node) == BF16 ? 2 : 4) << ", hct_t, x" << k << "[b]);\n";
          issue << "        HCT_STAGED_ISSUE_ONE(q" << k << ", " << staged_off << ", " << C * (rg.ext_dtype(e.node) == BF16 ? 2 : 4) << ")\n";
          staged_off += C * (rg.ext_dtype(e.node) == BF16 ? 2 : 4);
        } else {
          loads << "      float x" << k << "[HCT_B][HCT_E];\n      " << FORB << "hct_load_row(q" << k << ", HCT_ROWB(b), hct_t, x" << k
                << "[b], false);\n";
        }
        break;
      case Bcast::RowVec:
        if (reg_rowvec) {
          hoisted << "    float x" << k << "[HCT_E]; hct_load_row(q" << k << ", 0, hct_t, x" << k << ", true);\n";
        } else if (smem_rowvec) {
          fill << "    for (int i_ = threadIdx.x * 4; i_ < HCT_C; i_ += HCT_T * HCT_G * 4) {\n"
               << "      float t_[4]; hct_vecio<4>::ld_keep(q" << k << " + i_, t_);\n"
               << "      *(float4*)(hct_ring + " << rowvec_off << " + (size_t)i_ * 4) = make_float4(t_[0], t_[1], t_[2], t_[3]);\n    }\n";
          loads << "      float x" << k << "[HCT_E]; hct_read_staged<float>(hct_ring + " << rowvec_off << ", hct_t, x" << k << ");\n";
          rowvec_off += C * 4;
        } else {
          loads << "      float x" << k << "[HCT_E]; hct_load_row(q" << k << ", 0, hct_t, x" << k << ", true);\n";
        }
        break;
      case Bcast::Scalar:
        pre << "    const float c" << k << " = hct_ld1(q" << k << ");\n";
        break;
      case Bcast::RowIdx: {
        // index from the row's leading coordinates
        loads << "      float c" << k << "[HCT_B];\n      " << FORB << "{\n        long long r_ = HCT_ROWB(b), i_ = 0;\n";
        for (int d = (int)grp.full_shape.size() - 2; d >= 0; --d) {
          int64_t ext = grp.full_shape[d];
          int64_t st = e.lead_stride[d];
          if (st != 0) loads << "        i_ += (r_ % " << ext << "LL) * " << st << "LL;\n";
          loads << "        r_ /= " << ext << "LL;\n";
        }
        loads << "        c" << k << "[b] = hct_ld1(q" << k << " + i_);\n      }\n";
        break;
      }
    }
  }

  // ---- nodes
  // A layer normalisation whose input is a softmax of the same group knows its mean (1/C) and may take
  // its variance from the softmax's sum of squared terms when eps is large enough to absorb the
  // cancellation in mean(p^2) - 1/C^2 (C * eps >= 1/40: relative error of the result below 1.5e-6).
  auto ln_var_from_softmax = [&](int ln) {
    const Node& l = g.nodes[ln];
    if (l.cls != OpClass::RowLayernorm) return false;
    const Operand& x = l.args[0];
    return !x.is_literal() && p.group_of[x.node] == gi && g.nodes[x.node].cls == OpClass::RowSoftmax && (double)C * l.eps >= 0.025 &&
           !tun.row_no_softmax_ln_fusion;
  };
  auto softmax_feeds_fused_ln = [&](int sm) {
    for (int other : grp.nodes)
      if (ln_var_from_softmax(other) && g.nodes[other].args[0].node == sm) return true;
    return false;
  };
  bool refill_placed = false;
  for (int ni : grp.nodes) {
    const Node& nd = g.nodes[ni];
    std::string id = std::to_string(ni);
    const bool reduces = nd.cls == OpClass::RowReduce || nd.cls == OpClass::RowSoftmax || nd.cls == OpClass::RowLayernorm;
    b << "      // " << nd.name << " = " << nd.op << "\n";
    if (nd.cls == OpClass::Unary || nd.cls == OpClass::Binary) {
      std::vector<std::string> av;
      if (p.is_colv[ni]) {
        for (auto& a : nd.args) av.push_back(rg.ref(a, false));
        b << "      float s" << id << "[HCT_B];\n      " << FORB << "s" << id << "[b] = " << elementwise_call(nd, av, "hct_row0 + b") << ";\n";
      } else if (folded[ni]) {
        b << "      // (folded into the sum that consumes it)\n";
      } else if (packed && nd.cls == OpClass::Binary && (nd.op == "add" || nd.op == "sub" || nd.op == "mul")) {
        std::string e2;
        const int fa = nd.op == "mul" ? -1 : (!nd.args[0].is_literal() && folded[nd.args[0].node]) ? 0 : (!nd.args[1].is_literal() && folded[nd.args[1].node]) ? 1 : -1;
        if (fa >= 0) {
          // a * b + c, a * b - c, c - a * b as one packed multiply-add
          const Node& m = g.nodes[nd.args[fa].node];
          std::string ma = rg.ref(m.args[0], true), mb = rg.ref(m.args[1], true), c = rg.ref(nd.args[1 - fa], true);
          if (nd.op == "sub" && fa == 0) c = "-(" + c + ")";
          if (nd.op == "sub" && fa == 1) ma = "-(" + ma + ")";
          e2 = "hct_fma2(" + pk(ma) + ", " + pk(mb) + ", " + pk(c) + ")";
        } else {
          e2 = "hct_" + nd.op + "2(" + pk(rg.ref(nd.args[0], true)) + ", " + pk(rg.ref(nd.args[1], true)) + ")";
        }
        b << "      float v" << id << "[HCT_B][HCT_E];\n      " << FORB << FORP << upk_into(e2, "v" + id) << "\n";
      } else if (packed && nd.cls == OpClass::Unary && (nd.op == "sigmoid" || nd.op == "gelu_tanh")) {
        b << "      float v" << id << "[HCT_B][HCT_E];\n      " << FORB << FORP
          << upk_into("hct_" + nd.op + (nd.op == "sigmoid" && !xu_bound ? "2m(" : "2(") + pk(rg.ref(nd.args[0], true)) + ")", "v" + id) << "\n";
      } else {
        for (auto& a : nd.args) av.push_back(rg.ref(a, true));
        b << "      float v" << id << "[HCT_B][HCT_E];\n      " << FORB << FORE << "v" << id << "[b][e] = "
          << elementwise_call(nd, av, "(hct_row0 + b) * (long long)HCT_C + HCT_COL(e)") << ";\n";
      }
    } else if (nd.cls == OpClass::RowReduce && (nd.op == "row_argmax" || nd.op == "row_argmin")) {
      // column of the largest / smallest element (the first one among equals), delivered as an fp32 value
      std::string a = rg.ref(nd.args[0], true);
      const bool amax = nd.op == "row_argmax";
      b << "      float s" << id << "[HCT_B];\n      {\n        float bv_[HCT_B]; int bi_[HCT_B];\n        " << FORB << "{\n          bv_[b] = "
        << (amax ? "-HCT_INF" : "HCT_INF") << ";\n          bi_[b] = 0x7fffffff;\n          " << FORE << "if (HCT_HAS(e) && (" << a
        << (amax ? " > " : " < ") << "bv_[b] || bi_[b] == 0x7fffffff)) { bv_[b] = " << a << "; bi_[b] = HCT_COL(e); }\n        }\n"
        << "        hct_row_argreduce<" << (amax ? "true" : "false") << ">(bv_, bi_, hct_cx, HCT_SM_SMEM);\n"
        << (refill_placed ? "" : "@REFILL@")
        << "        " << FORB << "s" << id << "[b] = (float)bi_[b];\n      }\n";
    } else if (nd.cls == OpClass::RowReduce && nd.op == "row_min") {
      // min(x) = -max(-x): shares the maximum's exchange
      std::string a = rg.ref(nd.args[0], true);
      b << "      float s" << id << "[HCT_B];\n      " << FORB << "{\n        s" << id << "[b] = -HCT_INF;\n        "
        << FORE << "if (HCT_HAS(e)) s" << id << "[b] = fmaxf(s" << id << "[b], -(" << a << "));\n      }\n"
        << "      HCT_RMAX(s" << id << ");\n";
      if (!refill_placed) { b << "@REFILL@"; refill_placed = true; }
      b << "      " << FORB << "s" << id << "[b] = -s" << id << "[b];\n";
    } else if (nd.cls == OpClass::RowReduce) {
      std::string a = rg.ref(nd.args[0], true);
      bool is_max = nd.op == "row_max";
      b << "      float s" << id << "[HCT_B];\n      " << FORB << "{\n        s" << id << "[b] = " << (is_max ? "-HCT_INF" : "0.0f") << ";\n        "
        << FORE << "if (HCT_HAS(e)) s" << id << "[b] = " << (is_max ? "fmaxf(s" + id + "[b], " + a + ")" : "s" + id + "[b] + " + a) << ";\n      }\n"
        << "      " << (is_max ? "HCT_RMAX" : "HCT_RSUM") << "(s" << id << ");\n";
      if (!refill_placed) { b << "@REFILL@"; refill_placed = true; }
      if (nd.op == "row_mean")
        b << "      " << FORB << "s" << id << "[b] = s" << id << "[b] / (float)" << (p.reduce_count[ni] > 0 ? std::to_string(p.reduce_count[ni]) : std::string("HCT_C")) << ";\n";
    } else if (nd.cls == OpClass::RowSoftmax) {
      // One exchange between the warps of a row: every warp takes its exponentials relative to its own
      // maximum (found with shuffles alone), and the per-warp (maximum, sum) pairs are folded afterwards.
      // A layer normalisation that reads this softmax can take its variance from the sum of squared
      // terms gathered in the same exchange (see below); `sq<id>` then holds sum_j p_j^2 of the row.
      std::string a = rg.ref(nd.args[0], true);
      const bool with_q = softmax_feeds_fused_ln(ni);
      b << "      float v" << id << "[HCT_B][HCT_E];\n"
        << "      float sq" << id << "[HCT_B], kk" << id << "[HCT_B];\n"
        << "      {\n"
        << "        float m_[HCT_B];\n        " << FORB << "{\n          m_[b] = -HCT_INF;\n          " << FORE << "if (HCT_HAS(e)) m_[b] = fmaxf(m_[b], " << a
        << ");\n        }\n"
        << "        hct_warp_reduce<true>(m_);\n"
        // exp(x - m) as 2^(x*log2e - m*log2e) in one multiply-add: the product m*log2e is rounded on its own,
        // which scales the warp's terms by up to 2^(|m| * 1.45 * 2^-24).  Below |m| = 16 that is under 1e-6 and
        // harmless; above, the difference is taken first (exact where it matters, and safe for huge values).
        << "        float d_[HCT_B], q_[HCT_B];\n        " << FORB << "{\n          const float mr_ = m_[b] == -HCT_INF ? 0.0f : m_[b];\n"
        << "          d_[b] = 0.0f;\n          q_[b] = 0.0f;\n          if (fabsf(mr_) < 16.0f) {\n            const float ml_ = -mr_ * HCT_LOG2E;\n            ";
      if (packed_full) {
        // exponent, running sum and running sum of squares on pairs; the two partial sums are added at the end
        b << "hct_f2 d2_ = hct_pk(0.0f, 0.0f), q2_ = d2_;\n            " << FORP << "{ const hct_f2 t_ = hct_exp2_fast2(hct_fma2(" << pk(a)
          << ", hct_pk(HCT_LOG2E, HCT_LOG2E), hct_pk(ml_, ml_))); " << "hct_upk(t_, v" << id << "[b][2 * p_], v" << id << "[b][2 * p_ + 1]); d2_ = hct_add2(d2_, t_);"
          << (with_q ? " q2_ = hct_fma2(t_, t_, q2_);" : "") << " }\n            { float lo_, hi_; hct_upk(d2_, lo_, hi_); d_[b] = lo_ + hi_; hct_upk(q2_, lo_, hi_); q_[b] = lo_ + hi_; }\n";
      } else {
        b << FORE << "{ v" << id << "[b][e] = HCT_HAS(e) ? hct_exp2_fast(fmaf(" << a << ", HCT_LOG2E, ml_)) : 0.0f; d_[b] += v" << id << "[b][e];"
          << (with_q ? " q_[b] = fmaf(v" + id + "[b][e], v" + id + "[b][e], q_[b]);" : "") << " }\n";
      }
      b << "          } else {\n            " << FORE
        << "{ v" << id << "[b][e] = HCT_HAS(e) ? hct_exp2_fast((" << a << " - mr_) * HCT_LOG2E) : 0.0f; d_[b] += v" << id << "[b][e];"
        << (with_q ? " q_[b] = fmaf(v" + id + "[b][e], v" + id + "[b][e], q_[b]);" : "") << " }\n          }\n        }\n"
        << "        hct_warp_reduce<false>(d_);\n"
        << (with_q ? "        hct_warp_reduce<false>(q_);\n" : "")
        << "        float f_[HCT_B];\n"
        << "        hct_softmax_combine<" << (with_q ? "true" : "false") << ">(m_, d_, q_, f_, hct_cx, HCT_SM_SMEM);\n"
        << (refill_placed ? "" : "@REFILL@")
        << "        " << FORB << "{\n          const float inv_ = hct_rcp_fast(d_[b]);\n          const float k_ = f_[b] * inv_;\n          sq" << id
        << "[b] = q_[b] * inv_ * inv_;\n          ";
      // The factor that turns the terms into probabilities is left to a layer normalisation that is the only
      // reader of this softmax and folds it into its own scaling (one multiply-add per element for both).
      if (with_q && uses[ni] == 1 && !stored(ni))
        b << "kk" << id << "[b] = k_;\n";
      else if (packed)
        b << FORP << upk_into("hct_mul2(" + pk("v" + id + "[b][e]") + ", hct_pk(k_, k_))", "v" + id) << "\n";
      else
        b << FORE << "v" << id << "[b][e] *= k_;\n";
      b << "        }\n"
        << "      }\n";
    } else if (nd.cls == OpClass::RowLayernorm) {
      std::string a = rg.ref(nd.args[0], true);
      std::string ga = rg.ref(nd.args[1], true), be = rg.ref(nd.args[2], true);
      b << "      float v" << id << "[HCT_B][HCT_E];\n"
        << "      {\n"
        << "        float m_[HCT_B];\n";
      // A softmax row sums to one, so its mean is 1/C: no reduction is needed for it.
      const Operand& xin = nd.args[0];
      const bool mean_known = !xin.is_literal() && p.group_of[xin.node] == gi && g.nodes[xin.node].cls == OpClass::RowSoftmax;
      if (mean_known) {
        b << "        " << FORB << "m_[b] = 1.0f;\n";
      } else {
        b << "        " << FORB << "{\n          m_[b] = 0.0f;\n          " << FORE << "if (HCT_HAS(e)) m_[b] += " << a << ";\n        }\n"
          << "        HCT_RSUM(m_);\n"
          << (refill_placed ? "" : "@REFILL@");
      }
      if (mean_known && ln_var_from_softmax(ni)) {
        // variance = mean(p^2) - 1/C^2 with sum p^2 from the softmax's exchange: no reduction at all here.
        // Rounding of the difference is at most 2^-24 * mean(p^2) <= 2^-24 / C, which the eps under the
        // root keeps below 2^-24 / (2 C eps) of the result (the rule applies only when C * eps >= 1/40).
        b << "        " << FORB << "{\n          m_[b] = m_[b] / (float)HCT_C;\n          const float var_ = fmaxf(fmaf(sq" << xin.node
          << "[b], 1.0f / (float)HCT_C, -m_[b] * m_[b]), 0.0f);\n          const float r_ = hct_rsqrt_fast(var_ + " << float_lit(nd.eps) << ");\n          "
          ;
        const bool deferred = uses[xin.node] == 1 && !stored(xin.node);   // the softmax left its terms unscaled: kk holds the factor
        if (deferred && packed_full)
          b << "const float ka_ = kk" << xin.node << "[b] * r_, kb_ = -m_[b] * r_;\n          " << FORP
            << upk_into("hct_fma2(hct_fma2(" + pk(a) + ", hct_pk(ka_, ka_), hct_pk(kb_, kb_)), " + pk(ga) + ", " + pk(be) + ")", "v" + id) << "\n        }\n";
        else if (deferred)
          b << "const float ka_ = kk" << xin.node << "[b] * r_, kb_ = -m_[b] * r_;\n          " << FORE << "v" << id << "[b][e] = fmaf(fmaf(" << a
            << ", ka_, kb_), " << ga << ", " << be << ");\n        }\n";
        else
          b << FORE << "{ const float d_ = HCT_HAS(e) ? " << a << " - m_[b] : 0.0f; v" << id << "[b][e] = fmaf(d_ * r_, " << ga << ", " << be
            << "); }\n        }\n";
        b << "      }\n";
      } else {
        b << "        float q_[HCT_B];\n        " << FORB << "{\n          m_[b] = m_[b] / (float)HCT_C;\n          q_[b] = 0.0f;\n          " << FORE
          << "{ const float d_ = HCT_HAS(e) ? " << a << " - m_[b] : 0.0f; v" << id << "[b][e] = d_; q_[b] = fmaf(d_, d_, q_[b]); }\n        }\n"
          << "        HCT_RSUM(q_);\n"
          << "        " << FORB << "{\n          const float r_ = hct_rsqrt_fast(q_[b] * (1.0f / (float)HCT_C) + " << float_lit(nd.eps)
          << ");\n          " << FORE << "v" << id << "[b][e] = fmaf(v" << id << "[b][e] * r_, " << ga << ", " << be << ");\n        }\n"
          << "      }\n";
      }
    } else {
      throw Error(HCT_ERR_UNSUPPORTED, "operator " + nd.op + " cannot be part of a row kernel");
    }
    if (reduces) refill_placed = true;
  }

  // ---- stores
  std::ostringstream stores;
  for (auto& s : grp.stores) {
    int pi = rg.ptr_index(s.node, !s.to_output);
    const char* ct = ctype(s.dtype);
    std::string id = std::to_string(s.node);
    if (p.is_colv[s.node])
      stores << "      " << FORB << "if (HCT_LIVEB(b) && hct_t == 0) hct_st1((" << ct << "*)hct_p.ptr[" << pi << "] + hct_row0 + b, s" << id
             << "[b]);\n";
    else if (!s.to_output && p.split_store[s.node])
      stores << "      " << FORB << "if (HCT_LIVEB(b)) hct_store_row_split((float*)hct_p.ptr[" << pi << "], (float*)((char*)hct_p.ptr[" << pi << "] + "
             << p.split_lo_offset[s.node] << "LL), hct_row0 + b, hct_t, v" << id << "[b]);\n";
    else
      stores << "      " << FORB << "if (HCT_LIVEB(b)) hct_store_row((" << ct << "*)hct_p.ptr[" << pi << "], hct_row0 + b, hct_t, v" << id
             << "[b]);\n";
  }

  std::ostringstream src;
  const size_t nptr = rg.ptrs.size() + (staged ? 1 : 0);
  src << "#define HCT_T " << T << "\n#define HCT_G " << G << "\n#define HCT_V " << V << "\n#define HCT_NV " << NV << "\n"
      << "#define HCT_R " << R << "LL\n#define HCT_C " << C << "\n#define HCT_B " << B << "\n#define HCT_NPTR " << std::max<size_t>(1, nptr) << "\n";
  if (staged)
    src << "#define HCT_MINB " << (G * T <= 512 ? tun.row_min_blocks : 1) << "\n#define HCT_RING_OFF " << rowvec_bytes << "\n#define HCT_STAGED 1\n#define HCT_NSTG " << nstg << "\n#define HCT_STAGE_BYTES " << stage_bytes << "\n#define HCT_STATUS_SLOT "
        << rg.ptrs.size() << "\n";
  src << skeleton_source("common") << "\n" << skeleton_source("row") << "\n";
  if (!staged) {
    src << "HCT_ROW_KERNEL_BEGIN(" << name << ")\n"
        << pre.str() << "  HCT_ROW_LOOP_BEGIN\n"
        << loads.str() << strip_marker(b.str()) << stores.str() << "  HCT_ROW_LOOP_END\nHCT_ROW_KERNEL_END\n";
  } else {
    src << "HCT_STAGED_KERNEL_BEGIN(" << name << ")\n"
        << pre.str()
        << "    const long long hct_stride = (long long)gridDim.x * (HCT_G * HCT_B);\n"
        << "    if (hct_t == 0) {\n"
        << "      for (int s_ = 0; s_ < HCT_NSTG; ++s_) {\n"
        << "        HCT_STAGED_ISSUE_BEGIN(((long long)blockIdx.x * HCT_G + hct_cx.g) * HCT_B + s_ * hct_stride, s_)\n"
        << issue.str() << "        HCT_STAGED_ISSUE_END\n      }\n    }\n"
        << "    // row vectors become resident while the first rows are in flight\n"
        << fill.str() << (smem_rowvec ? "    __syncthreads();\n" : "") << hoisted.str()
        << "    int hct_it = 0;\n"
        << "  HCT_ROW_LOOP_BEGIN\n"
        << "    if (hct_live) {\n"
        << "      const int hct_s = hct_it % HCT_NSTG;\n"
        << "      hct_row_mbar_wait(hct_smem_u32(&hct_full[hct_cx.g][hct_s]), (hct_u32)((hct_it / HCT_NSTG) & 1), &hct_failed, hct_status);\n"
        << "      const unsigned char* hct_slot = hct_my_ring + (size_t)hct_s * (HCT_STAGE_BYTES * HCT_B);\n"
        << loads.str();
    // The slot may be refilled once every thread of the row has taken its share, i.e. after any
    // barrier of the row group: the first reduction's barrier if the chain has one, else one of its own.
    std::string refill = "      if (hct_t == 0) {\n        HCT_STAGED_ISSUE_BEGIN(hct_row0 + HCT_NSTG * hct_stride, hct_s)\n" + issue.str() +
                         "        HCT_STAGED_ISSUE_END\n      }\n";
    std::string body = b.str();
    size_t mark = body.find("@REFILL@");
    if (mark != std::string::npos && HCT_T_GT32(T))
      body.replace(mark, 8, refill);
    else {
      if (mark != std::string::npos) body.erase(mark, 8);
      src << "      HCT_GROUP_SYNC;\n" << refill;
    }
    src << body << stores.str() << "    }\n    ++hct_it;\n"
        << "  HCT_ROW_LOOP_END\nHCT_ROW_KERNEL_END\n";
  }

  KernelSpec k;
  k.name = name;
  k.source = src.str();
  k.block[0] = (unsigned)(G * T);
  k.persistent = true;
  k.max_grid = (unsigned)std::min<int64_t>((R + G * B - 1) / (G * B), 0x7fffffff);
  k.grid[0] = k.max_grid;
  k.ptrs = rg.ptrs;
  if (staged) {
    k.wants_status = true;
    k.smem_bytes = (unsigned)(rowvec_bytes + G * nstg * B * stage_bytes);
  }
  std::ostringstream d;
  d << "row kernel T=" << T << " G=" << G << " V=" << V << " NV=" << NV;
  if (B > 1) d << " B=" << B;
  if (staged) d << ", " << nstg << "-row bulk-copy ring";
  k.desc = d.str();
  out->push_back(k);
}

}  // namespace hct
