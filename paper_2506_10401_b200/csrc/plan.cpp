#include "plan.h"

#include <algorithm>
#include <sstream>

#include "../../include/hct.h"

namespace hct {

namespace {

std::vector<int64_t> col_shape(std::vector<int64_t> s) {
  s.back() = 1;
  return s;
}

bool all_ones(const std::vector<int64_t>& s) {
  for (auto d : s)
    if (d != 1) return false;
  return true;
}

// Classify operand shape `s` against the group's full shape.  Returns false if the pattern is unsupported.
bool classify(const std::vector<int64_t>& s, const std::vector<int64_t>& full, Bcast* kind, std::vector<int64_t>* lead_stride) {
  lead_stride->clear();
  if (s == full) {
    *kind = Bcast::Full;
    return true;
  }
  if (all_ones(s)) {
    *kind = Bcast::Scalar;
    return true;
  }
  if (s.size() > full.size()) return false;
  // right-align
  std::vector<int64_t> a(full.size(), 1);
  for (size_t i = 0; i < s.size(); ++i) a[full.size() - s.size() + i] = s[i];
  for (size_t i = 0; i < full.size(); ++i)
    if (a[i] != 1 && a[i] != full[i]) return false;
  bool lead_ones = true;
  for (size_t i = 0; i + 1 < a.size(); ++i) lead_ones = lead_ones && a[i] == 1;
  if (lead_ones && a.back() == full.back()) {
    *kind = Bcast::RowVec;
    return true;
  }
  if (a.back() == 1) {
    *kind = Bcast::RowIdx;
    lead_stride->assign(full.size() - 1, 0);
    int64_t st = 1;
    for (int i = (int)a.size() - 2; i >= 0; --i) {
      if (a[i] != 1) {
        (*lead_stride)[i] = st;
        st *= a[i];
      }
    }
    return true;
  }
  return false;  // e.g. [R,C] with [H,1,C]: broadcast along a middle axis of a full-width operand
}

}  // namespace

int find_ext(const Group& grp, int node) {
  for (size_t i = 0; i < grp.ext.size(); ++i)
    if (grp.ext[i].node == node) return (int)i;
  return -1;
}

Plan make_plan(const Graph& g) {
  Plan p;
  const int n = (int)g.nodes.size();
  p.group_of.assign(n, -1);
  p.ws_offset.assign(n, -1);
  p.is_colv.assign(n, 0);
  p.partial_cols.assign(n, 0);
  p.reduce_count.assign(n, 0);
  p.split_store.assign(n, 0);
  p.split_lo_offset.assign(n, 0);

  auto add_ext = [&](Group& grp, int node, int consumer) {
    if (find_ext(grp, node) >= 0) return;
    ExtOperand e;
    e.node = node;
    if (p.partial_cols[node] > 0) {   // arrives as [R, chunks] partial sums: a full-width operand of the rewritten group
      e.bcast = Bcast::Full;
      grp.ext.push_back(e);
      return;
    }
    if (!classify(g.nodes[node].shape, grp.full_shape, &e.bcast, &e.lead_stride))
      throw Error(HCT_ERR_UNSUPPORTED, "node '" + g.nodes[consumer].name + "': broadcast pattern of operand '" +
                                           g.nodes[node].name + "' is not supported");
    grp.ext.push_back(e);
  };

  // Can node i (elementwise or row op) live in group gi?
  auto can_join = [&](int gi, int i) -> bool {
    const Group& grp = p.groups[gi];
    const Node& nd = g.nodes[i];
    bool full = nd.shape == grp.full_shape;
    bool colv = nd.shape == col_shape(grp.full_shape);
    if (grp.kind != GroupKind::Row) {
      if (!(nd.cls == OpClass::Unary || nd.cls == OpClass::Binary) || !full) return false;
      for (auto& a : nd.args) {
        if (a.is_literal() || p.group_of[a.node] == gi) continue;
        Bcast b;
        std::vector<int64_t> ls;
        if (!classify(g.nodes[a.node].shape, grp.full_shape, &b, &ls)) return false;
        if (b == Bcast::RowIdx) {
          // contraction epilogues index per-row scalars by GEMM row, or by channel for NCHW outputs
          if (grp.kind == GroupKind::Conv) {
            const auto& s = g.nodes[a.node].shape;
            int64_t K = grp.full_shape[1];
            bool chan = (s.size() == 3 && s[0] == K && s[1] == 1 && s[2] == 1) ||
                        (s.size() == 4 && s[0] == 1 && s[1] == K && s[2] == 1 && s[3] == 1);
            if (!chan) return false;
          }
        }
        if (b == Bcast::RowVec && grp.kind == GroupKind::Conv) return false;
        if (b == Bcast::RowIdx && grp.kind == GroupKind::Permute && grp.full_shape.size() > 2) return false;
      }
      return true;
    }
    if (!full && !colv) return false;
    if (nd.cls == OpClass::RowSoftmax || nd.cls == OpClass::RowLayernorm || nd.cls == OpClass::RowReduce) {
      if (g.nodes[nd.args[0].node].shape != grp.full_shape) return false;
      if (grp.full_shape.size() != 2) return false;
    }
    for (auto& a : nd.args) {
      if (a.is_literal() || p.group_of[a.node] == gi) continue;
      Bcast b;
      std::vector<int64_t> ls;
      if (!classify(g.nodes[a.node].shape, grp.full_shape, &b, &ls)) return false;
    }
    return true;
  };

  for (int i = 0; i < n; ++i) {
    const Node& nd = g.nodes[i];
    if (nd.cls == OpClass::Input) continue;
    int gi = -1;
    if (nd.cls == OpClass::Gemm || nd.cls == OpClass::Conv || nd.cls == OpClass::Transpose || nd.cls == OpClass::Sort ||
        nd.cls == OpClass::Reshape || nd.cls == OpClass::Permute) {
      Group grp;
      grp.kind = nd.cls == OpClass::Gemm ? GroupKind::Gemm : nd.cls == OpClass::Conv ? GroupKind::Conv
                 : nd.cls == OpClass::Transpose ? GroupKind::Transpose : nd.cls == OpClass::Sort ? GroupKind::Sort
                 : nd.cls == OpClass::Permute ? GroupKind::Permute : GroupKind::Reshape;
      grp.full_shape = nd.shape;
      p.groups.push_back(grp);
      gi = (int)p.groups.size() - 1;
    } else {
      int cand = -1;
      for (auto& a : nd.args)
        if (!a.is_literal()) cand = std::max(cand, p.group_of[a.node]);
      if (cand >= 0 && can_join(cand, i)) {
        gi = cand;
      } else {
        Group grp;
        grp.kind = GroupKind::Row;
        if (nd.cls == OpClass::Unary || nd.cls == OpClass::Binary)
          grp.full_shape = nd.shape;
        else
          grp.full_shape = g.nodes[nd.args[0].node].shape;
        p.groups.push_back(grp);
        gi = (int)p.groups.size() - 1;
      }
    }
    Group& grp = p.groups[gi];
    grp.nodes.push_back(i);
    p.group_of[i] = gi;
    if (grp.kind == GroupKind::Row && nd.shape != grp.full_shape) p.is_colv[i] = 1;
    if (nd.cls == OpClass::RowSoftmax || nd.cls == OpClass::RowLayernorm || nd.cls == OpClass::RowReduce)
      grp.has_reduction = true;
  }

  // Row sums folded into a contraction's epilogue (the paper's first case study: matrix product, dropout, mean,
  // softmax in one fused group).  When a value of a tensor-core GEMM group is read only by row_sum / row_mean nodes
  // whose row group holds nothing but per-row values, the epilogue emits one partial sum per row and 32-column
  // chunk instead of the value, and that row group runs over [R, chunks].
  for (int v = 0; v < n; ++v) {
    const Node& nv = g.nodes[v];
    if (nv.cls == OpClass::Input || nv.output_index >= 0 || nv.dtype != F32) continue;
    const int gv = p.group_of[v];
    if (p.groups[gv].kind != GroupKind::Gemm) continue;
    const Node& an = g.nodes[p.groups[gv].nodes[0]];
    const Node& opa = g.nodes[an.args[0].node];
    const Node& opb = g.nodes[an.args[1].node];
    // (the operand types and extents for which the tensor-core kernels, whose epilogue works on 32-column chunks, are taken)
    const bool tc_bf16 = opa.dtype == BF16 && opb.dtype == BF16 && opa.shape[1] % 8 == 0;
    const bool tc_f32 = opa.dtype == F32 && opb.dtype == F32 && opa.shape[1] % 4 == 0;
    if (!(tc_bf16 || tc_f32) || an.shape[1] % 32 != 0) continue;
    int target = -1;
    bool ok = true, any = false;
    for (int u = 0; u < n && ok; ++u)
      for (auto& a : g.nodes[u].args) {
        if (a.is_literal() || a.node != v) continue;
        if (p.group_of[u] == gv) { ok = false; break; }   // also used inside the epilogue: stays an ordinary value
        const Node& nu = g.nodes[u];
        if (!(nu.cls == OpClass::RowReduce && (nu.op == "row_sum" || nu.op == "row_mean"))) { ok = false; break; }
        if (target >= 0 && p.group_of[u] != target) { ok = false; break; }
        target = p.group_of[u];
        any = true;
      }
    if (!ok || !any) continue;
    Group& tg = p.groups[target];
    if (tg.kind != GroupKind::Row) continue;
    for (int u : tg.nodes) {
      if (!p.is_colv[u]) ok = false;
      for (auto& a : g.nodes[u].args)   // no other full-width operand in that group
        if (!a.is_literal() && a.node != v && p.group_of[a.node] != target && g.nodes[a.node].shape == tg.full_shape) ok = false;
    }
    if (!ok) continue;
    p.partial_cols[v] = nv.shape[1] / 32;
    for (int u : tg.nodes)
      for (auto& a : g.nodes[u].args)
        if (!a.is_literal() && a.node == v) p.reduce_count[u] = nv.shape[1];
    tg.full_shape = {nv.shape[0], p.partial_cols[v]};
  }

  // TF32 head and tail written by the producing row kernel's store.
  for (int v = 0; v < n; ++v) {
    const Node& nv = g.nodes[v];
    if (nv.cls == OpClass::Input || nv.output_index >= 0 || nv.dtype != F32 || nv.shape.size() != 2) continue;
    const Group& gv = p.groups[p.group_of[v]];
    if (gv.kind != GroupKind::Row || p.is_colv[v] || nv.shape != gv.full_shape) continue;
    bool ok = true, any = false;
    for (int u = 0; u < n && ok; ++u)
      for (size_t ai = 0; ai < g.nodes[u].args.size(); ++ai) {
        const Operand& a = g.nodes[u].args[ai];
        if (a.is_literal() || a.node != v || p.group_of[u] == p.group_of[v]) continue;
        const Node& nu = g.nodes[u];
        const bool gemm_a = nu.cls == OpClass::Gemm && ai == 0 && g.nodes[nu.args[1].node].dtype == F32 && nv.shape[1] % 4 == 0;
        if (!gemm_a) ok = false;
        any = true;
      }
    if (ok && any) p.split_store[v] = 1;
  }

  // Iteration spaces, external operands.
  for (auto& grp : p.groups) {
    grp.C = grp.full_shape.back();
    grp.R = 1;
    for (size_t d = 0; d + 1 < grp.full_shape.size(); ++d) grp.R *= grp.full_shape[d];
  }
  for (int i = 0; i < n; ++i) {
    const Node& nd = g.nodes[i];
    if (nd.cls == OpClass::Input) continue;
    Group& grp = p.groups[p.group_of[i]];
    bool anchor = nd.cls == OpClass::Gemm || nd.cls == OpClass::Conv || nd.cls == OpClass::Transpose || nd.cls == OpClass::Sort ||
                  nd.cls == OpClass::Reshape || nd.cls == OpClass::Permute;
    for (auto& a : nd.args) {
      if (a.is_literal() || p.group_of[a.node] == p.group_of[i]) continue;
      if (anchor) continue;  // contraction operands are bound separately
      add_ext(grp, a.node, i);
    }
  }

  // Stores: a node is written if it is a graph output or read by another group.
  std::vector<char> cross(n, 0);
  for (int i = 0; i < n; ++i)
    for (auto& a : g.nodes[i].args)
      if (!a.is_literal() && g.nodes[a.node].cls != OpClass::Input && p.group_of[a.node] != p.group_of[i]) cross[a.node] = 1;
  size_t ws = 0;
  for (int i = 0; i < n; ++i) {
    const Node& nd = g.nodes[i];
    if (nd.cls == OpClass::Input) continue;
    Group& grp = p.groups[p.group_of[i]];
    bool out = nd.output_index >= 0;
    // consumers always read fp32; an output stored as bf16 cannot serve them
    bool need_ws = cross[i] && !(out && nd.out_dtype == nd.dtype);   // an output of the value's own width serves its consumers too
    if (out) grp.stores.push_back({i, nd.out_dtype, true});
    if (need_ws) {
      // intermediates are fp32, except values a cast has rounded to bf16, which keep that width
      p.ws_offset[i] = (int64_t)ws;
      if (p.split_store[i]) {
        p.split_lo_offset[i] = (int64_t)(((size_t)nd.numel() * 4 + 255) / 256 * 256);   // head, then tail
        ws += 2 * (size_t)p.split_lo_offset[i];
      } else if (p.partial_cols[i] > 0)
        ws += ((size_t)nd.shape[0] * p.partial_cols[i] * 4 + 255) / 256 * 256;   // fp32 partial row sums
      else
        ws += ((size_t)nd.numel() * (nd.dtype == BF16 ? 2 : 4) + 255) / 256 * 256;
      grp.stores.push_back({i, p.partial_cols[i] > 0 ? F32 : nd.dtype, false});
    }
  }
  p.workspace_bytes = ws;

  // Work accounting.
  auto dsize = [](DType d) { return d == BF16 ? 2.0 : 4.0; };
  for (int i : g.inputs) p.algorithmic_bytes += g.nodes[i].numel() * dsize(g.nodes[i].dtype);
  for (int i : g.outputs) p.algorithmic_bytes += g.nodes[i].numel() * dsize(g.nodes[i].out_dtype);
  for (int i = 0; i < n; ++i) {
    const Node& nd = g.nodes[i];
    if (nd.cls == OpClass::Gemm) {
      const auto& a = g.nodes[nd.args[0].node].shape;
      p.flops += 2.0 * a[0] * a[1] * nd.shape[1];
    } else if (nd.cls == OpClass::Conv) {
      const auto& w = g.nodes[nd.args[1].node].shape;
      p.flops += 2.0 * nd.numel() * w[1] * w[2] * w[3];
    }
    if (p.ws_offset[i] < 0) continue;
    // An intermediate counts (one write, one read) only where no single pass could keep it on chip:
    //  * a value that depends on a reduction (a row reduction of its group, or a contraction) and feeds a
    //    contraction or a transposition: every element of the operand needs the whole reduction first;
    //  * a contraction's result that feeds a row reduction over rows wider than one accumulator tile (512 columns).
    // Elementwise producers of a contraction could be applied while the operand is loaded, a sort is local to
    // its row, and a reshape moves no data: those edges are free.
    bool unavoidable = false;
    const Group& pg = p.groups[p.group_of[i]];
    const bool after_reduction = pg.kind == GroupKind::Gemm || pg.kind == GroupKind::Conv || (pg.kind == GroupKind::Row && pg.has_reduction);
    for (int j = 0; j < n; ++j)
      for (auto& a : g.nodes[j].args) {
        if (a.is_literal() || a.node != i || p.group_of[j] == p.group_of[i]) continue;
        bool into_contraction = (g.nodes[j].cls == OpClass::Gemm || g.nodes[j].cls == OpClass::Conv || g.nodes[j].cls == OpClass::Transpose ||
                                 g.nodes[j].cls == OpClass::Permute) &&
                                after_reduction;
        bool from_contraction = (pg.kind == GroupKind::Gemm || pg.kind == GroupKind::Conv) && p.groups[p.group_of[j]].has_reduction &&
                                nd.shape.back() > 512;
        unavoidable = unavoidable || into_contraction || from_contraction;
      }
    if (unavoidable) p.algorithmic_bytes += (nd.dtype == BF16 ? 4.0 : 8.0) * nd.numel();
  }

  std::ostringstream os;
  for (size_t gi = 0; gi < p.groups.size(); ++gi) {
    const Group& grp = p.groups[gi];
    os << "kernel " << gi << " " << (grp.kind == GroupKind::Row ? "row" : grp.kind == GroupKind::Gemm ? "gemm" : grp.kind == GroupKind::Conv ? "conv" : grp.kind == GroupKind::Transpose ? "transpose" : grp.kind == GroupKind::Sort ? "sort" : grp.kind == GroupKind::Permute ? "permute" : "reshape") << " [";
    for (size_t d = 0; d < grp.full_shape.size(); ++d) os << (d ? "," : "") << grp.full_shape[d];
    os << "]:";
    for (int i : grp.nodes) os << " " << g.nodes[i].name << "=" << g.nodes[i].op;
    os << " | stores:";
    for (auto& s : grp.stores)
      os << " " << g.nodes[s.node].name
         << (s.to_output ? "" : p.partial_cols[s.node] > 0 ? "(ws: row sums of 32-column chunks, folded into the epilogue)"
             : p.split_store[s.node] ? "(ws: TF32 head and tail for the GEMM that reads it)" : "(ws)");
    os << "\n";
  }
  p.text = os.str();
  return p;
}

}  // namespace hct
