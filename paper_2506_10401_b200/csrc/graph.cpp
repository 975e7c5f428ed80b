// Spec reader.  The checks are the validity rules of the paper's graph construction (§3.2):
// the graph is a DAG (an operand must be defined on an earlier line), every operator agrees
// with the shapes and dtypes of its operands, and no node dangles (all reach an output).
#include "graph.h"

#include <cctype>
#include <cerrno>
#include <cstdlib>
#include <cmath>
#include <cstdio>
#include <map>
#include <sstream>

#include "../../include/hct.h"

namespace hct {

static const char* kUnary[] = {"relu", "gelu_tanh", "gelu_erf", "sigmoid", "exp", "tanh", "sqrt", "sin", "cos", "neg", "abs",
                               "log", "rsqrt", "square", "reciprocal"};
static const char* kBinary[] = {"add", "sub", "mul", "div", "max", "min"};

bool is_unary(const std::string& op) {
  for (auto u : kUnary)
    if (op == u) return true;
  return false;
}
bool is_binary(const std::string& op) {
  for (auto b : kBinary)
    if (op == b) return true;
  return false;
}

namespace {
constexpr int64_t kMaxElements = (int64_t)1 << 40;

std::string trim(const std::string& s) {
  size_t a = 0, b = s.size();
  while (a < b && std::isspace((unsigned char)s[a])) ++a;
  while (b > a && std::isspace((unsigned char)s[b - 1])) --b;
  return s.substr(a, b - a);
}

bool valid_name(const std::string& s) {
  if (s.empty() || !(std::isalpha((unsigned char)s[0]) || s[0] == '_')) return false;
  for (char c : s)
    if (!(std::isalnum((unsigned char)c) || c == '_')) return false;
  return true;
}

[[noreturn]] void fail(int code, int line, const std::string& msg) {
  std::ostringstream os;
  os << "line " << line << ": " << msg;
  throw Error(code, os.str());
}

std::string shape_str(const std::vector<int64_t>& s) {
  std::ostringstream os;
  os << "[";
  for (size_t i = 0; i < s.size(); ++i) os << (i ? "," : "") << s[i];
  os << "]";
  return os.str();
}

bool parse_number(const std::string& s, double* out) {
  if (s.empty()) return false;
  char* end = nullptr;
  double v = std::strtod(s.c_str(), &end);
  if (end != s.c_str() + s.size()) return false;
  *out = v;
  return true;
}

bool parse_int(const std::string& s, int64_t* out) {
  if (s.empty()) return false;
  char* end = nullptr;
  errno = 0;
  long long v = std::strtoll(s.c_str(), &end, 10);
  if (end != s.c_str() + s.size() || errno == ERANGE) return false;   // not a number, or not representable
  *out = v;
  return true;
}

std::vector<std::string> split(const std::string& s, char sep) {
  std::vector<std::string> out;
  std::string cur;
  for (char c : s) {
    if (c == sep) {
      out.push_back(trim(cur));
      cur.clear();
    } else {
      cur.push_back(c);
    }
  }
  out.push_back(trim(cur));
  return out;
}

std::vector<int64_t> broadcast(const std::vector<int64_t>& a, const std::vector<int64_t>& b, int line) {
  size_t n = std::max(a.size(), b.size());
  std::vector<int64_t> out(n);
  for (size_t i = 0; i < n; ++i) {
    int64_t x = i + a.size() >= n ? a[i + a.size() - n] : 1;
    int64_t y = i + b.size() >= n ? b[i + b.size() - n] : 1;
    if (x == y || y == 1)
      out[i] = x;
    else if (x == 1)
      out[i] = y;
    else
      fail(HCT_ERR_GRAPH, line, "shapes " + shape_str(a) + " and " + shape_str(b) + " do not broadcast");
  }
  return out;
}

}  // namespace

Graph parse_spec(const std::string& text) {
  Graph g;
  std::map<std::string, int> index;
  std::istringstream in(text);
  std::string raw;
  int line = 0;
  bool header = false;

  auto lookup = [&](const std::string& tok, int ln, bool allow_literal) -> Operand {
    Operand o;
    auto it = index.find(tok);
    if (it != index.end()) {
      o.node = it->second;
      return o;
    }
    double v;
    if (parse_number(tok, &v)) {
      if (!allow_literal) fail(HCT_ERR_GRAPH, ln, "a number is not allowed as operand here");
      o.literal = v;
      return o;
    }
    if (!valid_name(tok)) fail(HCT_ERR_PARSE, ln, "malformed operand '" + tok + "'");
    fail(HCT_ERR_GRAPH, ln, "operand '" + tok + "' is not defined on an earlier line (dangling edge or cycle)");
  };

  while (std::getline(in, raw)) {
    ++line;
    size_t hash = raw.find('#');
    std::string s = trim(hash == std::string::npos ? raw : raw.substr(0, hash));
    if (s.empty()) continue;
    if (!header) {
      std::istringstream hs(s);
      std::string a, b, c;
      hs >> a >> b;
      if (a != "hct" || b != "1" || (hs >> c)) fail(HCT_ERR_PARSE, line, "expected header 'hct 1'");
      header = true;
      continue;
    }
    std::istringstream ls(s);
    std::string kw;
    ls >> kw;
    if (kw == "input") {
      std::string name, dtype;
      ls >> name >> dtype;
      std::string rest;
      std::getline(ls, rest);
      rest = trim(rest);
      if (!valid_name(name)) fail(HCT_ERR_PARSE, line, "malformed input name");
      if (index.count(name)) fail(HCT_ERR_GRAPH, line, "duplicate name '" + name + "'");
      Node n;
      n.name = name;
      n.op = "input";
      n.cls = OpClass::Input;
      if (dtype == "f32")
        n.dtype = F32;
      else if (dtype == "bf16")
        n.dtype = BF16;
      else
        fail(HCT_ERR_PARSE, line, "unknown dtype '" + dtype + "'");
      {  // optional layout word after the shape
        size_t rb = rest.find(']');
        if (rb != std::string::npos && rb + 1 < rest.size()) {
          std::string layout = trim(rest.substr(rb + 1));
          rest = rest.substr(0, rb + 1);
          if (layout == "nhwc")
            n.nhwc = true;
          else if (layout != "nchw")
            fail(HCT_ERR_PARSE, line, "unknown layout '" + layout + "' (nchw or nhwc)");
        }
      }
      if (rest.size() < 2 || rest.front() != '[' || rest.back() != ']') fail(HCT_ERR_PARSE, line, "malformed shape");
      for (auto& t : split(rest.substr(1, rest.size() - 2), ',')) {
        int64_t d;
        if (!parse_int(t, &d) || d < 0) fail(HCT_ERR_PARSE, line, "malformed shape extent '" + t + "'");
        n.shape.push_back(d);
      }
      if (n.shape.empty() || n.shape.size() > 4) fail(HCT_ERR_PARSE, line, "rank must be 1..4");
      if (n.nhwc && (n.shape.size() != 4 || n.dtype != BF16)) fail(HCT_ERR_UNSUPPORTED, line, "the nhwc layout is supported for bf16 inputs of rank 4");
      {  // tensors are capped at 2^40 elements, so that element counts, byte counts and workspace offsets stay far inside int64
        int64_t count = 1;
        for (int64_t d : n.shape) {
          if (d > kMaxElements || (d > 0 && count > kMaxElements / d)) fail(HCT_ERR_UNSUPPORTED, line, "tensors of more than 2^40 elements are not supported");
          count *= d;
        }
      }
      n.input_index = (int)g.inputs.size();
      index[name] = (int)g.nodes.size();
      g.inputs.push_back((int)g.nodes.size());
      g.nodes.push_back(n);
    } else if (kw == "node") {
      std::string rest;
      std::getline(ls, rest);
      size_t eq = rest.find('=');
      size_t lp = rest.find('(');
      size_t rp = rest.rfind(')');
      if (eq == std::string::npos || lp == std::string::npos || rp == std::string::npos || !(eq < lp && lp < rp) ||
          !trim(rest.substr(rp + 1)).empty())
        fail(HCT_ERR_PARSE, line, "malformed node, expected: node NAME = OP(args)");
      std::string name = trim(rest.substr(0, eq));
      std::string op = trim(rest.substr(eq + 1, lp - eq - 1));
      std::string argstr = trim(rest.substr(lp + 1, rp - lp - 1));
      if (!valid_name(name)) fail(HCT_ERR_PARSE, line, "malformed node name");
      if (!valid_name(op)) fail(HCT_ERR_PARSE, line, "malformed operator name");
      if (index.count(name)) fail(HCT_ERR_GRAPH, line, "duplicate name '" + name + "'");
      std::vector<std::string> pos;
      std::map<std::string, std::string> attrs;
      if (!argstr.empty()) {
        for (auto& t : split(argstr, ',')) {
          if (t.empty()) fail(HCT_ERR_PARSE, line, "empty argument");
          size_t e = t.find('=');
          if (e != std::string::npos) {
            attrs[trim(t.substr(0, e))] = trim(t.substr(e + 1));
          } else {
            if (!attrs.empty()) fail(HCT_ERR_PARSE, line, "positional argument after keyword argument");
            pos.push_back(t);
          }
        }
      }
      auto only_attrs = [&](std::initializer_list<const char*> allowed) {
        for (auto& kv : attrs) {
          bool ok = false;
          for (auto a : allowed) ok = ok || kv.first == a;
          if (!ok) fail(HCT_ERR_GRAPH, line, "unknown attribute '" + kv.first + "' for " + op);
        }
      };
      auto int_attr = [&](const char* key, int dflt) {
        auto it = attrs.find(key);
        if (it == attrs.end()) return dflt;
        int64_t v;
        if (!parse_int(it->second, &v)) fail(HCT_ERR_PARSE, line, std::string("attribute ") + key + " must be an integer");
        return (int)v;
      };
      Node n;
      n.name = name;
      n.op = op;
      n.dtype = F32;
      if (op == "cast_bf16") {
        // rounds to bfloat16 (nearest even); the value may then feed a bf16 gemm / conv2d, and is kept as
        // bf16 when it has to be materialised between kernels
        only_attrs({});
        if (pos.size() != 1) fail(HCT_ERR_GRAPH, line, "cast_bf16 takes one operand");
        n.cls = OpClass::Unary;
        n.args = {lookup(pos[0], line, false)};
        n.shape = g.nodes[n.args[0].node].shape;
        n.dtype = BF16;
      } else if (op == "dropout") {
        // Inverted dropout with a counter-based mask (the hash generator of the paper's first case study):
        // h = i + seed; h ^= h >> 17; h ^= h << 31; h ^= h >> 8 in 64-bit arithmetic, i the element's
        // row-major offset; the element is kept, scaled by 1/(1-p), when h mod 1000 >= round(1000 p).
        only_attrs({"p", "seed"});
        if (pos.size() != 1) fail(HCT_ERR_GRAPH, line, "dropout takes one operand");
        n.cls = OpClass::Unary;
        n.args = {lookup(pos[0], line, false)};
        n.shape = g.nodes[n.args[0].node].shape;
        n.drop_p = 0.5;
        if (attrs.count("p") && (!parse_number(attrs["p"], &n.drop_p) || !(n.drop_p >= 0.0 && n.drop_p < 1.0)))
          fail(HCT_ERR_PARSE, line, "p must be a number in [0,1)");
        int64_t seed = 0;
        if (attrs.count("seed") && (!parse_int(attrs["seed"], &seed) || seed < 0)) fail(HCT_ERR_PARSE, line, "seed must be a non-negative integer");
        n.drop_seed = (uint64_t)seed;
        n.drop_threshold = (unsigned)std::llround(n.drop_p * 1000.0);
        if (n.drop_threshold >= 1000) fail(HCT_ERR_PARSE, line, "p rounds to 1: nothing would be kept");
      } else if (is_unary(op)) {
        only_attrs({});
        if (pos.size() != 1) fail(HCT_ERR_GRAPH, line, op + " takes one operand");
        n.cls = OpClass::Unary;
        n.args = {lookup(pos[0], line, false)};
        n.shape = g.nodes[n.args[0].node].shape;
      } else if (is_binary(op)) {
        only_attrs({});
        if (pos.size() != 2) fail(HCT_ERR_GRAPH, line, op + " takes two operands");
        n.cls = OpClass::Binary;
        n.args = {lookup(pos[0], line, true), lookup(pos[1], line, true)};
        if (n.args[0].is_literal() && n.args[1].is_literal())
          fail(HCT_ERR_GRAPH, line, "at least one operand must be a tensor");
        if (n.args[0].is_literal())
          n.shape = g.nodes[n.args[1].node].shape;
        else if (n.args[1].is_literal())
          n.shape = g.nodes[n.args[0].node].shape;
        else
          n.shape = broadcast(g.nodes[n.args[0].node].shape, g.nodes[n.args[1].node].shape, line);
      } else if (op == "row_softmax" || op == "row_sum" || op == "row_mean" || op == "row_max" || op == "row_min" || op == "row_argmax" ||
                 op == "row_argmin") {
        only_attrs({});
        if (pos.size() != 1) fail(HCT_ERR_GRAPH, line, op + " takes one operand");
        n.cls = op == "row_softmax" ? OpClass::RowSoftmax : OpClass::RowReduce;
        n.args = {lookup(pos[0], line, false)};
        auto& s = g.nodes[n.args[0].node].shape;
        // a softmax over a single column is legal (and identically one); the reductions need two columns
        if (s.size() != 2 || s[1] < (op == "row_softmax" ? 1 : 2))
          fail(HCT_ERR_GRAPH, line, op + " needs a [R,C] operand with C >= " + (op == "row_softmax" ? "1" : "2") + ", got " + shape_str(s));
        n.shape = s;
        if (n.cls == OpClass::RowReduce) n.shape[1] = 1;
      } else if (op == "row_layernorm") {
        only_attrs({"eps"});
        if (pos.size() != 3) fail(HCT_ERR_GRAPH, line, "row_layernorm takes (x, gamma, beta)");
        n.cls = OpClass::RowLayernorm;
        for (auto& p : pos) n.args.push_back(lookup(p, line, false));
        auto& s = g.nodes[n.args[0].node].shape;
        if (s.size() != 2 || s[1] < 2) fail(HCT_ERR_GRAPH, line, "row_layernorm needs a [R,C] operand with C >= 2, got " + shape_str(s));
        for (int i = 1; i < 3; ++i) {
          auto& ps = g.nodes[n.args[i].node].shape;
          bool ok = (ps.size() == 1 && ps[0] == s[1]) || (ps.size() == 2 && ps[0] == 1 && ps[1] == s[1]);
          if (!ok) fail(HCT_ERR_GRAPH, line, "gamma/beta must have shape [C], got " + shape_str(ps));
        }
        if (attrs.count("eps") && (!parse_number(attrs["eps"], &n.eps) || !(n.eps >= 0)))
          fail(HCT_ERR_PARSE, line, "eps must be a non-negative number");
        n.shape = s;
      } else if (op == "transpose") {
        // layout transform (Table 1): y[j,i] = x[i,j] for a 2-D operand
        only_attrs({});
        if (pos.size() != 1) fail(HCT_ERR_GRAPH, line, "transpose takes one operand");
        n.cls = OpClass::Transpose;
        n.args = {lookup(pos[0], line, false)};
        auto& s = g.nodes[n.args[0].node].shape;
        if (s.size() != 2) fail(HCT_ERR_GRAPH, line, "transpose needs a [R,C] operand, got " + shape_str(s));
        n.shape = {s[1], s[0]};
      } else if (op == "permute") {
        // layout transform (Table 1): the axes of a tensor of rank 2..4 in another order; axes=0231 means
        // output axis d is input axis digit d (NCHW -> NHWC)
        only_attrs({"axes"});
        if (pos.size() != 1) fail(HCT_ERR_GRAPH, line, "permute takes one operand");
        n.cls = OpClass::Permute;
        n.args = {lookup(pos[0], line, false)};
        const Node& src = g.nodes[n.args[0].node];
        const size_t rank = src.shape.size();
        const std::string ax = attrs.count("axes") ? attrs["axes"] : "";
        if (rank < 2 || ax.size() != rank) fail(HCT_ERR_GRAPH, line, "permute needs a tensor of rank 2..4 and axes=<one digit per axis>");
        bool seen[4] = {false, false, false, false};
        n.shape.clear();
        for (size_t d = 0; d < rank; ++d) {
          const int a = ax[d] - '0';
          if (a < 0 || a >= (int)rank || seen[a]) fail(HCT_ERR_GRAPH, line, "axes must be a permutation of 0.." + std::to_string(rank - 1));
          seen[a] = true;
          n.shape.push_back(src.shape[a]);
          n.perm[4 - rank + d] = a + (int)(4 - rank);   // in the padded four-axis numbering
        }
        n.dtype = src.dtype;   // values are moved unchanged
      } else if (op == "reshape") {
        // layout transform (Table 1): the same elements in row-major order under a new 2-D shape, e.g. flattening
        // [N,C,H,W] into [N, C*H*W] in front of a gemm
        only_attrs({"rows", "cols"});
        if (pos.size() != 1) fail(HCT_ERR_GRAPH, line, "reshape takes one operand");
        n.cls = OpClass::Reshape;
        n.args = {lookup(pos[0], line, false)};
        const Node& src = g.nodes[n.args[0].node];
        int64_t rows, cols;
        if (!attrs.count("rows") || !attrs.count("cols") || !parse_int(attrs["rows"], &rows) || !parse_int(attrs["cols"], &cols) || rows < 1 || cols < 1)
          fail(HCT_ERR_PARSE, line, "reshape needs rows=R, cols=C (positive integers)");
        if (rows * cols != src.numel()) fail(HCT_ERR_GRAPH, line, "reshape of " + shape_str(src.shape) + " must keep the number of elements");
        n.shape = {rows, cols};
        n.dtype = src.dtype;   // values are moved unchanged, so a bf16 value stays bf16
      } else if (op == "row_sort" || op == "row_topk" || op == "row_argsort" || op == "row_topk_indices") {
        // logic-intensive operators (Table 1): the values of every row in order; row_topk keeps the k largest, largest first;
        // row_argsort / row_topk_indices deliver the columns those values came from (the smaller column first among equals)
        const bool topk = op == "row_topk" || op == "row_topk_indices";
        n.sort_indices = op == "row_argsort" || op == "row_topk_indices";
        if (topk) only_attrs({"k"}); else only_attrs({"descending"});
        if (pos.size() != 1) fail(HCT_ERR_GRAPH, line, op + " takes one operand");
        n.cls = OpClass::Sort;
        n.args = {lookup(pos[0], line, false)};
        auto& s = g.nodes[n.args[0].node].shape;
        if (s.size() != 2) fail(HCT_ERR_GRAPH, line, op + " needs a [R,C] operand, got " + shape_str(s));
        if (s[1] > 8192) fail(HCT_ERR_UNSUPPORTED, line, op + " supports rows of up to 8192 elements");
        n.descending = topk || int_attr("descending", 0) != 0;
        n.sort_k = topk ? int_attr("k", 1) : 0;
        if (topk && (n.sort_k < 1 || n.sort_k > s[1])) fail(HCT_ERR_GRAPH, line, op + " needs 1 <= k <= C");
        n.shape = {s[0], topk ? (int64_t)n.sort_k : s[1]};
      } else if (op == "gemm") {
        only_attrs({"precision"});
        if (pos.size() != 2) fail(HCT_ERR_GRAPH, line, "gemm takes (a, b)");
        n.cls = OpClass::Gemm;
        n.args = {lookup(pos[0], line, false), lookup(pos[1], line, false)};
        auto& a = g.nodes[n.args[0].node];
        auto& b = g.nodes[n.args[1].node];
        if (a.shape.size() != 2 || b.shape.size() != 2 || a.shape[1] != b.shape[0])
          fail(HCT_ERR_GRAPH, line, "gemm shapes " + shape_str(a.shape) + " x " + shape_str(b.shape) + " do not contract");
        if (a.dtype != b.dtype) fail(HCT_ERR_GRAPH, line, "gemm operands must have one dtype");
        n.shape = {a.shape[0], b.shape[1]};
      } else if (op == "conv2d") {
        only_attrs({"stride", "pad", "dilation", "groups"});
        if (pos.size() != 2) fail(HCT_ERR_GRAPH, line, "conv2d takes (x, w)");
        n.cls = OpClass::Conv;
        n.args = {lookup(pos[0], line, false), lookup(pos[1], line, false)};
        auto& a = g.nodes[n.args[0].node];
        auto& b = g.nodes[n.args[1].node];
        n.stride = int_attr("stride", 1);
        n.pad = int_attr("pad", 0);
        n.dilation = int_attr("dilation", 1);
        n.groups = int_attr("groups", 1);
        // channels and filters are cut into `groups` equal parts; a filter sees only its part's channels
        if (a.shape.size() != 4 || b.shape.size() != 4 || n.stride < 1 || n.pad < 0 || n.dilation < 1 || n.groups < 1 ||
            a.shape[1] != b.shape[1] * n.groups || b.shape[0] % n.groups != 0)
          fail(HCT_ERR_GRAPH, line, "conv2d operands " + shape_str(a.shape) + ", " + shape_str(b.shape) + " are inconsistent");
        if (a.dtype != b.dtype) fail(HCT_ERR_GRAPH, line, "conv2d operands must have one dtype");
        // a filter of R taps spaced `dilation` apart spans dilation * (R - 1) + 1 input rows
        const int64_t eh = a.shape[2] + 2 * n.pad - ((int64_t)n.dilation * (b.shape[2] - 1) + 1);
        const int64_t ew = a.shape[3] + 2 * n.pad - ((int64_t)n.dilation * (b.shape[3] - 1) + 1);
        if (eh < 0 || ew < 0) fail(HCT_ERR_GRAPH, line, "conv2d output is empty");
        int64_t ho = eh / n.stride + 1, wo = ew / n.stride + 1;
        n.shape = {a.shape[0], b.shape[0], ho, wo};
      } else {
        fail(HCT_ERR_GRAPH, line, "unknown operator '" + op + "'");
      }
      index[name] = (int)g.nodes.size();
      g.nodes.push_back(n);
    } else if (kw == "output") {
      std::string name, dtype, layout, extra;
      ls >> name;
      bool has_dtype = (bool)(ls >> dtype);
      bool has_layout = (bool)(ls >> layout);
      if (name.empty() || (ls >> extra)) fail(HCT_ERR_PARSE, line, "malformed output, expected: output NAME [DTYPE [LAYOUT]]");
      auto it = index.find(name);
      if (it == index.end()) fail(HCT_ERR_GRAPH, line, "output '" + name + "' is not defined");
      Node& n = g.nodes[it->second];
      if (n.cls == OpClass::Input) fail(HCT_ERR_GRAPH, line, "an input cannot be an output");
      if (n.output_index >= 0) fail(HCT_ERR_GRAPH, line, "duplicate output '" + name + "'");
      if (!has_dtype || dtype == "f32")
        n.out_dtype = F32;
      else if (dtype == "bf16")
        n.out_dtype = BF16;
      else
        fail(HCT_ERR_PARSE, line, "unknown dtype '" + dtype + "'");
      if (has_layout) {
        if (layout == "nhwc")
          n.out_nhwc = true;
        else if (layout != "nchw")
          fail(HCT_ERR_PARSE, line, "unknown layout '" + layout + "' (nchw or nhwc)");
        if (n.out_nhwc && n.shape.size() != 4) fail(HCT_ERR_UNSUPPORTED, line, "the nhwc layout is supported for outputs of rank 4");
      }
      n.output_index = (int)g.outputs.size();
      g.outputs.push_back(it->second);
    } else {
      fail(HCT_ERR_PARSE, line, "unknown statement '" + kw + "'");
    }
  }
  if (!header) throw Error(HCT_ERR_PARSE, "empty spec");
  if (g.outputs.empty()) throw Error(HCT_ERR_GRAPH, "the graph has no output");
  // a channels-last input is an activation tensor for convolutions: nothing else reads that layout
  for (const Node& nd : g.nodes)
    for (size_t ai = 0; ai < nd.args.size(); ++ai) {
      const Operand& a = nd.args[ai];
      if (a.is_literal() || !g.nodes[a.node].nhwc) continue;
      if (!(nd.cls == OpClass::Conv && ai == 0))
        throw Error(HCT_ERR_UNSUPPORTED, "input '" + g.nodes[a.node].name + "' is declared nhwc and may only be the first operand of conv2d");
    }

  // No dangling nodes: everything must reach an output.
  std::vector<char> live(g.nodes.size(), 0);
  std::vector<int> stack(g.outputs.begin(), g.outputs.end());
  while (!stack.empty()) {
    int i = stack.back();
    stack.pop_back();
    if (live[i]) continue;
    live[i] = 1;
    for (auto& a : g.nodes[i].args)
      if (!a.is_literal()) stack.push_back(a.node);
  }
  for (size_t i = 0; i < g.nodes.size(); ++i)
    if (!live[i]) throw Error(HCT_ERR_GRAPH, "node '" + g.nodes[i].name + "' does not reach any output");
  for (auto& n : g.nodes)
    if (n.numel() == 0) throw Error(HCT_ERR_UNSUPPORTED, "tensor '" + n.name + "' is empty");
  return g;
}

std::string elementwise_call(const Node& nd, const std::vector<std::string>& args, const std::string& flat_index) {
  std::string c = "hct_" + nd.op + "(";
  for (size_t i = 0; i < args.size(); ++i) c += (i ? ", " : "") + args[i];
  if (nd.op == "dropout") {
    char scale[32];
    std::snprintf(scale, sizeof scale, "%.9ef", (double)(float)(1.0 / (1.0 - nd.drop_p)));
    c += ", (unsigned long long)(" + flat_index + "), " + std::to_string((unsigned long long)nd.drop_seed) + "ULL, " +
         std::to_string(nd.drop_threshold) + "u, " + scale;
  }
  return c + ")";
}

}  // namespace hct
