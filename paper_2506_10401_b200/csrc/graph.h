// Typed operator DAG built from spec text: parsing, validation and shape inference.
#pragma once
#include <cstdint>
#include <stdexcept>
#include <string>
#include <vector>

namespace hct {

enum DType { F32 = 0, BF16 = 1 };

enum class OpClass { Input, Unary, Binary, RowSoftmax, RowLayernorm, RowReduce, Gemm, Conv, Transpose, Sort, Reshape, Permute };

struct Error : std::runtime_error {
  int code;
  Error(int c, const std::string& m) : std::runtime_error(m), code(c) {}
};

struct Operand {
  int node = -1;       // index into Graph::nodes, or -1 for a literal
  double literal = 0;  // used when node < 0
  bool is_literal() const { return node < 0; }
};

struct Node {
  std::string name;
  std::string op;  // "input" or the operator name
  OpClass cls = OpClass::Input;
  std::vector<Operand> args;
  std::vector<int64_t> shape;
  DType dtype = F32;  // storage dtype of an input; computed nodes are fp32 values (BF16: values rounded to bfloat16 by cast_bf16)
  double eps = 1e-5;
  int stride = 1, pad = 0, dilation = 1, groups = 1;
  int sort_k = 0;            // row_topk: number of leading elements kept (0: the whole sorted row)
  bool descending = false;   // row_sort / row_topk: largest first
  int perm[4] = {0, 1, 2, 3}; // permute: output axis d is input axis perm[d] (both padded to four axes with leading ones)
  bool sort_indices = false; // row_argsort / row_topk_indices: the columns of the ordered values instead of the values
  // dropout: element with flat index i is kept when hash(i + seed) mod 1000 >= drop_threshold (= round(1000 p))
  double drop_p = 0.0;
  uint64_t drop_seed = 0;
  unsigned drop_threshold = 0;
  int input_index = -1;   // position among `input` lines
  bool out_nhwc = false;  // output only: the output buffer of this rank-4 value is laid out [N,H,W,C]
  bool nhwc = false;      // input only: a rank-4 tensor [N,C,H,W] whose buffer is laid out [N,H,W,C] (channels contiguous)
  int output_index = -1;  // position among `output` lines
  DType out_dtype = F32;  // storage dtype when the node is a graph output
  int64_t numel() const {
    int64_t n = 1;
    for (auto d : shape) n *= d;
    return n;
  }
};

struct Graph {
  std::vector<Node> nodes;   // definition order is a topological order
  std::vector<int> inputs;   // node indices
  std::vector<int> outputs;  // node indices
};

// Throws Error(HCT_ERR_PARSE | HCT_ERR_GRAPH | HCT_ERR_UNSUPPORTED).
Graph parse_spec(const std::string& text);

bool is_unary(const std::string& op);
bool is_binary(const std::string& op);

// Source text of the call that evaluates elementwise node `nd` on the operand expressions `args`;
// `flat_index` is an expression for the element's row-major offset in the node's tensor (used by dropout).
std::string elementwise_call(const Node& nd, const std::vector<std::string>& args, const std::string& flat_index);

}  // namespace hct
