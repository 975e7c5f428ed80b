// Fusion planner: partitions the operator DAG into kernels.
//
// Two kinds of group exist.  A *row group* is a maximal set of elementwise, broadcast and
// row-reduction nodes that share one [R,C] iteration space, so a row can stay in registers from
// the first load to the last store.  A *contraction group* is one gemm or conv2d node together
// with the elementwise nodes that consume its result (its epilogue); a transpose anchors a group the same way.  Values that cross a group
// boundary are written once to caller-provided workspace (fp32).
#pragma once
#include <string>
#include <vector>

#include "graph.h"

namespace hct {

enum class GroupKind { Row, Gemm, Conv, Transpose, Sort, Reshape, Permute };

// How an operand indexes relative to the group's full shape [.., C].
enum class Bcast {
  Full,    // same shape: element (row, col)
  RowVec,  // [C] / [1,..,C]: indexed by col
  RowIdx,  // last extent 1: one scalar per row, index = sum of row coordinates times strides
  Scalar   // a single element
};

struct ExtOperand {
  int node;  // producing node (a graph input or a node materialised by an earlier group)
  Bcast bcast;
  // RowIdx: index = sum_d coord_d * stride[d] over the leading extents of the full shape
  std::vector<int64_t> lead_stride;
};

struct Store {
  int node;
  DType dtype;
  bool to_output;  // graph output buffer, else workspace
};

struct Group {
  GroupKind kind = GroupKind::Row;
  std::vector<int> nodes;           // topological; a contraction group starts with its anchor
  std::vector<int64_t> full_shape;  // shape of full-size values ([R,C], [M,N] or [N,K,H,W])
  int64_t R = 0, C = 0;             // rows = product of leading extents, cols = last extent
  std::vector<ExtOperand> ext;      // deduplicated external operands
  std::vector<Store> stores;
  bool has_reduction = false;
};

struct Plan {
  std::vector<Group> groups;
  std::vector<int> group_of;           // per node (-1 for inputs)
  std::vector<int64_t> ws_offset;      // per node, -1 if not in workspace
  std::vector<char> is_colv;           // per node: value is one scalar per row of its group
  // A contraction result that only feeds row sums is not materialised: the epilogue writes one partial sum per
  // row and 32-column chunk, and the row group sums those.  partial_cols[node] = chunks per row (0: stored whole);
  // reduce_count[node] = number of elements a row_mean divides by when its operand arrives as partial sums (0: its width).
  std::vector<int64_t> partial_cols, reduce_count;
  // A full-width fp32 value of a row group whose only readers are fp32 tensor-core GEMMs taking it as their first
  // operand is stored as the TF32 head and tail those GEMMs multiply (two arrays in its workspace slot, the tail
  // split_lo_offset bytes after the head) instead of as the value itself: the GEMM's split pre-pass skips it.
  std::vector<char> split_store;
  std::vector<int64_t> split_lo_offset;
  size_t workspace_bytes = 0;
  double algorithmic_bytes = 0, flops = 0;
  std::string text;
};

Plan make_plan(const Graph& g);

// Index of `node` in group.ext, or -1.
int find_ext(const Group& grp, int node);

}  // namespace hct
