// Host-side graph store: tensors as nodes, operators as multi-input/multi-output edges
// (Sec. 2.1, 2.2), gradient stages as sets of derivative pairs (Sec. 2.3).
#pragma once
#include <cstdint>
#include <string>
#include <unordered_set>
#include <vector>

#include "../../include/dragon.h"

namespace dragon {

struct Shape {
  int rank = 0;
  int64_t d[2] = {1, 1};
  int64_t numel() const { return (rank >= 1 ? d[0] : 1) * (rank >= 2 ? d[1] : 1); }
  int64_t rows() const { return rank == 2 ? d[0] : 1; }            // right-aligned view [rows, cols]
  int64_t cols() const { return rank == 2 ? d[1] : (rank == 1 ? d[0] : 1); }
  bool operator==(const Shape& o) const {
    if (rank != o.rank) return false;
    for (int i = 0; i < rank; ++i)
      if (d[i] != o.d[i]) return false;
    return true;
  }
  bool operator!=(const Shape& o) const { return !(*this == o); }
};

struct TensorInfo {
  std::string name;
  int dtype = DRAGON_F32;
  Shape shape;
  int producer = -1;      // operator id, -1 for a source
  bool consumed = false;  // some operator reads it
  int grad_stage = -1;    // >= 0: this tensor is d(objs of that stage)/d(grad_wrt)
  int grad_wrt = -1;
};

struct OpInfo {
  int type = 0;
  std::vector<int> in, out;
};

struct GradStage {
  std::vector<int> objs, wrts, grad_ids;
};

struct Graph {
  std::vector<TensorInfo> tensors;
  std::vector<OpInfo> ops;
  std::vector<GradStage> stages;
  std::unordered_set<std::string> names;
};

// Result of the two prunes for one function(inputs, outputs).
struct GradOpRef {
  int stage;
  int op;
  uint32_t mask;  // bit p: gradient w.r.t. operand position p is produced
};

struct PruneResult {
  std::vector<uint8_t> marked;              // per tensor id
  std::vector<int> fwd_ops;                 // creation order
  std::vector<GradOpRef> grad_ops;          // stage by stage, inverse creation order
  std::vector<uint8_t> used_inputs;         // per listed input
  std::vector<std::vector<uint8_t>> in_G;   // per stage, per tensor: on a chain wrt ~> obj
  std::vector<std::vector<uint8_t>> gmark;  // per stage, per tensor: gradient node marked
};

void set_error(const char* fmt, ...);
const char* last_error();

// right-aligned broadcast of two shapes restricted to the classes [], [C], [R,C]; false if incompatible
bool broadcast_shapes(const Shape& a, const Shape& b, Shape* out);

// chains wrt ~> obj for one stage (Algorithm 2, all pairs at once)
std::vector<uint8_t> backward_chain_marks(const Graph& g, const std::vector<int>& objs, const std::vector<int>& wrts);

// in-place structures of the pruned forward graph (Sec. 2.4, Algorithm 3): per tensor the ancestor
// it may be renamed to (itself when it starts a structure), -1 for an unmarked tensor
std::vector<int> inplace_rename(const Graph& g, const PruneResult& pr);

// both prunes over the two-stage DAG; returns a DRAGON_* code
int prune_function(const Graph& g, const std::vector<int>& inputs, const std::vector<int>& outputs, PruneResult* out);

}  // namespace dragon

struct dragon_graph {
  dragon::Graph g;
};
