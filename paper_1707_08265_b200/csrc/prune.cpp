// Forward prune (Algorithm 1) and backward prune (Algorithm 2) over the two-stage DAG of
// Sec. 2.3, iterative (explicit stacks) so that graph depth is not limited by the call stack.
#include <algorithm>
#include <cstdarg>
#include <cstdio>

#include "graph.h"

namespace dragon {

static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

const char* last_error() { return g_err; }

bool broadcast_shapes(const Shape& a, const Shape& b, Shape* out) {
  const Shape& hi = a.rank >= b.rank ? a : b;
  const Shape& lo = a.rank >= b.rank ? b : a;
  *out = hi;
  if (lo.rank == 0) return true;
  if (lo.rank == hi.rank) {
    if (lo == hi) return true;
    // [1,C] against [R,C]
    if (lo.rank == 2 && lo.d[1] == hi.d[1] && (lo.d[0] == 1 || hi.d[0] == 1)) {
      out->d[0] = lo.d[0] == 1 ? hi.d[0] : lo.d[0];
      return true;
    }
    return false;
  }
  // lo is [C], hi is [R,C]
  return lo.rank == 1 && hi.rank == 2 && lo.d[0] == hi.d[1];
}

namespace {

// multi-source reachability along `next`, written with an explicit stack
template <class NextFn>
void sweep(size_t n, const std::vector<int>& start, std::vector<uint8_t>* seen, NextFn next) {
  seen->assign(n, 0);
  std::vector<int> stack;
  for (int s : start)
    if (!(*seen)[s]) {
      (*seen)[s] = 1;
      stack.push_back(s);
    }
  while (!stack.empty()) {
    int x = stack.back();
    stack.pop_back();
    next(x, [&](int y) {
      if (!(*seen)[y]) {
        (*seen)[y] = 1;
        stack.push_back(y);
      }
    });
  }
}

}  // namespace

std::vector<uint8_t> backward_chain_marks(const Graph& g, const std::vector<int>& objs, const std::vector<int>& wrts) {
  // The union over all pairs (obj, wrt) of the nodes on a chain wrt ~> obj equals
  // descendants(wrts) intersected with ancestors(objs); two linear sweeps replace the per-pair
  // memoised search of Algorithm 2.
  const int n = (int)g.tensors.size();
  std::vector<std::vector<int>> consumers(n);
  for (int k = 0; k < (int)g.ops.size(); ++k)
    for (int i : g.ops[k].in) consumers[i].push_back(k);
  std::vector<uint8_t> down, up;
  sweep(n, wrts, &down, [&](int x, auto visit) {
    for (int k : consumers[x])
      for (int o : g.ops[k].out) visit(o);
  });
  sweep(n, objs, &up, [&](int x, auto visit) {
    int p = g.tensors[x].producer;
    if (p >= 0)
      for (int i : g.ops[p].in) visit(i);
  });
  std::vector<uint8_t> m(n);
  for (int i = 0; i < n; ++i) m[i] = down[i] && up[i];
  return m;
}

int prune_function(const Graph& g, const std::vector<int>& inputs, const std::vector<int>& outputs, PruneResult* out) {
  const int n = (int)g.tensors.size();
  const int n_ops = (int)g.ops.size();
  const int n_st = (int)g.stages.size();

  out->in_G.resize(n_st);
  std::vector<std::vector<uint8_t>> gop(n_st);  // gradient operator of op k exists in stage s
  for (int s = 0; s < n_st; ++s) {
    out->in_G[s] = backward_chain_marks(g, g.stages[s].objs, g.stages[s].wrts);
    const auto& G = out->in_G[s];
    gop[s].assign(n_ops, 0);
    for (int k = 0; k < n_ops; ++k) {
      bool o_in = false, i_in = false;
      for (int o : g.ops[k].out) o_in |= G[o] != 0;
      for (int i : g.ops[k].in) i_in |= G[i] != 0;
      gop[s][k] = o_in && i_in;
    }
  }
  // a fetched gradient needs a chain; feeding an intermediate tensor can have cut the last one
  for (int t : outputs) {
    const TensorInfo& ti = g.tensors[t];
    if (ti.grad_stage >= 0 && !out->in_G[ti.grad_stage][ti.grad_wrt]) {
      set_error("no chain is left from '%s' to any objective of its gradient stage in this function", g.tensors[ti.grad_wrt].name.c_str());
      return DRAGON_ERR_NO_PATH;
    }
  }
  std::vector<std::vector<int>> consumers(n);
  for (int k = 0; k < n_ops; ++k)
    for (int i : g.ops[k].in)
      if (consumers[i].empty() || consumers[i].back() != k) consumers[i].push_back(k);
  std::vector<std::vector<uint8_t>> is_obj(n_st, std::vector<uint8_t>(n, 0));
  for (int s = 0; s < n_st; ++s)
    for (int o : g.stages[s].objs) is_obj[s][o] = 1;

  // Algorithm 1 over forward nodes [0, n) and gradient nodes n*(1+s)+x, from the fetched targets
  std::vector<uint8_t> seen;
  sweep((size_t)n * (1 + n_st), outputs, &seen, [&](int node, auto visit) {
    if (node < n) {
      const TensorInfo& t = g.tensors[node];
      if (t.grad_stage >= 0) {
        visit(n * (1 + t.grad_stage) + t.grad_wrt);
      } else if (t.producer >= 0) {
        for (int i : g.ops[t.producer].in) visit(i);
      }
      return;
    }
    const int s = node / n - 1, x = node % n;
    if (is_obj[s][x]) visit(x);  // the chain starts at the objective itself
    for (int k : consumers[x])
      if (gop[s][k])
        for (int y : g.ops[k].out)
          if (out->in_G[s][y]) visit(n * (1 + s) + y);
  });

  out->marked.assign(n, 0);
  for (int t = 0; t < n; ++t) {
    const TensorInfo& ti = g.tensors[t];
    out->marked[t] = ti.grad_stage >= 0 ? seen[(size_t)n * (1 + ti.grad_stage) + ti.grad_wrt] : seen[t];
  }
  out->gmark.assign(n_st, std::vector<uint8_t>());
  for (int s = 0; s < n_st; ++s) out->gmark[s].assign(seen.begin() + (size_t)n * (1 + s), seen.begin() + (size_t)n * (2 + s));

  out->fwd_ops.clear();
  for (int k = 0; k < n_ops; ++k) {
    bool keep = false;
    for (int o : g.ops[k].out) keep |= out->marked[o] != 0;
    if (keep) out->fwd_ops.push_back(k);
  }
  out->grad_ops.clear();
  for (int s = 0; s < n_st; ++s)
    for (int k = n_ops - 1; k >= 0; --k) {
      if (!gop[s][k]) continue;
      const auto& in = g.ops[k].in;
      uint32_t mask = 0;
      for (int p = 0; p < (int)in.size() && p < 32; ++p) {
        bool first = true;
        for (int q = 0; q < p; ++q) first &= in[q] != in[p];
        if (first && out->in_G[s][in[p]] && out->gmark[s][in[p]]) mask |= 1u << p;
      }
      if (mask) out->grad_ops.push_back({s, k, mask});
    }
  out->used_inputs.clear();
  for (int i : inputs) out->used_inputs.push_back(out->marked[i]);
  // a marked source that is not listed cannot be fed
  std::vector<uint8_t> listed(n, 0);
  for (int i : inputs) listed[i] = 1;
  for (int t = 0; t < n; ++t)
    if (out->marked[t] && g.tensors[t].producer < 0 && g.tensors[t].grad_stage < 0 && !listed[t]) {
      set_error("tensor '%s' is needed by the targets but is not among the inputs", g.tensors[t].name.c_str());
      return DRAGON_ERR_MISSING_INPUT;
    }
  return DRAGON_OK;
}

// Algorithm 3 (Sec. 2.4).  A node with exactly one child hands its memory on to that child, so a
// path of such nodes is one in-place structure named after its first node.  Nodes are taken in
// creation order; from each node that has no name yet the walk follows only-children until it
// meets a node with several (or no) children, or one that already has a name: every node is named
// once, O(n + e).  Only marked tensors and kept forward operators take part (renaming comes after
// the prunes: it would make the graph cyclic).
std::vector<int> inplace_rename(const Graph& g, const PruneResult& pr) {
  const int n = (int)g.tensors.size();
  std::vector<std::vector<int>> child(n);
  for (int k : pr.fwd_ops) {
    const OpInfo& op = g.ops[k];
    for (int i : op.in) {
      if (!pr.marked[i]) continue;
      for (int o : op.out)
        if (pr.marked[o] && std::find(child[i].begin(), child[i].end(), o) == child[i].end()) child[i].push_back(o);
    }
  }
  std::vector<int> rd(n, -1);
  for (int start = 0; start < n; ++start) {
    if (!pr.marked[start]) continue;
    int x = start;
    while (rd[x] < 0) {
      rd[x] = start;
      if (child[x].size() != 1) break;
      x = child[x][0];
    }
  }
  return rd;
}

}  // namespace dragon
