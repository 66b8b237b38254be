// Host compiler, part 1: kept operators -> micro-operations -> fused segments -> launch plan.
//
// Forward operators are lowered in creating order, gradient operators in inverse order
// (Sec. 3.2).  A gradient operator reads forward values through its anchor (Sec. 3.3); inside
// one fused segment those are simply values that stay live, across segments they are
// workspace tensors.  Gradients with respect to broadcast operands are kept per domain element
// (the reverse sweep is linear in dy) and summed once, where the gradient tensor is written.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <map>
#include <set>

#include "plan.h"

namespace dragon {
namespace {

struct Lowerer {
  const Graph& g;
  const PruneResult& pr;
  Plan* plan;
  std::vector<Item> items;
  std::vector<Value> vals;
  std::vector<int> fval;                      // forward tensor -> value id
  std::vector<std::map<int, int>> gval;       // per stage: tensor -> gradient value id
  std::vector<int> fetch_of;                  // tensor -> fetch position or -1
  std::map<std::pair<int, int>, int> materialised;   // (value, dtype) -> memref
  std::vector<std::map<int, int>> pending;    // per stage: tensor -> gradient contributions still to come
  std::map<int, int> def_item;                // value -> index of the micro-operation that defines it
  int err = DRAGON_OK;

  Lowerer(const Graph& g_, const PruneResult& pr_, Plan* p) : g(g_), pr(pr_), plan(p) {}

  int new_mem(int where, int index, int dtype, const Shape& s) {
    MemRef m;
    m.where = where; m.index = index; m.dtype = dtype; m.shape = s;
    plan->mems.push_back(m);
    return (int)plan->mems.size() - 1;
  }
  int new_val(int kind, const Shape& s, int mem = -1, float c = 0.f) {
    Value v; v.kind = kind; v.shape = s; v.mem = mem; v.c = c;
    v.row_uniform = s.numel() == 1;     // scalars and constants; operations set it for their results
    vals.push_back(v);
    return (int)vals.size() - 1;
  }
  // the micro-operation that defines value v (through widenings), or null
  const Item* def_of(int v) const {
    for (;;) {
      auto it = def_item.find(v);
      if (it == def_item.end()) return nullptr;
      const Item& d = items[it->second];
      if (d.opc != M_WIDEN) return &d;
      v = d.a;
    }
  }
  int konst(float c) {
    int v = new_val(VK_CONST, Shape(), -1, c);
    vals[v].known_const = true;
    vals[v].lo = vals[v].hi = c;
    return v;
  }
  bool is_const(int v, float c) const { return vals[v].known_const && vals[v].c == c; }

  // the same value seen with a (wider) logical shape; emits no instruction
  int widen(int v, const Shape& want) {
    Shape s;
    if (!broadcast_shapes(vals[v].shape, want, &s) || s == vals[v].shape) return v;
    Item it; it.kind = IT_MOP; it.opc = M_WIDEN; it.a = v;
    it.dst = new_val(VK_OP, s);
    vals[it.dst].known_const = vals[v].known_const;
    vals[it.dst].c = vals[v].c;
    vals[it.dst].row_uniform = vals[v].row_uniform;
    vals[it.dst].lo = vals[v].lo;
    vals[it.dst].hi = vals[v].hi;
    def_item[it.dst] = (int)items.size();
    items.push_back(it);
    return it.dst;
  }

  // [lo, hi] of the result of a micro-operation from those of its operands (NaN aside); anything not known is
  // the whole line.  The bounds are rounded outwards by a relative 1e-6 so that fp32 rounding cannot breach them.
  void set_range(int dst, int opc, const Value& A, const Value* B) {
    const float inf = std::numeric_limits<float>::infinity();
    float lo = -inf, hi = inf;
    auto corners = [&](float (*f)(float, float)) {
      const float c[4] = {f(A.lo, B->lo), f(A.lo, B->hi), f(A.hi, B->lo), f(A.hi, B->hi)};
      lo = inf; hi = -inf;
      for (float x : c) {
        if (x != x) { lo = -inf; hi = inf; return; }      // 0 * inf, inf - inf: nothing is known
        lo = std::min(lo, x); hi = std::max(hi, x);
      }
    };
    const float m = std::max(std::fabs(A.lo), std::fabs(A.hi));
    switch (opc) {
      case M_ADD: corners([](float x, float y) { return x + y; }); break;
      case M_SUB: corners([](float x, float y) { return x - y; }); break;
      case M_MUL: corners([](float x, float y) { return x * y; }); break;
      case M_DIVP: lo = std::min(A.lo, 0.f); hi = std::max(A.hi, 0.f); break;          // |a / (1 + |b|)| <= |a|, same sign
      case M_SIN: case M_COS: case M_TANH: case M_TANHB: case M_DIVPGB: lo = -1.f; hi = 1.f; break;
      case M_SIGMOID: case M_SIGMOIDB: case M_STEP: case M_CLAMPMASK: lo = 0.f; hi = 1.f; break;
      case M_EXPC: case M_EXPCB: lo = 4.5e-5f; hi = 22027.f; break;                    // e^-10 .. e^10
      case M_RELU: lo = std::max(A.lo, 0.f); hi = std::max(A.hi, 0.f); break;
      case M_NEG: lo = -A.hi; hi = -A.lo; break;
      case M_ONEMSQ: hi = 1.f; lo = m < 1e18f ? 1.f - m * m : -inf; break;              // 1 - y^2
      case M_YOMY: hi = 0.25f;                                                          // y (1 - y), concave
        lo = m < 1e18f ? std::min(A.lo * (1.f - A.lo), A.hi * (1.f - A.hi)) : -inf; break;
      case M_RBF16: lo = A.lo - std::fabs(A.lo) / 128.f; hi = A.hi + std::fabs(A.hi) / 128.f; break;
      case M_ROWSUM: { const float n = (float)A.shape.cols(); lo = std::min(A.lo * n, A.lo); hi = std::max(A.hi * n, A.hi); break; }
      case M_SQRT: lo = std::sqrt(std::max(A.lo, 0.f)); hi = A.hi >= 0.f ? std::sqrt(A.hi) : 0.f; break;
      case M_RCP: if (A.lo > 0.f || A.hi < 0.f) { lo = 1.f / A.hi; hi = 1.f / A.lo; } break;
      default: break;
    }
    if (lo != lo || hi != hi) { lo = -inf; hi = inf; }
    vals[dst].lo = lo - std::fabs(lo) * 1e-6f;
    vals[dst].hi = hi + std::fabs(hi) * 1e-6f;
  }

  int mop(int opc, int a, int b = -1) {
    Shape s = vals[a].shape;
    if (b >= 0 && !broadcast_shapes(vals[a].shape, vals[b].shape, &s)) {
      set_error("internal: operands of a micro-operation do not broadcast");
      err = DRAGON_ERR_SHAPE;
      return a;
    }
    if (opc == M_MUL) {  // the seed of a gradient stage is one: dy * v folds to v
      if (is_const(a, 1.f)) return widen(b, s);
      if (is_const(b, 1.f)) return widen(a, s);
    }
    if (opc == M_NEG && vals[a].known_const) return widen(konst(-vals[a].c), s);
    if (opc == M_MUL && (vals[a].known_const != vals[b].known_const)) {
      // (x * c1) * c2 = x * (c1 * c2): a mean of a row-uniform value, a scaled sum of one
      const int x = vals[a].known_const ? b : a, c = vals[a].known_const ? a : b;
      const Item* d = def_of(x);
      if (d && d->opc == M_MUL && (vals[d->a].known_const != vals[d->b].known_const)) {
        const int dx = vals[d->a].known_const ? d->b : d->a, dc = vals[d->a].known_const ? d->a : d->b;
        return mop(M_MUL, widen(dx, vals[x].shape), konst(vals[dc].c * vals[c].c));
      }
    }
    // the sum over a row whose elements are all equal is that element times the row length: no reduction
    // (Sum of a Sum, Mean of a Mean, the gradient of a Mean that reaches it as one value per row)
    if (opc == M_ROWSUM && vals[a].row_uniform) return mop(M_MUL, a, konst((float)vals[a].shape.cols()));
    if (is_binary(opc) && vals[a].known_const && vals[b].known_const) {
      float x = vals[a].c, y = vals[b].c;
      float r = opc == M_ADD ? x + y : opc == M_SUB ? x - y : opc == M_MUL ? x * y : x / (1.f + std::fabs(y));
      return widen(konst(r), s);
    }
    // clamps that cannot act are left out: tanh keeps its argument inside [-10, 10] and its result inside [-1, 1]
    // (the rational fit stays below 1 well beyond |x| = 4), sigmoid and exp keep the exponential in range
    const float mag = std::max(std::fabs(vals[a].lo), std::fabs(vals[a].hi));
    if (opc == M_TANH && mag <= 4.01f) opc = M_TANHB;
    if (opc == M_SIGMOID && mag <= 80.f) opc = M_SIGMOIDB;
    if (opc == M_EXPC && mag <= 9.99f) opc = M_EXPCB;
    Item it; it.kind = IT_MOP; it.opc = opc; it.a = a; it.b = b;
    it.dst = new_val(VK_OP, s);
    set_range(it.dst, opc, vals[a], b >= 0 ? &vals[b] : nullptr);
    vals[it.dst].row_uniform = opc == M_ROWSUM || (vals[a].row_uniform && (b < 0 || vals[b].row_uniform));
    def_item[it.dst] = (int)items.size();
    items.push_back(it);
    return it.dst;
  }
  void store(int v, int mem) {
    Item it; it.kind = IT_MOP; it.opc = M_STORE; it.a = v; it.mem = mem;
    items.push_back(it);
  }
  void accum(int v, int mem) {
    Item it; it.kind = IT_MOP; it.opc = M_ACCUM; it.a = v; it.mem = mem;
    items.push_back(it);
  }
  // memory image of value v with the given dtype (dtype < 0: any float type)
  int materialise(int v, int dtype, int dtype_if_new) {
    const Value& val = vals[v];
    if (val.kind == VK_MEM && (dtype < 0 || plan->mems[val.mem].dtype == dtype)) return val.mem;
    const int want = dtype < 0 ? dtype_if_new : dtype;
    auto key = std::make_pair(v, want);
    auto it = materialised.find(key);
    if (it != materialised.end()) return it->second;   // one image per value and type
    int m = new_mem(MEM_WORK, -1, want, val.shape);
    store(v, m);
    materialised[key] = m;
    return m;
  }
  // C = opA * opB^T; tA / tB: the memory matrix of the operand is its transpose ([K, M] / [K, N])
  int gemm(int mA, int mB, int out_where, int out_index, int out_dtype, bool tA = false, bool tB = false) {
    Shape s; s.rank = 2; s.d[0] = plan->mems[mA].shape.d[tA ? 1 : 0]; s.d[1] = plan->mems[mB].shape.d[tB ? 1 : 0];
    int mC = new_mem(out_where, out_index, out_dtype, s);
    Item x; x.kind = IT_GEMM; x.mA = mA; x.mB = mB; x.mC = mC; x.tA = tA; x.tB = tB;
    items.push_back(x);
    return mC;
  }

  void accumulate_grad(int s, int x, int contrib) {
    auto it = gval[s].find(x);
    if (it == gval[s].end()) gval[s][x] = contrib;
    else it->second = mop(M_ADD, it->second, contrib);
  }

  void store_fetch(int v, int tensor) {
    const TensorInfo& t = g.tensors[tensor];
    int m = new_mem(MEM_FETCH, fetch_of[tensor], t.dtype, t.shape);
    if (vals[v].shape == t.shape) store(v, m);
    else accum(v, m);
  }

  void lower_forward(int k) {
    const OpInfo& op = g.ops[k];
    const int o = op.out[0];
    const TensorInfo& to = g.tensors[o];
    auto in = [&](int p) { return fval[op.in[p]]; };
    int v = -1;
    switch (op.type) {
      case DRAGON_OP_ADD: v = mop(M_ADD, in(0), in(1)); break;
      case DRAGON_OP_SUB: v = mop(M_SUB, in(0), in(1)); break;
      case DRAGON_OP_MUL: v = mop(M_MUL, in(0), in(1)); break;
      case DRAGON_OP_DIV: v = mop(M_DIVP, in(0), in(1)); break;
      case DRAGON_OP_SIN: v = mop(M_SIN, in(0)); break;
      case DRAGON_OP_EXP: v = mop(M_EXPC, in(0)); break;
      case DRAGON_OP_TANH: v = mop(M_TANH, in(0)); break;
      case DRAGON_OP_SIGMOID: v = mop(M_SIGMOID, in(0)); break;
      case DRAGON_OP_RELU: v = mop(M_RELU, in(0)); break;
      case DRAGON_OP_SQRT: v = mop(M_SQRT, in(0)); break;
      case DRAGON_OP_RECIPROCAL: v = mop(M_RCP, in(0)); break;
      case DRAGON_OP_SUM: v = mop(M_ROWSUM, in(0)); break;
      case DRAGON_OP_MEAN: v = mop(M_MUL, mop(M_ROWSUM, in(0)), konst(1.f / (float)to.shape.cols())); break;
      case DRAGON_OP_BIAS_ADD: v = mop(M_ADD, in(0), in(1)); break;
      case DRAGON_OP_INNER_PRODUCT: {
        int mA = materialise(in(0), DRAGON_BF16, DRAGON_BF16);
        int mB = materialise(in(1), DRAGON_BF16, DRAGON_BF16);
        bool direct = fetch_of[o] >= 0;
        int mC = gemm(mA, mB, direct ? MEM_FETCH : MEM_WORK, direct ? fetch_of[o] : -1, to.dtype);
        fval[o] = new_val(VK_MEM, to.shape, mC);
        return;
      }
      case DRAGON_OP_SOFTMAX_CROSS_ENTROPY: {
        int mZ = materialise(in(0), -1, g.tensors[op.in[0]].dtype);
        int mL = vals[in(1)].mem;
        bool direct = fetch_of[o] >= 0;
        int mC = new_mem(direct ? MEM_FETCH : MEM_WORK, direct ? fetch_of[o] : -1, DRAGON_F32, Shape());
        Item x; x.kind = IT_SCE_FWD; x.mA = mZ; x.mB = mL; x.mC = mC;
        items.push_back(x);
        fval[o] = new_val(VK_MEM, to.shape, mC);
        return;
      }
      default:
        set_error("operator type %d cannot be lowered", op.type);
        err = DRAGON_ERR_UNSUPPORTED;
        return;
    }
    if (to.dtype == DRAGON_BF16) v = mop(M_RBF16, v);
    fval[o] = v;
    if (fetch_of[o] >= 0) store_fetch(v, o);
  }

  void lower_gradient(const GradOpRef& r) {
    const OpInfo& op = g.ops[r.op];
    const int s = r.stage, o = op.out[0];
    auto gy = gval[s].find(o);
    if (gy == gval[s].end()) return;  // no gradient reaches this operator
    // a gradient value stands for a tensor of at least the output's shape (a folded seed or a
    // scalar factor is narrower); sums over broadcast axes count every element of that shape
    const int dy = widen(gy->second, g.tensors[o].shape);
    std::vector<bool> want(op.in.size(), false);
    for (size_t p = 0; p < op.in.size(); ++p)
      for (size_t q = 0; q < op.in.size(); ++q)
        if (((r.mask >> q) & 1u) && op.in[q] == op.in[p]) want[p] = true;
    auto in = [&](int p) { return fval[op.in[p]]; };
    auto add = [&](int p, int c) { accumulate_grad(s, op.in[p], c); };
    switch (op.type) {
      case DRAGON_OP_ADD: case DRAGON_OP_BIAS_ADD:
        if (want[0]) add(0, dy);
        if (want[1]) add(1, dy);
        break;
      case DRAGON_OP_SUB:
        if (want[0]) add(0, dy);
        if (want[1]) add(1, mop(M_NEG, dy));
        break;
      case DRAGON_OP_MUL:
        if (want[0]) add(0, mop(M_MUL, dy, in(1)));
        if (want[1]) add(1, mop(M_MUL, dy, in(0)));
        break;
      case DRAGON_OP_DIV:
        if (want[0]) add(0, mop(M_DIVP, dy, in(1)));
        if (want[1]) add(1, mop(M_MUL, mop(M_MUL, dy, in(0)), mop(M_DIVPGB, in(1))));
        break;
      case DRAGON_OP_SIN: add(0, mop(M_MUL, dy, mop(M_COS, in(0)))); break;
      case DRAGON_OP_EXP: add(0, mop(M_MUL, mop(M_MUL, dy, fval[o]), mop(M_CLAMPMASK, in(0)))); break;
      case DRAGON_OP_TANH: add(0, mop(M_MUL, dy, mop(M_ONEMSQ, fval[o]))); break;
      case DRAGON_OP_SIGMOID: add(0, mop(M_MUL, dy, mop(M_YOMY, fval[o]))); break;
      // [x > 0] = [relu(x) > 0]: reading the output keeps the input out of memory
      case DRAGON_OP_RELU: add(0, mop(M_MUL, dy, mop(M_STEP, fval[o]))); break;
      case DRAGON_OP_SQRT: add(0, mop(M_MUL, dy, mop(M_MUL, konst(0.5f), mop(M_RCP, fval[o])))); break;      // dy / (2 y)
      case DRAGON_OP_RECIPROCAL: add(0, mop(M_NEG, mop(M_MUL, dy, mop(M_MUL, fval[o], fval[o])))); break;     // -dy y^2
      case DRAGON_OP_SUM: case DRAGON_OP_MEAN: {
        int c = mop(M_ROWSUM, dy);
        if (op.type == DRAGON_OP_MEAN) c = mop(M_MUL, c, konst(1.f / (float)g.tensors[o].shape.cols()));
        add(0, c);
        break;
      }
      case DRAGON_OP_INNER_PRODUCT: {
        int mdY = materialise(dy, DRAGON_BF16, DRAGON_BF16);
        if (want[0]) {  // dX[M,K] = dY[M,N] * W[N,K]
          int mW = materialise(in(1), DRAGON_BF16, DRAGON_BF16);
          // the gradient of a bf16 activation is kept in bf16 (it feeds the next contraction);
          // a gradient that the caller asked for stays fp32
          const auto& wr = g.stages[s].wrts;
          const bool wanted = std::find(wr.begin(), wr.end(), op.in[0]) != wr.end();
          int mC = gemm(mdY, mW, MEM_WORK, -1,
                        (g.tensors[op.in[0]].dtype == DRAGON_BF16 && !wanted) ? DRAGON_BF16 : DRAGON_F32, false, true);
          add(0, new_val(VK_MEM, plan->mems[mC].shape, mC));
        }
        if (want[1]) {  // dW[N,K] = dY^T[N,M] * X[M,K]
          int mX = materialise(in(0), DRAGON_BF16, DRAGON_BF16);
          int mC = gemm(mdY, mX, MEM_WORK, -1, DRAGON_F32, true, true);
          add(1, new_val(VK_MEM, plan->mems[mC].shape, mC));
        }
        break;
      }
      case DRAGON_OP_SOFTMAX_CROSS_ENTROPY: {
        const TensorInfo& tz = g.tensors[op.in[0]];
        int mZ = materialise(in(0), -1, tz.dtype);
        int mdZ = new_mem(MEM_WORK, -1, tz.dtype, tz.shape);
        Item x; x.kind = IT_SCE_BWD; x.mA = mZ; x.mB = vals[in(1)].mem; x.mC = mdZ;
        if (vals[dy].known_const) x.scale = vals[dy].c;
        else x.mD = materialise(dy, DRAGON_F32, DRAGON_F32);
        items.push_back(x);
        add(0, new_val(VK_MEM, tz.shape, mdZ));
        break;
      }
      default:
        set_error("gradient of operator type %d cannot be lowered", op.type);
        err = DRAGON_ERR_UNSUPPORTED;
    }
  }
};

// true when a value/memory shape fits the fused domain `dom` (may widen it)
bool join_domain(Shape* dom, bool* has_dom, const Shape& s) {
  if (!*has_dom) { *dom = s; *has_dom = true; return true; }
  Shape out;
  if (!broadcast_shapes(*dom, s, &out)) return false;
  *dom = out;
  return true;
}

}  // namespace

static size_t share_workspace(Plan* plan, size_t off);

// per operand of a VM program: position (index into the code) of its last load and of its first store
std::vector<VmAccess> vm_operand_accesses(const VmSegment& sg) {
  std::vector<VmAccess> acc(sg.operand_mem.size());
  for (int i = 0; i < (int)sg.code.size(); ++i) {
    const uint32_t cs = sg.code[i] & 1023u, arg = sg.code[i] >> 14;
    if (cs == (uint32_t)vm::P_UCONST) { ++i; continue; }
    int opd = -1; bool store = false;
    const uint32_t jg = cs / vm::kJointStride;
    if (cs == (uint32_t)vm::P_GST || cs == (uint32_t)vm::P_GSTF || cs == (uint32_t)vm::P_GSTFL) { opd = (int)arg; store = true; }
    else if (cs < (uint32_t)vm::kFirstPlain && jg == (uint32_t)vm::J_FMAURSTL) { opd = (int)(arg >> 9); store = true; }
    else if (cs == (uint32_t)vm::P_GLD || cs == (uint32_t)vm::P_GLDF || (cs < (uint32_t)vm::kFirstPlain && jg == (uint32_t)vm::J_GLDR)) opd = (int)arg;
    else if (cs == (uint32_t)vm::P_GLDA0 || cs == (uint32_t)vm::P_GLDA || cs == (uint32_t)vm::P_LDSW || cs == (uint32_t)vm::P_LDSWA ||
             cs == (uint32_t)vm::P_GLDA0H || cs == (uint32_t)vm::P_LDSWAH ||
             (cs < (uint32_t)vm::kFirstPlain && (jg == (uint32_t)vm::J_LDSWR || jg == (uint32_t)vm::J_LDSWAR || jg == (uint32_t)vm::J_LDSWARF))) opd = (int)(arg & 63u);
    else if (cs == (uint32_t)vm::P_ULOAD) opd = (int)(arg >> 9);
    if (opd < 0 || opd >= (int)acc.size()) continue;
    if (store) acc[opd].first_store = std::min(acc[opd].first_store, i);
    else acc[opd].last_load = i;
  }
  return acc;
}

static int lower_with_cuts(const Graph& g, const PruneResult& pr, const std::vector<int>& inputs, const std::vector<int>& outputs,
                           int sm_count, Plan* plan, const std::set<int>& cuts, int* cut_here);

// A fused segment that exceeds what one VM program can hold (memory operands, stream length, uniforms,
// reduced outputs) is cut in two at its middle micro-operation and everything is lowered again; values that
// cross the new boundary become workspace tensors like any others.
int lower_function(const Graph& g, const PruneResult& pr, const std::vector<int>& inputs,
                   const std::vector<int>& outputs, int sm_count, Plan* plan) {
  std::set<int> cuts;
  for (int round = 0; round < 64; ++round) {
    Plan trial;
    int cut_here = -1;
    const int rc = lower_with_cuts(g, pr, inputs, outputs, sm_count, &trial, cuts, &cut_here);
    if (rc != kVmErrTooLarge) {
      if (rc == DRAGON_OK) *plan = std::move(trial);
      return rc;
    }
    if (cut_here < 0 || !cuts.insert(cut_here).second) break;
  }
  return DRAGON_ERR_UNSUPPORTED;   // the message of the last attempt stands
}

static int lower_with_cuts(const Graph& g, const PruneResult& pr, const std::vector<int>& inputs, const std::vector<int>& outputs,
                           int sm_count, Plan* plan, const std::set<int>& cuts, int* cut_here) {
  Lowerer L(g, pr, plan);
  plan->sm_count = sm_count;
  const int n = (int)g.tensors.size();
  L.fval.assign(n, -1);
  L.fetch_of.assign(n, -1);
  L.gval.resize(g.stages.size());
  for (int j = 0; j < (int)outputs.size(); ++j) {
    if (L.fetch_of[outputs[j]] >= 0) {
      set_error("tensor '%s' is fetched twice", g.tensors[outputs[j]].name.c_str());
      return DRAGON_ERR_INVALID_ARG;
    }
    L.fetch_of[outputs[j]] = j;
  }
  for (int j = 0; j < (int)inputs.size(); ++j) {
    const TensorInfo& t = g.tensors[inputs[j]];
    if (!pr.marked[inputs[j]]) continue;
    int m = L.new_mem(MEM_FEED, j, t.dtype, t.shape);
    L.fval[inputs[j]] = L.new_val(VK_MEM, t.shape, m);
    if (L.fetch_of[inputs[j]] >= 0) {  // a fetched input is copied
      int mo = L.new_mem(MEM_FETCH, L.fetch_of[inputs[j]], t.dtype, t.shape);
      Item x; x.kind = IT_COPY; x.mA = m; x.mC = mo;
      L.items.push_back(x);
    }
  }
  for (int k : pr.fwd_ops) {
    L.lower_forward(k);
    if (L.err) return L.err;
  }
  auto seed_stage = [&](int s) {  // one for every element of every objective of a live stage
    auto& gv = L.gval[s];
    if (gv.empty())
      for (int o : g.stages[s].objs)
        if (pr.in_G[s][o]) gv[o] = L.konst(1.f);
  };
  // a fetched gradient is written as soon as its last contribution is in (it then joins the
  // segment that produced it instead of a trailing one that would re-read everything)
  auto produced = [&](const GradOpRef& r) {
    std::vector<int> t;
    const OpInfo& op = g.ops[r.op];
    for (size_t p = 0; p < op.in.size(); ++p)
      if ((r.mask >> p) & 1u) t.push_back(op.in[p]);
    return t;
  };
  L.pending.resize(g.stages.size());
  for (const GradOpRef& r : pr.grad_ops)
    for (int t : produced(r)) ++L.pending[r.stage][t];
  std::vector<std::vector<uint8_t>> fetched_early(g.stages.size(), std::vector<uint8_t>(n, 0));
  for (const GradOpRef& r : pr.grad_ops) {
    seed_stage(r.stage);
    L.lower_gradient(r);
    if (L.err) return L.err;
    for (int t : produced(r)) {
      if (--L.pending[r.stage][t] != 0) continue;
      const GradStage& st = g.stages[r.stage];
      for (size_t j = 0; j < st.wrts.size(); ++j)
        if (st.wrts[j] == t && L.fetch_of[st.grad_ids[j]] >= 0 && !fetched_early[r.stage][t]) {
          auto it = L.gval[r.stage].find(t);
          if (it == L.gval[r.stage].end()) continue;
          L.store_fetch(L.widen(it->second, g.tensors[t].shape), st.grad_ids[j]);
          fetched_early[r.stage][t] = 1;
        }
    }
  }
  for (int s = 0; s < (int)g.stages.size(); ++s) {
    const GradStage& st = g.stages[s];
    for (size_t j = 0; j < st.wrts.size(); ++j) {
      int gid = st.grad_ids[j];
      if (L.fetch_of[gid] < 0 || fetched_early[s][st.wrts[j]]) continue;
      seed_stage(s);
      auto it = L.gval[s].find(st.wrts[j]);
      int v = it == L.gval[s].end() ? L.konst(0.f) : it->second;
      L.store_fetch(L.widen(v, g.tensors[st.wrts[j]].shape), gid);
    }
  }
  if (L.err) return L.err;

  std::vector<Item>& items = L.items;
  std::vector<Value>& vals = L.vals;
  std::vector<MemRef>& mems = plan->mems;
  const int n_lowered = (int)items.size();     // items appended later (stores of crossing values) have indices beyond

  // A workspace image that is written once and then only copied to a fetch buffer by a plain
  // full-shape store is written to the fetch buffer directly (gradient tensors produced by a
  // contraction, fetched logits...).
  for (size_t i = 0; i < items.size(); ++i) {
    Item& st = items[i];
    if (st.kind != IT_MOP || st.opc != M_STORE || vals[st.a].kind != VK_MEM) continue;
    int src = vals[st.a].mem, dst = st.mem;
    if (mems[src].where != MEM_WORK || mems[dst].where != MEM_FETCH) continue;
    if (mems[src].dtype != mems[dst].dtype || mems[src].shape != mems[dst].shape) continue;
    int writers = 0;
    for (const Item& w : items)
      if ((w.kind != IT_MOP && w.mC == src) || (w.kind == IT_MOP && (w.opc == M_STORE || w.opc == M_ACCUM) && w.mem == src)) ++writers;
    if (writers != 1) continue;
    mems[src].where = MEM_FETCH;
    mems[src].index = mems[dst].index;
    st.opc = -1;  // removed
  }
  items.erase(std::remove_if(items.begin(), items.end(), [](const Item& x) { return x.kind == IT_MOP && x.opc < 0; }), items.end());

  // dead-code elimination, roots = everything that reaches a fetch buffer
  std::vector<uint8_t> val_live(vals.size(), 0);
  for (auto& m : mems) m.live = m.where == MEM_FETCH;
  auto use_val = [&](int v) {
    if (v < 0) return;
    val_live[v] = 1;
    if (vals[v].kind == VK_MEM) mems[vals[v].mem].live = true;
  };
  for (int i = (int)items.size() - 1; i >= 0; --i) {
    Item& it = items[i];
    if (it.kind == IT_MOP) {
      if (it.opc == M_STORE || it.opc == M_ACCUM) it.live = mems[it.mem].live;
      else it.live = val_live[it.dst] != 0;
      if (it.live) { use_val(it.a); use_val(it.b); }
    } else {
      it.live = mems[it.mC].live;
      if (it.live)
        for (int m : {it.mA, it.mB, it.mD, it.mE})
          if (m >= 0) mems[m].live = true;
      // (mF is set by a later pass, from an accumulation that is live itself)
    }
  }

  // segmentation: maximal runs of live micro-operations whose shapes share one domain
  std::vector<std::vector<int>> seg_items;
  {
    Shape dom; bool has_dom = false; int cur = -1;
    for (int i = 0; i < (int)items.size(); ++i) {
      Item& it = items[i];
      if (!it.live) continue;
      if (it.kind != IT_MOP) { cur = -1; has_dom = false; continue; }
      Shape s = (it.opc == M_STORE || it.opc == M_ACCUM) ? vals[it.a].shape : vals[it.dst].shape;
      if (cur < 0 || cuts.count(i) || !join_domain(&dom, &has_dom, s)) {
        seg_items.emplace_back();
        cur = (int)seg_items.size() - 1;
        has_dom = false;
        join_domain(&dom, &has_dom, s);
      }
      it.segment = cur;
      seg_items[cur].push_back(i);
    }
  }
  // values that cross a segment boundary become workspace tensors
  {
    std::vector<int> def_seg(vals.size(), -1), def_item(vals.size(), -1);
    for (int i = 0; i < (int)items.size(); ++i)
      if (items[i].live && items[i].kind == IT_MOP && items[i].dst >= 0) { def_seg[items[i].dst] = items[i].segment; def_item[items[i].dst] = i; }
    std::map<int, int> spilled;  // value -> VK_MEM value
    const int n_items = (int)items.size();
    for (int i = 0; i < n_items; ++i) {
      if (!items[i].live || items[i].kind != IT_MOP) continue;
      for (int which = 0; which < 2; ++which) {
        int v = which == 0 ? items[i].a : items[i].b;
        if (v < 0 || vals[v].kind != VK_OP || def_seg[v] == items[i].segment) continue;
        auto f = spilled.find(v);
        if (f == spilled.end()) {
          int dt = items[def_item[v]].opc == M_RBF16 ? DRAGON_BF16 : DRAGON_F32;
          // an image of this value that its own segment already writes serves as well
          auto have = L.materialised.find(std::make_pair(v, dt));
          if (have != L.materialised.end() && mems[have->second].live) {
            bool same_seg = false;
            for (int j = 0; j < n_items; ++j)
              if (items[j].live && items[j].kind == IT_MOP && items[j].opc == M_STORE && items[j].mem == have->second && items[j].a == v)
                same_seg = items[j].segment == def_seg[v];
            if (same_seg) {
              Value nv; nv.kind = VK_MEM; nv.shape = vals[v].shape; nv.mem = have->second;
              vals.push_back(nv);
              f = spilled.emplace(v, (int)vals.size() - 1).first;
            }
          }
        }
        if (f == spilled.end()) {
          int dt = items[def_item[v]].opc == M_RBF16 ? DRAGON_BF16 : DRAGON_F32;
          MemRef m; m.where = MEM_WORK; m.dtype = dt; m.shape = vals[v].shape; m.live = true;
          mems.push_back(m);
          int mid = (int)mems.size() - 1;
          Item st; st.kind = IT_MOP; st.opc = M_STORE; st.a = v; st.mem = mid; st.live = true; st.segment = def_seg[v];
          items.push_back(st);
          auto& lst = seg_items[def_seg[v]];  // right after the definition, while the value is at hand
          lst.insert(std::find(lst.begin(), lst.end(), def_item[v]) + 1, (int)items.size() - 1);
          Value nv; nv.kind = VK_MEM; nv.shape = vals[v].shape; nv.mem = mid;
          vals.push_back(nv);
          f = spilled.emplace(v, (int)vals.size() - 1).first;
        }
        if (which == 0) items[i].a = f->second; else items[i].b = f->second;
      }
    }
  }

  // a segment runs where its first item stands (items appended later for values that cross
  // segments belong to the segment of the value's definition)
  auto runs_at = [&](int i) {
    const Item& it = items[i];
    if (it.kind != IT_MOP || it.segment < 0 || seg_items[it.segment].empty()) return i;
    return *std::min_element(seg_items[it.segment].begin(), seg_items[it.segment].end());
  };
  // position of the last live item that writes memory m (-1: a feed, or never written)
  auto last_writer = [&](int m) {
    int w = -1;
    for (int i = 0; i < (int)items.size(); ++i) {
      const Item& it = items[i];
      if (!it.live) continue;
      if (it.kind != IT_MOP) { if (it.mC == m || (it.kind == IT_SCE_FWD && it.mD == m)) w = std::max(w, i); }
      else if ((it.opc == M_STORE || it.opc == M_ACCUM) && it.mem == m) w = std::max(w, runs_at(i));
    }
    return w;
  };
  // A segment that only adds a row vector to the product of an InnerProduct, optionally clamps
  // it at zero and rounds it, and stores the result, runs in the epilogue of that product: the
  // fp32 product then never reaches memory.
  for (size_t s = 0; s < seg_items.size(); ++s) {
    std::vector<int> body;
    for (int i : seg_items[s])
      if (items[i].live && items[i].opc != M_WIDEN) body.push_back(i);
    if (body.size() < 2 || body.size() > 4) continue;
    auto root = [&](int v) {   // through the widenings to the value they show
      for (bool again = true; again && v >= 0 && vals[v].kind == VK_OP;) {
        again = false;
        for (int i : seg_items[s])
          if (items[i].opc == M_WIDEN && items[i].dst == v) { v = items[i].a; again = true; break; }
      }
      return v;
    };
    const Item& add = items[body[0]];
    const Item& st = items[body.back()];
    if (add.opc != M_ADD || st.opc != M_STORE) continue;
    int prod = root(add.a), bias = root(add.b);
    if (prod < 0 || bias < 0) continue;
    if (!(vals[prod].kind == VK_MEM && vals[prod].shape.rank == 2)) std::swap(prod, bias);
    if (vals[prod].kind != VK_MEM || vals[bias].kind != VK_MEM || vals[prod].shape.rank != 2) continue;
    const int mP = vals[prod].mem, mBias = vals[bias].mem, mOut = st.mem;
    const Shape& sp = mems[mP].shape;
    const Shape& sb = mems[mBias].shape;
    const bool row_vector = (sb.rank == 1 && sb.d[0] == sp.d[1]) || (sb.rank == 2 && sb.d[0] == 1 && sb.d[1] == sp.d[1]);
    if (mems[mP].where != MEM_WORK || mems[mP].dtype != DRAGON_F32 || !row_vector || !(mems[mOut].shape == sp)) continue;
    if (mems[mBias].dtype != DRAGON_F32 && mems[mBias].dtype != DRAGON_BF16) continue;
    bool relu = false, rounded = false, chain = true;
    int last = add.dst;
    for (size_t k = 1; k + 1 < body.size() && chain; ++k) {
      const Item& u = items[body[k]];
      if (u.a != last) chain = false;
      else if (u.opc == M_RELU && !relu && !rounded) relu = true;
      else if (u.opc == M_RBF16 && !rounded) rounded = true;
      else chain = false;
      last = u.dst;
    }
    if (!chain || st.a != last) continue;
    if (rounded != (mems[mOut].dtype == DRAGON_BF16) || (!rounded && mems[mOut].dtype != DRAGON_F32)) continue;
    int producer = -1, readers = 0;
    for (int i = 0; i < (int)items.size(); ++i) {
      const Item& it = items[i];
      if (!it.live) continue;
      if (it.kind == IT_GEMM && it.mC == mP) producer = i;
      if (it.kind != IT_MOP) { readers += (it.mA == mP) + (it.mB == mP) + (it.mD == mP); continue; }
      if (it.opc == M_WIDEN) continue;
      for (int v : {it.a, it.b})
        if (v >= 0 && root(v) >= 0 && vals[root(v)].kind == VK_MEM && vals[root(v)].mem == mP) ++readers;
    }
    if (producer < 0 || producer > runs_at(body[0]) || readers != 1 || items[producer].mD >= 0 || last_writer(mBias) > producer) continue;
    items[producer].mC = mOut;
    items[producer].mD = mBias;
    items[producer].relu = relu;
    mems[mBias].live = true;
    mems[mP].live = false;
    for (int i : seg_items[s]) items[i].live = false;
    seg_items[s].clear();
  }

  // The general form of the above (a chain of elementwise operators behind an InnerProduct, Sec. 3.3's
  // operator-at-a-time execution being what is avoided): a segment whose only tensor of the product's shape
  // that it computes on is the product itself, each operation taking the running value and at most a
  // constant, a scalar, a row vector or one more tensor of that shape, ending in one store, becomes the
  // product's epilogue program; the arithmetic is that of the VM's leaves (vm_math.h) in the same order.
  for (size_t s = 0; s < seg_items.size(); ++s) {
    std::vector<int> body;
    for (int i : seg_items[s])
      if (items[i].live && items[i].opc != M_WIDEN) body.push_back(i);
    if (body.size() < 2 || (int)body.size() > kMaxEpiOps + 1) continue;
    auto root = [&](int v) {
      for (bool again = true; again && v >= 0 && vals[v].kind == VK_OP;) {
        again = false;
        for (int i : seg_items[s])
          if (items[i].opc == M_WIDEN && items[i].dst == v) { v = items[i].a; again = true; break; }
      }
      return v;
    };
    const Item& st = items[body.back()];
    if (st.opc != M_STORE) continue;
    // the product: the first operation's operand that is a rank-2 f32 workspace tensor written by a live contraction
    const Item& first = items[body[0]];
    int prod = -1;
    for (int v : {root(first.a), first.b >= 0 ? root(first.b) : -1})
      if (v >= 0 && vals[v].kind == VK_MEM && mems[vals[v].mem].where == MEM_WORK && mems[vals[v].mem].dtype == DRAGON_F32 &&
          mems[vals[v].mem].shape.rank == 2 && prod < 0) {
        for (const Item& it : items)
          if (it.live && it.kind == IT_GEMM && it.mC == vals[v].mem) prod = v;
      }
    if (prod < 0) continue;
    const int mP = vals[prod].mem, mOut = st.mem;
    const Shape sp = mems[mP].shape;
    if (!(mems[mOut].shape == sp)) continue;
    int producer = -1, readers = 0;
    for (int i = 0; i < (int)items.size(); ++i) {
      const Item& it = items[i];
      if (!it.live) continue;
      if (it.kind == IT_GEMM && it.mC == mP) producer = i;
      if (it.kind != IT_MOP) { readers += (it.mA == mP) + (it.mB == mP) + (it.mD == mP) + (it.mE == mP); continue; }
      if (it.opc == M_WIDEN) continue;
      for (int v : {it.a, it.b})
        if (v >= 0 && root(v) >= 0 && vals[root(v)].kind == VK_MEM && vals[root(v)].mem == mP) ++readers;
    }
    if (producer < 0 || producer > runs_at(body[0]) || readers != 1 || items[producer].mD >= 0 || items[producer].mE >= 0 ||
        !items[producer].epi.empty() || items[producer].relu) continue;
    std::vector<EpiSpec> prog;
    int cur = prod;
    bool ok = true, rounded = false;
    for (size_t k = 0; k + 1 < body.size() && ok; ++k) {
      const Item& u = items[body[k]];
      const int ua = root(u.a), ub = u.b >= 0 ? root(u.b) : -1;
      EpiSpec e;
      if (rounded) { ok = false; break; }                      // the rounding to bf16 is the last operation
      if (u.b < 0) {
        if (ua != cur) { ok = false; break; }
        switch (u.opc) {
          case M_RELU: e.opc = E_RELU; break;
          case M_TANH: case M_TANHB: e.opc = E_TANH; break;          // the epilogue keeps the clamped forms
          case M_SIGMOID: case M_SIGMOIDB: e.opc = E_SIGMOID; break;
          case M_EXPC: case M_EXPCB: e.opc = E_EXPC; break;
          case M_SIN: e.opc = E_SIN; break;
          case M_NEG: e.opc = E_NEG; break;
          case M_SQRT: e.opc = E_SQRT; break;
          case M_RCP: e.opc = E_RCP; break;
          case M_RBF16: e.opc = E_RBF16; rounded = true; break;
          default: ok = false;
        }
      } else {
        if ((ua == cur) == (ub == cur)) { ok = false; break; }  // the running value exactly once
        const bool value_first = ua == cur;
        const int o = value_first ? ub : ua;
        switch (u.opc) {
          case M_ADD: e.opc = E_ADD; break;
          case M_MUL: e.opc = E_MUL; break;
          case M_SUB: e.opc = value_first ? E_SUB : E_RSUB; break;
          default: ok = false;
        }
        if (!ok) break;
        const Value& ov = vals[o];
        if (ov.known_const) { e.operand = EO_CONST; e.c = ov.c; }
        else if (ov.kind != VK_MEM) ok = false;
        else {
          const MemRef& om = mems[ov.mem];
          const bool row_vector = (om.shape.rank == 1 && om.shape.d[0] == sp.d[1]) || (om.shape.rank == 2 && om.shape.d[0] == 1 && om.shape.d[1] == sp.d[1]);
          if (om.dtype != DRAGON_F32 && om.dtype != DRAGON_BF16) ok = false;
          else if (om.shape.numel() == 1) e.operand = EO_SCALAR;
          else if (row_vector) e.operand = EO_ROW;
          else if (om.shape == sp && ov.mem != mP) e.operand = EO_FULL;
          else ok = false;
          e.mem = ov.mem;
          if (ok && last_writer(ov.mem) > producer) ok = false;   // it must be in memory before the product runs
        }
      }
      if (!ok) break;
      // nothing else may read an intermediate value of the chain
      int uses = 0;
      for (const Item& it : items)
        if (it.live && it.kind == IT_MOP && it.opc != M_WIDEN)
          uses += (it.a >= 0 && root(it.a) == u.dst) + (it.b >= 0 && root(it.b) == u.dst);
      if (uses != 1) { ok = false; break; }
      prog.push_back(e);
      cur = u.dst;
    }
    if (!ok || root(st.a) != cur || prog.empty()) continue;
    if (rounded != (mems[mOut].dtype == DRAGON_BF16) || (!rounded && mems[mOut].dtype != DRAGON_F32)) continue;
    items[producer].mC = mOut;
    items[producer].epi = prog;
    for (const EpiSpec& e : prog)
      if (e.mem >= 0) mems[e.mem].live = true;
    mems[mP].live = false;
    for (int i : seg_items[s]) items[i].live = false;
    seg_items[s].clear();
  }

  // The backward of ReLU behind a product: a segment that multiplies the product by step(h), h a
  // bf16 tensor of the same shape already in memory, stores that (and perhaps sums it as well),
  // leaves the multiplication to the product's epilogue; what remains of the segment reads the
  // stored result.
  for (size_t s = 0; s < seg_items.size(); ++s) {
    std::vector<int> body;
    for (int i : seg_items[s])
      if (items[i].live && items[i].opc != M_WIDEN) body.push_back(i);
    int i_step = -1, i_mul = -1, i_store = -1, n_accum = 0, n_other = 0;
    for (int i : body) {
      const int opc = items[i].opc;
      if (opc == M_STEP && i_step < 0) i_step = i;
      else if (opc == M_MUL && i_mul < 0) i_mul = i;
      else if (opc == M_STORE && i_store < 0) i_store = i;
      else if (opc == M_ACCUM) ++n_accum;
      else ++n_other;
    }
    if (i_step < 0 || i_mul < 0 || i_store < 0 || n_other) continue;
    const Item& stp = items[i_step];
    const Item& mul = items[i_mul];
    if (vals[stp.a].kind != VK_MEM) continue;
    int prod = mul.a == stp.dst ? mul.b : mul.b == stp.dst ? mul.a : -1;
    if (prod < 0 || vals[prod].kind != VK_MEM) continue;
    const int mH = vals[stp.a].mem, mP = vals[prod].mem, mOut = items[i_store].mem;
    bool uses_ok = items[i_store].a == mul.dst;
    for (int i : body)
      if (items[i].opc == M_ACCUM) uses_ok &= items[i].a == mul.dst;
    if (!uses_ok) continue;
    if (mems[mP].where != MEM_WORK || mems[mP].shape.rank != 2 || !(mems[mH].shape == mems[mP].shape) || !(mems[mOut].shape == mems[mP].shape)) continue;
    if (mems[mH].dtype != DRAGON_BF16 || mems[mP].dtype != mems[mOut].dtype) continue;
    int producer = -1, readers = 0;
    for (int i = 0; i < (int)items.size(); ++i) {
      const Item& it = items[i];
      if (!it.live) continue;
      if (it.kind == IT_GEMM && it.mC == mP) producer = i;
      if (it.kind != IT_MOP) {
        readers += (it.mA == mP) + (it.mB == mP) + (it.mD == mP) + (it.mE == mP);
        continue;
      }
      if (it.opc == M_WIDEN) continue;
      for (int v : {it.a, it.b})
        if (v >= 0 && vals[v].kind == VK_MEM && vals[v].mem == mP) ++readers;
    }
    if (producer < 0 || producer > runs_at(body[0]) || readers != 1 || items[producer].mE >= 0 || last_writer(mH) > producer) continue;
    items[producer].mC = mOut;
    items[producer].mE = mH;
    mems[mH].live = true;
    mems[mP].live = false;
    items[i_step].live = items[i_mul].live = items[i_store].live = false;
    Value nv; nv.kind = VK_MEM; nv.shape = mems[mOut].shape; nv.mem = mOut;
    vals.push_back(nv);
    std::vector<int> rest;
    for (int i : seg_items[s]) {
      if (!items[i].live) continue;
      if (items[i].opc == M_ACCUM) { items[i].a = (int)vals.size() - 1; rest.push_back(i); }
    }
    for (int i : seg_items[s])
      if (items[i].live && items[i].opc != M_ACCUM) items[i].live = false;   // widenings of what is gone
    seg_items[s] = rest;
  }

  // A segment that is nothing but the column sums of a tensor that a contraction or the softmax gradient has
  // just written (a bias gradient) leaves the summing to that kernel: its CTAs write partial column sums of
  // the values they hold anyway, and the fixed-order finishing kernel adds them.  The tensor is not read again.
  for (size_t s = 0; s < seg_items.size(); ++s) {
    std::vector<int> body;
    for (int i : seg_items[s])
      if (items[i].live && items[i].opc != M_WIDEN) body.push_back(i);
    if (body.size() != 1 || items[body[0]].opc != M_ACCUM) continue;
    const Item& ac = items[body[0]];
    if (vals[ac.a].kind != VK_MEM) continue;
    const int m = vals[ac.a].mem, mT = ac.mem;
    const Shape& sm = mems[m].shape;
    const Shape& stg = mems[mT].shape;
    if (sm.rank != 2 || !(stg.rank == 1 && stg.d[0] == sm.d[1]) || (mems[mT].dtype != DRAGON_F32 && mems[mT].dtype != DRAGON_BF16)) continue;
    int producer = -1;
    for (int i = 0; i < (int)items.size(); ++i) {
      const Item& it = items[i];
      if (it.live && (it.kind == IT_GEMM || it.kind == IT_SCE_BWD) && it.mC == m) producer = i;
    }
    if (producer < 0 || producer > runs_at(body[0]) || items[producer].mF >= 0) continue;
    if (items[producer].kind == IT_SCE_BWD && (sm.d[1] & 7 || sm.d[1] > 4096 || items[producer].mD >= 0)) continue;   // the in-register row kernel only
    items[producer].mF = mT;
    for (int i : seg_items[s]) items[i].live = false;
    seg_items[s].clear();
  }

  // steps in execution order
  std::vector<int> seg_step(seg_items.size(), -1);
  plan->segs.resize(seg_items.size());
  std::vector<bool> fused_away(items.size(), false);
  for (int i = 0; i < (int)items.size(); ++i) {
    const Item& it = items[i];
    if (!it.live || fused_away[i]) continue;
    if (it.kind == IT_MOP) {
      if (it.segment >= 0 && seg_step[it.segment] < 0) {
        seg_step[it.segment] = (int)plan->steps.size();
        Step st; st.kind = ST_VM; st.seg = it.segment;
        plan->steps.push_back(st);
      }
      continue;
    }
    Step st;
    st.kind = it.kind == IT_GEMM ? ST_GEMM : it.kind == IT_TRANSPOSE ? ST_TRANSPOSE : it.kind == IT_SCE_FWD ? ST_SCE_FWD
              : it.kind == IT_SCE_BWD ? ST_SCE_BWD : ST_COPY;
    st.mA = it.mA; st.mB = it.mB; st.mC = it.mC; st.mD = it.mD; st.mE = it.mE; st.scale = it.scale; st.tA = it.tA; st.tB = it.tB;
    st.relu = it.relu;
    st.epi = it.epi;
    st.mF = it.mF;
    if (it.kind == IT_SCE_FWD) {
      // the gradient with respect to the same logits, scaled by a constant, comes out of the same
      // pass: the step then carries the gradient tensor in mD
      st.mD = -1;
      for (int j = i + 1; j < (int)items.size(); ++j) {
        const Item& b = items[j];
        if (b.live && b.kind == IT_SCE_BWD && b.mA == it.mA && b.mB == it.mB && b.mD < 0) {
          st.mD = b.mC;
          st.scale = b.scale;
          st.mF = b.mF;
          fused_away[j] = true;
          break;
        }
      }
    }
    plan->steps.push_back(st);
  }
  for (size_t s = 0; s < seg_items.size(); ++s) {
    if (seg_items[s].empty()) continue;   // ran in a product's epilogue
    int rc = codegen_segment(items, seg_items[s], vals, mems, sm_count, &plan->segs[s]);
    if (rc == kVmErrTooLarge) {
      // the middle of the segment's own micro-operations (stores that were appended for crossing values sit at
      // the end of the item list and are not cut points)
      std::vector<int> own;
      for (int i : seg_items[s])
        if (i < n_lowered) own.push_back(i);
      std::sort(own.begin(), own.end());
      if (own.size() >= 2) *cut_here = own[own.size() / 2];
    }
    if (rc) return rc;
  }

  // workspace layout: the status word, live workspace tensors, then per-segment scratch
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 255) & ~(size_t)255; return o; };
  plan->status_off = take(256);
  off = share_workspace(plan, off);
  for (auto& sg : plan->segs) {
    sg.spill_off = take((size_t)sg.grid * sg.n_spill * kVmTile * sizeof(float));
    sg.colpart_off = take((size_t)sg.n_colacc * sg.grid * sg.cols * sizeof(float));
    sg.scalpart_off = take((size_t)kHostChunks * sg.n_scalacc * sg.grid * sizeof(double));   // a set per chunk of a chunked host run
  }
  for (auto& st : plan->steps) {
    if (st.kind == ST_SCE_FWD) st.scratch_off = take((size_t)mems[st.mA].shape.d[0] * sizeof(float));
    if (st.mF >= 0) {   // partial column sums: one row per 32 output rows of a contraction, one per CTA of the softmax kernel
      const Shape& sc = mems[st.kind == ST_SCE_FWD ? st.mD : st.mC].shape;
      st.n_colpart = st.kind == ST_GEMM ? (int)((sc.d[0] + 127) / 128) * 4 : (int)std::min<int64_t>(sc.d[0], (int64_t)sm_count * 4);
      st.colpart_off = take((size_t)st.n_colpart * sc.d[1] * sizeof(float));
    }
  }
  plan->workspace_bytes = off;
  return DRAGON_OK;
}

// Memory sharing between the tensors that cross kernels (the purpose of Sec. 2.4, at the granularity of
// plan steps).  Every workspace tensor lives from the first step that touches it to the last one.
//  * In place (the paper's in-place structure): the output of an elementwise VM step takes the region
//    of an input of that step that dies there, when both have the domain's shape and the same element
//    size and the program reads the input for the last time before it first writes the output, so
//    every thread overwrites only what it has already read.
//  * Otherwise a region is handed on once its tensor is dead: regions are taken in step order from
//    the free list (smallest that fits, the remainder stays free), new space only when none fits.
static size_t share_workspace(Plan* plan, size_t off) {
  std::vector<MemRef>& mems = plan->mems;
  const int n_steps = (int)plan->steps.size();
  std::vector<std::vector<int>> reads(n_steps), writes(n_steps);
  auto touch = [&](int si, int m, bool w) {
    if (m < 0 || mems[m].where != MEM_WORK || !mems[m].live) return;
    (w ? writes : reads)[si].push_back(m);
    if (mems[m].first_step < 0) mems[m].first_step = si;
    mems[m].last_step = si;
  };
  // positions of the last load and the first store of every operand of a VM program
  std::vector<std::vector<VmAccess>> acc(n_steps);
  for (int si = 0; si < n_steps; ++si) {
    const Step& st = plan->steps[si];
    if (st.kind != ST_VM) {
      touch(si, st.mA, false); touch(si, st.mB, false);
      if (st.kind == ST_SCE_BWD || st.kind == ST_GEMM) touch(si, st.mD, false);
      if (st.kind == ST_GEMM) touch(si, st.mE, false);
      if (st.kind == ST_GEMM)
        for (const EpiSpec& e : st.epi) touch(si, e.mem, false);
      if (st.kind == ST_SCE_FWD) touch(si, st.mD, true);
      touch(si, st.mC, true);
      touch(si, st.mF, true);
      continue;
    }
    const VmSegment& sg = plan->segs[st.seg];
    acc[si] = vm_operand_accesses(sg);
    for (size_t i = 0; i < sg.operand_mem.size(); ++i) {
      if (acc[si][i].last_load >= 0) touch(si, sg.operand_mem[i], false);
      if (acc[si][i].first_store < (1 << 30)) touch(si, sg.operand_mem[i], true);
    }
    for (const FinishJob& j : sg.finish) touch(si, j.mem, true);
  }
  std::vector<std::pair<size_t, size_t>> free_list;   // (offset, bytes), 256-byte granules
  auto round = [](size_t b) { return (b + 255) & ~(size_t)255; };
  std::vector<char> placed(mems.size(), 0);
  for (int si = 0; si < n_steps; ++si) {
    const Step& st = plan->steps[si];
    // 1. outputs of an elementwise step over inputs that die here
    std::vector<int> taken;    // inputs whose region was handed to an output
    if (st.kind == ST_VM) {
      const VmSegment& sg = plan->segs[st.seg];
      for (size_t o = 0; o < sg.operand_mem.size(); ++o) {
        const int y = sg.operand_mem[o];
        if (mems[y].where != MEM_WORK || !mems[y].live || placed[y] || mems[y].first_step != si) continue;
        if (acc[si][o].first_store >= (1 << 30) || acc[si][o].last_load >= 0 || sg.operand_kind[o] != (uint32_t)vm::K_FULL) continue;
        for (size_t i = 0; i < sg.operand_mem.size(); ++i) {
          const int x = sg.operand_mem[i];
          if (x == y || mems[x].where != MEM_WORK || !placed[x] || mems[x].last_step != si || sg.operand_kind[i] != (uint32_t)vm::K_FULL) continue;
          if (std::find(taken.begin(), taken.end(), x) != taken.end()) continue;
          if (mems[x].bytes() != mems[y].bytes() || mems[x].dtype != mems[y].dtype) continue;
          if (acc[si][i].first_store < (1 << 30) || acc[si][i].last_load < 0 || acc[si][i].last_load > acc[si][o].first_store) continue;
          mems[y].offset = mems[x].offset;
          mems[y].shares_input = 1;
          placed[y] = 1;
          taken.push_back(x);
          break;
        }
      }
    }
    // 2. everything else that starts here
    for (int m : writes[si]) {
      if (placed[m] || mems[m].first_step != si) continue;
      const size_t need = round(mems[m].bytes());
      int best = -1;
      for (int k = 0; k < (int)free_list.size(); ++k)
        if (free_list[k].second >= need && (best < 0 || free_list[k].second < free_list[best].second)) best = k;
      if (best >= 0) {
        mems[m].offset = free_list[best].first;
        free_list[best].first += need;
        free_list[best].second -= need;
        if (free_list[best].second == 0) free_list.erase(free_list.begin() + best);
      } else {
        mems[m].offset = off;
        off += need;
      }
      placed[m] = 1;
    }
    // 3. what dies here is free from the next step on (unless an output took it over)
    for (int pass = 0; pass < 2; ++pass)
      for (int m : (pass ? writes[si] : reads[si])) {
        if (mems[m].last_step != si || !placed[m] || std::find(taken.begin(), taken.end(), m) != taken.end()) continue;
        bool listed = false;
        for (auto& fr : free_list) listed |= fr.first == mems[m].offset;
        if (listed) continue;
        bool inherited = false;   // a region that an in-place output still holds stays taken
        for (size_t k = 0; k < mems.size(); ++k)
          inherited |= (int)k != m && placed[k] && mems[k].where == MEM_WORK && mems[k].live && mems[k].offset == mems[m].offset && mems[k].last_step > si;
        if (!inherited) free_list.emplace_back(mems[m].offset, round(mems[m].bytes()));
      }
  }
  for (auto& m : mems)     // a live workspace tensor that no step touches keeps a region of its own
    if (m.where == MEM_WORK && m.live && m.first_step < 0) { m.offset = off; off += round(m.bytes()); }
  return off;
}

// one mnemonic per instruction word of a segment
static std::string disassemble(const VmSegment& sg) {
  static const char* jn[] = {"ldr", "str", "add", "sub", "rsub", "mul", "divp", "rdivp", "addto", "accum", "fmaur", "rtos", "stor", "spillr", "fillr",
                             "gldr", "sincosr", "cossinr", "macc0", "macc1", "macc2", "macc3", "ldswr", "ldswar",
                             "stld0", "stld1", "stld2", "stld3", "stld4", "stld5", "stld6", "stld7", "ldswarf", "fmaurst}loop", "strlds"};
  static const char* pn[] = {"ldu", "addu", "subu", "rsubu", "mulu", "divpu", "rdivpu", "fmau", "lds", "sts", "adds", "subs", "rsubs", "muls",
                             "divps", "rdivps", "sin", "cos", "sincos", "cossin", "expc", "tanh", "sigmoid", "relu", "neg", "step", "clampmask", "onemsq",
                             "yomy", "divpgb", "rbf16", "rowsum", "gld", "gst", "gldf", "gstf", "fill", "spill", "uload", "uconst", "loop{", "}loop", "colout",
                             "scalout", "sacc0", "sacc1", "sacc2", "sacc3", "ascal0", "ascal1", "ascal2", "ascal3", "glda0", "glda", "ldsw", "ldswa", "gstf}loop", "glda0h", "ldswah", "rowsumu", "accums", "sqrt", "rcp", "tanhb", "sigmoidb", "expcb", "end"};
  std::string s;
  char buf[64];
  for (size_t i = 0; i < sg.code.size(); ++i) {
    const uint32_t w = sg.code[i];
    const int cs = (int)(w & 1023u);
    const uint32_t arg = w >> 14;
    if (cs < vm::kFirstPlain) snprintf(buf, sizeof(buf), "%s r%d", jn[cs / vm::kJointStride], cs % vm::kJointStride);
    else if (cs < vm::P_COUNT_) snprintf(buf, sizeof(buf), "%s", pn[cs - vm::kFirstPlain]);
    else snprintf(buf, sizeof(buf), "?%d", cs);
    s += buf;
    if (arg || (cs >= vm::kFirstPlain && cs != vm::P_LOOP_BEGIN && cs != vm::P_LOOP_END && cs != vm::P_END && !(cs >= vm::P_SIN && cs <= vm::P_ROWSUM && cs != vm::P_SINCOS && cs != vm::P_COSSIN) && !(cs >= vm::P_SACC0 && cs <= vm::P_SACC3))) {
      snprintf(buf, sizeof(buf), " %u", arg);
      s += buf;
    }
    s += "; ";
    if (cs == vm::P_UCONST) ++i;
    if (cs == vm::P_END) break;
  }
  return s;
}

std::string describe_plan(const Plan& p) {
  std::string s;
  char buf[256];
  for (const Step& st : p.steps) {
    switch (st.kind) {
      case ST_VM: {
        const VmSegment& sg = p.segs[st.seg];
        snprintf(buf, sizeof(buf), "vm[%s %s n=%lld cols=%d instr=%d body=%d operands=%d smem=%d spill=%d colacc=%d scalacc=%d grid=%d]\n",
                 sg.row_mode ? "row" : "flat", sg.dense ? "dense" : "wide", sg.n, sg.cols, (int)sg.code.size(), sg.n_instr_body,
                 (int)sg.operand_mem.size(), sg.n_smem, sg.n_spill, sg.n_colacc, sg.n_scalacc, sg.grid);
        s += buf;
        if (sg.code.size() <= 96) s += "  code: " + disassemble(sg) + "\n";
        buf[0] = 0;
        break;
      }
      case ST_GEMM: {
        static const char* en[] = {"add", "sub", "rsub", "mul", "relu", "tanh", "sigmoid", "expc", "sin", "neg", "sqrt", "rcp", "rbf16"};
        static const char* on[] = {"", "c", "s", "row", "full"};
        std::string ep;
        for (const EpiSpec& e : st.epi) ep += std::string(ep.empty() ? " epilogue: " : ", ") + en[e.opc] + (e.operand ? std::string(" ") + on[e.operand] : "");
        snprintf(buf, sizeof(buf), "gemm[%lldx%lldx%lld%s%s%s%s%s -> %s%s]\n", (long long)p.mems[st.mC].shape.d[0], (long long)p.mems[st.mC].shape.d[1],
                 (long long)p.mems[st.mA].shape.d[st.tA ? 0 : 1], st.tA ? " A^T" : "", st.tB ? " B^T" : "", st.mD >= 0 ? " +bias" : "",
                 st.relu ? " relu" : "", st.mE >= 0 ? " *step" : "", p.mems[st.mC].dtype == DRAGON_BF16 ? "bf16" : "f32",
                 (ep + (st.mF >= 0 ? " +colsum" : "")).c_str());
        break;
      }
      case ST_TRANSPOSE:
        snprintf(buf, sizeof(buf), "transpose[%lldx%lld]\n", (long long)p.mems[st.mA].shape.d[0], (long long)p.mems[st.mA].shape.d[1]);
        break;
      case ST_SCE_FWD: snprintf(buf, sizeof(buf), st.mD >= 0 ? "softmax_ce_fwd+bwd%s\n" : "softmax_ce_fwd%s\n", st.mF >= 0 ? " +colsum" : ""); break;
      case ST_SCE_BWD: snprintf(buf, sizeof(buf), "softmax_ce_bwd%s\n", st.mF >= 0 ? " +colsum" : ""); break;
      default: snprintf(buf, sizeof(buf), "copy\n");
    }
    s += buf;
  }
  return s;
}

}  // namespace dragon
