// C ABI of libdragon.so: graph capture, compile (prune + lower), run.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>

#include "plan.h"
#include "vm_math.h"

namespace dragon {
cudaError_t launch_vm(const vm::Params& p, int grid, int n_smem_slots, bool dense, cudaStream_t st, void* spec_kernel);
void load_specialized(VmSegment* sg);
void unload_specialized(VmSegment* sg);
cudaError_t launch_finish(const VmSegment& sg, const std::vector<MemRef>& mems, void* const* mem_ptr, char* ws, cudaStream_t st, int chunks);
cudaError_t launch_sce_fwd(const void* z, int zdtype, const int* labels, int rows, int cols, float* rowloss, float* out,
                           int* status, cudaStream_t st, void* dz, int dzdtype, float dl_imm, float* colpart, int n_colpart);
cudaError_t launch_sce_bwd(const void* z, int zdtype, const int* labels, int rows, int cols, void* dz, int dzdtype,
                           const float* dl_ptr, float dl_imm, int* status, cudaStream_t st, float* colpart, int n_colpart);
cudaError_t launch_colsum_finish(const float* part, int n_part, int cols, void* out, int dtype, cudaStream_t st);
cudaError_t launch_transpose16(const void* in, void* out, int rows, int cols, cudaStream_t st);
int launch_gemm_bf16(const void* A, const void* B, void* C, int c_dtype, int M, int N, int K, bool a_mn, bool b_mn, int* status,
                     cudaStream_t st, const void* bias, int bias_dtype, bool relu, const void* mask,
                     const std::vector<EpiSpec>& epi, const std::vector<MemRef>& mems, void* const* mem_ptr, float* colpart);
}  // namespace dragon

using namespace dragon;

namespace {

bool valid_tensor(const dragon_graph_t* g, dragon_id t) { return t >= 0 && t < (int)g->g.tensors.size(); }

int infer_shape(const Graph& g, int type, const dragon_id* in, int n_in, Shape* out) {
  auto T = [&](int p) -> const TensorInfo& { return g.tensors[in[p]]; };
  auto is_float = [&](int p) { return T(p).dtype == DRAGON_F32 || T(p).dtype == DRAGON_BF16; };
  switch (type) {
    case DRAGON_OP_ADD: case DRAGON_OP_SUB: case DRAGON_OP_MUL: case DRAGON_OP_DIV:
      if (n_in != 2) { set_error("binary operator takes 2 inputs"); return DRAGON_ERR_INVALID_ARG; }
      if (!is_float(0) || !is_float(1)) { set_error("elementwise operators take f32/bf16 tensors"); return DRAGON_ERR_DTYPE; }
      if (!broadcast_shapes(T(0).shape, T(1).shape, out)) { set_error("operands '%s' and '%s' do not broadcast", T(0).name.c_str(), T(1).name.c_str()); return DRAGON_ERR_SHAPE; }
      return DRAGON_OK;
    case DRAGON_OP_SIN: case DRAGON_OP_EXP: case DRAGON_OP_TANH: case DRAGON_OP_SIGMOID: case DRAGON_OP_RELU:
    case DRAGON_OP_SQRT: case DRAGON_OP_RECIPROCAL:
    case DRAGON_OP_SUM: case DRAGON_OP_MEAN:
      if (n_in != 1) { set_error("unary operator takes 1 input"); return DRAGON_ERR_INVALID_ARG; }
      if (!is_float(0)) { set_error("elementwise operators take f32/bf16 tensors"); return DRAGON_ERR_DTYPE; }
      if ((type == DRAGON_OP_SUM || type == DRAGON_OP_MEAN) && T(0).shape.rank == 0) { set_error("Sum/Mean need rank >= 1"); return DRAGON_ERR_SHAPE; }
      *out = T(0).shape;
      return DRAGON_OK;
    case DRAGON_OP_INNER_PRODUCT:
      if (n_in != 2) { set_error("InnerProduct takes 2 inputs"); return DRAGON_ERR_INVALID_ARG; }
      if (!is_float(0) || !is_float(1)) { set_error("InnerProduct takes f32/bf16 tensors"); return DRAGON_ERR_DTYPE; }
      if (T(0).shape.rank != 2 || T(1).shape.rank != 2 || T(0).shape.d[1] != T(1).shape.d[1]) { set_error("InnerProduct needs X[M,K], W[N,K]"); return DRAGON_ERR_SHAPE; }
      out->rank = 2; out->d[0] = T(0).shape.d[0]; out->d[1] = T(1).shape.d[0];
      return DRAGON_OK;
    case DRAGON_OP_BIAS_ADD:
      if (n_in != 2) { set_error("BiasAdd takes 2 inputs"); return DRAGON_ERR_INVALID_ARG; }
      if (!is_float(0) || !is_float(1)) { set_error("BiasAdd takes f32/bf16 tensors"); return DRAGON_ERR_DTYPE; }
      if (T(0).shape.rank != 2 || T(1).shape.rank != 1 || T(0).shape.d[1] != T(1).shape.d[0]) { set_error("BiasAdd needs Y[M,N], b[N]"); return DRAGON_ERR_SHAPE; }
      *out = T(0).shape;
      return DRAGON_OK;
    case DRAGON_OP_SOFTMAX_CROSS_ENTROPY:
      if (n_in != 2) { set_error("SoftmaxCrossEntropy takes 2 inputs"); return DRAGON_ERR_INVALID_ARG; }
      if (!is_float(0) || T(1).dtype != DRAGON_I32) { set_error("SoftmaxCrossEntropy takes float logits and int32 labels"); return DRAGON_ERR_DTYPE; }
      if (T(0).shape.rank != 2 || T(1).shape.rank != 1 || T(0).shape.d[0] != T(1).shape.d[0]) { set_error("SoftmaxCrossEntropy needs Z[M,N], labels[M]"); return DRAGON_ERR_SHAPE; }
      *out = Shape();
      return DRAGON_OK;
    default:
      set_error("unknown operator type %d", type);
      return DRAGON_ERR_INVALID_ARG;
  }
}

int query_sm_count() {
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess || n <= 0) { cudaGetLastError(); return kDefaultSmCount; }
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
    cudaGetLastError();
    return kDefaultSmCount;
  }
  return sms;
}

}  // namespace

extern "C" {

dragon_graph_t* dragon_graph_create(void) { return new (std::nothrow) dragon_graph_t(); }
void dragon_graph_destroy(dragon_graph_t* g) { delete g; }

dragon_id dragon_add_tensor(dragon_graph_t* g, const char* name, int dtype, int rank, const int64_t* shape) {
  if (!g || !name || rank < 0 || rank > 2 || (rank > 0 && !shape)) { set_error("dragon_add_tensor: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  if (dtype != DRAGON_F32 && dtype != DRAGON_BF16 && dtype != DRAGON_I32) { set_error("dragon_add_tensor: unknown dtype %d", dtype); return DRAGON_ERR_DTYPE; }
  TensorInfo t;
  t.name = name;
  t.dtype = dtype;
  t.shape.rank = rank;
  for (int i = 0; i < rank; ++i) {
    if (shape[i] <= 0) { set_error("dragon_add_tensor: dimension %d of '%s' is not positive", i, name); return DRAGON_ERR_SHAPE; }
    t.shape.d[i] = shape[i];
  }
  if (!g->g.names.insert(t.name).second) { set_error("dragon_add_tensor: name '%s' is already taken", name); return DRAGON_ERR_INVALID_ARG; }
  g->g.tensors.push_back(t);
  return (dragon_id)g->g.tensors.size() - 1;
}

dragon_id dragon_add_op(dragon_graph_t* g, int op_type, const dragon_id* in, int n_in, const dragon_id* out, int n_out,
                        const double* attrs, int n_attrs) {
  (void)attrs;
  if (!g || !in || !out || n_in <= 0 || n_out <= 0 || n_attrs < 0) { set_error("dragon_add_op: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  for (int i = 0; i < n_in; ++i)
    if (!valid_tensor(g, in[i])) { set_error("dragon_add_op: input id %d is not a tensor", in[i]); return DRAGON_ERR_INVALID_ARG; }
  for (int i = 0; i < n_out; ++i)
    if (!valid_tensor(g, out[i])) { set_error("dragon_add_op: output id %d is not a tensor", out[i]); return DRAGON_ERR_INVALID_ARG; }
  if (n_out != 1 && op_type != DRAGON_OP_OPAQUE) { set_error("dragon_add_op: every executable operator type has one output (DRAGON_OP_OPAQUE takes several)"); return DRAGON_ERR_INVALID_ARG; }
  for (int i = 0; i < n_in; ++i)
    if (g->g.tensors[in[i]].grad_stage >= 0) { set_error("dragon_add_op: gradient tensors cannot be consumed by operators"); return DRAGON_ERR_UNSUPPORTED; }
  for (int j = 0; j < n_out; ++j) {
    const TensorInfo& to = g->g.tensors[out[j]];
    if (to.producer >= 0 || to.grad_stage >= 0) { set_error("dragon_add_op: tensor '%s' already has a producer", to.name.c_str()); return DRAGON_ERR_NOT_SSA; }
    for (int i = 0; i < n_in; ++i)
      if (in[i] == out[j]) { set_error("dragon_add_op: operator reads its own output '%s'", to.name.c_str()); return DRAGON_ERR_NOT_SSA; }
    for (int i = 0; i < j; ++i)
      if (out[i] == out[j]) { set_error("dragon_add_op: output '%s' is listed twice", to.name.c_str()); return DRAGON_ERR_NOT_SSA; }
    // a tensor that was read before it got a producer would let the new operator close a cycle
    if (to.consumed) { set_error("dragon_add_op: tensor '%s' is already read by an earlier operator", to.name.c_str()); return DRAGON_ERR_NOT_SSA; }
    if (to.dtype == DRAGON_I32) { set_error("dragon_add_op: operators produce f32/bf16 tensors"); return DRAGON_ERR_DTYPE; }
  }
  if (op_type != DRAGON_OP_OPAQUE) {
    const TensorInfo& to = g->g.tensors[out[0]];
    Shape s;
    int rc = infer_shape(g->g, op_type, in, n_in, &s);
    if (rc != DRAGON_OK) return rc;
    if (s != to.shape) { set_error("dragon_add_op: declared shape of '%s' differs from the inferred one", to.name.c_str()); return DRAGON_ERR_SHAPE; }
  }
  OpInfo op;
  op.type = op_type;
  op.in.assign(in, in + n_in);
  op.out.assign(out, out + n_out);
  g->g.ops.push_back(op);
  for (int i = 0; i < n_in; ++i) g->g.tensors[in[i]].consumed = true;
  for (int j = 0; j < n_out; ++j) g->g.tensors[out[j]].producer = (int)g->g.ops.size() - 1;
  return (dragon_id)g->g.ops.size() - 1;
}

int dragon_add_grad(dragon_graph_t* g, const dragon_id* objs, int n_obj, const dragon_id* wrts, int n_wrt,
                    dragon_id* out_grad_tensor_ids) {
  if (!g || !objs || !wrts || !out_grad_tensor_ids || n_obj <= 0 || n_wrt <= 0) { set_error("dragon_add_grad: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  GradStage st;
  for (int i = 0; i < n_obj; ++i) {
    if (!valid_tensor(g, objs[i]) || g->g.tensors[objs[i]].grad_stage >= 0) { set_error("dragon_add_grad: bad objective id %d", objs[i]); return DRAGON_ERR_INVALID_ARG; }
    if (g->g.tensors[objs[i]].dtype == DRAGON_I32) { set_error("dragon_add_grad: objective must be a float tensor"); return DRAGON_ERR_DTYPE; }
    st.objs.push_back(objs[i]);
  }
  for (int i = 0; i < n_wrt; ++i) {
    if (!valid_tensor(g, wrts[i]) || g->g.tensors[wrts[i]].grad_stage >= 0) { set_error("dragon_add_grad: bad derivative target id %d", wrts[i]); return DRAGON_ERR_INVALID_ARG; }
    if (g->g.tensors[wrts[i]].dtype == DRAGON_I32) { set_error("dragon_add_grad: derivative target must be a float tensor"); return DRAGON_ERR_DTYPE; }
    st.wrts.push_back(wrts[i]);
  }
  std::vector<uint8_t> G = backward_chain_marks(g->g, st.objs, st.wrts);
  for (int w : st.wrts)
    if (!G[w]) { set_error("dragon_add_grad: no chain from '%s' to any objective", g->g.tensors[w].name.c_str()); return DRAGON_ERR_NO_PATH; }
  const int s = (int)g->g.stages.size();
  for (int i = 0; i < n_wrt; ++i) {
    TensorInfo t;
    t.name = "grad" + std::to_string(s) + "/" + g->g.tensors[wrts[i]].name;
    while (!g->g.names.insert(t.name).second) t.name += "'";
    t.dtype = DRAGON_F32;
    t.shape = g->g.tensors[wrts[i]].shape;
    t.grad_stage = s;
    t.grad_wrt = wrts[i];
    g->g.tensors.push_back(t);
    st.grad_ids.push_back((int)g->g.tensors.size() - 1);
    out_grad_tensor_ids[i] = st.grad_ids.back();
  }
  g->g.stages.push_back(st);
  return DRAGON_OK;
}

int dragon_graph_num_tensors(const dragon_graph_t* g) { return g ? (int)g->g.tensors.size() : DRAGON_ERR_INVALID_ARG; }
int dragon_graph_num_ops(const dragon_graph_t* g) { return g ? (int)g->g.ops.size() : DRAGON_ERR_INVALID_ARG; }

dragon_function_t* dragon_function(dragon_graph_t* g, const dragon_id* inputs, int n_in, const dragon_id* outputs, int n_out) {
  if (!g || (n_in > 0 && !inputs) || !outputs || n_in < 0 || n_out <= 0) { set_error("dragon_function: bad argument"); return nullptr; }
  std::vector<int> in(inputs, inputs + n_in), out(outputs, outputs + n_out);
  std::vector<uint8_t> seen(g->g.tensors.size(), 0);
  for (int t : in) {
    if (!valid_tensor(g, t)) { set_error("dragon_function: input id %d is not a tensor", t); return nullptr; }
    if (g->g.tensors[t].grad_stage >= 0) { set_error("dragon_function: input '%s' is a gradient tensor and cannot be fed", g->g.tensors[t].name.c_str()); return nullptr; }
    if (seen[t]) { set_error("dragon_function: input '%s' is listed twice", g->g.tensors[t].name.c_str()); return nullptr; }
    seen[t] = 1;
  }
  for (int t : out)
    if (!valid_tensor(g, t)) { set_error("dragon_function: output id %d is not a tensor", t); return nullptr; }
  dragon_function_t* f = new (std::nothrow) dragon_function_t();
  if (!f) return nullptr;
  f->n_tensors = (int)g->g.tensors.size();
  f->n_in = n_in;
  f->n_out = n_out;
  if (const char* tier = std::getenv("DRAGON_VM_TIER")) f->tier = tier[0] == '0' ? 0 : 1;
  for (int t : in) f->in_info.push_back(g->g.tensors[t]);
  for (int t : out) f->out_info.push_back(g->g.tensors[t]);
  // A listed input that an operator produces is given, not solved (Sec. 3.1: any tensor can be fed): in
  // this function's graph it is a source, and the operator that would have produced it loses it as an
  // output.  The cut is made on a copy; the caller's graph stays as it is.
  const dragon::Graph* fg = &g->g;
  dragon::Graph cut;
  bool feeds_intermediate = false;
  for (int t : in) feeds_intermediate |= g->g.tensors[t].producer >= 0;
  if (feeds_intermediate) {
    cut = g->g;
    for (int t : in) {
      const int p = cut.tensors[t].producer;
      if (p < 0) continue;
      auto& o = cut.ops[p].out;
      o.erase(std::remove(o.begin(), o.end(), t), o.end());
      cut.tensors[t].producer = -1;
    }
    fg = &cut;
  }
  if (prune_function(*fg, in, out, &f->prune) != DRAGON_OK) { delete f; return nullptr; }
  f->rename = inplace_rename(*fg, f->prune);
  // a kept operator that is only an edge set (Sec. 2.2) can be pruned around but not executed: the
  // function keeps its prune results and refuses to run
  for (int k : f->prune.fwd_ops)
    if (fg->ops[k].type == DRAGON_OP_OPAQUE) {
      f->not_executable = "the function keeps an opaque operator (operator " + std::to_string(k) + "): it can be pruned but not executed";
      return f;
    }
  if (lower_function(*fg, f->prune, in, out, query_sm_count(), &f->plan) != DRAGON_OK) { delete f; return nullptr; }
  return f;
}

void dragon_function_destroy(dragon_function_t* f) {
  if (!f) return;
  for (void* ev : f->prof_ev) cudaEventDestroy(reinterpret_cast<cudaEvent_t>(ev));
  for (void* ev : f->h_event) cudaEventDestroy(reinterpret_cast<cudaEvent_t>(ev));
  for (void* s : f->h_stream) if (s) cudaStreamDestroy(reinterpret_cast<cudaStream_t>(s));
  for (auto& sg : f->plan.segs) {
    if (sg.d_code) cudaFree(sg.d_code);
    unload_specialized(&sg);
  }
  delete f;
}

int dragon_function_marked(const dragon_function_t* f, uint8_t* flags, int n_tensors) {
  if (!f || !flags || n_tensors != f->n_tensors) { set_error("dragon_function_marked: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  std::memcpy(flags, f->prune.marked.data(), (size_t)n_tensors);
  return DRAGON_OK;
}

int dragon_function_kept_ops(const dragon_function_t* f, dragon_id* fwd_ops, int cap_f, int* n_f, dragon_id* grad_ops,
                             uint32_t* grad_input_mask, int cap_g, int* n_g) {
  if (!f || !n_f || !n_g || cap_f < 0 || cap_g < 0) { set_error("dragon_function_kept_ops: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  *n_f = (int)f->prune.fwd_ops.size();
  *n_g = (int)f->prune.grad_ops.size();
  for (int i = 0; i < *n_f && i < cap_f && fwd_ops; ++i) fwd_ops[i] = f->prune.fwd_ops[i];
  for (int i = 0; i < *n_g && i < cap_g; ++i) {
    if (grad_ops) grad_ops[i] = f->prune.grad_ops[i].op;
    if (grad_input_mask) grad_input_mask[i] = f->prune.grad_ops[i].mask;
  }
  return DRAGON_OK;
}

int dragon_function_used_inputs(const dragon_function_t* f, uint8_t* flags, int n_in) {
  if (!f || (n_in > 0 && !flags) || n_in != f->n_in) { set_error("dragon_function_used_inputs: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  if (n_in) std::memcpy(flags, f->prune.used_inputs.data(), (size_t)n_in);
  return DRAGON_OK;
}

int dragon_function_can_alias(const dragon_function_t* f, int input, int output) {
  if (!f || input < 0 || input >= f->n_in || output < 0 || output >= f->n_out) { set_error("dragon_function_can_alias: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  const Plan& P = f->plan;
  if (!f->not_executable.empty() || P.steps.size() != 1 || P.steps[0].kind != ST_VM) return 0;
  const VmSegment& sg = P.segs[P.steps[0].seg];
  if (sg.row_mode) return 0;
  const std::vector<VmAccess> acc = vm_operand_accesses(sg);
  int oi = -1, oo = -1;
  for (size_t k = 0; k < sg.operand_mem.size(); ++k) {
    const MemRef& m = P.mems[sg.operand_mem[k]];
    if (sg.operand_kind[k] != (uint32_t)vm::K_FULL) continue;
    if (m.where == MEM_FEED && m.index == input) oi = (int)k;
    if (m.where == MEM_FETCH && m.index == output) oo = (int)k;
  }
  if (oi < 0 || oo < 0) return 0;
  const MemRef &mi = P.mems[sg.operand_mem[oi]], &mo = P.mems[sg.operand_mem[oo]];
  if (mi.dtype != mo.dtype || mi.shape.numel() != mo.shape.numel() || mi.shape.numel() != sg.n) return 0;
  // several memrefs may name the same position: every load of the input, every store of the output
  int last_load = -1, first_store = 1 << 30;
  for (size_t k = 0; k < sg.operand_mem.size(); ++k) {
    const MemRef& m = P.mems[sg.operand_mem[k]];
    if (m.where == MEM_FEED && m.index == input) { if (sg.operand_kind[k] != (uint32_t)vm::K_FULL) return 0; last_load = std::max(last_load, acc[k].last_load); }
    if (m.where == MEM_FETCH && m.index == output) { if (acc[k].last_load >= 0) return 0; first_store = std::min(first_store, acc[k].first_store); }
  }
  return (last_load >= 0 && last_load < first_store) ? 1 : 0;
}

int dragon_function_rename_dictionary(const dragon_function_t* f, dragon_id* ancestor, int n_tensors) {
  if (!f || !ancestor || n_tensors != f->n_tensors) { set_error("dragon_function_rename_dictionary: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  for (int i = 0; i < n_tensors; ++i) ancestor[i] = f->rename[i];
  return DRAGON_OK;
}

int dragon_function_workspace_tensors(const dragon_function_t* f, int64_t* out, int cap) {
  if (!f || (cap > 0 && !out) || cap < 0) { set_error("dragon_function_workspace_tensors: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  int n = 0;
  for (const MemRef& m : f->plan.mems) {
    if (m.where != MEM_WORK || !m.live) continue;
    if (n < cap) {
      out[5 * n + 0] = (int64_t)m.offset;
      out[5 * n + 1] = (int64_t)m.bytes();
      out[5 * n + 2] = m.first_step;
      out[5 * n + 3] = m.last_step;
      out[5 * n + 4] = m.shares_input;
    }
    ++n;
  }
  return n;
}

int dragon_function_num_launches(const dragon_function_t* f) {
  if (!f) return DRAGON_ERR_INVALID_ARG;
  int n = 0;
  for (const Step& st : f->plan.steps) {
    if (st.kind == ST_VM) n += 1 + (f->plan.segs[st.seg].finish.empty() ? 0 : 1);
    else if (st.kind == ST_SCE_FWD) n += 2 + (st.mF >= 0 ? 1 : 0);
    else if (st.kind != ST_COPY) n += 1 + (st.mF >= 0 ? 1 : 0);
  }
  return n;
}

int dragon_function_describe(const dragon_function_t* f, char* buf, int cap) {
  if (!f || !buf || cap <= 0) return DRAGON_ERR_INVALID_ARG;
  std::string s = f->not_executable.empty() ? describe_plan(f->plan) : "not executable: " + f->not_executable + "\n";
  for (size_t k = 0; k < f->plan.steps.size(); ++k)
    if (f->plan.steps[k].kind == ST_VM && f->plan.segs[f->plan.steps[k].seg].spec_state < 0)
      s += "note: the program of step " + std::to_string(k) + " runs interpreted: " + f->plan.segs[f->plan.steps[k].seg].spec_log + "\n";
  std::strncpy(buf, s.c_str(), (size_t)cap - 1);
  buf[cap - 1] = 0;
  return DRAGON_OK;
}

int dragon_function_vm_step(const dragon_function_t* f, int step, int64_t* info, uint32_t* code, int cap_code,
                            int64_t* operands, int cap_operands, int64_t* reduced, int cap_reduced) {
  if (!f || !info || step < 0 || step >= (int)f->plan.steps.size() || f->plan.steps[step].kind != ST_VM || cap_code < 0 || cap_operands < 0) {
    set_error("dragon_function_vm_step: not a graph-VM step");
    return DRAGON_ERR_INVALID_ARG;
  }
  const VmSegment& sg = f->plan.segs[f->plan.steps[step].seg];
  info[0] = (int64_t)sg.code.size(); info[1] = sg.row_mode; info[2] = sg.cols; info[3] = (int64_t)sg.operand_mem.size();
  info[4] = sg.n_spill; info[5] = sg.n_smem; info[6] = sg.n & 0xffffffffLL; info[7] = sg.n >> 32;
  info[8] = (int64_t)sg.finish.size();
  info[9] = sg.dense ? vm::kVmRegsDense : vm::kVmRegsWide;
  for (int i = 0; reduced && i < cap_reduced && i < (int)sg.finish.size(); ++i) {
    const MemRef& m = f->plan.mems[sg.finish[i].mem];
    reduced[3 * i + 0] = sg.finish[i].kind;
    reduced[3 * i + 1] = sg.finish[i].acc;
    reduced[3 * i + 2] = m.where == MEM_FETCH ? m.index : -1;
  }
  for (int i = 0; code && i < cap_code && i < (int)sg.code.size(); ++i) code[i] = sg.code[i];
  for (int i = 0; operands && i < cap_operands && i < (int)sg.operand_mem.size(); ++i) {
    const MemRef& m = f->plan.mems[sg.operand_mem[i]];
    operands[4 * i + 0] = m.where;
    operands[4 * i + 1] = m.where == MEM_WORK ? (int64_t)(m.offset / 256) : m.index;
    operands[4 * i + 2] = sg.operand_kind[i];
    operands[4 * i + 3] = m.dtype;
  }
  return DRAGON_OK;
}

size_t dragon_function_workspace_bytes(const dragon_function_t* f) { return f ? f->plan.workspace_bytes : 0; }

int dragon_function_set_workspace(dragon_function_t* f, void* dev_ptr, size_t bytes) {
  if (!f) { set_error("dragon_function_set_workspace: NULL function"); return DRAGON_ERR_INVALID_ARG; }
  if (!dev_ptr || ((uintptr_t)dev_ptr & 255) || bytes < f->plan.workspace_bytes) {
    set_error("workspace must be 256-byte aligned device memory of at least %zu bytes", f->plan.workspace_bytes);
    return DRAGON_ERR_WORKSPACE;
  }
  f->workspace = dev_ptr;
  f->workspace_bytes = bytes;
  f->status_ready = false;
  return DRAGON_OK;
}

// First run: device copies of the instruction streams and, unless the function is held to the interpreter,
// the kernels specialised for them.  A program whose specialised kernel cannot be made (no assembler in
// the driver, an assembler error) stays with the interpreter; dragon_function_describe() says why.
static int upload_programs(dragon_function_t* f) {
  for (auto& sg : f->plan.segs) {
    if (sg.code.empty()) continue;
    if (!sg.d_code && (cudaMalloc(&sg.d_code, sg.code.size() * 4) != cudaSuccess ||
                       cudaMemcpy(sg.d_code, sg.code.data(), sg.code.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess)) {
      set_error("dragon_run: cannot upload the instruction stream: %s", cudaGetErrorString(cudaGetLastError()));
      sg.d_code = nullptr;
      return DRAGON_ERR_CUDA;
    }
    if (f->tier && sg.spec_state == 0) load_specialized(&sg);
  }
  f->uploaded = true;
  return DRAGON_OK;
}

int dragon_function_specialize(dragon_function_t* f, int mode) {
  if (!f || mode < 0 || mode > 2) { set_error("dragon_function_specialize: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  f->tier = mode ? 1 : 0;
  if (mode != 2) return DRAGON_OK;
  if (!f->not_executable.empty()) { set_error("dragon_function_specialize: %s", f->not_executable.c_str()); return DRAGON_ERR_UNSUPPORTED; }
  int n = 0;
  for (auto& sg : f->plan.segs) {
    if (sg.code.empty()) continue;
    if (sg.spec_state == 0) load_specialized(&sg);
    if (sg.spec_state != 1) { set_error("dragon_function_specialize: %s", sg.spec_log.c_str()); return DRAGON_ERR_CUDA; }
    ++n;
  }
  return n;
}

int dragon_function_num_specialized(const dragon_function_t* f) {
  if (!f) { set_error("dragon_function_num_specialized: NULL function"); return DRAGON_ERR_INVALID_ARG; }
  int n = 0;
  for (const auto& sg : f->plan.segs) n += f->tier && sg.spec_state == 1;
  return n;
}

int dragon_verify_vm_program(const uint32_t* code, int n_code, int loop_start, int register_slots, int n_operands,
                             int n_smem_slots, int n_spill_slots, int n_column_accs, int n_scalar_accs, int row_mode) {
  return verify_program(code, n_code, loop_start, register_slots, n_operands, n_smem_slots, n_spill_slots, n_column_accs,
                        n_scalar_accs, row_mode != 0);
}

int dragon_function_vm_ptx(const dragon_function_t* f, int step, char* buf, int cap) {
  if (!f || step < 0 || step >= (int)f->plan.steps.size() || f->plan.steps[step].kind != ST_VM || cap < 0 || (cap > 0 && !buf)) {
    set_error("dragon_function_vm_ptx: not a graph-VM step");
    return DRAGON_ERR_INVALID_ARG;
  }
  std::string ptx;
  const int rc = specialize_ptx(f->plan.segs[f->plan.steps[step].seg], "dragon_vm_spec", &ptx);
  if (rc != DRAGON_OK) return rc;
  if (cap > 0) {
    const size_t k = std::min(ptx.size(), (size_t)cap - 1);
    std::memcpy(buf, ptx.data(), k);
    buf[k] = 0;
  }
  return (int)ptx.size();
}

int dragon_run(dragon_function_t* f, const void* const* feeds, void* const* fetches, void* cuda_stream) {
  if (!f || !fetches || (f->n_in > 0 && !feeds)) { set_error("dragon_run: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  Plan& P = f->plan;
  if (!f->not_executable.empty()) { set_error("dragon_run: %s", f->not_executable.c_str()); return DRAGON_ERR_UNSUPPORTED; }
  if (!f->workspace) { set_error("dragon_run: no workspace set (need %zu bytes)", P.workspace_bytes); return DRAGON_ERR_WORKSPACE; }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  char* ws = reinterpret_cast<char*>(f->workspace);
  std::vector<void*> ptr(P.mems.size(), nullptr);
  for (size_t m = 0; m < P.mems.size(); ++m) {
    const MemRef& mr = P.mems[m];
    if (mr.where == MEM_WORK) { ptr[m] = ws + mr.offset; continue; }
    if (!mr.live) continue;
    void* q = mr.where == MEM_FEED ? const_cast<void*>(feeds[mr.index]) : fetches[mr.index];
    if (!q || ((uintptr_t)q & 15)) {
      set_error("dragon_run: %s %d is NULL or not 16-byte aligned", mr.where == MEM_FEED ? "feed" : "fetch", mr.index);
      return DRAGON_ERR_INVALID_ARG;
    }
    ptr[m] = q;
  }
  if (upload_programs(f) != DRAGON_OK) return DRAGON_ERR_CUDA;
  // this run's status word, and the other one, which it clears for the next run
  int* const word0 = reinterpret_cast<int*>(ws + P.status_off);
  cudaError_t e = cudaSuccess;
  if (!f->status_ready) {
    e = cudaMemsetAsync(word0, 0, 256, st);
    f->status_ready = true;
    f->run_parity = 0;
  }
  int* const status = word0 + 16 * f->run_parity;
  int* const status_next = word0 + 16 * (f->run_parity ^ 1);
  bool next_cleared = false;
  for (size_t si = 0; si < P.steps.size(); ++si) {
    const Step& s = P.steps[si];
    if (e != cudaSuccess) break;
    const bool prof = (int)si == f->prof_step && 2 * (f->prof_used + 1) <= (int)f->prof_ev.size();
    if (prof && s.kind != ST_VM) cudaEventRecord(reinterpret_cast<cudaEvent_t>(f->prof_ev[2 * f->prof_used]), st);
    switch (s.kind) {
      case ST_VM: {
        VmSegment& sg = P.segs[s.seg];
        vm::Params p;
        std::memset(&p, 0, sizeof(p));
        p.code = sg.d_code;
        p.n_code = (int)sg.code.size();
        p.row_mode = sg.row_mode;
        p.n = sg.n;
        p.cols = sg.cols;
        p.n_spill = sg.n_spill;
        p.n_tiles = (uint32_t)(sg.row_mode ? sg.n : (sg.n + kVmTile - 1) / kVmTile);
        p.loop_start = (uint32_t)sg.loop_start;
        p.grid = (uint32_t)sg.grid;
        p.n_full_tiles = sg.row_mode ? (sg.cols == kVmTile ? p.n_tiles : 0u) : (uint32_t)(sg.n / kVmTile);
        p.spill = reinterpret_cast<float*>(ws + sg.spill_off);
        p.colpart = reinterpret_cast<float*>(ws + sg.colpart_off);
        p.scalpart = reinterpret_cast<double*>(ws + sg.scalpart_off);
        p.status = status;
        p.status_clear = next_cleared ? nullptr : status_next;
        next_cleared = true;
        for (size_t i = 0; i < sg.operand_mem.size(); ++i) {
          p.operand[i].ptr = ptr[sg.operand_mem[i]];
          p.operand[i].kind = sg.operand_kind[i];
          p.operand[i].dtype = (uint32_t)P.mems[sg.operand_mem[i]].dtype;
        }
        if (prof) cudaEventRecord(reinterpret_cast<cudaEvent_t>(f->prof_ev[2 * f->prof_used]), st);
        e = launch_vm(p, sg.grid, sg.n_smem, sg.dense, st, f->tier ? sg.spec_kernel : nullptr);
        if (prof) cudaEventRecord(reinterpret_cast<cudaEvent_t>(f->prof_ev[2 * f->prof_used + 1]), st);
        if (e == cudaSuccess) e = launch_finish(sg, P.mems, ptr.data(), ws, st, 1);
        break;
      }
      case ST_GEMM: {
        const MemRef &A = P.mems[s.mA], &C = P.mems[s.mC];
        const int kc = (int)(s.tA ? A.shape.d[0] : A.shape.d[1]);
        int rc = launch_gemm_bf16(ptr[s.mA], ptr[s.mB], ptr[s.mC], C.dtype, (int)C.shape.d[0], (int)C.shape.d[1], kc, s.tA, s.tB, status, st,
                                  s.mD >= 0 ? ptr[s.mD] : nullptr, s.mD >= 0 ? P.mems[s.mD].dtype : DRAGON_F32, s.relu, s.mE >= 0 ? ptr[s.mE] : nullptr,
                                  s.epi, P.mems, ptr.data(), s.mF >= 0 ? reinterpret_cast<float*>(ws + s.colpart_off) : nullptr);
        if (rc != DRAGON_OK) { f->status_ready = false; return rc; }
        break;
      }
      case ST_TRANSPOSE:
        e = launch_transpose16(ptr[s.mA], ptr[s.mC], (int)P.mems[s.mA].shape.d[0], (int)P.mems[s.mA].shape.d[1], st);
        break;
      case ST_SCE_FWD:
        e = launch_sce_fwd(ptr[s.mA], P.mems[s.mA].dtype, reinterpret_cast<const int*>(ptr[s.mB]), (int)P.mems[s.mA].shape.d[0],
                           (int)P.mems[s.mA].shape.d[1], reinterpret_cast<float*>(ws + s.scratch_off), reinterpret_cast<float*>(ptr[s.mC]), status, st,
                           s.mD >= 0 ? ptr[s.mD] : nullptr, s.mD >= 0 ? P.mems[s.mD].dtype : 0, s.scale,
                           s.mF >= 0 ? reinterpret_cast<float*>(ws + s.colpart_off) : nullptr, s.n_colpart);
        break;
      case ST_SCE_BWD:
        e = launch_sce_bwd(ptr[s.mA], P.mems[s.mA].dtype, reinterpret_cast<const int*>(ptr[s.mB]), (int)P.mems[s.mA].shape.d[0],
                           (int)P.mems[s.mA].shape.d[1], ptr[s.mC], P.mems[s.mC].dtype,
                           s.mD >= 0 ? reinterpret_cast<const float*>(ptr[s.mD]) : nullptr, s.scale, status, st,
                           s.mF >= 0 ? reinterpret_cast<float*>(ws + s.colpart_off) : nullptr, s.n_colpart);
        break;
      case ST_COPY:
        e = cudaMemcpyAsync(ptr[s.mC], ptr[s.mA], P.mems[s.mA].bytes(), cudaMemcpyDeviceToDevice, st);
        break;
    }
    if (prof) {
      if (s.kind != ST_VM) cudaEventRecord(reinterpret_cast<cudaEvent_t>(f->prof_ev[2 * f->prof_used + 1]), st);
      ++f->prof_used;
    }
    if (e == cudaSuccess && s.mF >= 0 && s.kind != ST_VM)     // the partial column sums that the kernel left -> the row vector
      e = launch_colsum_finish(reinterpret_cast<const float*>(ws + s.colpart_off), s.n_colpart, (int)P.mems[s.mF].shape.d[0], ptr[s.mF],
                               P.mems[s.mF].dtype, st);
  }
  if (e != cudaSuccess) {
    f->status_ready = false;   // both status words are cleared again before the next run
    set_error("dragon_run: CUDA error: %s", cudaGetErrorString(e));
    return DRAGON_ERR_CUDA;
  }
  if (!next_cleared && cudaMemsetAsync(status_next, 0, sizeof(int), st) != cudaSuccess) {
    set_error("dragon_run: CUDA error: %s", cudaGetErrorString(cudaGetLastError()));
    return DRAGON_ERR_CUDA;
  }
  f->last_status_word = f->run_parity;
  f->run_parity ^= 1;
  f->last_stream = cuda_stream;
  return DRAGON_OK;
}

size_t dragon_function_staging_bytes(const dragon_function_t* f) {
  if (!f) return 0;
  size_t n = 0;
  for (const MemRef& m : f->plan.mems)
    if (m.live && m.where != MEM_WORK) n += (m.bytes() + 255) & ~(size_t)255;
  return n;
}

namespace {

// A function that is one flat elementwise VM launch over many tiles, whose tensors all have the
// domain's shape or are scalars, can run in chunks of the element range: the copy-in of chunk c+1,
// the kernel of chunk c and the copy-out of chunk c-1 then overlap (the link is full duplex).
bool chunkable(const dragon_function_t* f) {
  const Plan& P = f->plan;
  if (P.steps.size() != 1 || P.steps[0].kind != ST_VM) return false;
  const VmSegment& sg = P.segs[P.steps[0].seg];
  if (sg.row_mode || sg.n_spill || sg.n_colacc) return false;
  const long long tiles = (sg.n + kVmTile - 1) / kVmTile;
  if (tiles / kHostChunks < sg.grid) return false;          // every chunk keeps all CTAs busy
  for (uint32_t k : sg.operand_kind) if (k != vm::K_FULL && k != vm::K_SCALAR) return false;
  for (int m : sg.operand_mem) if (P.mems[m].where == MEM_WORK) return false;
  for (const FinishJob& j : sg.finish) if (j.kind != 1) return false;
  for (const MemRef& m : P.mems)
    if (m.live && m.where != MEM_WORK && m.shape.numel() != sg.n && m.shape.numel() != 1) return false;
  return true;
}

#define HOST_TRY(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { f->status_ready = false; \
  set_error("dragon_run_host: CUDA error: %s", cudaGetErrorString(e_)); return DRAGON_ERR_CUDA; } } while (0)

int run_host_chunked(dragon_function_t* f, const std::vector<const void*>& dev_feeds, const std::vector<void*>& dev_fetches,
                     const void* const* host_feeds, void* const* host_fetches, cudaStream_t st) {
  Plan& P = f->plan;
  VmSegment& sg = P.segs[P.steps[0].seg];
  if (!f->workspace) { set_error("dragon_run_host: no workspace set (need %zu bytes)", P.workspace_bytes); return DRAGON_ERR_WORKSPACE; }
  char* ws = reinterpret_cast<char*>(f->workspace);
  if (!f->h_stream[0]) {
    for (void*& s : f->h_stream) {
      cudaStream_t ns;
      HOST_TRY(cudaStreamCreateWithFlags(&ns, cudaStreamNonBlocking));
      s = ns;
    }
    for (int i = 0; i < 2 * kHostChunks + 2; ++i) {
      cudaEvent_t ev;
      HOST_TRY(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
      f->h_event.push_back(ev);
    }
  }
  cudaStream_t s_in = reinterpret_cast<cudaStream_t>(f->h_stream[0]), s_out = reinterpret_cast<cudaStream_t>(f->h_stream[1]);
  auto ev = [&](int i) { return reinterpret_cast<cudaEvent_t>(f->h_event[i]); };
  cudaEvent_t ev_start = ev(2 * kHostChunks), ev_done = ev(2 * kHostChunks + 1);
  if (upload_programs(f) != DRAGON_OK) return DRAGON_ERR_CUDA;
  int* const word0 = reinterpret_cast<int*>(ws + P.status_off);
  if (!f->status_ready) {
    HOST_TRY(cudaMemsetAsync(word0, 0, 256, st));
    f->status_ready = true;
    f->run_parity = 0;
  }
  int* const status = word0 + 16 * f->run_parity;
  int* const status_next = word0 + 16 * (f->run_parity ^ 1);
  // the copy-in stream starts after everything already queued on the caller's stream (the previous run reads the staging area)
  HOST_TRY(cudaEventRecord(ev_start, st));
  HOST_TRY(cudaStreamWaitEvent(s_in, ev_start, 0));
  HOST_TRY(cudaStreamWaitEvent(s_out, ev_start, 0));
  // scalars go first, whole
  for (const MemRef& m : P.mems)
    if (m.live && m.where == MEM_FEED && m.shape.numel() == 1 && sg.n != 1)
      HOST_TRY(cudaMemcpyAsync(const_cast<void*>(dev_feeds[m.index]), host_feeds[m.index], m.bytes(), cudaMemcpyHostToDevice, s_in));
  const long long tiles = (sg.n + kVmTile - 1) / kVmTile, base_tiles = tiles / kHostChunks, extra = tiles % kHostChunks;
  long long tile0 = 0;
  for (int c = 0; c < kHostChunks; ++c) {
    const long long ntile = base_tiles + (c < extra ? 1 : 0);
    const long long e0 = tile0 * kVmTile, e1 = std::min<long long>(sg.n, (tile0 + ntile) * kVmTile), cn = e1 - e0;
    tile0 += ntile;
    std::vector<uint8_t> done_in(f->n_in, 0), done_out(f->n_out, 0);
    for (const MemRef& m : P.mems) {
      if (!m.live || m.where != MEM_FEED || m.shape.numel() == 1 || done_in[m.index]) continue;
      done_in[m.index] = 1;
      const size_t es = m.dtype == DRAGON_BF16 ? 2 : 4;
      HOST_TRY(cudaMemcpyAsync(reinterpret_cast<char*>(const_cast<void*>(dev_feeds[m.index])) + e0 * es,
                               reinterpret_cast<const char*>(host_feeds[m.index]) + e0 * es, (size_t)cn * es, cudaMemcpyHostToDevice, s_in));
    }
    HOST_TRY(cudaEventRecord(ev(c), s_in));
    HOST_TRY(cudaStreamWaitEvent(st, ev(c), 0));
    vm::Params p;
    std::memset(&p, 0, sizeof(p));
    p.code = sg.d_code;
    p.n_code = (int)sg.code.size();
    p.n = cn;
    p.n_tiles = (uint32_t)ntile;
    p.loop_start = (uint32_t)sg.loop_start;
    p.grid = (uint32_t)sg.grid;
    p.n_full_tiles = (uint32_t)(cn / kVmTile);
    p.spill = reinterpret_cast<float*>(ws + sg.spill_off);
    p.colpart = reinterpret_cast<float*>(ws + sg.colpart_off);
    p.scalpart = reinterpret_cast<double*>(ws + sg.scalpart_off) + (size_t)c * sg.n_scalacc * sg.grid;
    p.status = status;
    p.status_clear = c == 0 ? status_next : nullptr;
    for (size_t i = 0; i < sg.operand_mem.size(); ++i) {
      const MemRef& m = P.mems[sg.operand_mem[i]];
      char* q = reinterpret_cast<char*>(m.where == MEM_FEED ? const_cast<void*>(dev_feeds[m.index]) : dev_fetches[m.index]);
      if (sg.operand_kind[i] == vm::K_FULL) q += e0 * (m.dtype == DRAGON_BF16 ? 2 : 4);
      p.operand[i].ptr = q;
      p.operand[i].kind = sg.operand_kind[i];
      p.operand[i].dtype = (uint32_t)m.dtype;
    }
    HOST_TRY(launch_vm(p, sg.grid, sg.n_smem, sg.dense, st, f->tier ? sg.spec_kernel : nullptr));
    HOST_TRY(cudaEventRecord(ev(kHostChunks + c), st));
    HOST_TRY(cudaStreamWaitEvent(s_out, ev(kHostChunks + c), 0));
    for (const MemRef& m : P.mems) {
      if (!m.live || m.where != MEM_FETCH || m.shape.numel() == 1 || done_out[m.index]) continue;
      done_out[m.index] = 1;
      const size_t es = m.dtype == DRAGON_BF16 ? 2 : 4;
      HOST_TRY(cudaMemcpyAsync(reinterpret_cast<char*>(host_fetches[m.index]) + e0 * es,
                               reinterpret_cast<char*>(dev_fetches[m.index]) + e0 * es, (size_t)cn * es, cudaMemcpyDeviceToHost, s_out));
    }
  }
  // sums over the whole domain: the partials of all chunks, then their copy to the host
  std::vector<void*> mem_ptr(P.mems.size(), nullptr);
  for (size_t m = 0; m < P.mems.size(); ++m)
    if (P.mems[m].live && P.mems[m].where == MEM_FETCH) mem_ptr[m] = dev_fetches[P.mems[m].index];
  HOST_TRY(launch_finish(sg, P.mems, mem_ptr.data(), ws, st, kHostChunks));
  std::vector<uint8_t> done_out(f->n_out, 0);
  for (const MemRef& m : P.mems) {
    if (!m.live || m.where != MEM_FETCH || m.shape.numel() != 1 || done_out[m.index]) continue;
    done_out[m.index] = 1;
    HOST_TRY(cudaMemcpyAsync(host_fetches[m.index], dev_fetches[m.index], m.bytes(), cudaMemcpyDeviceToHost, st));
  }
  // the caller's stream ends after the last copy-out
  HOST_TRY(cudaEventRecord(ev_done, s_out));
  HOST_TRY(cudaStreamWaitEvent(st, ev_done, 0));
  f->last_status_word = f->run_parity;
  f->run_parity ^= 1;
  f->last_stream = st;
  return DRAGON_OK;
}

}  // namespace

int dragon_run_host(dragon_function_t* f, const void* const* host_feeds, void* const* host_fetches, void* staging_dev,
                    size_t staging_bytes, void* cuda_stream) {
  if (!f || !host_fetches || (f->n_in > 0 && !host_feeds)) { set_error("dragon_run_host: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  if (!f->not_executable.empty()) { set_error("dragon_run_host: %s", f->not_executable.c_str()); return DRAGON_ERR_UNSUPPORTED; }
  if (!staging_dev || ((uintptr_t)staging_dev & 255) || staging_bytes < dragon_function_staging_bytes(f)) {
    set_error("dragon_run_host: staging area must be 256-byte aligned device memory of at least %zu bytes", dragon_function_staging_bytes(f));
    return DRAGON_ERR_WORKSPACE;
  }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  const bool chunked = chunkable(f) && f->prof_step < 0;
  std::vector<const void*> feeds(f->n_in, nullptr);
  std::vector<void*> fetches(f->n_out, nullptr);
  char* base = reinterpret_cast<char*>(staging_dev);
  size_t off = 0;
  // several memrefs may name the same feed / fetch position: one staging slot per position
  for (const MemRef& m : f->plan.mems) {
    if (!m.live || m.where == MEM_WORK) continue;
    const size_t sz = (m.bytes() + 255) & ~(size_t)255;
    if (m.where == MEM_FEED && !feeds[m.index]) {
      if (!host_feeds[m.index]) { set_error("dragon_run_host: feed %d is NULL", m.index); return DRAGON_ERR_INVALID_ARG; }
      feeds[m.index] = base + off;
      if (!chunked && cudaMemcpyAsync(base + off, host_feeds[m.index], m.bytes(), cudaMemcpyHostToDevice, st) != cudaSuccess) {
        set_error("dragon_run_host: host-to-device copy failed: %s", cudaGetErrorString(cudaGetLastError()));
        return DRAGON_ERR_CUDA;
      }
    } else if (m.where == MEM_FETCH && !fetches[m.index]) {
      if (!host_fetches[m.index]) { set_error("dragon_run_host: fetch %d is NULL", m.index); return DRAGON_ERR_INVALID_ARG; }
      fetches[m.index] = base + off;
    }
    off += sz;
  }
  if (chunked) return run_host_chunked(f, feeds, fetches, host_feeds, host_fetches, st);
  int rc = dragon_run(f, feeds.data(), fetches.data(), cuda_stream);
  if (rc != DRAGON_OK) return rc;
  std::vector<uint8_t> copied(f->n_out, 0);
  for (const MemRef& m : f->plan.mems) {
    if (!m.live || m.where != MEM_FETCH || copied[m.index]) continue;
    copied[m.index] = 1;
    if (cudaMemcpyAsync(host_fetches[m.index], fetches[m.index], m.bytes(), cudaMemcpyDeviceToHost, st) != cudaSuccess) {
      set_error("dragon_run_host: device-to-host copy failed: %s", cudaGetErrorString(cudaGetLastError()));
      return DRAGON_ERR_CUDA;
    }
  }
  return DRAGON_OK;
}

int dragon_function_profile(dragon_function_t* f, int step, int capacity) {
  if (!f || step >= (int)f->plan.steps.size() || (step >= 0 && (capacity <= 0 || capacity > 65536))) {
    set_error("dragon_function_profile: bad argument");
    return DRAGON_ERR_INVALID_ARG;
  }
  f->prof_step = step;
  f->prof_used = 0;
  if (step < 0) return DRAGON_OK;
  while ((int)f->prof_ev.size() < 2 * capacity) {
    cudaEvent_t ev;
    if (cudaEventCreate(&ev) != cudaSuccess) { set_error("dragon_function_profile: cudaEventCreate failed"); return DRAGON_ERR_CUDA; }
    f->prof_ev.push_back(ev);
  }
  return DRAGON_OK;
}

int dragon_function_profile_read(dragon_function_t* f, double* total_ms, int* runs) {
  if (!f || !total_ms || !runs) { set_error("dragon_function_profile_read: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  double tot = 0.0;
  for (int i = 0; i < f->prof_used; ++i) {
    cudaEvent_t a = reinterpret_cast<cudaEvent_t>(f->prof_ev[2 * i]), b = reinterpret_cast<cudaEvent_t>(f->prof_ev[2 * i + 1]);
    float ms = 0.f;
    if (cudaEventSynchronize(b) != cudaSuccess || cudaEventElapsedTime(&ms, a, b) != cudaSuccess) {
      set_error("dragon_function_profile_read: %s", cudaGetErrorString(cudaGetLastError()));
      return DRAGON_ERR_CUDA;
    }
    tot += ms;
  }
  *total_ms = tot;
  *runs = f->prof_used;
  f->prof_used = 0;
  return DRAGON_OK;
}

int dragon_function_status(dragon_function_t* f) {
  if (!f || !f->workspace) { set_error("dragon_function_status: no run yet"); return DRAGON_ERR_INVALID_ARG; }
  int v = 0;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(f->last_stream);
  if (cudaStreamSynchronize(st) != cudaSuccess ||
      cudaMemcpy(&v, reinterpret_cast<char*>(f->workspace) + f->plan.status_off + 64 * f->last_status_word, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) {
    set_error("dragon_function_status: CUDA error: %s", cudaGetErrorString(cudaGetLastError()));
    return DRAGON_ERR_CUDA;
  }
  return v;
}

int dragon_host_math(int fn, const float* x, float* y, int n) {
  if (!x || !y || n < 0) { set_error("dragon_host_math: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  for (int i = 0; i < n; ++i) {
    switch (fn) {
      case DRAGON_OP_SIN: y[i] = vmmath::sin_f(x[i]); break;
      case 100 + DRAGON_OP_SIN: y[i] = vmmath::cos_f(x[i]); break;
      case DRAGON_OP_EXP: y[i] = vmmath::exp_clamped10(x[i]); break;
      case DRAGON_OP_TANH: y[i] = vmmath::tanh_f(x[i]); break;
      case DRAGON_OP_SIGMOID: y[i] = vmmath::sigmoid_f(x[i]); break;
      case DRAGON_OP_DIV: y[i] = vmmath::divp_f(1.f, x[i]); break;
      case DRAGON_OP_SQRT: y[i] = vmmath::sqrt_f(x[i]); break;
      case DRAGON_OP_RECIPROCAL: y[i] = vmmath::f_rcp(x[i]); break;
      default: set_error("dragon_host_math: unknown function %d", fn); return DRAGON_ERR_INVALID_ARG;
    }
  }
  return DRAGON_OK;
}

const char* dragon_last_error(void) { return dragon::last_error(); }

}  // extern "C"
