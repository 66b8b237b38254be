// Compiled form of a pruned function: a list of launch steps produced by the host compiler
// (lower.cpp builds the micro-operation list from the kept operators, codegen.cpp turns each
// fused segment into a VM instruction stream).
#pragma once
#include <limits>
#include <string>
#include <vector>

#include "graph.h"
#include "vm_isa.h"

namespace dragon {

// geometry of the VM kernel: every CTA owns tiles of kVmTile elements, kVmVec per thread
constexpr int kVmThreads = DRAGON_VM_THREADS;
constexpr int kVmVec = DRAGON_VM_VEC;
constexpr int kVmTile = kVmThreads * kVmVec;  // 4096
constexpr int kVmCodeMaxWords = 8 * 1024;     // instruction stream held in shared memory (8 bytes per word once decoded)
constexpr int kVmSmemSlots = 13;              // V-wide shared-memory slots per thread at most (wide build: one CTA per SM, 227 KB)
constexpr int kVmSmemSlotsLongCode = 9;       // the same when the instruction stream is too long for that many
constexpr int kVmSmemSlotsDense = 6;          // the same for the dense build (two CTAs share the SM's shared memory)
constexpr int kVmReduceBytes = 1024;          // shared memory for the per-warp partials of row sums and block sums
constexpr int kDefaultSmCount = 148;
constexpr int kVmErrTooLarge = -100;          // codegen_segment: the segment exceeds a capacity of one program (operands, stream
                                              // length, uniforms, reduced outputs); the lowering cuts it in two and tries again
constexpr int kHostChunks = 16;               // dragon_run_host pipelines a large elementwise function in this many chunks

enum MemWhere { MEM_FEED = 0, MEM_FETCH = 1, MEM_WORK = 2 };

struct MemRef {
  int where = MEM_WORK;
  int index = -1;        // feed / fetch position; unused for workspace buffers
  int dtype = DRAGON_F32;
  Shape shape;
  size_t offset = 0;     // byte offset inside the workspace (MEM_WORK)
  bool live = false;
  int first_step = -1, last_step = -1;   // plan steps that touch it first and last (MEM_WORK)
  int shares_input = 0;  // 1: written in place over an input of its producing step that dies there (Sec. 2.4)
  size_t bytes() const { return (size_t)shape.numel() * (dtype == DRAGON_BF16 ? 2 : 4); }
};

enum MOpc {
  M_ADD, M_SUB, M_MUL, M_DIVP,
  M_SIN, M_COS, M_EXPC, M_TANH, M_SIGMOID, M_RELU, M_NEG, M_STEP, M_CLAMPMASK, M_ONEMSQ, M_YOMY,
  M_DIVPGB, M_RBF16, M_ROWSUM, M_SQRT, M_RCP,
  M_TANHB, M_SIGMOIDB, M_EXPCB,   // the same functions where the argument is proven inside the range in which the clamps do nothing
  M_WIDEN,  // same value, wider logical shape (no instruction)
  M_STORE,  // write value a to memory mem
  M_ACCUM   // sum value a over the axes along which mem is smaller, write to mem
};
inline bool is_binary(int opc) { return opc <= M_DIVP; }

enum ValKind { VK_MEM, VK_OP, VK_CONST };
struct Value {
  int kind = VK_OP;
  Shape shape;
  int mem = -1;
  float c = 0.f;
  bool known_const = false;  // VK_CONST, or a widened view of one
  bool row_uniform = false;  // the same value in every element of a row: a row sum, a scalar, or an elementwise function of such
  // every element lies in [lo, hi] whatever is fed (NaN aside): interval arithmetic over the micro-operations
  float lo = -std::numeric_limits<float>::infinity(), hi = std::numeric_limits<float>::infinity();
};

// One operation of a product's epilogue program: the running value v of an output element (the fp32
// accumulator) becomes v op x, x a constant, a scalar tensor, a row vector of N elements or a tensor of the
// product's shape, or f(v).  Sub and Div keep the operand order of the graph (R = the value is the second operand).
enum EpiOpc { E_ADD, E_SUB, E_RSUB, E_MUL, E_RELU, E_TANH, E_SIGMOID, E_EXPC, E_SIN, E_NEG, E_SQRT, E_RCP, E_RBF16 };
enum EpiOperand { EO_NONE, EO_CONST, EO_SCALAR, EO_ROW, EO_FULL };
struct EpiSpec {
  int opc = E_ADD, operand = EO_NONE, mem = -1;
  float c = 0.f;
};
constexpr int kMaxEpiOps = 8;

enum ItemKind { IT_MOP, IT_GEMM, IT_TRANSPOSE, IT_SCE_FWD, IT_SCE_BWD, IT_COPY };
struct Item {
  int kind = IT_MOP;
  // IT_MOP
  int opc = 0, a = -1, b = -1, dst = -1, mem = -1;
  // heavy items: memory operands.  GEMM: C = act(A * B^T + D) * step(E) with D an optional row
  // vector, act the identity or max(., 0), E an optional bf16 tensor of C's shape; TRANSPOSE: C = A^T;
  // SCE: A = logits, B = labels, C = out, D = scalar dL (gradient)
  int mA = -1, mB = -1, mC = -1, mD = -1, mE = -1;
  int mF = -1;                             // GEMM, SCE_BWD: row vector that receives the column sums of the tensor written to mC
  float scale = 1.f;                       // SCE_BWD: immediate dL when mD < 0
  bool tA = false, tB = false;             // GEMM: operand given transposed ([K, M] / [K, N] row-major)
  bool relu = false;                       // GEMM: max(., 0) in the epilogue
  std::vector<EpiSpec> epi;                // GEMM: further elementwise operations on the accumulator, in order
  bool live = false;
  int segment = -1;
};

// ---- launch steps -------------------------------------------------------------------------

struct FinishJob {
  int kind;       // 0: column sums of colpart[acc] -> mem; 1: scalar sum of scalpart[acc] -> mem
  int acc;        // accumulator index inside the segment
  int mem;
};

struct VmSegment {
  std::vector<uint32_t> code;
  std::vector<int> operand_mem;     // operand table: memref ids
  std::vector<uint32_t> operand_kind;
  bool row_mode = false;
  bool dense = false;               // kernel build: dense (3 register slots, 2 CTAs per SM) or wide (7, 1)
  long long n = 0;                  // flat: elements; row: rows
  int cols = 0;
  int n_spill = 0, n_colacc = 0, n_scalacc = 0, n_smem = 0;
  int grid = 0;
  size_t spill_off = 0, colpart_off = 0, scalpart_off = 0;  // workspace offsets
  std::vector<FinishJob> finish;
  uint32_t* d_code = nullptr;       // device copy
  int n_instr_body = 0;
  int loop_start = 0;               // index in code of the first instruction of the per-tile body
  // the kernel specialised for this instruction stream (specialize.cpp), made from PTX at the first run
  int spec_state = 0;               // 0 not tried yet, 1 loaded, -1 failed (the interpreter runs the program)
  void* spec_lib = nullptr;         // cudaLibrary_t
  void* spec_kernel = nullptr;      // cudaKernel_t
  std::string spec_log;             // why it failed
};

enum StepKind { ST_VM, ST_GEMM, ST_TRANSPOSE, ST_SCE_FWD, ST_SCE_BWD, ST_COPY };
struct Step {
  int kind;
  int seg = -1;                          // ST_VM
  int mA = -1, mB = -1, mC = -1, mD = -1, mE = -1;   // mE: ST_GEMM epilogue mask (step(E) multiplies the product)
  float scale = 1.f;
  bool tA = false, tB = false;
  bool relu = false;                     // ST_GEMM: epilogue max(., 0); its bias row vector is mD
  std::vector<EpiSpec> epi;              // ST_GEMM: the epilogue program that follows bias / max / mask
  int mF = -1;                           // ST_GEMM / ST_SCE_*: row vector receiving the column sums of the written tensor
  int n_colpart = 0;                     // ... partial rows the kernel writes for it (fixed by the launch shape)
  size_t colpart_off = 0;                // ... and where: float [n_colpart][cols] in the workspace
  size_t scratch_off = 0;                // SCE_FWD: per-row losses
};

struct Plan {
  std::vector<MemRef> mems;
  std::vector<VmSegment> segs;
  std::vector<Step> steps;
  size_t workspace_bytes = 0;
  size_t status_off = 0;
  int sm_count = kDefaultSmCount;
};

int lower_function(const Graph& g, const PruneResult& pr, const std::vector<int>& inputs,
                   const std::vector<int>& outputs, int sm_count, Plan* plan);

// codegen.cpp: instruction stream for the micro-operations items[idx[..]] (all IT_MOP, one domain)
int codegen_segment(const std::vector<Item>& items, const std::vector<int>& idx, const std::vector<Value>& vals,
                    const std::vector<MemRef>& mems, int sm_count, VmSegment* seg);

std::string describe_plan(const Plan& p);

// verify.cpp: static range check of every index an instruction stream uses, and of its structure
int verify_program(const uint32_t* code, int n, int loop_start, int register_slots, int n_operands, int n_smem,
                   int n_spill, int n_colacc, int n_scalacc, bool row_mode);
int verify_segment(const VmSegment& sg);

// specialize.cpp: PTX of the kernel that runs sg's instruction stream as straight-line code
int specialize_ptx(const VmSegment& sg, const char* entry, std::string* ptx);

// per operand of a VM program: position (index into the code) of its last load and of its first store
struct VmAccess { int last_load = -1, first_store = 1 << 30; };
std::vector<VmAccess> vm_operand_accesses(const VmSegment& sg);

}  // namespace dragon

struct dragon_function {
  dragon::PruneResult prune;
  dragon::Plan plan;
  std::vector<int> rename;   // Algorithm 3 on the pruned graph (per tensor id)
  std::string not_executable;   // non-empty: why dragon_run refuses this function (it still answers every prune query)
  int n_tensors = 0, n_in = 0, n_out = 0;
  int tier = 1;              // 1: graph-VM programs run as specialised kernels (made at the first run), 0: interpreted
  std::vector<dragon::TensorInfo> in_info, out_info;   // name, type and shape of every listed input and output
  void* workspace = nullptr;
  size_t workspace_bytes = 0;
  void* last_stream = nullptr;
  bool uploaded = false;
  // two status words used by alternate runs: a run reports into one and clears the other for the
  // run after it, so that no run needs a memset of its own
  bool status_ready = false;
  int run_parity = 0, last_status_word = 0;
  // dragon_run_host, chunked: copy-in and copy-out streams and the events that order them (made on first use)
  void* h_stream[2] = {nullptr, nullptr};
  std::vector<void*> h_event;
  // profiling ring (dragon_function_profile)
  int prof_step = -1, prof_used = 0;
  std::vector<void*> prof_ev;   // 2 * capacity cudaEvent_t
};
