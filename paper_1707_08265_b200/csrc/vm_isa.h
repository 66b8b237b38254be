// Instruction set of the graph-VM kernel.  One 32-bit word per instruction:
//   bits 0..9   case id (for register-operand instructions: base + register slot)
//   bits 10..13 reserved
//   bits 14..31 arg (uniform / shared-memory slot / operand / spill index)
// The machine is an accumulator machine: every thread owns V elements of the current tile;
// "acc" and the register slots R[0..NR) are V-wide and live in registers, shared-memory slots
// S[.] are V-wide per thread, uniforms U[.] are one float per CTA.
#pragma once
#include <cstdint>

// geometry of the VM kernel (threads per CTA, elements per thread, register slots)
#ifndef DRAGON_VM_REGS
#define DRAGON_VM_REGS 7
#endif
#ifndef DRAGON_VM_THREADS
#define DRAGON_VM_THREADS 512
#define DRAGON_VM_VEC 8
#endif

namespace dragon {
namespace vm {

constexpr int kMaxOperands = 40;   // memory operands per kernel launch
constexpr int kMaxUniforms = 512;

enum Joint : int {  // each occupies kJointStride consecutive case ids, one per register slot
  J_LDR = 0,   // acc = R
  J_STR,       // R = acc
  J_ADD,       // acc = acc + R
  J_SUB,       // acc = acc - R
  J_RSUB,      // acc = R - acc
  J_MUL,       // acc = acc * R
  J_DIVP,      // acc = acc / (1 + |R|)
  J_RDIVP,     // acc = R / (1 + |acc|)
  J_ADDTO,     // R = R + acc
  J_ACCUM,     // R = R + (lane valid ? acc : 0)   (loop-carried accumulators)
  J_FMAUR,     // acc = acc * U[arg] + R
  J_RTOS,      // S[arg] = R
  J_STOR,      // R = S[arg]
  J_SPILL,     // spill[arg] = R
  J_FILL,      // R = spill[arg]
  J_COUNT
};
constexpr int kJointStride = DRAGON_VM_REGS;  // case ids are dense, so the dispatch is one indexed jump
constexpr int kFirstPlain = J_COUNT * kJointStride;

enum Plain : int {
  P_LDU = kFirstPlain,  // acc = U[arg]
  P_ADDU, P_SUBU, P_RSUBU, P_MULU, P_DIVPU, P_RDIVPU,
  P_FMAU,               // acc = acc * U[arg & 511] + U[arg >> 9]
  P_LDS,                // acc = S[arg]
  P_STS,                // S[arg] = acc
  P_ADDS, P_SUBS, P_RSUBS, P_MULS, P_DIVPS, P_RDIVPS,
  P_SIN, P_COS,
  P_SINCOS,             // S[arg] = cos(acc); acc = sin(acc)
  P_EXPC, P_TANH, P_SIGMOID, P_RELU, P_NEG,
  P_STEP,               // acc = acc > 0 ? 1 : 0
  P_CLAMPMASK,          // acc = (-10 <= acc <= 10) ? 1 : 0
  P_ONEMSQ,             // acc = 1 - acc^2
  P_YOMY,               // acc = acc * (1 - acc)
  P_DIVPGB,             // acc = -sgn(acc) / (1 + |acc|)^2
  P_RBF16,              // acc = float(bf16(acc)), round to nearest even
  P_ROWSUM,             // acc = sum of acc over the whole row (all lanes, all threads), row mode only
  P_GLD,                // acc = operand[arg] at this tile
  P_GST,                // operand[arg] at this tile = acc
  P_FILL,               // acc = spill[arg]
  P_SPILL,              // spill[arg] = acc
  P_ULOAD,              // U[arg & 511] = scalar operand[arg >> 9]   (prologue)
  P_UCONST,             // U[arg] = next word reinterpreted as float (prologue)
  P_LOOP_BEGIN,         // start of the per-tile body
  P_LOOP_END,           // next tile; jumps back to the body or falls through to the epilogue
  P_COLOUT,             // column partial sums: colpart[arg][cta][c] = acc
  P_SCALOUT,            // scalar partial sum: scalpart[arg][cta] = block sum of acc in fp64
  P_END,
  P_COUNT_
};

inline uint32_t encode(int case_id, int r, uint32_t arg) {
  return (uint32_t)case_id | ((uint32_t)r << 10) | (arg << 14);
}

enum OperandKind : uint32_t { K_FULL = 0, K_ROW = 1, K_SCALAR = 2 };

struct Operand {        // 16 bytes
  void* ptr;
  uint32_t kind;        // OperandKind
  uint32_t dtype;       // DRAGON_F32 / DRAGON_BF16
};

struct Params {
  const uint32_t* code;     // device copy of the instruction stream
  int n_code;
  int row_mode;             // 0: flat domain of n elements; 1: rows x cols, one row per tile
  long long n;              // flat: element count; row mode: row count
  int cols;                 // row mode: row length
  int n_spill;              // spill slots per CTA
  float* spill;             // [grid][n_spill][tile]
  float* colpart;           // [n_colacc][grid][cols]
  double* scalpart;         // [n_scalacc][grid]
  int* status;
  Operand operand[kMaxOperands];
};

}  // namespace vm
}  // namespace dragon
