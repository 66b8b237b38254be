// Instruction set of the graph-VM kernel.  One 32-bit word per instruction:
//   bits 0..9   case id (for register-operand instructions: base + register slot)
//   bits 10..13 reserved
//   bits 14..31 arg (uniform / shared-memory slot / operand / spill index)
// The machine is an accumulator machine: every thread owns V elements of the current tile;
// "acc" and the register slots R[0..NR) are V-wide and live in registers, shared-memory slots
// S[.] are V-wide per thread, uniforms U[.] are one float per CTA.
#pragma once
#include <cstdint>

// geometry of the VM kernel (threads per CTA, elements per thread)
#define DRAGON_VM_THREADS 512
#define DRAGON_VM_VEC 8

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
  J_GLDR,      // R = acc = operand[arg] at this tile
  J_SINCOSR,   // R = cos(acc); acc = sin(acc)
  J_COSSINR,   // R = sin(acc); acc = cos(acc)
  J_MACC0, J_MACC1, J_MACC2, J_MACC3,   // A[i] += sum over this thread's valid lanes of acc * R   (acc unchanged)
  J_LDSWR,     // R = acc = staged operand (P_LDSW)
  J_LDSWAR,    // J_LDSWR, then P_GLDA for the same operand and slot
  // R[a] = acc; acc = R: the most frequent pair of instructions ("put this away, take that") as one,
  // one group per a (the slot index of the case id is the register that is loaded)
  J_STLD0, J_STLD1, J_STLD2, J_STLD3, J_STLD4, J_STLD5, J_STLD6, J_STLD7,
  // two frequent pairs as one instruction each (one dispatch less per tile):
  J_LDSWARF,   // J_LDSWAR (arg bits 0..9: operand | slot << 6), then acc = R * U[u] + U[u + 1], u = arg >> 10
  J_FMAURSTL,  // J_FMAUR with U[arg & 511], then P_GSTFL to operand arg >> 9
  J_STRLDS,    // R = acc; acc = S[arg]   (J_STR, then P_LDS)
  J_COUNT
};
// The kernel exists in two builds that share this encoding: "wide" (7 register slots, one CTA per
// SM) and "dense" (3 register slots, two CTAs per SM, for programs with few live values: twice
// the warps hide the latency of the dispatch).  A case id whose slot a build lacks is never emitted.
constexpr int kJointStride = 8;
constexpr int kVmRegsWide = 7, kVmRegsDense = 3;
constexpr int kVmScalarAccs = 4;             // A[0..4): per-thread scalar accumulators (packed pair of partial sums)
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
  P_COSSIN,             // S[arg] = sin(acc); acc = cos(acc)
  P_EXPC, P_TANH, P_SIGMOID, P_RELU, P_NEG,
  P_STEP,               // acc = acc > 0 ? 1 : 0
  P_CLAMPMASK,          // acc = (-10 <= acc <= 10) ? 1 : 0
  P_ONEMSQ,             // acc = 1 - acc^2
  P_YOMY,               // acc = acc * (1 - acc)
  P_DIVPGB,             // acc = -sgn(acc) / (1 + |acc|)^2
  P_RBF16,              // acc = float(bf16(acc)), round to nearest even
  P_ROWSUM,             // acc = sum of acc over the whole row (all lanes, all threads), row mode only;
                        // arg bits 0..1: scratch buffer (successive row sums differ), bit 2: barrier after the read too
  P_GLD,                // acc = operand[arg] at this tile
  P_GST,                // operand[arg] at this tile = acc
  P_GLDF,               // P_GLD for an fp32 operand of the full domain shape
  P_GSTF,               // P_GST for an fp32 operand of the full domain shape
  P_FILL,               // acc = spill[arg]
  P_SPILL,              // spill[arg] = acc
  P_ULOAD,              // U[arg & 511] = scalar operand[arg >> 9]   (prologue)
  P_UCONST,             // U[arg] = next word reinterpreted as float (prologue)
  P_LOOP_BEGIN,         // start of the per-tile body
  P_LOOP_END,           // next tile; jumps back to the body or falls through to the epilogue
  P_COLOUT,             // column partial sums: colpart[arg][cta][c] = acc
  P_SCALOUT,            // scalar partial sum: scalpart[arg][cta] = block sum of acc in fp64
  P_SACC0, P_SACC1, P_SACC2, P_SACC3,       // A[i] += sum over this thread's valid lanes of acc
  P_ASCAL0, P_ASCAL1, P_ASCAL2, P_ASCAL3,   // scalpart[arg][cta] = block sum of A[i] in fp64
  // Staged loads of an fp32 operand of the full domain shape (arg = operand | slot << 6): every thread
  // copies its own 32 bytes of a tile into S[slot] with asynchronous copies one iteration ahead, so
  // the latency of the global load is spent while the previous tile is computed.  A thread reads only
  // what it copied itself, so no barrier is involved.
  P_GLDA0,              // start the copy of the current tile (before the first iteration; full tiles only)
  P_GLDA,               // start the copy of this CTA's next tile, if it has a whole one
  P_LDSW,               // acc = the current tile: waits for this thread's copies and reads S[slot]
                        // (a ragged tile was not staged and is loaded directly)
  P_LDSWA,              // P_LDSW, then P_GLDA for the same operand and slot (the tile is read once per iteration)
  P_GSTFL,              // P_GSTF followed by P_LOOP_END (a body that ends in a store)
  P_GLDA0H,             // P_GLDA0 for a bf16 operand (8 bytes per thread and half of the tile)
  P_LDSWAH,             // P_LDSWA for a bf16 operand: converts to fp32 at the read; such an operand is read once per iteration
  P_ROWSUMU,            // P_ROWSUM with arg & 7, then acc = acc * U[arg >> 3]   (a row mean)
  P_ACCUMS,             // S[arg] = S[arg] + (lane valid ? acc : 0): a loop-carried accumulator kept in shared memory
                        // (reduced outputs beyond the pinned register slots)
  P_SQRT,               // acc = sqrt(acc)
  P_RCP,                // acc = 1 / acc
  // tanh, sigmoid and clamped exp without their clamps, for arguments that the host's interval analysis has
  // proven inside the range where the clamps do nothing (|x| <= 4.01, |x| <= 80, |x| <= 9.99)
  P_TANHB, P_SIGMOIDB, P_EXPCB,
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

struct Params {             // kernel parameter block; the PTX generator (vm_ptxgen.py) uses the same offsets
  const uint32_t* code;     //  0  device copy of the instruction stream
  float* spill;             //  8  [grid][n_spill][tile]
  float* colpart;           // 16  [n_colacc][grid][cols]
  double* scalpart;         // 24  [n_scalacc][grid]
  int* status;              // 32
  long long n;              // 40  flat: element count; row mode: row count
  int n_code;               // 48
  int row_mode;             // 52  0: flat domain of n elements; 1: rows x cols, one row per tile
  int cols;                 // 56  row mode: row length
  int n_spill;              // 60  spill slots per CTA
  uint32_t n_tiles;         // 64
  uint32_t loop_start;      // 68  index of the first instruction of the per-tile body
  uint32_t grid;            // 72  CTAs launched
  uint32_t n_full_tiles;    // 76  tiles [0, n_full_tiles) hold all kVmTile elements (row mode: rows of exactly kVmTile)
  int* status_clear;        // 80  word that CTA 0 sets to 0 (the status word of the next run), or null
  unsigned long long reserved2;   // 88
  Operand operand[kMaxOperands];   // 96
};
static_assert(sizeof(Operand) == 16 && sizeof(Params) == 96 + 16 * kMaxOperands, "layout shared with the PTX generator");


}  // namespace vm
}  // namespace dragon
