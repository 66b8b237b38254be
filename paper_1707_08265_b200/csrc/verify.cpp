// Static verification of a graph-VM instruction stream.  A program is fixed when dragon_function()
// returns and every index it uses (register slot, shared-memory slot, uniform, memory operand, spill
// slot, accumulator) is a field of an instruction word, so checking each word once on the host gives
// what a range check in every leaf of the kernel would give at run time, at no cost per element.
// codegen runs it on every program it emits; dragon_verify_vm_program() exposes it for tests.
#include <cstdio>

#include "plan.h"
#include "vm_isa.h"

namespace dragon {

namespace {

struct Limits {
  int nr, n_operands, n_smem, n_spill, n_colacc, n_scalacc;
  bool row_mode;
};

bool fail(int pc, const char* what, unsigned got, int limit) {
  set_error("program word %d: %s %u is out of range (limit %d)", pc, what, got, limit);
  return false;
}

// one instruction word; *literal: the next word is data, not an instruction
bool check_word(int pc, uint32_t w, const Limits& L, bool* literal, bool* ends_loop) {
  using namespace vm;
  const int cs = (int)(w & 1023u);
  const uint32_t arg = w >> 14;
  *literal = *ends_loop = false;
  auto U = [&](uint32_t i) { return i < (uint32_t)kMaxUniforms || fail(pc, "uniform", i, kMaxUniforms); };
  auto S = [&](uint32_t i) { return i < (uint32_t)L.n_smem || fail(pc, "shared-memory slot", i, L.n_smem); };
  auto O = [&](uint32_t i) { return i < (uint32_t)L.n_operands || fail(pc, "memory operand", i, L.n_operands); };
  auto X = [&](uint32_t i) { return i < (uint32_t)L.n_spill || fail(pc, "spill slot", i, L.n_spill); };
  if (cs >= P_COUNT_) return fail(pc, "case id", (unsigned)cs, P_COUNT_);
  if (cs < kFirstPlain) {
    const int j = cs / kJointStride, r = cs % kJointStride;
    if (r >= L.nr) return fail(pc, "register slot", (unsigned)r, L.nr);
    if (j >= J_STLD0 && j <= J_STLD7 && j - J_STLD0 >= L.nr) return fail(pc, "register slot", (unsigned)(j - J_STLD0), L.nr);
    switch (j) {
      case J_FMAUR: return U(arg);
      case J_RTOS: case J_STOR: case J_STRLDS: return S(arg);
      case J_SPILL: case J_FILL: return X(arg);
      case J_GLDR: return O(arg);
      case J_LDSWR: case J_LDSWAR: return O(arg & 63u) && S(arg >> 6);
      case J_LDSWARF: return O(arg & 63u) && S((arg >> 6) & 15u) && U((arg >> 10) + 1);
      case J_FMAURSTL: *ends_loop = true; return U(arg & 511u) && O(arg >> 9);
      default: return true;
    }
  }
  switch (cs) {
    case P_LDU: case P_ADDU: case P_SUBU: case P_RSUBU: case P_MULU: case P_DIVPU: case P_RDIVPU: return U(arg);
    case P_FMAU: return U(arg & 511u) && U(arg >> 9);
    case P_LDS: case P_STS: case P_ADDS: case P_SUBS: case P_RSUBS: case P_MULS: case P_DIVPS: case P_RDIVPS:
    case P_SINCOS: case P_COSSIN: case P_ACCUMS: return S(arg);
    case P_ROWSUM:
      if (!L.row_mode) { set_error("program word %d: a row sum in a flat program", pc); return false; }
      return arg < 8u || fail(pc, "row-sum argument", arg, 8);
    case P_ROWSUMU:
      if (!L.row_mode) { set_error("program word %d: a row sum in a flat program", pc); return false; }
      return U(arg >> 3);
    case P_GLD: case P_GST: case P_GLDF: case P_GSTF: return O(arg);
    case P_GSTFL: *ends_loop = true; return O(arg);
    case P_FILL: case P_SPILL: return X(arg);
    case P_ULOAD: return U(arg & 511u) && O(arg >> 9);
    case P_UCONST: *literal = true; return U(arg);
    case P_LOOP_END: *ends_loop = true; return true;
    case P_COLOUT: return arg < (uint32_t)L.n_colacc || fail(pc, "column accumulator", arg, L.n_colacc);
    case P_SCALOUT: case P_ASCAL0: case P_ASCAL1: case P_ASCAL2: case P_ASCAL3:
      return arg < (uint32_t)L.n_scalacc || fail(pc, "scalar accumulator", arg, L.n_scalacc);
    case P_GLDA0: case P_GLDA: case P_LDSW: case P_LDSWA: case P_GLDA0H: case P_LDSWAH: return O(arg & 63u) && S(arg >> 6);
    default: return true;
  }
}

}  // namespace

// Whole program: every word in range, one loop_begin before the per-tile body, the body closed by a
// loop end, the stream closed by P_END, nothing but P_END after it.
int verify_program(const uint32_t* code, int n, int loop_start, int register_slots, int n_operands, int n_smem,
                   int n_spill, int n_colacc, int n_scalacc, bool row_mode) {
  using namespace vm;
  if (!code || n <= 0) { set_error("empty program"); return DRAGON_ERR_INVALID_ARG; }
  if (register_slots != kVmRegsWide && register_slots != kVmRegsDense) { set_error("no kernel build has %d register slots", register_slots); return DRAGON_ERR_INVALID_ARG; }
  if (n_operands < 0 || n_operands > kMaxOperands || n_smem < 0 || n_smem > kVmSmemSlots || n_spill < 0 || n_colacc < 0 || n_scalacc < 0) {
    set_error("program limits out of range");
    return DRAGON_ERR_INVALID_ARG;
  }
  const Limits L = {register_slots, n_operands, n_smem, n_spill, n_colacc, n_scalacc, row_mode};
  int begin_at = -1, end_loop_at = -1;
  bool start_is_instruction = false;
  for (int pc = 0; pc < n; ++pc) {
    bool literal = false, ends_loop = false;
    if (!check_word(pc, code[pc], L, &literal, &ends_loop)) return DRAGON_ERR_INVALID_ARG;
    const int cs = (int)(code[pc] & 1023u);
    if (pc == loop_start) start_is_instruction = true;
    if (cs == P_LOOP_BEGIN) {
      if (begin_at >= 0) { set_error("program word %d: second loop_begin", pc); return DRAGON_ERR_INVALID_ARG; }
      begin_at = pc;
    }
    if (ends_loop) {
      if (end_loop_at >= 0) { set_error("program word %d: second loop end", pc); return DRAGON_ERR_INVALID_ARG; }
      end_loop_at = pc;
    }
    if (cs == P_END) {   // the stream may be padded with further end words, nothing else
      for (int q = pc + 1; q < n; ++q)
        if ((int)(code[q] & 1023u) != P_END) { set_error("program word %d: instructions behind the end", q); return DRAGON_ERR_INVALID_ARG; }
      break;
    }
    if (literal) {
      if (pc + 1 >= n) { set_error("program word %d: uconst without its literal", pc); return DRAGON_ERR_INVALID_ARG; }
      ++pc;
    }
    if (pc == n - 1) { set_error("the program does not end with the end instruction"); return DRAGON_ERR_INVALID_ARG; }
  }
  if (begin_at < 0 || loop_start <= begin_at || loop_start >= n || !start_is_instruction) {
    set_error("the per-tile body (start %d) does not lie behind a loop_begin", loop_start);
    return DRAGON_ERR_INVALID_ARG;
  }
  if (end_loop_at < loop_start) { set_error("the per-tile body is not closed by a loop end"); return DRAGON_ERR_INVALID_ARG; }
  return DRAGON_OK;
}

int verify_segment(const VmSegment& sg) {
  return verify_program(sg.code.data(), (int)sg.code.size(), sg.loop_start, sg.dense ? vm::kVmRegsDense : vm::kVmRegsWide,
                        (int)sg.operand_mem.size(), sg.n_smem, sg.n_spill, sg.n_colacc, sg.n_scalacc, sg.row_mode);
}

}  // namespace dragon
