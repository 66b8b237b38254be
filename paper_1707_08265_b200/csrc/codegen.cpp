// Host compiler, part 2: one fused segment of micro-operations -> VM instruction stream.
//
// The VM is an accumulator machine (vm_isa.h).  Values that outlive the accumulator get a
// home: a register slot, then a shared-memory slot, then a per-CTA spill slot in the workspace;
// the victim of an eviction is the value whose next use is farthest away.  Tensors that are
// memory operands can be re-read instead of being kept; scalars and constants live in the
// uniform table.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <map>
#include <string>

#include "plan.h"

namespace dragon {
namespace {

using namespace vm;

enum HomeKind { H_NONE, H_REG, H_SMEM, H_SPILL };
constexpr int kFar = 1 << 30;

struct VInfo {
  std::vector<int> uses;   // positions (index into the segment's item list), ascending
  int home = H_NONE, home_idx = -1;
  int uni = -1;            // uniform-table index (scalars, constants)
  int operand = -1;        // operand-table index (memory tensors that are not scalars)
};

struct Gen {
  const std::vector<Item>& items;
  const std::vector<int>& idx;
  const std::vector<Value>& vals;
  const std::vector<MemRef>& mems;
  VmSegment* seg;
  Shape dom;
  std::vector<int> canon;
  std::map<int, VInfo> info;
  std::vector<uint32_t> pro, preamble, body, epi;
  const int nr;                  // register slots of the kernel build this program is for
  const int n_smem_max;          // shared-memory slots that build can hold
  int reg_owner[kJointStride];   // value id, -1 free, -2 pinned accumulator
  int smem_owner[kVmSmemSlots];
  std::vector<int> free_spill;
  int n_uni = 0;
  int acc_val = -1;
  std::vector<bool> done;        // item already produced by a fused instruction
  std::vector<std::pair<int, int>> accs;  // (item position of an accumulation, its pinned register)
  std::vector<std::pair<int, int>> saccs; // (item position of an accumulation to a scalar, its scalar accumulator)
  std::vector<std::pair<int, int>> maccs; // (item position of an accumulation, its pinned shared-memory slot)
  int err = DRAGON_OK;

  Gen(const std::vector<Item>& it, const std::vector<int>& ix, const std::vector<Value>& v,
      const std::vector<MemRef>& m, VmSegment* s, int n_regs, int n_smem)
      : items(it), idx(ix), vals(v), mems(m), seg(s), nr(n_regs), n_smem_max(n_smem) {}

  int C(int v) const { return v < 0 ? v : canon[v]; }

  int class_of(const Shape& s) const {
    if (s == dom) return K_FULL;
    if (s.numel() == 1) return K_SCALAR;
    if (dom.rank == 2 && s.rows() == 1 && s.cols() == dom.cols()) return K_ROW;
    return -1;
  }
  int operand_for(int mem, int kind) {
    for (size_t i = 0; i < seg->operand_mem.size(); ++i)
      if (seg->operand_mem[i] == mem && seg->operand_kind[i] == (uint32_t)kind) return (int)i;
    seg->operand_mem.push_back(mem);
    seg->operand_kind.push_back((uint32_t)kind);
    return (int)seg->operand_mem.size() - 1;
  }
  int next_use(int v, int pos) const {  // first use strictly after pos
    auto it = info.find(v);
    if (it == info.end()) return kFar;
    auto u = std::upper_bound(it->second.uses.begin(), it->second.uses.end(), pos);
    return u == it->second.uses.end() ? kFar : *u;
  }
  bool is_input(int v) const { auto it = info.find(v); return it != info.end() && it->second.operand >= 0; }
  bool addressable(int v) { VInfo& f = info[v]; return f.uni >= 0 || f.home == H_REG || f.home == H_SMEM; }

  void emit(int c, int r = 0, uint32_t arg = 0) { body.push_back(encode(c, r, arg)); }
  void emit_str(int k) { emit(J_STR * kJointStride + k); }
  // the accumulation at item position q of the value in the accumulator
  bool emit_accum(int q) {
    for (auto& a : accs) if (a.first == q) { emit(J_ACCUM * kJointStride + a.second); return true; }
    for (auto& a : saccs) if (a.first == q) { emit(P_SACC0 + a.second); return true; }
    for (auto& a : maccs) if (a.first == q) { emit(P_ACCUMS, 0, (uint32_t)a.second); return true; }
    return false;
  }
  int scalar_acc_at(int q) const {
    for (auto& a : saccs) if (a.first == q) return a.second;
    return -1;
  }

  void release(int v) {
    VInfo& f = info[v];
    if (f.home == H_REG) reg_owner[f.home_idx] = -1;
    else if (f.home == H_SMEM) smem_owner[f.home_idx] = -1;
    else if (f.home == H_SPILL) free_spill.push_back(f.home_idx);
    f.home = H_NONE;
  }
  void release_dead(int v, int pos) {
    if (v >= 0 && next_use(v, pos) == kFar) {
      release(v);
      if (acc_val == v) acc_val = -1;
    }
  }
  int new_spill() {
    if (!free_spill.empty()) { int g = free_spill.back(); free_spill.pop_back(); return g; }
    return seg->n_spill++;
  }
  int free_smem() {
    for (int s = 0; s < n_smem_max; ++s)
      if (smem_owner[s] == -1) { seg->n_smem = std::max(seg->n_smem, s + 1); return s; }
    return -1;
  }
  int free_reg() const {
    for (int k = 0; k < nr; ++k)
      if (reg_owner[k] == -1) return k;
    return -1;
  }
  // a free register slot; may evict the resident value whose next use is farthest
  int alloc_reg(int pos, int keep1 = -1, int keep2 = -1) {
    int k0 = free_reg();
    if (k0 >= 0) return k0;
    int best = -1, best_use = -1;
    for (int k = 0; k < nr; ++k) {
      int v = reg_owner[k];
      if (v < 0 || v == keep1 || v == keep2) continue;
      int u = next_use(v, pos - 1);
      if (is_input(v)) u = kFar - 1;  // a cached memory operand is dropped for free
      if (u > best_use) { best_use = u; best = k; }
    }
    if (best < 0) { err = kVmErrTooLarge; set_error("graph VM: out of register slots"); return 0; }
    int v = reg_owner[best];
    VInfo& f = info[v];
    if (is_input(v)) {
      f.home = H_NONE;
    } else {
      int s = free_smem();
      if (s >= 0) { emit(J_RTOS * kJointStride + best, 0, s); f.home = H_SMEM; f.home_idx = s; smem_owner[s] = v; }
      else { int gsl = new_spill(); emit(J_SPILL * kJointStride + best, 0, gsl); f.home = H_SPILL; f.home_idx = gsl; }
    }
    reg_owner[best] = -1;
    return best;
  }
  void give_reg(int v, int k) { VInfo& f = info[v]; f.home = H_REG; f.home_idx = k; reg_owner[k] = v; }

  // the accumulator is about to be overwritten: keep its value if it is used after position pos
  void save_acc(int pos, int keep1 = -1, int keep2 = -1) {
    int v = acc_val;
    if (v < 0) return;
    VInfo& f = info[v];
    if (f.uni >= 0 || f.home != H_NONE) return;
    int nu = next_use(v, pos);
    if (nu == kFar) return;
    const bool have_free = free_reg() >= 0;
    if (is_input(v) && !have_free) return;  // re-read later
    if (!have_free) {
      // if every register holds something needed sooner, the accumulator itself goes down a level
      int farthest = -1;
      for (int k = 0; k < nr; ++k) {
        int w = reg_owner[k];
        if (w < 0 || w == keep1 || w == keep2) continue;
        farthest = std::max(farthest, is_input(w) ? kFar - 1 : next_use(w, pos));
      }
      if (farthest >= 0 && farthest <= nu) {
        int s = free_smem();
        if (s >= 0) { emit(P_STS, 0, s); f.home = H_SMEM; f.home_idx = s; smem_owner[s] = v; }
        else { int gsl = new_spill(); emit(P_SPILL, 0, gsl); f.home = H_SPILL; f.home_idx = gsl; }
        return;
      }
    }
    int k = alloc_reg(pos + 1, keep1, keep2);
    emit_str(k);
    give_reg(v, k);
  }
  void load_acc(int v, int pos, int keep1 = -1, int keep2 = -1) {
    if (acc_val == v) return;
    save_acc(pos - 1, keep1, keep2);
    VInfo& f = info[v];
    if (f.uni >= 0) emit(P_LDU, 0, f.uni);
    else if (f.home == H_REG) emit(J_LDR * kJointStride + f.home_idx);
    else if (f.home == H_SMEM) emit(P_LDS, 0, f.home_idx);
    else if (f.home == H_SPILL) emit(P_FILL, 0, f.home_idx);
    else if (f.operand >= 0) emit(P_GLD, 0, f.operand);
    else { err = DRAGON_ERR_UNSUPPORTED; set_error("graph VM: value has no location"); }
    acc_val = v;
  }
  // a spilled value comes back into a register slot without touching the accumulator
  bool fill_to_reg(int v, int pos, int keep1, int keep2) {
    VInfo& f = info[v];
    if (f.home != H_SPILL) return false;
    int k = alloc_reg(pos, keep1, keep2);
    emit(J_FILL * kJointStride + k, 0, f.home_idx);
    free_spill.push_back(f.home_idx);
    give_reg(v, k);
    return true;
  }
  // acc holds v: give it a register home now
  void home_acc(int v, int pos, int keep1, int keep2) {
    int k = alloc_reg(pos, keep1, keep2);
    emit_str(k);
    give_reg(v, k);
  }
  // acc holds x and is about to be overwritten by a result: give x a home if it is needed again
  // (a memory operand only while a register slot is free; it can be re-read otherwise)
  void keep_operand(int x, int pos, int other) {
    if (next_use(x, pos) == kFar || addressable(x) || info[x].home != H_NONE) return;
    if (!is_input(x)) {
      int k = alloc_reg(pos, x, other);
      emit_str(k);
      give_reg(x, k);
      return;
    }
    int k = free_reg();
    if (k >= 0) { emit_str(k); give_reg(x, k); }
  }

  // scalar accumulator that takes the product d = acc * y directly, or -1: d's only use must be a
  // sum over the whole domain and y must sit in a register slot
  int macc_target(const Item& it, int d, int y) {
    if (it.opc != M_MUL) return -1;
    const VInfo& fy = info[y];
    if (fy.uni >= 0 || fy.home != H_REG || info[d].uses.size() != 1) return -1;
    const int q = info[d].uses[0];
    const Item& o2 = items[idx[q]];
    return (!done[q] && o2.opc == M_ACCUM && C(o2.a) == d) ? scalar_acc_at(q) : -1;
  }

  void binary(const Item& it, int pos) {
    static const int jop[4] = {J_ADD, J_SUB, J_MUL, J_DIVP}, jrev[4] = {J_ADD, J_RSUB, J_MUL, J_RDIVP};
    static const int uop[4] = {P_ADDU, P_SUBU, P_MULU, P_DIVPU}, urev[4] = {P_ADDU, P_RSUBU, P_MULU, P_RDIVPU};
    static const int sop[4] = {P_ADDS, P_SUBS, P_MULS, P_DIVPS}, srev[4] = {P_ADDS, P_RSUBS, P_MULS, P_RDIVPS};
    const int a = C(it.a), b = C(it.b), d = C(it.dst);
    int x, y;  // x goes through the accumulator, y is addressed
    if (a == b) { x = a; y = a; }
    else if (acc_val == a) { x = a; y = b; }
    else if (acc_val == b) { x = b; y = a; }
    else {
      bool aa = addressable(a), ab = addressable(b);
      if (aa && !ab) { x = b; y = a; }
      else if (ab && !aa) { x = a; y = b; }
      else if (aa && ab) {
        // a uniform stays the addressed operand (multiply-by-uniform then add fuses later);
        // otherwise keep the one that is needed again where it is
        bool a_dies = next_use(a, pos) == kFar, b_dies = next_use(b, pos) == kFar;
        if (info[a].uni >= 0 && info[b].uni < 0) { x = b; y = a; }
        else if (info[b].uni >= 0 && info[a].uni < 0) { x = a; y = b; }
        else if (b_dies && !a_dies) { x = b; y = a; } else { x = a; y = b; }
      } else { x = a; y = b; }
    }
    if (a == b) {
      load_acc(x, pos, x);
      if (!addressable(x)) home_acc(x, pos, x, -1);
    } else {
      if (!addressable(y)) fill_to_reg(y, pos, x, y);
      if (!addressable(y)) {
        // y is a memory operand: it has to pass through the accumulator, so the roles swap
        if (acc_val == x) {
          if (!addressable(x)) home_acc(x, pos, x, y);
        } else if (!addressable(x) && !fill_to_reg(x, pos, x, y)) {
          load_acc(x, pos, x, y);
          home_acc(x, pos, x, y);
        }
        std::swap(x, y);
      }
      load_acc(x, pos, x, y);
      if (macc_target(it, d, y) < 0) keep_operand(x, pos, y);   // a fused multiply-accumulate leaves x in the accumulator
    }
    const bool rev = (x == b && a != b);
    const int o = it.opc - M_ADD;
    VInfo& fy = info[y];
    // a product whose only use is a sum over the whole domain goes straight into the scalar
    // accumulator; the accumulator register keeps x
    {
      const int sa = macc_target(it, d, y);
      if (sa >= 0) {
        const int q = info[d].uses[0];
        emit((J_MACC0 + sa) * kJointStride + fy.home_idx);
        done[q] = true;
        info[d].uses.clear();
        acc_val = x;
        release_dead(a, pos);
        if (b != a) release_dead(b, pos);
        return;
      }
    }
    if (fy.uni >= 0) emit(rev ? urev[o] : uop[o], 0, fy.uni);
    else if (fy.home == H_REG) emit((rev ? jrev[o] : jop[o]) * kJointStride + fy.home_idx);
    else emit(rev ? srev[o] : sop[o], 0, fy.home_idx);
    acc_val = d;
    release_dead(a, pos);
    if (b != a) release_dead(b, pos);
  }

  void unary(const Item& it, int pos) {
    static const std::map<int, int> op = {{M_SIN, P_SIN}, {M_COS, P_COS}, {M_EXPC, P_EXPC}, {M_TANH, P_TANH},
      {M_SIGMOID, P_SIGMOID}, {M_RELU, P_RELU}, {M_NEG, P_NEG}, {M_STEP, P_STEP}, {M_CLAMPMASK, P_CLAMPMASK},
      {M_ONEMSQ, P_ONEMSQ}, {M_YOMY, P_YOMY}, {M_DIVPGB, P_DIVPGB}, {M_RBF16, P_RBF16}, {M_ROWSUM, P_ROWSUM},
      {M_SQRT, P_SQRT}, {M_RCP, P_RCP}, {M_TANHB, P_TANHB}, {M_SIGMOIDB, P_SIGMOIDB}, {M_EXPCB, P_EXPCB}};
    const int a = C(it.a), d = C(it.dst);
    load_acc(a, pos, a);
    // sin and cos of the same value share one range reduction
    if (it.opc == M_SIN || it.opc == M_COS) {
      for (int q = pos + 1; q < (int)idx.size() && q < pos + 4096; ++q) {
        const Item& o2 = items[idx[q]];
        if (done[q] || o2.kind != IT_MOP || (o2.opc != M_SIN && o2.opc != M_COS) || o2.opc == it.opc || C(o2.a) != a) continue;
        int dsin = it.opc == M_SIN ? d : C(o2.dst), dcos = it.opc == M_SIN ? C(o2.dst) : d;
        auto& ua = info[a].uses;  // the partner's use of a is consumed here
        ua.erase(std::remove(ua.begin(), ua.end(), q), ua.end());
        keep_operand(a, pos, -1);
        // the one needed first stays in the accumulator, the other goes to a register slot (a
        // shared-memory slot when none is free)
        const bool cos_first = next_use(dcos, pos) < next_use(dsin, pos);
        const int dacc = cos_first ? dcos : dsin, dother = cos_first ? dsin : dcos;
        const int k = free_reg();
        if (k >= 0) {
          emit((cos_first ? J_COSSINR : J_SINCOSR) * kJointStride + k);
          give_reg(dother, k);
        } else {
          int sl = free_smem();
          if (sl < 0) { ua.push_back(q); std::sort(ua.begin(), ua.end()); break; }  // two separate instructions
          smem_owner[sl] = dother;
          emit(cos_first ? P_COSSIN : P_SINCOS, 0, sl);
          info[dother].home = H_SMEM; info[dother].home_idx = sl;
        }
        acc_val = dacc;
        done[q] = true;
        release_dead(a, pos);
        if (next_use(dother, pos) == kFar) release(dother);
        if (next_use(dacc, pos) == kFar) acc_val = -1;
        return;
      }
    }
    keep_operand(a, pos, -1);
    emit(op.at(it.opc));
    acc_val = d;
    release_dead(a, pos);
  }

  // the accumulator holds a fresh value: stores and accumulations of it that come later in the
  // list are issued right away (they depend on nothing else), which saves a store/reload pair
  void drain_acc(int pos) {
    const int v = acc_val;
    if (v < 0) return;
    for (int q = pos + 1; q < (int)idx.size() && q < pos + 4096; ++q) {
      const Item& o2 = items[idx[q]];
      if (done[q] || (o2.opc != M_STORE && o2.opc != M_ACCUM) || C(o2.a) != v) continue;
      if (o2.opc == M_STORE) {
        int cls = class_of(mems[o2.mem].shape);
        if (cls < 0) continue;
        emit(P_GST, 0, operand_for(o2.mem, cls));
      } else if (!emit_accum(q)) {
        continue;
      }
      done[q] = true;
      auto& u = info[v].uses;
      u.erase(std::remove(u.begin(), u.end(), q), u.end());
    }
    if (next_use(v, pos) == kFar) { release(v); acc_val = -1; }
  }

  // Loads of fp32 tensors of the full domain shape are staged through free shared-memory slots:
  // the copy of a tile starts one iteration ahead (P_GLDA after the slot's last read, P_GLDA0
  // before the first iteration) and the read (P_LDSW / J_LDSWR) finds it on chip.
  void stage_loads() {
    const char* off = std::getenv("DRAGON_VM_STAGING");
    if (off && std::string(off) == "0") return;
    auto load_operand = [&](uint32_t w, int* k) -> int {   // operand of a short fp32 load, or -1
      const uint32_t cs = w & 1023u;
      *k = -1;
      if (cs == (uint32_t)P_GLDF) return (int)(w >> 14);
      if (cs >= (uint32_t)(J_GLDR * kJointStride) && cs < (uint32_t)(J_GLDR * kJointStride + nr)) { *k = (int)(cs - J_GLDR * kJointStride); return (int)(w >> 14); }
      return -1;
    };
    std::map<int, int> slot_of;                 // operand -> staging slot
    std::map<int, size_t> last_read;            // operand -> position of its last load in the body
    for (size_t i = 0; i < body.size(); ++i) {
      int k, opd = load_operand(body[i], &k);
      if (opd < 0 || opd >= 64) continue;
      if (!slot_of.count(opd)) {
        if (seg->n_smem >= n_smem_max) continue;  // no free slot: this operand keeps its direct loads
        slot_of[opd] = seg->n_smem++;
      }
      last_read[opd] = i;
    }
    std::vector<uint32_t> out;
    std::map<int, bool> seen;
    for (size_t i = 0; i < body.size(); ++i) {
      int k, opd = load_operand(body[i], &k);
      if (opd < 0 || !slot_of.count(opd)) { out.push_back(body[i]); continue; }
      const uint32_t sl = (uint32_t)slot_of[opd], arg = (uint32_t)opd | (sl << 6);
      if (!seen[opd]) {                          // first read of the iteration: wait for the copy
        if (last_read[opd] == i) {               // the only read: the next copy starts in the same instruction
          out.push_back(k < 0 ? encode(P_LDSWA, 0, arg) : encode(J_LDSWAR * kJointStride + k, 0, arg));
          seen[opd] = true;
          continue;
        }
        out.push_back(k < 0 ? encode(P_LDSW, 0, arg) : encode(J_LDSWR * kJointStride + k, 0, arg));
        seen[opd] = true;
      } else {                                   // the slot still holds the tile
        out.push_back(encode(P_LDS, 0, sl));
        if (k >= 0) out.push_back(encode(J_STR * kJointStride + k, 0, 0));
      }
      if (last_read[opd] == i) out.push_back(encode(P_GLDA, 0, arg));
    }
    body.swap(out);
    for (auto& so : slot_of) preamble.push_back(encode(P_GLDA0, 0, (uint32_t)so.first | ((uint32_t)so.second << 6)));
    // bf16 operands of the full domain shape that the body reads exactly once
    std::map<int, int> reads;
    for (uint32_t w : body)
      if ((w & 1023u) == (uint32_t)P_GLD) ++reads[(int)(w >> 14)];
    for (uint32_t& w : body) {
      const int opd = (int)(w >> 14);
      if ((w & 1023u) != (uint32_t)P_GLD || opd >= 64 || reads[opd] != 1) continue;
      if (seg->operand_kind[opd] != (uint32_t)K_FULL || mems[seg->operand_mem[opd]].dtype != DRAGON_BF16) continue;
      if (seg->n_smem >= n_smem_max) break;
      const uint32_t arg = (uint32_t)opd | ((uint32_t)seg->n_smem++ << 6);
      w = encode(P_LDSWAH, 0, arg);
      preamble.push_back(encode(P_GLDA0H, 0, arg));
    }
  }

  int run() {
    // 1. aliases (WIDEN) and the fused domain
    canon.resize(vals.size());
    for (size_t v = 0; v < vals.size(); ++v) canon[v] = (int)v;
    bool has_dom = false, any_rowsum = false;
    auto join = [&](const Shape& s) {
      if (!has_dom) { dom = s; has_dom = true; return; }
      Shape o;
      if (broadcast_shapes(dom, s, &o)) dom = o;
    };
    for (int i : idx) {
      const Item& it = items[i];
      if (it.opc == M_WIDEN) canon[it.dst] = canon[it.a];
      if (it.opc == M_STORE || it.opc == M_ACCUM) join(vals[it.a].shape);
      else join(vals[it.dst].shape);
      any_rowsum |= it.opc == M_ROWSUM;
    }
    // 2. uses and static locations
    std::fill(reg_owner, reg_owner + kJointStride, -1);
    std::fill(smem_owner, smem_owner + kVmSmemSlots, -1);
    bool any_row_class = false;
    auto note = [&](int v, int pos) {
      if (v < 0) return;
      v = C(v);
      VInfo& f = info[v];
      f.uses.push_back(pos);
      const Value& val = vals[v];
      if (val.kind == VK_CONST && f.uni < 0) {
        f.uni = n_uni++;
        pro.push_back(encode(P_UCONST, 0, f.uni));
        uint32_t bits; std::memcpy(&bits, &val.c, 4);
        pro.push_back(bits);
      } else if (val.kind == VK_MEM && f.uni < 0 && f.operand < 0) {
        int cls = class_of(mems[val.mem].shape);
        if (cls < 0) { err = DRAGON_ERR_UNSUPPORTED; set_error("graph VM: operand shape does not fit the fused domain"); return; }
        if (cls == K_SCALAR) {
          f.uni = n_uni++;
          pro.push_back(encode(P_ULOAD, 0, (uint32_t)f.uni | ((uint32_t)operand_for(val.mem, K_SCALAR) << 9)));
        } else {
          f.operand = operand_for(val.mem, cls);
          any_row_class |= cls == K_ROW;
        }
      }
    };
    for (int p = 0; p < (int)idx.size(); ++p) {
      const Item& it = items[idx[p]];
      if (it.opc == M_WIDEN) continue;
      note(it.a, p);
      note(it.b, p);
      if ((it.opc == M_STORE || it.opc == M_ACCUM) && class_of(mems[it.mem].shape) == K_ROW) any_row_class = true;
    }
    if (err) return err;
    if (n_uni > 511) { set_error("graph VM: too many scalars and constants"); return kVmErrTooLarge; }
    seg->row_mode = any_rowsum || any_row_class;
    if (seg->row_mode) {
      seg->n = dom.rows();
      seg->cols = (int)dom.cols();
      if (dom.cols() > kVmTile) { set_error("graph VM: rows longer than %d elements are not supported", kVmTile); return DRAGON_ERR_UNSUPPORTED; }
    } else {
      seg->n = dom.numel();
      seg->cols = 0;
    }
    // 3. accumulators get pinned registers
    for (int p = 0; p < (int)idx.size(); ++p)
      if (items[idx[p]].opc == M_ACCUM) {
        // a sum over the whole domain needs one running value per thread; a column sum one per lane
        if (class_of(mems[items[idx[p]].mem].shape) == K_SCALAR && (int)saccs.size() < kVmScalarAccs) {
          saccs.emplace_back(p, (int)saccs.size());
          continue;
        }
        int k = (int)accs.size();
        if (k >= nr - 2) {
          // no register slot left to pin: the running sum lives in a shared-memory slot (two slots stay free for values)
          int sl = (int)maccs.size() + 2 < n_smem_max ? free_smem() : -1;
          if (sl < 0) { set_error("graph VM: too many reduced outputs in one segment"); return kVmErrTooLarge; }
          smem_owner[sl] = -2;
          maccs.emplace_back(p, sl);
          continue;
        }
        reg_owner[k] = -2;
        accs.emplace_back(p, k);
      }
    if (!maccs.empty()) {   // those slots start at zero
      const float zero = 0.f;
      const int uz = n_uni++;
      pro.push_back(encode(P_UCONST, 0, uz));
      uint32_t bits; std::memcpy(&bits, &zero, 4);
      pro.push_back(bits);
      preamble.push_back(encode(P_LDU, 0, uz));
      for (auto& a : maccs) preamble.push_back(encode(P_STS, 0, (uint32_t)a.second));
      if (n_uni > 511) { set_error("graph VM: too many scalars and constants"); return kVmErrTooLarge; }
    }
    // 4. body
    done.assign(idx.size(), false);
    for (int p = 0; p < (int)idx.size() && !err; ++p) {
      if (done[p]) continue;
      const Item& it = items[idx[p]];
      if (it.opc == M_WIDEN) continue;
      if (is_binary(it.opc)) { binary(it, p); drain_acc(p); }
      else if (it.opc == M_STORE) {
        int v = C(it.a);
        int cls = class_of(mems[it.mem].shape);
        if (cls < 0) { set_error("graph VM: store shape does not fit the fused domain"); return DRAGON_ERR_UNSUPPORTED; }
        int opd = operand_for(it.mem, cls);
        load_acc(v, p, v);
        emit(P_GST, 0, opd);
        release_dead(v, p);
      } else if (it.opc == M_ACCUM) {
        int v = C(it.a);
        load_acc(v, p, v);
        emit_accum(p);
        release_dead(v, p);
      } else { unary(it, p); drain_acc(p); }
    }
    if (err) return err;
    // 5. peephole: multiply by a uniform followed by an add fuses into one instruction
    std::vector<uint32_t> fused;
    for (size_t i = 0; i < body.size(); ++i) {
      uint32_t w = body[i];
      if ((w & 1023u) == (uint32_t)P_MULU && i + 1 < body.size()) {
        uint32_t nx = body[i + 1], ncase = nx & 1023u, ui = w >> 14;
        if (ncase == (uint32_t)P_ADDU && ui < 512 && (nx >> 14) < 512) { fused.push_back(encode(P_FMAU, 0, ui | ((nx >> 14) << 9))); ++i; continue; }
        if (ncase >= (uint32_t)(J_ADD * kJointStride) && ncase < (uint32_t)(J_ADD * kJointStride + nr)) {
          fused.push_back(encode(J_FMAUR * kJointStride + (int)(ncase - J_ADD * kJointStride), 0, ui)); ++i; continue;
        }
      }
      fused.push_back(w);
    }
    body.swap(fused);
    fused.clear();
    // loads and stores of fp32 tensors of the full domain shape have their own, shorter instructions
    auto plain_f32 = [&](uint32_t opd) {
      return seg->operand_kind[opd] == (uint32_t)K_FULL && mems[seg->operand_mem[opd]].dtype == DRAGON_F32;
    };
    for (uint32_t& w : body) {
      if ((w & 1023u) == (uint32_t)P_GLD && plain_f32(w >> 14)) w = encode(P_GLDF, 0, w >> 14);
      else if ((w & 1023u) == (uint32_t)P_GST && plain_f32(w >> 14)) w = encode(P_GSTF, 0, w >> 14);
    }
    for (size_t i = 0; i < body.size(); ++i) {   // a load that is kept in a register slot is one instruction
      const uint32_t w = body[i], nx = i + 1 < body.size() ? body[i + 1] : 0u, ncase = nx & 1023u;
      if ((w & 1023u) == (uint32_t)P_GLDF && i + 1 < body.size() && ncase >= (uint32_t)(J_STR * kJointStride) && ncase < (uint32_t)(J_STR * kJointStride + nr)) {
        fused.push_back(encode(J_GLDR * kJointStride + (int)(ncase - J_STR * kJointStride), 0, w >> 14));
        ++i;
        continue;
      }
      fused.push_back(w);
    }
    body.swap(fused);
    fused.clear();
    for (size_t i = 0; i < body.size(); ++i) {   // "R[a] = acc; acc = R[b]" is one instruction
      const uint32_t c0 = body[i] & 1023u, c1 = i + 1 < body.size() ? (body[i + 1] & 1023u) : ~0u;
      if (c0 >= (uint32_t)(J_STR * kJointStride) && c0 < (uint32_t)(J_STR * kJointStride + nr) &&
          c1 < (uint32_t)(J_LDR * kJointStride + nr)) {   // J_LDR is the first group: case ids [0, nr)
        const int a = (int)(c0 - J_STR * kJointStride), b = (int)(c1 - J_LDR * kJointStride);
        if (a != b) { fused.push_back(encode((J_STLD0 + a) * kJointStride + b, 0, 0)); ++i; continue; }
      }
      fused.push_back(body[i]);
    }
    body.swap(fused);
    {   // row sums alternate between scratch buffers so that each needs one barrier only; successive
        // ones (the last of an iteration and the first of the next included) never share a buffer
      std::vector<size_t> rs;
      for (size_t i = 0; i < body.size(); ++i)
        if ((body[i] & 1023u) == (uint32_t)P_ROWSUM) rs.push_back(i);
      for (size_t j = 0; j < rs.size(); ++j) {
        uint32_t arg = (uint32_t)(j & 1);
        if (rs.size() == 1) arg = 4;                                   // alone in the body: barrier after the read too
        else if ((rs.size() & 1) && j + 1 == rs.size()) arg = 2;        // odd count: the last one takes a third buffer
        body[rs[j]] = encode(P_ROWSUM, 0, arg);
      }
    }
    stage_loads();
    {   // a staged load kept in a register slot followed by an affine map with adjacent uniforms
      std::vector<uint32_t> out;
      for (size_t i = 0; i < body.size(); ++i) {
        const uint32_t w = body[i], cs = w & 1023u, nx = i + 1 < body.size() ? body[i + 1] : 0u;
        if (cs >= (uint32_t)(J_LDSWAR * kJointStride) && cs < (uint32_t)(J_LDSWAR * kJointStride + nr) && i + 1 < body.size() &&
            (nx & 1023u) == (uint32_t)P_FMAU) {
          const uint32_t ui = (nx >> 14) & 511u, uj = nx >> 23, a = w >> 14;
          if (uj == ui + 1 && ui < 256 && a < 1024) {
            out.push_back(encode(J_LDSWARF * kJointStride + (int)(cs - J_LDSWAR * kJointStride), 0, a | (ui << 10)));
            ++i;
            continue;
          }
        }
        out.push_back(w);
      }
      body.swap(out);
    }
    {   // "R = acc; acc = S[slot]" and "row sum, times a uniform" (a mean) are one instruction each
      std::vector<uint32_t> out;
      for (size_t i = 0; i < body.size(); ++i) {
        const uint32_t w = body[i], cs = w & 1023u, nx = i + 1 < body.size() ? body[i + 1] : 0u, nc = nx & 1023u;
        if (i + 1 < body.size() && cs >= (uint32_t)(J_STR * kJointStride) && cs < (uint32_t)(J_STR * kJointStride + nr) && nc == (uint32_t)P_LDS) {
          out.push_back(encode(J_STRLDS * kJointStride + (int)(cs - J_STR * kJointStride), 0, nx >> 14));
          ++i;
        } else if (i + 1 < body.size() && cs == (uint32_t)P_ROWSUM && nc == (uint32_t)P_MULU && (nx >> 14) < 512) {
          out.push_back(encode(P_ROWSUMU, 0, ((w >> 14) & 7u) | ((nx >> 14) << 3)));
          ++i;
        } else {
          out.push_back(w);
        }
      }
      body.swap(out);
    }
    // 6. epilogue: accumulators leave as per-CTA partial sums
    for (auto& a : accs) {
      const Item& it = items[idx[a.first]];
      int cls = class_of(mems[it.mem].shape);
      FinishJob job; job.mem = it.mem;
      epi.push_back(encode(J_LDR * kJointStride + a.second, 0, 0));
      if (cls == K_SCALAR) { job.kind = 1; job.acc = seg->n_scalacc++; epi.push_back(encode(P_SCALOUT, 0, job.acc)); }
      else if (cls == K_ROW) { job.kind = 0; job.acc = seg->n_colacc++; epi.push_back(encode(P_COLOUT, 0, job.acc)); }
      else { set_error("graph VM: reduction target shape is not supported"); return DRAGON_ERR_UNSUPPORTED; }
      seg->finish.push_back(job);
    }
    for (auto& a : maccs) {
      const Item& it = items[idx[a.first]];
      int cls = class_of(mems[it.mem].shape);
      FinishJob job; job.mem = it.mem;
      epi.push_back(encode(P_LDS, 0, (uint32_t)a.second));
      if (cls == K_SCALAR) { job.kind = 1; job.acc = seg->n_scalacc++; epi.push_back(encode(P_SCALOUT, 0, job.acc)); }
      else if (cls == K_ROW) { job.kind = 0; job.acc = seg->n_colacc++; epi.push_back(encode(P_COLOUT, 0, job.acc)); }
      else { set_error("graph VM: reduction target shape is not supported"); return DRAGON_ERR_UNSUPPORTED; }
      seg->finish.push_back(job);
    }
    for (auto& a : saccs) {
      const Item& it = items[idx[a.first]];
      FinishJob job; job.mem = it.mem; job.kind = 1; job.acc = seg->n_scalacc++;
      epi.push_back(encode(P_ASCAL0 + a.second, 0, job.acc));
      seg->finish.push_back(job);
    }
    seg->code = pro;
    seg->code.push_back(encode(P_LOOP_BEGIN, 0, 0));
    seg->code.insert(seg->code.end(), preamble.begin(), preamble.end());
    seg->loop_start = (int)seg->code.size();
    seg->code.insert(seg->code.end(), body.begin(), body.end());
    if (!body.empty() && (body.back() & 1023u) == (uint32_t)P_GSTF) {   // store and loop end in one instruction
      const uint32_t opd = body.back() >> 14, pv = body.size() > 1 ? body[body.size() - 2] : 0u, pc = pv & 1023u;
      if (body.size() > 1 && pc >= (uint32_t)(J_FMAUR * kJointStride) && pc < (uint32_t)(J_FMAUR * kJointStride + nr) && (pv >> 14) < 512 && opd < 64) {
        seg->code.pop_back();    // ... and the multiply-add before it as well
        seg->code.back() = encode(J_FMAURSTL * kJointStride + (int)(pc - J_FMAUR * kJointStride), 0, (pv >> 14) | (opd << 9));
      } else {
        seg->code.back() = encode(P_GSTFL, 0, opd);
      }
    } else {
      seg->code.push_back(encode(P_LOOP_END, 0, 0));
    }
    seg->code.insert(seg->code.end(), epi.begin(), epi.end());
    seg->code.push_back(encode(P_END, 0, 0));
    seg->code.push_back(encode(P_END, 0, 0));  // the interpreter prefetches one word ahead
    seg->n_instr_body = (int)body.size();
    // the kernel jumps through a table indexed by the case id without a range check
    for (size_t i = 0; i < seg->code.size(); ++i) {
      const int cs = (int)(seg->code[i] & 1023u);
      if (cs >= P_COUNT_) { set_error("graph VM: internal error, invalid case id %d", cs); return DRAGON_ERR_UNSUPPORTED; }
      if (cs == P_UCONST) ++i;  // the next word is a literal
    }
    if ((int)seg->code.size() > kVmCodeMaxWords) { set_error("graph VM: instruction stream too long (%d words)", (int)seg->code.size()); return kVmErrTooLarge; }
    if ((int)seg->finish.size() > kVmScalarAccs + kVmRegsWide - 2 + kVmSmemSlots - 2) { set_error("graph VM: too many reduced outputs in one segment"); return kVmErrTooLarge; }
    if ((int)seg->operand_mem.size() > kMaxOperands) { set_error("graph VM: too many memory operands in one segment"); return kVmErrTooLarge; }
    return DRAGON_OK;
  }
};

}  // namespace

int codegen_segment(const std::vector<Item>& items, const std::vector<int>& idx, const std::vector<Value>& vals,
                    const std::vector<MemRef>& mems, int sm_count, VmSegment* seg) {
  // the dense build (few register slots, two CTAs per SM) when the program keeps everything on
  // chip with it, else the wide one; DRAGON_VM_BUILD=wide|dense forces the choice
  const char* force = std::getenv("DRAGON_VM_BUILD");
  const bool only_wide = force && std::string(force) == "wide", only_dense = force && std::string(force) == "dense";
  int rc = DRAGON_ERR_UNSUPPORTED;
  (void)only_dense;      // the dense build is tried first anyway; a program that does not fit it goes to the wide one
  if (!only_wide) {
    VmSegment trial = *seg;
    Gen gen(items, idx, vals, mems, &trial, kVmRegsDense, kVmSmemSlotsDense);
    rc = gen.run();
    // it must keep everything on chip, within half an SM's shared memory
    const size_t smem = (size_t)((trial.code.size() + 3) & ~(size_t)3) * 8 + kMaxUniforms * 4 + kVmReduceBytes + kMaxOperands * 16 + (size_t)trial.n_smem * kVmTile * 4;
    if (rc == DRAGON_OK && trial.n_spill == 0 && smem <= 113 * 1024) { *seg = trial; seg->dense = true; }
    else rc = DRAGON_ERR_UNSUPPORTED;
  }
  if (rc != DRAGON_OK) {
    // as many shared-memory slots as fit beside the instruction stream (whose length depends a
    // little on the slot count: second attempt with the count that fits the first one's stream)
    auto smem_of = [](const VmSegment& g, int slots) {
      return (size_t)((g.code.size() + 3) & ~(size_t)3) * 8 + kMaxUniforms * 4 + kVmReduceBytes + kMaxOperands * 16 + (size_t)slots * kVmTile * 4;
    };
    for (int slots = kVmSmemSlots;; slots = kVmSmemSlotsLongCode) {
      VmSegment trial = *seg;
      Gen gen(items, idx, vals, mems, &trial, kVmRegsWide, slots);
      rc = gen.run();
      if (rc) return rc;
      if (smem_of(trial, trial.n_smem) <= (size_t)227 * 1024 || slots == kVmSmemSlotsLongCode) { *seg = trial; break; }
    }
    seg->dense = false;
  }
  long long tiles = seg->row_mode ? seg->n : (seg->n + kVmTile - 1) / kVmTile;
  if (tiles >= (1LL << 31)) { set_error("graph VM: more than 2^31 tiles"); return DRAGON_ERR_UNSUPPORTED; }
  seg->grid = (int)std::max<long long>(1, std::min<long long>(tiles, (long long)sm_count * (seg->dense ? 2 : 1)));
  // no program leaves here unverified: an index that a leaf would use out of range is a compiler error, not a fault
  if (verify_segment(*seg) != DRAGON_OK) return DRAGON_ERR_UNSUPPORTED;
  return DRAGON_OK;
}

}  // namespace dragon
