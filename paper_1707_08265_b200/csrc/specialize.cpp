// Specialisation of one instruction stream of the graph VM: the leaves of its instructions, taken from
// the generated templates, strung together in program order as one straight-line PTX kernel.  What the
// interpreter fetches and decodes at run time (case id, argument word, the literal behind a uconst, the
// start of the per-tile body) is a constant here, and the indexed branch between two instructions is
// gone, so the assembler folds the argument arithmetic, drops the register moves between leaves and
// schedules across them.  Every leaf computes with explicitly rounded operations, so the specialised
// kernel returns the interpreter's results bit for bit.  Host code only.
#include <cstring>
#include <string>
#include <vector>

#include "plan.h"
#include "vm_isa.h"
#include "vm_templates.h"

namespace dragon {

namespace {

// text with every #KEY# replaced; unknown keys are an error of the generator, reported to the caller
bool fill(const char* text, const std::vector<std::pair<std::string, std::string>>& sub, std::string* out) {
  for (const char* p = text; *p;) {
    const char* h = std::strchr(p, '#');
    if (!h) { out->append(p); break; }
    out->append(p, h - p);
    const char* e = std::strchr(h + 1, '#');
    if (!e) return false;
    const std::string key(h + 1, e - h - 1);
    bool found = false;
    for (const auto& kv : sub)
      if (kv.first == key) { out->append(kv.second); found = true; break; }
    if (!found) return false;
    p = e + 1;
  }
  return true;
}

std::string label_of(int pc, int n) { return pc < n ? "$I_" + std::to_string(pc) : std::string("$I_END"); }

}  // namespace

int specialize_ptx(const VmSegment& sg, const char* entry, std::string* ptx) {
  const vmt::Variant* v = nullptr;
  for (int i = 0; i < vmt::kNumVariants; ++i)
    if (vmt::kVariants[i].register_slots == (sg.dense ? vm::kVmRegsDense : vm::kVmRegsWide)) v = &vmt::kVariants[i];
  const int n = (int)sg.code.size();
  if (!v || n == 0 || sg.loop_start < 0 || sg.loop_start >= n) { set_error("specialize: no template set for this program"); return DRAGON_ERR_INVALID_ARG; }
  std::string body, cold, sites;
  body.reserve((size_t)n * 4096);
  int n_sites = 0;
  for (int pc = 0; pc < n;) {
    const uint32_t w = sg.code[pc], c = w & 1023u;
    if ((int)c >= v->n_cases || !v->leaves[c].text) { set_error("specialize: instruction %d has case id %u, which this build does not have", pc, c); return DRAGON_ERR_INVALID_ARG; }
    const vmt::Leaf& leaf = v->leaves[c];
    const bool literal = c == (uint32_t)vm::P_UCONST;
    const int next = pc + (literal ? 2 : 1);
    if (literal && pc + 1 >= n) { set_error("specialize: uconst without its literal"); return DRAGON_ERR_INVALID_ARG; }
    std::vector<std::pair<std::string, std::string>> sub = {
        {"I", std::to_string(pc)},
        {"NEXT", label_of(next, n)},
        {"NEXTARG", std::to_string(next < n ? sg.code[next] >> 14 : 0u)},
        {"LOOP", label_of(sg.loop_start, n)},
        {"LOOPARG", std::to_string(sg.code[sg.loop_start] >> 14)},
        {"LITERAL", std::to_string(literal ? sg.code[pc + 1] : 0u)}};
    for (int k = 0; k < leaf.n_sites; ++k) sub.push_back({"SITE" + std::to_string(k), std::to_string(n_sites + k)});
    n_sites += leaf.n_sites;
    body += label_of(pc, n) + ":\n";
    std::string labels;
    if (!fill(leaf.text, sub, &body) || !fill(leaf.cold, sub, &cold) || !fill(leaf.site_labels, sub, &labels)) {
      set_error("specialize: malformed template for case id %u", c);
      return DRAGON_ERR_INVALID_ARG;
    }
    if (!labels.empty()) sites += (sites.empty() ? "" : ", ") + labels;
    pc = next;
  }
  ptx->clear();
  ptx->reserve(body.size() + cold.size() + 65536);
  *ptx += vmt::kModuleHead;
  if (!fill(v->head, {{"ENTRY", entry}}, ptx)) { set_error("specialize: malformed head template"); return DRAGON_ERR_INVALID_ARG; }
  *ptx += v->prologue;
  *ptx += "\tmov.u32 %arg, " + std::to_string(sg.code[0] >> 14) + ";\n";
  *ptx += body;
  *ptx += "$I_END:\n\texit;\n";
  *ptx += cold;
  if (n_sites > 0 && !fill(v->reduction, {{"PHRET", sites}}, ptx)) { set_error("specialize: malformed reduction template"); return DRAGON_ERR_INVALID_ARG; }
  *ptx += "}\n";
  return DRAGON_OK;
}

}  // namespace dragon
