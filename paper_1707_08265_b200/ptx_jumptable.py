"""Build step: turns the VM kernel's dispatch tree into one indexed jump.

nvcc emits no indexed branch for a C++ switch, so vm_kernel.cu dispatches through a balanced tree
of compares.  Its PTX carries two kinds of markers (comments written by inline asm):
``// VMDISPATCH %r<N>`` where the case id is known, and ``// VMLEAF <id>`` at the top of the code
of every case.  This script gives every leaf block a label, checks that the tree between the
dispatch point and the leaves consists of compares and branches only (so that skipping it skips
no work; otherwise it refuses and the library keeps the tree), and replaces the dispatch point by
``brx.idx`` over a ``.branchtargets`` table.  The result is assembled with ptxas and loaded at
run time; the compiled-in tree kernel stays as the fallback.
"""
import re
import sys

LABEL = re.compile(r"^\s*(\$?[A-Za-z_][\w$]*):\s*$")
BRANCH = re.compile(r"^\s*(@!?%p\d+\s+)?(bra(\.uni)?|brx\.idx|ret|exit|trap)\b")
# compares, branches, and integer arithmetic on the case id (the compiler narrows and offsets it)
SPECIAL = re.compile(r"^\s*mov\.u32\s+(%r\d+),\s*%(tid|ctaid|ntid|nctaid)\.[xyz];")
TREE_OK = re.compile(r"^\s*(@!?%p\d+\s+)?(setp\.|bra\b|bra\.uni\b|cvt\.[us]\d+\.[us]\d+\s|and\.b(16|32)\s|(add|sub)\.s(16|32)\s|shr\.[us]32\s)")


def rewrite(ptx, kernel_substr="vm_kernel", thread=True):
    lines = ptx.split("\n")
    # body of the kernel entry
    start = next(i for i, l in enumerate(lines) if ".entry" in l and kernel_substr in l)
    depth, body_lo, body_hi = 0, None, None
    for i in range(start, len(lines)):
        depth += lines[i].count("{") - lines[i].count("}")
        if body_lo is None and "{" in lines[i]:
            body_lo = i
        if body_lo is not None and depth == 0:
            body_hi = i
            break
    disp = [i for i in range(body_lo, body_hi) if "// VMDISPATCH" in lines[i]]
    if len(disp) != 1:
        raise RuntimeError("expected one dispatch marker, found %d" % len(disp))
    disp = disp[0]
    reg = re.search(r"VMDISPATCH\s+(%r\d+)", lines[disp]).group(1)
    leaves = {}
    for i in range(body_lo, body_hi):
        m = re.search(r"// VMLEAF (\d+)", lines[i])
        if m:
            n = int(m.group(1))
            if n in leaves:
                raise RuntimeError("leaf %d appears twice" % n)
            leaves[n] = i
    n_leaves = max(leaves) + 1
    if sorted(leaves) != list(range(n_leaves)):
        raise RuntimeError("leaf ids are not dense")

    def is_code(l):
        s = l.strip()
        return bool(s) and not s.startswith("//") and not s.startswith(".") and not LABEL.match(l) and s not in ("{", "}")

    # label of the basic block that holds each leaf marker (insert one when the block is a fall-through)
    inserts = {}          # line index -> label to insert before that line
    leaf_label = {}
    for n, at in leaves.items():
        j = at - 1
        while True:
            if LABEL.match(lines[j]):
                leaf_label[n] = LABEL.match(lines[j]).group(1)
                break
            if is_code(lines[j]) and BRANCH.match(lines[j]):
                lab = "VMLEAF_%d" % n
                inserts[j + 1] = lab
                leaf_label[n] = lab
                break
            j -= 1
            if j <= body_lo:
                raise RuntimeError("no block start for leaf %d" % n)
    # safety: from the dispatch marker to every leaf block only compares and branches may run
    label_at = {LABEL.match(lines[i]).group(1): i for i in range(body_lo, body_hi) if LABEL.match(lines[i])}
    leaf_starts = set()
    for n, at in leaves.items():
        j = at
        while not (LABEL.match(lines[j]) or (is_code(lines[j]) and BRANCH.match(lines[j]))):
            j -= 1
        leaf_starts.add(j if LABEL.match(lines[j]) else j + 1)
    hoisted = set()

    def n_defs(reg):
        pat = re.compile(r"^\s*(@!?%p\d+\s+)?[a-z][\w.]*\s+(\{[^}]*)?" + re.escape(reg) + r"\b[,;}]")
        return sum(1 for j in range(body_lo, body_hi) if pat.match(lines[j]))

    seen, work = set(), [disp + 1]
    while work:
        i = work.pop()
        if i in seen:
            continue
        seen.add(i)
        while True:
            if i in leaf_starts:
                break
            l = lines[i]
            if "// VMLEAF" in l:
                break
            if is_code(l) and i not in hoisted:
                m = SPECIAL.match(l)
                if m and n_defs(m.group(1)) == 1:
                    hoisted.add(i)      # a re-read of a special register: defined once, so it can move to the entry
                elif not TREE_OK.match(l):
                    raise RuntimeError("dispatch tree holds other work: %r (line %d)" % (l.strip(), i))
                m = re.search(r"bra(\.uni)?\s+(\$?[\w$]+);", l)
                if m:
                    work.append(label_at[m.group(2)])
                    if not l.strip().startswith("@"):
                        break        # unconditional: no fall-through
            i += 1
            if i >= body_hi:
                raise RuntimeError("ran off the kernel body while checking the tree")
    # threaded dispatch: the decode of the next instruction (the loop head, a straight block that
    # ends at the dispatch point) is copied to the end of every leaf in place of the jump back,
    # so that it can be scheduled among the leaf's own arithmetic
    h = disp
    while not LABEL.match(lines[h]):
        h -= 1
        if h <= body_lo:
            raise RuntimeError("no label at the loop head")
    head_label = LABEL.match(lines[h]).group(1)
    head = [l for l in lines[h + 1:disp] if is_code(l)]
    for l in head:
        if BRANCH.match(l) and not l.strip().startswith("@"):
            raise RuntimeError("loop head is not a straight block")
    back = re.compile(r"^\s*bra(\.uni)?\s+" + re.escape(head_label) + r";\s*$")
    # rewrite
    out = []
    n_threaded = 0
    first_code = next(i for i in range(body_lo + 1, body_hi) if is_code(lines[i]))
    head = [l for l in head if l not in [lines[j] for j in hoisted]]
    for i, l in enumerate(lines):
        if i == first_code:
            out.extend(lines[j] for j in sorted(hoisted))
        if i in hoisted:
            continue
        if i in inserts:
            out.append(inserts[i] + ":")
        if i == disp:
            out.append("\tVMJT: .branchtargets " + ", ".join(leaf_label[n] for n in range(n_leaves)) + ";")
            out.append("\tbrx.idx.uni " + reg + ", VMJT;")
            continue
        if thread and body_lo < i < body_hi and back.match(l) and i > disp:
            out.extend(head)
            out.append("\tbrx.idx.uni " + reg + ", VMJT;")
            n_threaded += 1
            continue
        out.append(l)
    return "\n".join(out), n_leaves


if __name__ == "__main__":
    src, dst = sys.argv[1], sys.argv[2]
    text, n = rewrite(open(src).read())
    open(dst, "w").write(text)
    print("jump table over %d leaves written to %s" % (n, dst))
