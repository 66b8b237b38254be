"""Generator of the graph-VM kernel, written directly in PTX for sm_100a.

The VM (csrc/vm_isa.h) is an accumulator machine whose instructions work on V-wide per-thread
values.  An interpreter spends its time in two places: the arithmetic of the instructions and the
dispatch between them.  Both are written out here instruction by instruction instead of leaving
them to a C++ compiler:

* dispatch is one 64-bit shared-memory load of the pre-decoded {case, argument} pair, a pointer
  increment and a jump to the one dispatch block, which holds the kernel's only indexed branch
  (``brx.idx.uni`` over a table of leaf labels); the fetch of the next pair is issued at the top of
  a leaf, ahead of its arithmetic;
* every V-wide value lives in named registers as packed pairs (``.b64`` = two fp32), so additions,
  multiplications and fused multiply-adds are ``f32x2`` instructions: half the issue slots of
  scalar code for the same rounding (each lane is an IEEE fp32 operation);
* each (opcode, register slot) pair is its own leaf, so no register is ever selected at run time.

The elementary functions follow csrc/vm_math.h operation by operation (same constants, same
order), so the host instantiation of that header predicts the kernel's rounding.

Running this file writes the PTX to the path given as its first argument.
"""
import struct
import sys

TILE = 4096         # elements per tile = threads per CTA x elements per thread (512 x 8 or 1024 x 4)
SLOT_BYTES = TILE * 4
MAX_OPERANDS = 40
MAX_UNIFORMS = 512

# Params (csrc/vm_isa.h): byte offsets
P_CODE, P_SPILL, P_COLPART, P_SCALPART, P_STATUS, P_N = 0, 8, 16, 24, 32, 40
P_NCODE, P_ROWMODE, P_COLS, P_NSPILL, P_NTILES, P_LOOPSTART, P_GRID, P_NFULL, P_STATUSCLEAR, P_OPERAND = 48, 52, 56, 60, 64, 68, 72, 76, 80, 96
P_SIZE = P_OPERAND + 16 * MAX_OPERANDS
# shared memory behind the decoded instruction stream: uniforms | reduction scratch | operand table | slots
RED_BYTES = 1024    # per-warp partials of the row sums (three buffers of up to 32 floats) and of the fp64 block sums (32 doubles)
OFF_RED, OFF_OPB, OFF_SLOTS = MAX_UNIFORMS * 4, MAX_UNIFORMS * 4 + RED_BYTES, MAX_UNIFORMS * 4 + RED_BYTES + MAX_OPERANDS * 16

JOINT = ["ldr", "str", "add", "sub", "rsub", "mul", "divp", "rdivp", "addto", "accum", "fmaur", "rtos", "stor", "spillr", "fillr",
         "gldr", "sincosr", "cossinr", "macc0", "macc1", "macc2", "macc3", "ldswr", "ldswar",
         "stld0", "stld1", "stld2", "stld3", "stld4", "stld5", "stld6", "stld7", "ldswarf", "fmaurstl", "strlds"]
# Leaves that end in their own indexed branch instead of a jump to the shared dispatch block: one
# taken branch less per dispatch.  Measured, not derived: every further site makes the assembler add
# branch-table code and changes its register allocation, and larger sets ran slower on all three
# large workloads (16 more short leaves: +3 % on the sin/cos graph, +3 % on the random DAG), so the
# list holds the short arithmetic, store and staged-load leaves it was first tried with.
HOT = {"fmau", "mul", "sacc0", "macc1", "fmaur", "gstf", "gstfl", "cossinr", "ldswar", "ldswarf", "fmaurstl"}
JOINT_STRIDE = 8    # case id of a joint instruction = index * JOINT_STRIDE + register slot
N_SACC = 4          # scalar accumulators
PLAIN = ["ldu", "addu", "subu", "rsubu", "mulu", "divpu", "rdivpu", "fmau", "lds", "sts", "adds", "subs", "rsubs", "muls", "divps",
         "rdivps", "sin", "cos", "sincos", "cossin", "expc", "tanh", "sigmoid", "relu", "neg", "step", "clampmask", "onemsq", "yomy", "divpgb",
         "rbf16", "rowsum", "gld", "gst", "gldf", "gstf", "fill", "spill", "uload", "uconst", "loop_begin", "loop_end", "colout", "scalout",
         "sacc0", "sacc1", "sacc2", "sacc3", "ascal0", "ascal1", "ascal2", "ascal3", "glda0", "glda", "ldsw", "ldswa", "gstfl", "glda0h", "ldswah", "rowsumu", "accums", "sqrt", "rcp", "tanhb", "sigmoidb", "expcb", "end"]


def f32bits(x):
    return struct.unpack("<I", struct.pack("<f", x))[0]


def fc(x):
    return "0f%08X" % f32bits(x)


class Kernel:
    def __init__(self, name, nr, ctas_per_sm, threads=512, template=False):
        self.name, self.nr, self.ctas = name, nr, ctas_per_sm
        # template mode: every leaf is generated on its own, with placeholders (#...#) where the interpreter
        # fetches and dispatches; csrc/specialize.cpp strings such leaves together for one instruction stream
        self.template = template
        self.leaf_sites = []  # template mode: return labels of the sin/cos sites of the leaf being generated
        # geometry: a thread owns V elements of a tile as V/4 groups of four consecutive ones (a group is one
        # 16-byte vector, the groups of a warp are contiguous), held as NP = V/2 packed pairs
        self.NT = threads
        self.V = TILE // threads
        self.NP = self.V // 2
        self.NH = self.V // 4               # 16-byte groups per thread
        self.HALF_BYTES = threads * 16      # distance between a thread's groups
        self.red_shift = 6 if threads == 512 else 7     # log2 of the bytes of one buffer of per-warp row-sum partials
        assert 3 * (threads // 32) * 4 <= 512 and 512 + (threads // 32) * 8 <= RED_BYTES
        self.lines = []
        self.ph_sites = []    # return labels of the sin/cos sites (reduce_pio2)
        self.PX = ["%%PX%d" % i for i in range(self.NP)]
        self.PR = ["%%PR%d" % i for i in range(self.NP)]
        self.PK = ["%%PK%d" % i for i in range(self.NP)]
        self.cold = []        # rarely executed blocks, placed behind all leaves so that the hot leaves stay short and close together
        self.cnt = {"f": 0, "r": 0, "rd": 0, "p": 0, "fd": 0, "h": 0}
        self.nlabel = 0
        self.kt = []          # packed constants (u64 words)
        self.A = ["%%A%d" % i for i in range(self.NP)]
        self.R = [["%%R%d_%d" % (k, i) for i in range(self.NP)] for k in range(nr)]
        self.S = ["%%S%d" % i for i in range(N_SACC)]     # scalar accumulators (.f32)

    # ---- plumbing -------------------------------------------------------------------------
    def e(self, s):
        self.lines.append("\t" + s)

    def label(self, s):
        self.lines.append(s + ":")

    def begin_cold(self):
        self.hot_lines, self.lines = self.lines, self.cold

    def end_cold(self):
        self.lines = self.hot_lines

    def newlabel(self, stem="L"):
        self.nlabel += 1
        return "$%s_%s_%d%s" % (stem, self.name, self.nlabel, "_#I#" if self.template else "")

    def t(self, kind):
        self.cnt[kind] += 1
        return "%%%s%d" % ({"f": "f", "r": "r", "rd": "rd", "p": "p", "fd": "fd", "h": "h"}[kind], self.cnt[kind] - 1)

    def f(self): return self.t("f")
    def r(self): return self.t("r")
    def rd(self): return self.t("rd")
    def p(self): return self.t("p")
    def fd(self): return self.t("fd")

    def K(self, x, y=None):
        """packed constant {x, y} (y defaults to x), an immediate the assembler places as it sees fit"""
        w = f32bits(x) | (f32bits(x if y is None else y) << 32)
        d = self.rd()
        self.e("mov.b64 %s, 0x%016X;" % (d, w))
        return d

    # ---- packed helpers --------------------------------------------------------------------
    def fma2(self, a, b, c, d=None):
        d = d or self.rd()
        self.e("fma.rn.f32x2 %s, %s, %s, %s;" % (d, a, b, c))
        return d

    def mul2(self, a, b, d=None):
        d = d or self.rd()
        self.e("mul.rn.f32x2 %s, %s, %s;" % (d, a, b))
        return d

    # In a specialised kernel a packed product of one leaf can meet a packed sum of the next, and the
    # assembler was seen to contract such a pair into one fused multiply-add although both name their
    # rounding (a*b + c*d then differed from the interpreter in the last place; so did the sum written as
    # a*1 + b).  The scalar forms with an explicit rounding are never contracted, so there the packed sums
    # and differences are written as two scalar ones: the same bits as add.rn.f32x2 / sub.rn.f32x2.
    def add2(self, a, b, d=None):
        d = d or self.rd()
        if self.template:
            self.scalar_pair("add", a, b, d)
        else:
            self.e("add.rn.f32x2 %s, %s, %s;" % (d, a, b))
        return d

    def sub2(self, a, b, d=None):
        d = d or self.rd()
        if self.template:
            self.scalar_pair("sub", a, b, d)
        else:
            self.e("sub.rn.f32x2 %s, %s, %s;" % (d, a, b))
        return d

    def scalar_pair(self, op, a, b, d):
        (al, ah), (bl, bh) = self.unpack(a), self.unpack(b)
        lo, hi = self.f(), self.f()
        self.e("%s.rn.f32 %s, %s, %s;" % (op, lo, al, bl))
        self.e("%s.rn.f32 %s, %s, %s;" % (op, hi, ah, bh))
        self.e("mov.b64 %s, {%s, %s};" % (d, lo, hi))

    def unpack(self, a):
        lo, hi = self.f(), self.f()
        self.e("mov.b64 {%s, %s}, %s;" % (lo, hi, a))
        return lo, hi

    def pack(self, lo, hi, d=None):
        d = d or self.rd()
        self.e("mov.b64 %s, {%s, %s};" % (d, lo, hi))
        return d

    def splat(self, s):
        return self.pack(s, s)

    def scalars(self, vals):
        out = []
        for a in vals:
            out.extend(self.unpack(a))
        return out

    def packs(self, sc, dst=None):
        return [self.pack(sc[2 * i], sc[2 * i + 1], dst[i] if dst else None) for i in range(self.NP)]

    def rcp(self, x):
        d = self.f()
        self.e("rcp.approx.ftz.f32 %s, %s;" % (d, x))
        return d

    def rcp1pabs(self, x):
        """1 / (1 + |x|)"""
        a = self.f()
        self.e("abs.f32 %s, %s;" % (a, x))
        self.e("add.rn.f32 %s, %s, 0f3F800000;" % (a, a))
        return self.rcp(a)

    # ---- dispatch ---------------------------------------------------------------------------
    def fetch(self):
        if self.template:       # the next instruction's argument is a constant of the specialised kernel
            self.e("mov.u32 %arg, #NEXTARG#;")
            return
        self.e("ld.shared.v2.u32 {%case, %arg}, [%ip];")
        self.e("add.u32 %ip, %ip, 8;")

    def param(self, off, ty="u32"):
        d = self.rd() if ty in ("u64", "s64") else self.r()
        self.e("ld.param.%s %s, [VP+%d];" % (ty, d, off))
        return d

    def tx_is_zero(self):
        pr = self.p()
        self.e("setp.eq.u32 %s, %%pos0, 0;" % pr)
        return pr

    def pos0_64(self):
        d = self.rd()
        self.e("cvt.u64.u32 %s, %%pos0;" % d)
        return d

    def jump(self):
        # every leaf leaves through the one dispatch block: the assembler gives each indexed branch
        # its own table of branch instructions (about 2 KB per site), which with one site per leaf
        # made the code image four times larger and scattered the hot leaves
        if self.template:       # straight to the next instruction's leaf (the assembler drops a branch to the next line)
            self.e("bra.uni #NEXT#;")
            return
        if getattr(self, "own_brx", False):
            self.e("brx.idx.uni %%case, JT_%s;" % self.name)
            return
        self.e("bra.uni $DISPATCH_%s;" % self.name)

    # addresses that depend on the argument (taken before the fetch overwrites %arg)
    def slot_addr(self):
        a = self.r()
        self.e("mad.lo.u32 %s, %%arg, %d, %%sa;" % (a, SLOT_BYTES))
        return a

    def spill_addr(self):
        a = self.rd()
        self.e("mul.wide.u32 %s, %%arg, %d;" % (a, SLOT_BYTES))
        self.e("add.u64 %s, %s, %%spb;" % (a, a))
        return a

    def uniform(self, idx_reg=None):
        a, u = self.r(), self.f()
        self.e("shl.b32 %s, %s, 2;" % (a, idx_reg or "%arg"))
        self.e("add.u32 %s, %s, %%ub;" % (a, a))
        self.e("ld.shared.f32 %s, [%s];" % (u, a))
        return u

    def lds_v(self, addr, dst=None):
        d = dst or [self.rd() for _ in range(self.NP)]
        for h in range(self.NH):
            self.e("ld.shared.v2.b64 {%s, %s}, [%s+%d];" % (d[2 * h], d[2 * h + 1], addr, h * self.HALF_BYTES))
        return d

    def sts_v(self, addr, src):
        for h in range(self.NH):
            self.e("st.shared.v2.b64 [%s+%d], {%s, %s};" % (addr, h * self.HALF_BYTES, src[2 * h], src[2 * h + 1]))

    def ldg_v(self, addr, dst=None):
        d = dst or [self.rd() for _ in range(self.NP)]
        for h in range(self.NH):
            self.e("ld.global.v2.b64 {%s, %s}, [%s+%d];" % (d[2 * h], d[2 * h + 1], addr, h * self.HALF_BYTES))
        return d

    def stg_v(self, addr, src):
        for h in range(self.NH):
            self.e("st.global.v2.b64 [%s+%d], {%s, %s};" % (addr, h * self.HALF_BYTES, src[2 * h], src[2 * h + 1]))

    def mov_v(self, dst, src):
        for i in range(self.NP):
            self.e("mov.b64 %s, %s;" % (dst[i], src[i]))

    # ---- elementary functions (csrc/vm_math.h, operation by operation) -----------------------
    RANGE = 1048576.0     # 2^20: beyond it the two-constant reduction hands over to the exact one

    def reduce_pio2(self, xs):
        """-> (r, kb): remainders of the packed pairs xs modulo pi/2 and the words whose two low bits are
        the quadrant.  Common case (every lane of this thread within 2^20 in magnitude: one 3-input
        maximum per two or three lanes and a branch that is not taken): the two-constant reduction,
        packed.  Otherwise the thread leaves for the one copy of the general reduction that the kernel
        holds (emit_general_reduction), which returns here behind the packed code."""
        big = 12582912.0
        n = len(xs)
        assert n == self.NP
        r, kb = self.PR, self.PK
        lanes = []
        for x in xs:
            for s in self.unpack(x):
                a = self.f()
                self.e("abs.f32 %s, %s;" % (a, s))
                lanes.append(a)
        m = lanes[0]
        rest = lanes[1:]
        while rest:
            d = self.f()
            if len(rest) >= 2:
                self.e("max.NaN.f32 %s, %s, %s, %s;" % (d, m, rest[0], rest[1]))
                rest = rest[2:]
            else:
                self.e("max.NaN.f32 %s, %s, %s;" % (d, m, rest[0]))
                rest = rest[1:]
            m = d
        ok, stub, join = self.p(), self.newlabel("rng"), self.newlabel("rng")
        self.e("setp.le.f32 %s, %s, %s;" % (ok, m, fc(self.RANGE)))
        self.e("@!%s bra %s;" % (ok, stub))
        self.begin_cold()
        self.label(stub)
        for i in range(n):
            self.e("mov.b64 %s, %s;" % (self.PX[i], xs[i]))
        if self.template:
            self.e("mov.u32 %%phsite, #SITE%d#;" % len(self.leaf_sites))
            self.leaf_sites.append(join)
        else:
            self.e("mov.u32 %%phsite, %d;" % len(self.ph_sites))
        self.e("bra $PH_%s;" % self.name)
        self.end_cold()
        self.ph_sites.append(join)
        c = self.K(0.636619772367581343); cb = self.K(big)
        for x, d in zip(xs, kb):
            self.fma2(x, c, cb, d)
        c = self.K(-big)
        k = [self.add2(t, c) for t in kb]
        c = self.K(-1.57079637050628662109375)
        for ki, x, d in zip(k, xs, r):
            self.fma2(ki, c, x, d)
        c = self.K(4.371138828673793e-8)
        for ki, d in zip(k, r):
            self.fma2(ki, c, d, d)
        self.label(join)
        return list(r), list(kb)

    def emit_general_reduction(self):
        """The reduction modulo pi/2 for threads that hold a lane beyond 2^20, inf or NaN; one copy per
        kernel, entered from every sin/cos site with the argument in %PX and the site's number in
        %phsite, left through an indexed branch back to that site with r in %PR and the quadrant words
        in %PK.  The eight lanes are walked in a loop over a small local array.  A lane within range
        takes the two-constant reduction (the same operations as the packed code, hence the same
        results); inf/NaN give r = x - x (NaN); a large finite lane takes the exact reduction of
        csrc/vm_math.h (reduce_pio2_large): x = m * 2^s, a 96-bit window of 2/pi starting at bit
        s + 30 of the table times m modulo 2^96, whose top two bits are the quadrant and whose next
        64 the signed fraction of a quadrant."""
        if not self.ph_sites:
            return
        big = 12582912.0
        n = self.NP
        self.e("PHRET_%s: .branchtargets %s;" % (self.name, "#PHRET#" if self.template else ", ".join(self.ph_sites)))
        self.label("$PH_%s" % self.name)
        base = self.rd()
        self.e("mov.u64 %s, PHBUF;" % base)
        for i in range(n):
            self.e("st.local.b64 [%s+%d], %s;" % (base, 8 * i, self.PX[i]))
        loop, nxt, special, large = self.newlabel("rng"), self.newlabel("rng"), self.newlabel("rng"), self.newlabel("rng")
        i_, adr = self.r(), self.rd()
        self.e("mov.u32 %s, 0;" % i_)
        self.label(loop)
        xb, ax, pin, pnf = self.r(), self.r(), self.p(), self.p()
        self.e("mad.wide.u32 %s, %s, 4, %s;" % (adr, i_, base))
        self.e("ld.local.b32 %s, [%s];" % (xb, adr))
        self.e("and.b32 %s, %s, 0x7fffffff;" % (ax, xb))
        self.e("setp.le.u32 %s, %s, 0x%08X;" % (pin, ax, f32bits(self.RANGE)))
        self.e("@!%s bra %s;" % (pin, large))
        xs_, kbs, ks, rs = self.f(), self.f(), self.f(), self.f()
        self.e("mov.b32 %s, %s;" % (xs_, xb))
        self.e("fma.rn.f32 %s, %s, %s, %s;" % (kbs, xs_, fc(0.636619772367581343), fc(big)))
        self.e("add.rn.f32 %s, %s, %s;" % (ks, kbs, fc(-big)))
        self.e("fma.rn.f32 %s, %s, %s, %s;" % (rs, ks, fc(-1.57079637050628662109375), xs_))
        self.e("fma.rn.f32 %s, %s, %s, %s;" % (rs, ks, fc(4.371138828673793e-8), rs))
        self.e("st.local.f32 [%s+%d], %s;" % (adr, 8 * n, rs))
        self.e("st.local.f32 [%s+%d], %s;" % (adr, 16 * n, kbs))
        self.e("bra %s;" % nxt)
        self.label(large)
        self.e("setp.ge.u32 %s, %s, 0x7f800000;" % (pnf, ax))
        self.e("@%s bra %s;" % (pnf, special))
        # x = m * 2^s; window of 2/pi from bit s + 30
        mm, st, idx, sh, tb = self.r(), self.r(), self.r(), self.r(), self.rd()
        self.e("and.b32 %s, %s, 0x007fffff;" % (mm, ax))
        self.e("or.b32 %s, %s, 0x00800000;" % (mm, mm))
        self.e("shr.u32 %s, %s, 23;" % (st, ax))
        self.e("sub.u32 %s, %s, 120;" % (st, st))            # (exponent - 150) + 30
        self.e("shr.u32 %s, %s, 5;" % (idx, st))
        self.e("and.b32 %s, %s, 31;" % (sh, st))
        self.e("mov.u64 %s, TWO_OVER_PI;" % tb)
        self.e("mad.wide.u32 %s, %s, 4, %s;" % (tb, idx, tb))
        w = [self.r() for _ in range(4)]
        for j in range(4):
            self.e("ld.const.b32 %s, [%s+%d];" % (w[j], tb, 4 * j))
        h2, h1, h0 = self.r(), self.r(), self.r()
        self.e("shf.l.wrap.b32 %s, %s, %s, %s;" % (h2, w[1], w[0], sh))
        self.e("shf.l.wrap.b32 %s, %s, %s, %s;" % (h1, w[2], w[1], sh))
        self.e("shf.l.wrap.b32 %s, %s, %s, %s;" % (h0, w[3], w[2], sh))
        p0, p1, t, c, r2, r1, r0 = self.rd(), self.rd(), self.rd(), self.r(), self.r(), self.r(), self.r()
        self.e("mul.wide.u32 %s, %s, %s;" % (p0, mm, h0))
        self.e("shr.u64 %s, %s, 32;" % (t, p0))
        self.e("mad.wide.u32 %s, %s, %s, %s;" % (p1, mm, h1, t))
        self.e("shr.u64 %s, %s, 32;" % (t, p1))
        self.e("cvt.u32.u64 %s, %s;" % (c, t))
        self.e("mad.lo.u32 %s, %s, %s, %s;" % (r2, mm, h2, c))
        self.e("cvt.u32.u64 %s, %s;" % (r1, p1))
        self.e("cvt.u32.u64 %s, %s;" % (r0, p0))
        qi, fh, fl, frac, pneg, td, rf, px = self.r(), self.r(), self.r(), self.rd(), self.p(), self.fd(), self.f(), self.p()
        self.e("shr.u32 %s, %s, 30;" % (qi, r2))
        self.e("shf.l.wrap.b32 %s, %s, %s, 2;" % (fh, r1, r2))
        self.e("shf.l.wrap.b32 %s, %s, %s, 2;" % (fl, r0, r1))
        self.e("mov.b64 %s, {%s, %s};" % (frac, fl, fh))
        self.e("setp.lt.s64 %s, %s, 0;" % (pneg, frac))
        self.e("@%s add.u32 %s, %s, 1;" % (pneg, qi, qi))
        self.e("cvt.rn.f64.s64 %s, %s;" % (td, frac))
        self.e("mul.f64 %s, %s, 0d%016X;" % (td, td, struct.unpack("<Q", struct.pack("<d", 8.5153039502163865e-20))[0]))   # pi/2 * 2^-64
        self.e("cvt.rn.f32.f64 %s, %s;" % (rf, td))
        self.e("setp.ne.u32 %s, %s, %s;" % (px, xb, ax))     # sign bit set
        self.e("@%s neg.f32 %s, %s;" % (px, rf, rf))
        self.e("@%s neg.s32 %s, %s;" % (px, qi, qi))
        self.e("and.b32 %s, %s, 3;" % (qi, qi))
        self.e("or.b32 %s, %s, 0x%08X;" % (qi, qi, f32bits(big)))
        self.e("st.local.f32 [%s+%d], %s;" % (adr, 8 * n, rf))
        self.e("st.local.b32 [%s+%d], %s;" % (adr, 16 * n, qi))
        self.e("bra %s;" % nxt)
        self.label(special)
        xf, z, kq = self.f(), self.f(), self.r()
        self.e("mov.b32 %s, %s;" % (xf, xb))
        self.e("sub.rn.f32 %s, %s, %s;" % (z, xf, xf))
        self.e("mov.u32 %s, 0x%08X;" % (kq, f32bits(big)))
        self.e("st.local.f32 [%s+%d], %s;" % (adr, 8 * n, z))
        self.e("st.local.b32 [%s+%d], %s;" % (adr, 16 * n, kq))
        self.label(nxt)
        plp = self.p()
        self.e("add.u32 %s, %s, 1;" % (i_, i_))
        self.e("setp.lt.u32 %s, %s, %d;" % (plp, i_, 2 * n))
        self.e("@%s bra %s;" % (plp, loop))
        for i in range(n):
            self.e("ld.local.b64 %s, [%s+%d];" % (self.PR[i], base, 8 * n + 8 * i))
            self.e("ld.local.b64 %s, [%s+%d];" % (self.PK[i], base, 16 * n + 8 * i))
        self.e("brx.idx %%phsite, PHRET_%s;" % self.name)

    def sincos(self, xs, want_sin=True, want_cos=True):
        """sin and cos of the packed pairs xs, stage by stage over all pairs.  Reduction by multiples of
        pi/2 held in two parts (the part left out is 1.7e-15 per quadrant, 1.1e-9 at 2^20); lanes
        beyond 2^20 are redone exactly by fix_range."""
        r, kb = self.reduce_pio2(xs)
        z = [self.mul2(ri, ri) for ri in r]
        c0, c1 = self.K(-1.9515285269243e-4), self.K(8.33216077944338e-3)
        p = [self.fma2(zi, c0, c1) for zi in z]
        c = self.K(-1.6666654609873324e-1)
        p = [self.fma2(zi, pi, c) for zi, pi in zip(z, p)]
        rz = [self.mul2(ri, zi) for ri, zi in zip(r, z)]
        sp = [self.fma2(a, pi, ri) for a, pi, ri in zip(rz, p, r)]
        c0, c1 = self.K(2.4433150705502356e-5), self.K(-1.3887316189460366e-3)
        p = [self.fma2(zi, c0, c1) for zi in z]
        c = self.K(4.1666645681363114e-2)
        p = [self.fma2(zi, pi, c) for zi, pi in zip(z, p)]
        c0, c1 = self.K(-0.5), self.K(1.0)
        h = [self.fma2(zi, c0, c1) for zi in z]
        zz = [self.mul2(zi, zi) for zi in z]
        cp = [self.fma2(a, pi, hi) for a, pi, hi in zip(zz, p, h)]
        S, C = [], []
        cm = self.K(-1.0) if want_cos else None
        for i in range(len(xs)):
            ps, pc = self.unpack(sp[i]), self.unpack(cp[i])
            # quadrant q = k mod 4: sin = (q0 ? pc : ps) * (-1)^q1, cos = (q0 ? -ps : pc) * (-1)^q1
            nps = self.unpack(self.mul2(sp[i], cm)) if want_cos else None
            q = [self.r(), self.r()]
            self.e("mov.b64 {%s, %s}, %s;" % (q[0], q[1], kb[i]))
            so, co = [], []
            for j in range(2):
                b, u, pr = self.r(), self.r(), self.p()
                self.e("and.b32 %s, %s, 1;" % (b, q[j]))
                self.e("setp.ne.u32 %s, %s, 0;" % (pr, b))
                self.e("shl.b32 %s, %s, 30;" % (u, q[j]))
                if want_sin:
                    s = self.f()
                    self.e("selp.f32 %s, %s, %s, %s;" % (s, pc[j], ps[j], pr))
                    self.e("lop3.b32 %s, %s, %s, 0x80000000, 0x78;" % (s, s, u))   # s ^ (u & signbit)
                    so.append(s)
                if want_cos:
                    c = self.f()
                    self.e("selp.f32 %s, %s, %s, %s;" % (c, nps[j], pc[j], pr))
                    self.e("lop3.b32 %s, %s, %s, 0x80000000, 0x78;" % (c, c, u))
                    co.append(c)
            if want_sin:
                S.append(self.pack(so[0], so[1]))
            if want_cos:
                C.append(self.pack(co[0], co[1]))
        return S, C

    def exp_core(self, x):
        """x packed, already clamped so that the result is a normal number: e^x = 2^t with t = x * log2(e) held as
        t_hi + e: t_hi the rounded product, e its exact residue (one fused multiply-add) plus x times the part of
        log2(e) that fp32 leaves out; 2^t_hi by the hardware approximation (relative error 2^-22 at most over the
        whole range), times 1 + e * ln 2"""
        l_hi, l_lo = 1.44269502162933349609375, 1.9259629911266175e-8
        kl, kn = self.K(l_hi), self.K(-1.0)
        t = self.mul2(x, kl)
        e = self.fma2(x, kl, self.mul2(t, kn))
        e = self.fma2(x, self.K(l_lo), e)
        e = self.mul2(e, self.K(0.693147180559945309))
        lo, hi = self.unpack(t)
        p = []
        for s in (lo, hi):
            d = self.f()
            self.e("ex2.approx.ftz.f32 %s, %s;" % (d, s))
            p.append(d)
        pp = self.pack(p[0], p[1])
        return self.fma2(pp, e, pp)

    def clamp(self, s, lo, hi):
        d = self.f()
        self.e("max.NaN.f32 %s, %s, %s;" % (d, s, fc(lo)))      # a NaN stays a NaN (as in the reference arithmetic)
        self.e("min.NaN.f32 %s, %s, %s;" % (d, d, fc(hi)))
        return d

    EXP_LO, EXP_HI = -86.0, 88.7   # e^x stays a normal fp32 number on this range

    # The "b" forms of expc, sigmoid and tanh (bounded=True) leave the clamps out: the host emits them only where
    # its interval analysis has proven the argument inside the range in which the clamps do nothing.
    def expc(self, xs, bounded=False):
        out = []
        for x in xs:
            if bounded:
                out.append(self.exp_core(x))
                continue
            lo, hi = self.unpack(x)
            out.append(self.exp_core(self.pack(self.clamp(lo, -10.0, 10.0), self.clamp(hi, -10.0, 10.0))))
        return out

    def sigmoid(self, xs, bounded=False):
        out = []
        for x in xs:
            if bounded:
                e = self.exp_core(self.mul2(x, self.K(-1.0)))
                l2, h2 = self.unpack(self.add2(e, self.K(1.0)))
                out.append(self.pack(self.rcp(l2), self.rcp(h2)))
                continue
            lo, hi = self.unpack(self.mul2(x, self.K(-1.0)))
            e = self.exp_core(self.pack(self.clamp(lo, self.EXP_LO, self.EXP_HI), self.clamp(hi, self.EXP_LO, self.EXP_HI)))
            l2, h2 = self.unpack(self.add2(e, self.K(1.0)))
            out.append(self.pack(self.rcp(l2), self.rcp(h2)))
        return out

    def tanh(self, xs, bounded=False):
        """x * P(x^2) / Q(x^2) (a rational fit on |x| <= 9, about 5 ulp; beyond 9.07 it exceeds 1), argument
        clamped at 10 and result clamped to [-1, 1], so that a saturated tanh is exactly +-1; NaN stays NaN"""
        def clamp2(v, lim):
            out = []
            for s in self.unpack(v):
                d = self.f()
                self.e("max.NaN.f32 %s, %s, %s;" % (d, s, fc(-lim)))
                self.e("min.NaN.f32 %s, %s, %s;" % (d, d, fc(lim)))
                out.append(d)
            return self.pack(out[0], out[1])
        cs = list(xs) if bounded else [clamp2(x, 10.0) for x in xs]
        z = [self.mul2(c, c) for c in cs]
        k0, k1 = self.K(1.3442309683456469e-08), self.K(2.0679596671714183e-05)
        p = [self.fma2(zi, k0, k1) for zi in z]
        for c in (3.5001979607618507e-03, 1.3385017810927272e-01, 1.0):
            k = self.K(c)
            p = [self.fma2(zi, pi, k) for zi, pi in zip(z, p)]
        k0, k1 = self.K(7.814557141497938e-07), self.K(3.2929435375013785e-04)
        q = [self.fma2(zi, k0, k1) for zi in z]
        for c in (2.5894861704209737e-02, 4.6718338985166813e-01, 1.0):
            k = self.K(c)
            q = [self.fma2(zi, qi, k) for zi, qi in zip(z, q)]
        out = []
        for c, pi, qi in zip(cs, p, q):
            ql, qh = self.unpack(qi)
            y = self.mul2(self.mul2(c, pi), self.pack(self.rcp(ql), self.rcp(qh)))
            out.append(y if bounded else clamp2(y, 1.0))
        return out

    def divp(self, num, den, dst):
        """dst = num / (1 + |den|), packed lists"""
        for i in range(self.NP):
            lo, hi = self.unpack(den[i])
            self.mul2(num[i], self.pack(self.rcp1pabs(lo), self.rcp1pabs(hi)), dst[i])

    # ---- tile context -----------------------------------------------------------------------
    # Kept per thread between instructions: %tile (index), %tb4 (byte offset of this thread's first
    # element of the tile in an fp32 FULL tensor), %limit (valid elements in the tile), %tnext
    # (elements to this CTA's next tile, 0 when there is none), %pfull (limit == TILE; then every
    # 4-element group is whole and 16-byte aligned).
    def set_tile(self):
        done, flat = self.newlabel("st"), self.newlabel("st")
        prow, pn = self.p(), self.p()
        rowmode, gs, nt, tbase = self.param(P_ROWMODE), self.param(P_GRID), self.r(), self.rd()
        self.e("setp.ne.s32 %s, %s, 0;" % (prow, rowmode))
        self.e("add.u32 %s, %%tile, %s;" % (nt, gs))
        self.e("mov.u32 %tnext, 0;")
        self.e("@!%s bra.uni %s;" % (prow, flat))
        cols, ntiles = self.param(P_COLS), self.param(P_NTILES)
        self.e("mul.wide.u32 %s, %%tile, %s;" % (tbase, cols))
        self.e("mov.u32 %%limit, %s;" % cols)
        self.e("setp.lt.u32 %s, %s, %s;" % (pn, nt, ntiles))
        self.e("@%s mul.lo.u32 %%tnext, %s, %s;" % (pn, gs, cols))
        self.e("bra.uni %s;" % done)
        self.label(flat)
        n, left, end = self.param(P_N, "s64"), self.rd(), self.rd()
        self.e("mul.wide.u32 %s, %%tile, %d;" % (tbase, TILE))
        self.e("sub.s64 %s, %s, %s;" % (left, n, tbase))
        self.e("min.s64 %s, %s, %d;" % (left, left, TILE))
        self.e("cvt.u32.u64 %%limit, %s;" % left)
        self.e("add.u32 %s, %s, 1;" % (nt, nt))
        self.e("mul.wide.u32 %s, %s, %d;" % (end, nt, TILE))     # the whole next tile must exist
        self.e("setp.le.s64 %s, %s, %s;" % (pn, end, n))
        self.e("@%s shl.b32 %%tnext, %s, 12;" % (pn, gs))
        self.label(done)
        self.e("setp.eq.u32 %%pfull, %%limit, %d;" % TILE)
        p64 = self.pos0_64()
        self.e("add.u64 %s, %s, %s;" % (tbase, tbase, p64))
        self.e("shl.b64 %%tb4, %s, 2;" % tbase)

    def pvec(self):
        """4-element groups are 16-byte aligned: always in flat mode, in row mode when cols % 4 == 0"""
        pr, p2, t = self.p(), self.p(), self.r()
        self.e("setp.eq.s32 %s, %s, 0;" % (pr, self.param(P_ROWMODE)))
        self.e("and.b32 %s, %s, 3;" % (t, self.param(P_COLS)))
        self.e("setp.eq.u32 %s, %s, 0;" % (p2, t))
        self.e("or.pred %s, %s, %s;" % (pr, pr, p2))
        return pr

    # position of element j of this thread inside the tile
    def lane_pos(self, j):
        d = self.r()
        self.e("add.u32 %s, %%pos0, %d;" % (d, (j >> 2) * self.NT * 4 + (j & 3)))
        return d

    def mask_tail(self, sc):
        """scalars with the lanes beyond %limit replaced by 0"""
        out = []
        for j, s in enumerate(sc):
            pr, d = self.p(), self.f()
            self.e("setp.lt.u32 %s, %s, %%limit;" % (pr, self.lane_pos(j)))
            self.e("selp.f32 %s, %s, 0f00000000, %s;" % (d, s, pr))
            out.append(d)
        return out

    # ---- global loads and stores of one operand ----------------------------------------------
    def operand(self, want_meta=True, idx_reg=None):
        """-> (ptr u64, kind u32, dtype u32) of operand[%arg] (or [idx_reg]) from the shared-memory copy of the table"""
        a, ptr = self.r(), self.rd()
        self.e("shl.b32 %s, %s, 4;" % (a, idx_reg or "%arg"))
        if self.template:       # the index is a constant there: the entry is read straight from the kernel's parameters
            a64, base = self.rd(), self.rd()
            self.e("cvt.u64.u32 %s, %s;" % (a64, a))
            self.e("mov.u64 %s, VP;" % base)
            self.e("add.u64 %s, %s, %s;" % (base, base, a64))
            self.e("ld.param.u64 %s, [%s+%d];" % (ptr, base, P_OPERAND))
            if not want_meta:
                return ptr, None, None
            kind, dt = self.r(), self.r()
            self.e("ld.param.v2.u32 {%s, %s}, [%s+%d];" % (kind, dt, base, P_OPERAND + 8))
            return ptr, kind, dt
        self.e("add.u32 %s, %s, %%ub;" % (a, a))
        self.e("ld.shared.u64 %s, [%s+%d];" % (ptr, a, OFF_OPB))
        if not want_meta:
            return ptr, None, None
        kind, dt = self.r(), self.r()
        self.e("ld.shared.v2.u32 {%s, %s}, [%s+%d];" % (kind, dt, a, OFF_OPB + 8))
        return ptr, kind, dt

    def prefetch(self, adr, esize, cond=None):
        """pulls this CTA's next tile of a FULL operand into L2 while the current one is processed"""
        pr, pa, off = self.p(), self.rd(), self.rd()
        self.e("setp.ne.u32 %s, %%tnext, 0;" % pr)
        if cond:
            self.e("and.pred %s, %s, %s;" % (pr, pr, cond))
        self.e("mul.wide.u32 %s, %%tnext, %d;" % (off, esize))
        self.e("add.u64 %s, %s, %s;" % (pa, adr, off))
        for h in range(self.NH):
            ph, ps = self.p(), self.r()
            self.e("add.u32 %s, %%pos0, %d;" % (ps, h * self.NT * 4))
            self.e("setp.lt.u32 %s, %s, %%limit;" % (ph, ps))
            self.e("and.pred %s, %s, %s;" % (ph, ph, pr))
            self.e("@%s prefetch.global.L2 [%s+%d];" % (ph, pa, h * self.NT * 4 * esize))

    def leaf_gldf(self, dst, copy_to=None):
        """fp32 FULL operand -> dst (and copy_to)"""
        ptr, _, _ = self.operand(False)
        self.fetch()
        adr = self.rd()
        self.e("add.u64 %s, %s, %%tb4;" % (adr, ptr))
        slow = self.newlabel("gldf")
        self.e("@!%%pfull bra.uni %s;" % slow)
        pr, pa, off = self.p(), self.rd(), self.rd()
        self.e("setp.ne.u32 %s, %%tnext, 0;" % pr)
        self.e("mul.wide.u32 %s, %%tnext, 4;" % off)
        self.e("add.u64 %s, %s, %s;" % (pa, adr, off))
        for h in range(self.NH):
            self.e("@%s prefetch.global.L2 [%s+%d];" % (pr, pa, h * self.HALF_BYTES))
        for h in range(self.NH):
            self.e("ld.global.nc.v2.b64 {%s, %s}, [%s+%d];" % (dst[2 * h], dst[2 * h + 1], adr, h * self.HALF_BYTES))
        if copy_to:
            self.mov_v(copy_to, dst)
        self.jump()
        self.label(slow)
        self.prefetch(adr, 4)
        self.load_f32_slow(adr, dst)
        if copy_to:
            self.mov_v(copy_to, dst)
        self.jump()

    # ---- staged loads: arg = operand | slot << 6 ------------------------------------------------
    def staged_operand(self, masked=False):
        """-> (ptr u64 of the operand, shared address of this thread's 16 bytes of the slot); before the fetch.
        masked: the slot is a 4-bit field (the argument carries more above it)"""
        a, ptr, sl, sadr = self.r(), self.rd(), self.r(), self.r()
        self.e("and.b32 %s, %%arg, 63;" % a)
        self.e("shl.b32 %s, %s, 4;" % (a, a))
        if self.template:
            a64, base = self.rd(), self.rd()
            self.e("cvt.u64.u32 %s, %s;" % (a64, a))
            self.e("mov.u64 %s, VP;" % base)
            self.e("add.u64 %s, %s, %s;" % (base, base, a64))
            self.e("ld.param.u64 %s, [%s+%d];" % (ptr, base, P_OPERAND))
        else:
            self.e("add.u32 %s, %s, %%ub;" % (a, a))
            self.e("ld.shared.u64 %s, [%s+%d];" % (ptr, a, OFF_OPB))
        if masked:
            self.e("bfe.u32 %s, %%arg, 6, 4;" % sl)
        else:
            self.e("shr.u32 %s, %%arg, 6;" % sl)
        self.e("mad.lo.u32 %s, %s, %d, %%sa;" % (sadr, sl, SLOT_BYTES))
        return ptr, sadr

    def async_copy(self, sadr, gadr, pred):
        """this thread's two 16-byte pieces of a tile: global -> shared, asynchronously"""
        for h in range(self.NH):
            self.e("@%s cp.async.cg.shared.global [%s+%d], [%s+%d], 16;" % (pred, sadr, h * self.HALF_BYTES, gadr, h * self.HALF_BYTES))
        self.e("cp.async.commit_group;")

    def leaf_glda(self, first):
        ptr, sadr = self.staged_operand()
        self.fetch()
        adr, pr = self.rd(), self.p()
        self.e("add.u64 %s, %s, %%tb4;" % (adr, ptr))
        if first:
            self.e("mov.pred %s, %%pfull;" % pr)
        else:       # %tnext is non-zero only when the whole next tile exists
            off = self.rd()
            self.e("setp.ne.u32 %s, %%tnext, 0;" % pr)
            self.e("mul.wide.u32 %s, %%tnext, 4;" % off)
            self.e("add.u64 %s, %s, %s;" % (adr, adr, off))
        self.async_copy(sadr, adr, pr)
        self.jump()

    def next_copy(self, ptr, sadr):
        """start the copy of this CTA's next tile (when it has a whole one) into the slot"""
        adr, off, pr = self.rd(), self.rd(), self.p()
        self.e("setp.ne.u32 %s, %%tnext, 0;" % pr)
        self.e("mul.wide.u32 %s, %%tnext, 4;" % off)
        self.e("add.u64 %s, %s, %%tb4;" % (adr, ptr))
        self.e("add.u64 %s, %s, %s;" % (adr, adr, off))
        self.async_copy(sadr, adr, pr)

    # bf16 operands, read once per iteration: 8 bytes per thread and half, converted at the read
    def async_copy_h(self, sadr, gadr, pred):
        for h in range(self.NH):
            self.e("@%s cp.async.ca.shared.global [%s+%d], [%s+%d], 8;" % (pred, sadr, h * self.HALF_BYTES, gadr, h * self.NT * 8))
        self.e("cp.async.commit_group;")

    def tile_adr_h(self, ptr):
        adr, off = self.rd(), self.rd()
        self.e("shr.u64 %s, %%tb4, 1;" % off)
        self.e("add.u64 %s, %s, %s;" % (adr, ptr, off))
        return adr

    def leaf_glda0h(self):
        ptr, sadr = self.staged_operand()
        self.fetch()
        pr = self.p()
        self.e("mov.pred %s, %%pfull;" % pr)
        self.async_copy_h(sadr, self.tile_adr_h(ptr), pr)
        self.jump()

    def leaf_ldswah(self):
        A = self.A
        ptr, sadr = self.staged_operand()
        self.fetch()
        adr = self.tile_adr_h(ptr)
        slow = self.newlabel("ldswh")
        self.e("@!%%pfull bra.uni %s;" % slow)
        self.e("cp.async.wait_all;")
        for h in range(self.NH):
            w0, w1 = self.r(), self.r()
            self.e("ld.shared.v2.u32 {%s, %s}, [%s+%d];" % (w0, w1, sadr, h * self.HALF_BYTES))
            for i, w in enumerate((w0, w1)):
                lo, hi = self.r(), self.r()
                self.e("shl.b32 %s, %s, 16;" % (lo, w))
                self.e("and.b32 %s, %s, 0xffff0000;" % (hi, w))
                self.pack(lo, hi, A[2 * h + i])
        nadr, off, pr = self.rd(), self.rd(), self.p()      # the copy of the next tile, when it exists as a whole
        self.e("setp.ne.u32 %s, %%tnext, 0;" % pr)
        self.e("mul.wide.u32 %s, %%tnext, 2;" % off)
        self.e("add.u64 %s, %s, %s;" % (nadr, adr, off))
        self.async_copy_h(sadr, nadr, pr)
        self.jump()
        self.label(slow)       # a ragged tile is never staged
        self.load_bf16_slow(adr, A)
        self.jump()

    def leaf_ldsw(self, dst, copy_to=None, then_copy=False, affine=False):
        """affine: copy_to = dst * U[u] + U[u + 1] with u = arg >> 10 instead of a plain copy"""
        ptr, sadr = self.staged_operand(masked=affine)
        uu = vv = None
        if affine:
            iu, a = self.r(), self.r()
            self.e("shr.u32 %s, %%arg, 10;" % iu)
            self.e("shl.b32 %s, %s, 2;" % (a, iu))
            self.e("add.u32 %s, %s, %%ub;" % (a, a))
            u0, u1 = self.f(), self.f()
            self.e("ld.shared.f32 %s, [%s];" % (u0, a))
            self.e("ld.shared.f32 %s, [%s+4];" % (u1, a))
        self.fetch()
        if affine:
            uu, vv = self.splat(u0), self.splat(u1)

        def copy():
            if affine:
                for i in range(self.NP):
                    self.fma2(dst[i], uu, vv, copy_to[i])
            elif copy_to:
                self.mov_v(copy_to, dst)

        slow = self.newlabel("ldsw")
        self.e("@!%%pfull bra.uni %s;" % slow)
        self.e("cp.async.wait_all;")
        self.lds_v(sadr, dst)
        copy()
        if then_copy:      # the slot has been read (the loads above are ahead of the copy in this thread's order)
            self.next_copy(ptr, sadr)
        self.jump()
        self.label(slow)       # a ragged tile is never staged: load it and leave it in the slot for later reads
        adr = self.rd()
        self.e("add.u64 %s, %s, %%tb4;" % (adr, ptr))
        self.load_f32_slow(adr, dst)
        if not then_copy:      # (read once: nothing to keep; a ragged tile is followed by ragged tiles only, never staged)
            self.sts_v(sadr, dst)
        copy()
        self.jump()

    def load_f32_slow(self, adr, dst):
        pvec = self.pvec()
        for h in range(self.NH):
            lv, ln = self.newlabel("ld"), self.newlabel("ld")
            pv, pos3 = self.p(), self.r()
            self.e("add.u32 %s, %%pos0, %d;" % (pos3, h * self.NT * 4 + 3))
            self.e("setp.lt.u32 %s, %s, %%limit;" % (pv, pos3))
            self.e("and.pred %s, %s, %s;" % (pv, pv, pvec))
            self.e("@%s bra %s;" % (pv, lv))
            sc = []
            for e_ in range(4):
                pe, d = self.p(), self.f()
                self.e("setp.lt.u32 %s, %s, %%limit;" % (pe, self.lane_pos(4 * h + e_)))
                self.e("mov.f32 %s, 0f00000000;" % d)
                self.e("@%s ld.global.nc.f32 %s, [%s+%d];" % (pe, d, adr, h * self.HALF_BYTES + 4 * e_))
                sc.append(d)
            self.pack(sc[0], sc[1], dst[2 * h])
            self.pack(sc[2], sc[3], dst[2 * h + 1])
            self.e("bra %s;" % ln)
            self.label(lv)
            self.e("ld.global.nc.v2.b64 {%s, %s}, [%s+%d];" % (dst[2 * h], dst[2 * h + 1], adr, h * self.HALF_BYTES))
            self.label(ln)

    def leaf_gld(self):
        """any operand -> acc"""
        A = self.A
        ptr, kind, dt = self.operand()
        self.fetch()
        pfullk, pbf = self.p(), self.p()
        off, p64 = self.rd(), self.pos0_64()
        self.e("setp.eq.u32 %s, %s, 0;" % (pfullk, kind))
        self.e("shl.b64 %s, %s, 2;" % (p64, p64))
        self.e("selp.b64 %s, %%tb4, %s, %s;" % (off, p64, pfullk))     # FULL: this tile; ROW: the row itself
        self.e("setp.ne.u32 %s, %s, 0;" % (pbf, dt))
        lbf = self.newlabel("gld")
        self.e("@%s bra.uni %s;" % (pbf, lbf))
        adr = self.rd()
        self.e("add.u64 %s, %s, %s;" % (adr, ptr, off))
        slow = self.newlabel("gld")
        self.e("@!%%pfull bra.uni %s;" % slow)     # a full tile: whole, aligned vectors (ROW operands too)
        for h in range(self.NH):
            self.e("ld.global.nc.v2.b64 {%s, %s}, [%s+%d];" % (A[2 * h], A[2 * h + 1], adr, h * self.HALF_BYTES))
        self.jump()
        self.label(slow)
        self.prefetch(adr, 4, pfullk)
        self.load_f32_slow(adr, A)
        self.jump()
        # ---- bf16 ----
        self.label(lbf)
        adr = self.rd()
        self.e("shr.u64 %s, %s, 1;" % (off, off))
        self.e("add.u64 %s, %s, %s;" % (adr, ptr, off))
        slowb = self.newlabel("gld")
        self.e("@!%%pfull bra.uni %s;" % slowb)
        for h in range(self.NH):
            w0, w1 = self.r(), self.r()
            self.e("ld.global.nc.v2.u32 {%s, %s}, [%s+%d];" % (w0, w1, adr, h * self.NT * 8))
            for i, w in enumerate((w0, w1)):
                lo, hi = self.r(), self.r()
                self.e("shl.b32 %s, %s, 16;" % (lo, w))
                self.e("and.b32 %s, %s, 0xffff0000;" % (hi, w))
                self.pack(lo, hi, A[2 * h + i])
        self.jump()
        self.label(slowb)
        self.prefetch(adr, 2, pfullk)
        self.load_bf16_slow(adr, A)
        self.jump()

    def load_bf16_slow(self, adr, A):
        pvec = self.pvec()
        for h in range(self.NH):
            lv, ln = self.newlabel("gld"), self.newlabel("gld")
            pv, pos3 = self.p(), self.r()
            self.e("add.u32 %s, %%pos0, %d;" % (pos3, h * self.NT * 4 + 3))
            self.e("setp.lt.u32 %s, %s, %%limit;" % (pv, pos3))
            self.e("and.pred %s, %s, %s;" % (pv, pv, pvec))
            self.e("@%s bra %s;" % (pv, lv))
            sc = []
            for e_ in range(4):
                pe, d, hh = self.p(), self.r(), self.t("h")
                self.e("setp.lt.u32 %s, %s, %%limit;" % (pe, self.lane_pos(4 * h + e_)))
                self.e("mov.b16 %s, 0;" % hh)
                self.e("@%s ld.global.nc.u16 %s, [%s+%d];" % (pe, hh, adr, h * self.NT * 8 + 2 * e_))
                self.e("cvt.u32.u16 %s, %s;" % (d, hh))
                self.e("shl.b32 %s, %s, 16;" % (d, d))
                sc.append(d)
            self.pack(sc[0], sc[1], A[2 * h])
            self.pack(sc[2], sc[3], A[2 * h + 1])
            self.e("bra %s;" % ln)
            self.label(lv)
            w0, w1 = self.r(), self.r()
            self.e("ld.global.nc.v2.u32 {%s, %s}, [%s+%d];" % (w0, w1, adr, h * self.NT * 8))
            for i, w in enumerate((w0, w1)):
                lo, hi = self.r(), self.r()
                self.e("shl.b32 %s, %s, 16;" % (lo, w))
                self.e("and.b32 %s, %s, 0xffff0000;" % (hi, w))
                self.pack(lo, hi, A[2 * h + i])
            self.label(ln)

    def store_f32_slow(self, adr):
        A = self.A
        pvec = self.pvec()
        for h in range(self.NH):
            lv, ln = self.newlabel("st"), self.newlabel("st")
            pv, pos3 = self.p(), self.r()
            self.e("add.u32 %s, %%pos0, %d;" % (pos3, h * self.NT * 4 + 3))
            self.e("setp.lt.u32 %s, %s, %%limit;" % (pv, pos3))
            self.e("and.pred %s, %s, %s;" % (pv, pv, pvec))
            self.e("@%s bra %s;" % (pv, lv))
            sc = self.unpack(A[2 * h]) + self.unpack(A[2 * h + 1])
            for e_ in range(4):
                pe = self.p()
                self.e("setp.lt.u32 %s, %s, %%limit;" % (pe, self.lane_pos(4 * h + e_)))
                self.e("@%s st.global.f32 [%s+%d], %s;" % (pe, adr, h * self.HALF_BYTES + 4 * e_, sc[e_]))
            self.e("bra %s;" % ln)
            self.label(lv)
            self.e("st.global.v2.b64 [%s+%d], {%s, %s};" % (adr, h * self.HALF_BYTES, A[2 * h], A[2 * h + 1]))
            self.label(ln)

    def leaf_gstf(self, then_loop_end=False, ptr=None):
        """acc -> fp32 FULL operand (and, fused, the end of the per-tile body)"""
        if ptr is None:
            ptr, _, _ = self.operand(False)
        if not then_loop_end:
            self.fetch()
        adr = self.rd()
        self.e("add.u64 %s, %s, %%tb4;" % (adr, ptr))
        slow, done = self.newlabel("gstf"), self.newlabel("gstf")
        self.e("@!%%pfull bra.uni %s;" % slow)
        self.stg_v(adr, self.A)
        if then_loop_end:
            self.e("bra.uni %s;" % done)
        else:
            self.jump()
        self.label(slow)
        self.store_f32_slow(adr)
        if then_loop_end:
            self.label(done)
            self.leaf_loop_end()
        else:
            self.jump()

    def leaf_gst(self):
        """acc -> any operand"""
        A = self.A
        ptr, kind, dt = self.operand()
        self.fetch()
        lout = self.newlabel("gst")
        pfullk, pscal, pbf, pr, pfirst = self.p(), self.p(), self.p(), self.p(), self.p()
        off, p64 = self.rd(), self.pos0_64()
        self.e("setp.eq.u32 %s, %s, 0;" % (pfullk, kind))
        self.e("setp.eq.u32 %s, %s, 2;" % (pscal, kind))
        self.e("setp.ne.u32 %s, %s, 0;" % (pbf, dt))
        self.e("shl.b64 %s, %s, 2;" % (p64, p64))
        self.e("selp.b64 %s, %%tb4, %s, %s;" % (off, p64, pfullk))
        # ROW and SCALAR shaped outputs are written by the first tile only
        self.e("setp.eq.u32 %s, %%tile, 0;" % pfirst)
        self.e("or.pred %s, %s, %s;" % (pr, pfullk, pfirst))
        self.e("@!%s bra.uni %s;" % (pr, lout))
        lscal, lbf = self.newlabel("gst"), self.newlabel("gst")
        self.e("@%s bra.uni %s;" % (pscal, lscal))
        self.e("@%s bra.uni %s;" % (pbf, lbf))
        adr = self.rd()
        self.e("add.u64 %s, %s, %s;" % (adr, ptr, off))
        slow = self.newlabel("gst")
        self.e("@!%%pfull bra.uni %s;" % slow)
        self.stg_v(adr, A)
        self.jump()
        self.label(slow)
        self.store_f32_slow(adr)
        self.jump()
        # bf16 tensors
        self.label(lbf)
        adr = self.rd()
        self.e("shr.u64 %s, %s, 1;" % (off, off))
        self.e("add.u64 %s, %s, %s;" % (adr, ptr, off))
        slowb = self.newlabel("gst")
        self.e("@!%%pfull bra.uni %s;" % slowb)
        for h in range(self.NH):
            sc = self.unpack(A[2 * h]) + self.unpack(A[2 * h + 1])
            w0, w1 = self.r(), self.r()
            self.e("cvt.rn.bf16x2.f32 %s, %s, %s;" % (w0, sc[1], sc[0]))
            self.e("cvt.rn.bf16x2.f32 %s, %s, %s;" % (w1, sc[3], sc[2]))
            self.e("st.global.v2.u32 [%s+%d], {%s, %s};" % (adr, h * self.NT * 8, w0, w1))
        self.jump()
        self.label(slowb)
        pvec = self.pvec()
        for h in range(self.NH):
            lv, ln = self.newlabel("gst"), self.newlabel("gst")
            pv, pos3 = self.p(), self.r()
            sc = self.unpack(A[2 * h]) + self.unpack(A[2 * h + 1])
            w0, w1 = self.r(), self.r()
            self.e("cvt.rn.bf16x2.f32 %s, %s, %s;" % (w0, sc[1], sc[0]))
            self.e("cvt.rn.bf16x2.f32 %s, %s, %s;" % (w1, sc[3], sc[2]))
            self.e("add.u32 %s, %%pos0, %d;" % (pos3, h * self.NT * 4 + 3))
            self.e("setp.lt.u32 %s, %s, %%limit;" % (pv, pos3))
            self.e("and.pred %s, %s, %s;" % (pv, pv, pvec))
            self.e("@%s bra %s;" % (pv, lv))
            for e_ in range(4):
                pe, hh, w = self.p(), self.t("h"), (w0, w1)[e_ >> 1]
                self.e("setp.lt.u32 %s, %s, %%limit;" % (pe, self.lane_pos(4 * h + e_)))
                if e_ & 1:
                    self.e("{ .reg .b16 %%lo; mov.b32 {%%lo, %s}, %s; }" % (hh, w))
                else:
                    self.e("{ .reg .b16 %%hi; mov.b32 {%s, %%hi}, %s; }" % (hh, w))
                self.e("@%s st.global.u16 [%s+%d], %s;" % (pe, adr, h * self.NT * 8 + 2 * e_, hh))
            self.e("bra %s;" % ln)
            self.label(lv)
            self.e("st.global.v2.u32 [%s+%d], {%s, %s};" % (adr, h * self.NT * 8, w0, w1))
            self.label(ln)
        self.jump()
        # one scalar, written by thread 0
        self.label(lscal)
        skip, sb = self.newlabel("gst"), self.newlabel("gst")
        self.e("@!%s bra %s;" % (self.tx_is_zero(), skip))
        a0, _ = self.unpack(A[0])
        self.e("@%s bra.uni %s;" % (pbf, sb))
        self.e("st.global.f32 [%s], %s;" % (ptr, a0))
        self.e("bra %s;" % skip)
        self.label(sb)
        hh = self.t("h")
        self.e("cvt.rn.bf16.f32 %s, %s;" % (hh, a0))
        self.e("st.global.u16 [%s], %s;" % (ptr, hh))
        self.label(skip)
        self.label(lout)
        self.jump()

    # ---- leaves -------------------------------------------------------------------------------
    def lane_sum(self, vals):
        """sum of the 8 lanes of a packed self.V-wide value, as one scalar"""
        v = list(vals)
        while len(v) > 1:
            v = [self.add2(v[2 * i], v[2 * i + 1]) for i in range(len(v) // 2)]
        lo, hi = self.unpack(v[0])
        d = self.f()
        self.e("add.rn.f32 %s, %s, %s;" % (d, lo, hi))
        return d

    def leaf_joint(self, op, k):
        A, R = self.A, self.R[k]
        if op in ("rtos", "stor"):
            a = self.slot_addr()
            self.fetch()
            if op == "rtos":
                self.sts_v(a, R)
            else:
                self.lds_v(a, R)
        elif op in ("spillr", "fillr"):
            a = self.spill_addr()
            self.fetch()
            if op == "spillr":
                self.stg_v(a, R)
            else:
                self.ldg_v(a, R)
        elif op == "gldr":
            self.leaf_gldf(R, A)
            return
        elif op == "ldswr":
            self.leaf_ldsw(R, A)
            return
        elif op == "ldswar":
            self.leaf_ldsw(R, A, True)
            return
        elif op == "ldswarf":
            self.leaf_ldsw(R, A, True, affine=True)
            return
        elif op == "fmaurstl":     # acc = acc * U[arg & 511] + R; store to operand arg >> 9; end of the body
            iu, io = self.r(), self.r()
            self.e("and.b32 %s, %%arg, 511;" % iu)
            self.e("shr.u32 %s, %%arg, 9;" % io)
            u = self.uniform(iu)
            ptr, _, _ = self.operand(False, io)
            uu = self.splat(u)
            for i in range(self.NP):
                self.fma2(A[i], uu, R[i], A[i])
            self.leaf_gstf(True, ptr)
            return
        elif op == "strlds":            # R = acc; acc = S[arg]
            a = self.slot_addr()
            self.fetch()
            self.mov_v(R, A)
            self.lds_v(a, A)
        elif op.startswith("stld"):     # R[a] = acc; acc = R[k]
            self.fetch()
            self.mov_v(self.R[int(op[4])], A)
            self.mov_v(A, R)
        elif op in ("sincosr", "cossinr"):
            self.fetch()
            S, C = self.sincos(A)
            self.mov_v(R, C if op == "sincosr" else S)
            self.mov_v(A, S if op == "sincosr" else C)
        elif op.startswith("macc"):
            self.fetch()
            acc = self.S[int(op[4])]
            tail = self.newlabel("ma")
            self.e("@!%%pfull bra.uni %s;" % tail)
            t = self.mul2(A[0], R[0])
            for i in range(1, self.NP): t = self.fma2(A[i], R[i], t)
            lo, hi = self.unpack(t)
            self.e("add.rn.f32 %s, %s, %s;" % (lo, lo, hi))
            self.e("add.rn.f32 %s, %s, %s;" % (acc, acc, lo))
            self.jump()
            self.label(tail)
            m = self.packs(self.mask_tail(self.scalars(A)))
            t = self.mul2(m[0], R[0])
            for i in range(1, self.NP): t = self.fma2(m[i], R[i], t)
            lo, hi = self.unpack(t)
            self.e("add.rn.f32 %s, %s, %s;" % (lo, lo, hi))
            self.e("add.rn.f32 %s, %s, %s;" % (acc, acc, lo))
        elif op == "fmaur":
            u = self.uniform()
            self.fetch()
            uu = self.splat(u)
            for i in range(self.NP):
                self.fma2(A[i], uu, R[i], A[i])
        else:
            self.fetch()
            if op == "ldr":
                self.mov_v(A, R)
            elif op == "str":
                self.mov_v(R, A)
            elif op == "add":
                for i in range(self.NP): self.add2(A[i], R[i], A[i])
            elif op == "sub":
                for i in range(self.NP): self.sub2(A[i], R[i], A[i])
            elif op == "rsub":
                for i in range(self.NP): self.sub2(R[i], A[i], A[i])
            elif op == "mul":
                for i in range(self.NP): self.mul2(A[i], R[i], A[i])
            elif op == "divp":
                self.divp(A, R, A)
            elif op == "rdivp":
                self.divp(R, A, A)
            elif op == "addto":
                for i in range(self.NP): self.add2(R[i], A[i], R[i])
            elif op == "accum":
                tail = self.newlabel("acc")
                self.e("@!%%pfull bra.uni %s;" % tail)
                for i in range(self.NP): self.add2(R[i], A[i], R[i])
                self.jump()
                self.label(tail)
                m = self.packs(self.mask_tail(self.scalars(A)))
                for i in range(self.NP): self.add2(R[i], m[i], R[i])
            else:
                raise ValueError(op)
        self.jump()

    def leaf_plain(self, op):
        A = self.A
        if op in ("ldu", "addu", "subu", "rsubu", "mulu", "divpu", "rdivpu"):
            u = self.uniform()
            self.fetch()
            if op == "divpu":
                u = self.rcp1pabs(u)
            uu = self.splat(u)
            if op == "rdivpu":
                self.divp([uu] * self.NP, A, A)
            for i in range(self.NP):
                if op == "ldu": self.e("mov.b64 %s, %s;" % (A[i], uu))
                elif op == "addu": self.add2(A[i], uu, A[i])
                elif op == "subu": self.sub2(A[i], uu, A[i])
                elif op == "rsubu": self.sub2(uu, A[i], A[i])
                elif op in ("mulu", "divpu"): self.mul2(A[i], uu, A[i])
        elif op == "fmau":
            ia, ib = self.r(), self.r()
            self.e("and.b32 %s, %%arg, 511;" % ia)
            self.e("shr.u32 %s, %%arg, 9;" % ib)
            ua, ub = self.uniform(ia), self.uniform(ib)
            self.fetch()
            uu, vv = self.splat(ua), self.splat(ub)
            for i in range(self.NP): self.fma2(A[i], uu, vv, A[i])
        elif op == "lds":
            a = self.slot_addr(); self.fetch(); self.lds_v(a, A)
        elif op == "sts":
            a = self.slot_addr(); self.fetch(); self.sts_v(a, A)
        elif op in ("adds", "subs", "rsubs", "muls", "divps", "rdivps"):
            a = self.slot_addr(); self.fetch()
            T = self.lds_v(a)
            for i in range(self.NP):
                if op == "adds": self.add2(A[i], T[i], A[i])
                elif op == "subs": self.sub2(A[i], T[i], A[i])
                elif op == "rsubs": self.sub2(T[i], A[i], A[i])
                elif op == "muls": self.mul2(A[i], T[i], A[i])
            if op == "divps": self.divp(A, T, A)
            if op == "rdivps": self.divp(T, A, A)
        elif op == "sin":
            self.fetch(); S, _ = self.sincos(A, True, False); self.mov_v(A, S)
        elif op == "cos":
            self.fetch(); _, C = self.sincos(A, False, True); self.mov_v(A, C)
        elif op in ("sincos", "cossin"):
            a = self.slot_addr(); self.fetch()
            S, C = self.sincos(A)
            self.sts_v(a, C if op == "sincos" else S)
            self.mov_v(A, S if op == "sincos" else C)
        elif op == "expc":
            self.fetch(); self.mov_v(A, self.expc(A))
        elif op == "tanh":
            self.fetch(); self.mov_v(A, self.tanh(A))
        elif op == "sigmoid":
            self.fetch(); self.mov_v(A, self.sigmoid(A))
        elif op == "expcb":
            self.fetch(); self.mov_v(A, self.expc(A, bounded=True))
        elif op == "tanhb":
            self.fetch(); self.mov_v(A, self.tanh(A, bounded=True))
        elif op == "sigmoidb":
            self.fetch(); self.mov_v(A, self.sigmoid(A, bounded=True))
        elif op in ("relu", "step", "clampmask", "divpgb"):
            self.fetch()
            out = []
            for s in self.scalars(A):
                d = self.f()
                if op == "relu":
                    self.e("max.f32 %s, %s, 0f00000000;" % (d, s))
                elif op == "step":
                    pr = self.p()
                    self.e("setp.gt.f32 %s, %s, 0f00000000;" % (pr, s))
                    self.e("selp.f32 %s, 0f3F800000, 0f00000000, %s;" % (d, pr))
                elif op == "clampmask":
                    p1, p2 = self.p(), self.p()
                    self.e("setp.ge.f32 %s, %s, %s;" % (p1, s, fc(-10.0)))
                    self.e("setp.le.and.f32 %s, %s, %s, %s;" % (p2, s, fc(10.0), p1))
                    self.e("selp.f32 %s, 0f3F800000, 0f00000000, %s;" % (d, p2))
                else:   # -sgn(b) / (1 + |b|)^2, sgn(0) = 0
                    rr = self.rcp1pabs(s)
                    p1, p2, g = self.p(), self.p(), self.f()
                    self.e("setp.gt.f32 %s, %s, 0f00000000;" % (p1, s))
                    self.e("setp.lt.f32 %s, %s, 0f00000000;" % (p2, s))
                    self.e("selp.f32 %s, 0f3F800000, 0f00000000, %s;" % (g, p2))      # -sgn
                    self.e("selp.f32 %s, 0fBF800000, %s, %s;" % (g, g, p1))
                    self.e("mul.rn.f32 %s, %s, %s;" % (g, g, rr))
                    self.e("mul.rn.f32 %s, %s, %s;" % (d, g, rr))
                out.append(d)
            self.packs(out, A)
        elif op in ("sqrt", "rcp"):
            self.fetch()
            out = []
            for s in self.scalars(A):
                d = self.f()
                self.e("%s.approx.ftz.f32 %s, %s;" % (op, d, s))
                out.append(d)
            self.packs(out, A)
        elif op == "neg":
            self.fetch()
            m = self.K(-1.0)
            for i in range(self.NP): self.mul2(A[i], m, A[i])
        elif op == "onemsq":
            self.fetch()
            m, one = self.K(-1.0), self.K(1.0)
            for i in range(self.NP): self.fma2(self.mul2(A[i], m), A[i], one, A[i])
        elif op == "yomy":
            self.fetch()
            m, one = self.K(-1.0), self.K(1.0)
            for i in range(self.NP): self.mul2(A[i], self.fma2(A[i], m, one), A[i])
        elif op == "rbf16":
            self.fetch()
            for i in range(self.NP):
                lo, hi = self.unpack(A[i])
                w, l2, h2 = self.r(), self.r(), self.r()
                self.e("cvt.rn.bf16x2.f32 %s, %s, %s;" % (w, hi, lo))
                self.e("shl.b32 %s, %s, 16;" % (l2, w))
                self.e("and.b32 %s, %s, 0xffff0000;" % (h2, w))
                self.pack(l2, h2, A[i])
        elif op == "rowsum":     # arg: scratch buffer (bits 0..1), barrier after the read as well (bit 2)
            boff, t, psync = self.r(), self.r(), self.p()
            self.e("and.b32 %s, %%arg, 3;" % boff)
            self.e("shl.b32 %s, %s, %d;" % (boff, boff, self.red_shift))
            self.e("and.b32 %s, %%arg, 4;" % t)
            self.e("setp.ne.u32 %s, %s, 0;" % (psync, t))
            self.fetch()
            self.leaf_rowsum(boff, psync)
        elif op == "rowsumu":    # the same with arg & 7, then acc = acc * U[arg >> 3]
            boff, t, psync, iu = self.r(), self.r(), self.p(), self.r()
            self.e("and.b32 %s, %%arg, 3;" % boff)
            self.e("shl.b32 %s, %s, %d;" % (boff, boff, self.red_shift))
            self.e("and.b32 %s, %%arg, 4;" % t)
            self.e("setp.ne.u32 %s, %s, 0;" % (psync, t))
            self.e("shr.u32 %s, %%arg, 3;" % iu)
            u = self.uniform(iu)
            self.fetch()
            self.leaf_rowsum(boff, psync, u)
        elif op == "gld":
            self.leaf_gld(); return
        elif op == "gst":
            self.leaf_gst(); return
        elif op == "gldf":
            self.leaf_gldf(A); return
        elif op == "glda0":
            self.leaf_glda(True); return
        elif op == "glda":
            self.leaf_glda(False); return
        elif op == "ldsw":
            self.leaf_ldsw(A); return
        elif op == "ldswa":
            self.leaf_ldsw(A, None, True); return
        elif op == "glda0h":
            self.leaf_glda0h(); return
        elif op == "ldswah":
            self.leaf_ldswah(); return
        elif op == "gstf":
            self.leaf_gstf(); return
        elif op == "gstfl":
            self.leaf_gstf(True); return
        elif op == "fill":
            a = self.spill_addr(); self.fetch(); self.ldg_v(a, A)
        elif op == "spill":
            a = self.spill_addr(); self.fetch(); self.stg_v(a, A)
        elif op == "uload":
            self.leaf_uload()
        elif op == "uconst":
            self.leaf_uconst(); return
        elif op == "loop_begin":
            self.fetch()
            self.e("bar.sync 0;")          # uniforms written by thread 0 are visible from here on
        elif op == "loop_end":
            self.leaf_loop_end(); return
        elif op == "colout":
            self.leaf_colout()
        elif op == "scalout":
            self.leaf_scalout()
        elif op.startswith("sacc"):
            self.fetch()
            acc = self.S[int(op[4])]
            tail = self.newlabel("sa")
            self.e("@!%%pfull bra.uni %s;" % tail)
            self.e("add.rn.f32 %s, %s, %s;" % (acc, acc, self.lane_sum(A)))
            self.jump()
            self.label(tail)
            self.e("add.rn.f32 %s, %s, %s;" % (acc, acc, self.lane_sum(self.packs(self.mask_tail(self.scalars(A))))))
        elif op == "accums":     # S[arg] += acc over the valid lanes
            a = self.slot_addr(); self.fetch()
            T = self.lds_v(a)
            tail, st = self.newlabel("as"), self.newlabel("as")
            self.e("@!%%pfull bra.uni %s;" % tail)
            for i in range(self.NP): self.add2(T[i], A[i], T[i])
            self.e("bra.uni %s;" % st)
            self.label(tail)
            m = self.packs(self.mask_tail(self.scalars(A)))
            for i in range(self.NP): self.add2(T[i], m[i], T[i])
            self.label(st)
            self.sts_v(a, T)
        elif op.startswith("ascal"):
            self.leaf_scalout([self.S[int(op[5])]])
        elif op == "end":
            self.e("exit;")
            return
        else:
            raise ValueError(op)
        self.jump()

    def warp_and_lane(self):
        lane, warp, t = self.r(), self.r(), self.r()
        self.e("shr.u32 %s, %%pos0, 2;" % t)
        self.e("and.b32 %s, %s, 31;" % (lane, t))
        self.e("shr.u32 %s, %s, 5;" % (warp, t))
        return warp, lane

    def leaf_rowsum(self, boff, psync, scale=None):
        """acc = sum of acc over the row (times the scalar register scale, if given).  Successive row sums write their per-warp partials to
        different scratch buffers (the host alternates them), so one barrier per sum is enough: a
        buffer is written again only after another row sum's barrier, which every warp passes after
        it has read this one."""
        A = self.A
        full, go = self.newlabel("rs"), self.newlabel("rs")
        s = self.f()
        self.e("@%%pfull bra.uni %s;" % full)
        self.e("mov.f32 %s, %s;" % (s, self.lane_sum(self.packs(self.mask_tail(self.scalars(A))))))
        self.e("bra.uni %s;" % go)
        self.label(full)
        self.e("mov.f32 %s, %s;" % (s, self.lane_sum(A)))      # pairwise, with packed additions
        self.label(go)
        for o in (16, 8, 4, 2, 1):
            t = self.f()
            self.e("shfl.sync.bfly.b32 %s, %s, %d, 0x1f, 0xffffffff;" % (t, s, o))
            self.e("add.rn.f32 %s, %s, %s;" % (s, s, t))
        warp, lane = self.warp_and_lane()
        pr, a = self.p(), self.r()
        self.e("setp.eq.u32 %s, %s, 0;" % (pr, lane))
        base = self.r()
        self.e("add.u32 %s, %%ub, %s;" % (base, boff))
        self.e("shl.b32 %s, %s, 2;" % (a, warp))
        self.e("add.u32 %s, %s, %s;" % (a, a, base))
        self.e("@%s st.shared.f32 [%s+%d], %s;" % (pr, a, OFF_RED, s))
        self.e("bar.sync 0;")
        q = [self.rd() for _ in range(self.NT // 64)]       # the 16 per-warp partials as 8 packed pairs, summed pairwise
        for i in range(self.NT // 128):
            self.e("ld.shared.v2.b64 {%s, %s}, [%s+%d];" % (q[2 * i], q[2 * i + 1], base, OFF_RED + 16 * i))
        while len(q) > 1:
            q = [self.add2(q[2 * i], q[2 * i + 1]) for i in range(len(q) // 2)]
        lo, hi = self.unpack(q[0])
        tot = self.f()
        self.e("add.rn.f32 %s, %s, %s;" % (tot, lo, hi))
        nosync = self.newlabel("rs")
        self.e("@!%s bra.uni %s;" % (psync, nosync))
        self.e("bar.sync 0;")
        self.label(nosync)
        if scale:
            self.e("mul.rn.f32 %s, %s, %s;" % (tot, tot, scale))
        tt = self.splat(tot)
        for i in range(self.NP): self.e("mov.b64 %s, %s;" % (A[i], tt))

    def leaf_uload(self):
        """U[arg & 511] = scalar operand[arg >> 9], by thread 0"""
        skip, lb, lst = self.newlabel("ul"), self.newlabel("ul"), self.newlabel("ul")
        ui, oi, a, ptr, dt, pb, v = self.r(), self.r(), self.r(), self.rd(), self.r(), self.p(), self.f()
        self.e("and.b32 %s, %%arg, 511;" % ui)
        self.e("shr.u32 %s, %%arg, 9;" % oi)
        self.fetch()
        self.e("@!%s bra %s;" % (self.tx_is_zero(), skip))
        if self.template:
            ptr, _, dt = self.operand(idx_reg=oi)
        else:
            self.e("shl.b32 %s, %s, 4;" % (a, oi))
            self.e("add.u32 %s, %s, %%ub;" % (a, a))
            self.e("ld.shared.u64 %s, [%s+%d];" % (ptr, a, OFF_OPB))
            self.e("ld.shared.u32 %s, [%s+%d];" % (dt, a, OFF_OPB + 12))
        self.e("setp.ne.u32 %s, %s, 0;" % (pb, dt))
        self.e("@%s bra %s;" % (pb, lb))
        self.e("ld.global.nc.f32 %s, [%s];" % (v, ptr))
        self.e("bra %s;" % lst)
        self.label(lb)
        hh, w = self.t("h"), self.r()
        self.e("ld.global.nc.u16 %s, [%s];" % (hh, ptr))
        self.e("cvt.u32.u16 %s, %s;" % (w, hh))
        self.e("shl.b32 %s, %s, 16;" % (w, w))
        self.e("mov.b32 %s, %s;" % (v, w))
        self.label(lst)
        self.e("shl.b32 %s, %s, 2;" % (ui, ui))
        self.e("add.u32 %s, %s, %%ub;" % (ui, ui))
        self.e("st.shared.f32 [%s], %s;" % (ui, v))
        self.label(skip)

    def leaf_uconst(self):
        """U[arg] = the raw word that follows in the undecoded stream, by thread 0"""
        skip = self.newlabel("uc")
        ui, idx, ga, w, cb = self.r(), self.r(), self.rd(), self.r(), self.r()
        self.e("shl.b32 %s, %%arg, 2;" % ui)
        self.e("add.u32 %s, %s, %%ub;" % (ui, ui))
        if self.template:       # the literal is a constant; "next" is the instruction behind it
            self.fetch()
            self.e("@!%s bra %s;" % (self.tx_is_zero(), skip))
            self.e("mov.u32 %s, #LITERAL#;" % w)
            self.e("st.shared.u32 [%s], %s;" % (ui, w))
            self.label(skip)
            self.jump()
            return
        self.e("mov.u32 %s, dsm;" % cb)
        self.e("sub.u32 %s, %%ip, %s;" % (idx, cb))    # ip points at the literal's entry: 8 bytes per word
        self.e("shr.u32 %s, %s, 1;" % (idx, idx))          # -> byte offset in the 4-byte stream
        self.e("add.u32 %ip, %ip, 8;")
        self.fetch()
        self.e("@!%s bra %s;" % (self.tx_is_zero(), skip))
        self.e("cvt.u64.u32 %s, %s;" % (ga, idx))
        self.e("add.u64 %s, %s, %s;" % (ga, ga, self.param(P_CODE, "u64")))
        self.e("ld.global.nc.u32 %s, [%s];" % (w, ga))
        self.e("st.shared.u32 [%s], %s;" % (ui, w))
        self.label(skip)
        self.jump()

    def leaf_loop_end(self):
        out = self.newlabel("le")
        pr, cb = self.p(), self.r()
        self.e("add.u32 %%tile, %%tile, %s;" % self.param(P_GRID))
        self.e("setp.ge.u32 %s, %%tile, %s;" % (pr, self.param(P_NTILES)))
        self.e("@%s bra.uni %s;" % (pr, out))
        # a full tile (the common case) only moves the offsets on; a ragged one takes the general path
        slow, join = self.newlabel("le"), self.newlabel("le")
        pf, pn, nt, stride, gs, nfull = self.p(), self.p(), self.r(), self.rd(), self.param(P_GRID), self.param(P_NFULL)
        self.e("setp.lt.u32 %s, %%tile, %s;" % (pf, nfull))
        self.e("@!%s bra.uni %s;" % (pf, slow))
        self.e("mul.wide.u32 %s, %s, %d;" % (stride, gs, SLOT_BYTES))
        self.e("add.u64 %%tb4, %%tb4, %s;" % stride)
        self.e("add.u32 %s, %%tile, %s;" % (nt, gs))
        self.e("setp.lt.u32 %s, %s, %s;" % (pn, nt, nfull))
        self.e("shl.b32 %s, %s, 12;" % (nt, gs))
        self.e("selp.u32 %%tnext, %s, 0, %s;" % (nt, pn))
        self.e("bra.uni %s;" % join)
        self.label(slow)
        self.set_tile()
        self.label(join)
        if self.template:
            self.e("mov.u32 %arg, #LOOPARG#;")
            self.e("bra.uni #LOOP#;")
        else:
            self.e("mov.u32 %s, dsm;" % cb)
            self.e("mad.lo.u32 %%ip, %s, 8, %s;" % (self.param(P_LOOPSTART), cb))
        self.label(out)
        self.fetch()
        self.jump()

    def partial_index(self):
        """arg * grid + cta (taken before the fetch)"""
        o, t, cta = self.rd(), self.rd(), self.r()
        self.e("mul.wide.u32 %s, %%arg, %s;" % (o, self.param(P_GRID)))
        self.e("mov.u32 %s, %%ctaid.x;" % cta)
        self.e("cvt.u64.u32 %s, %s;" % (t, cta))
        self.e("add.u64 %s, %s, %s;" % (o, o, t))
        return o

    def leaf_colout(self):
        """column partial sums: colpart[arg][cta][c] = acc"""
        A = self.A
        o = self.partial_index()
        self.fetch()
        cols, c64 = self.param(P_COLS), self.rd()
        self.e("cvt.u64.u32 %s, %s;" % (c64, cols))
        self.e("mul.lo.u64 %s, %s, %s;" % (o, o, c64))
        self.e("add.u64 %s, %s, %s;" % (o, o, self.pos0_64()))
        self.e("shl.b64 %s, %s, 2;" % (o, o))
        self.e("add.u64 %s, %s, %s;" % (o, o, self.param(P_COLPART, "u64")))
        sc = self.scalars(A)
        for j in range(self.V):
            pr = self.p()
            self.e("setp.lt.u32 %s, %s, %s;" % (pr, self.lane_pos(j), cols))
            self.e("@%s st.global.f32 [%s+%d], %s;" % (pr, o, ((j >> 2) * self.NT * 4 + (j & 3)) * 4, sc[j]))

    def leaf_scalout(self, values=None):
        """scalar partial sum: scalpart[arg][cta] = block sum in fp64 of acc (or of the given scalars)"""
        A = self.A
        o = self.partial_index()
        self.fetch()
        self.e("shl.b64 %s, %s, 3;" % (o, o))
        self.e("add.u64 %s, %s, %s;" % (o, o, self.param(P_SCALPART, "u64")))
        s = self.fd()
        self.e("mov.f64 %s, 0d0000000000000000;" % s)
        for x in (values if values is not None else self.scalars(A)):
            d = self.fd()
            self.e("cvt.f64.f32 %s, %s;" % (d, x))
            self.e("add.f64 %s, %s, %s;" % (s, s, d))
        for off in (16, 8, 4, 2, 1):
            lo, hi, l2, h2, d = self.r(), self.r(), self.r(), self.r(), self.fd()
            self.e("mov.b64 {%s, %s}, %s;" % (lo, hi, s))
            self.e("shfl.sync.bfly.b32 %s, %s, %d, 0x1f, 0xffffffff;" % (l2, lo, off))
            self.e("shfl.sync.bfly.b32 %s, %s, %d, 0x1f, 0xffffffff;" % (h2, hi, off))
            self.e("mov.b64 %s, {%s, %s};" % (d, l2, h2))
            self.e("add.f64 %s, %s, %s;" % (s, s, d))
        warp, lane = self.warp_and_lane()
        pr, a = self.p(), self.r()
        self.e("setp.eq.u32 %s, %s, 0;" % (pr, lane))
        self.e("shl.b32 %s, %s, 3;" % (a, warp))
        self.e("add.u32 %s, %s, %%ub;" % (a, a))
        self.e("@%s st.shared.f64 [%s+%d], %s;" % (pr, a, OFF_RED + 512, s))
        self.e("bar.sync 0;")
        skip = self.newlabel("so")
        self.e("@!%s bra %s;" % (self.tx_is_zero(), skip))
        tot = self.fd()
        self.e("mov.f64 %s, 0d0000000000000000;" % tot)
        for i in range(self.NT // 32):
            d = self.fd()
            self.e("ld.shared.f64 %s, [%%ub+%d];" % (d, OFF_RED + 512 + 8 * i))
            self.e("add.f64 %s, %s, %s;" % (tot, tot, d))
        self.e("st.global.f64 [%s], %s;" % (o, tot))
        self.label(skip)
        self.e("bar.sync 0;")

    # ---- the kernel ---------------------------------------------------------------------------
    def cases(self):
        """case id -> ("j", op, slot) | ("p", op, 0) | ("bad", op, slot)"""
        out = []
        for op in JOINT:
            for k in range(JOINT_STRIDE):
                no_slot = op.startswith("stld") and int(op[4]) >= self.nr
                out.append(("j", op, k) if k < self.nr and not no_slot else ("bad", op, k))
        for op in PLAIN:
            out.append(("p", op, 0))
        return out

    def prologue(self):
        e = self.e
        tx = self.r()
        e("mov.u32 %s, %%tid.x;" % tx)
        e("shl.b32 %%pos0, %s, 2;" % tx)
        # shared memory: decoded code | uniforms | reduction scratch | operand table | slots
        e("mov.u32 %ub, dsm;")
        if not self.template:       # a specialised kernel holds no instruction stream: its uniforms start the area
            ncode, t0 = self.param(P_NCODE, "s32"), self.r()
            e("add.s32 %s, %s, 3;" % (t0, ncode))
            e("and.b32 %s, %s, 0xfffffffc;" % (t0, t0))
            e("shl.b32 %s, %s, 3;" % (t0, t0))
            e("add.u32 %%ub, %%ub, %s;" % t0)
        e("mad.lo.u32 %%sa, %s, 16, %%ub;" % tx)
        e("add.u32 %%sa, %%sa, %d;" % OFF_SLOTS)
        # operand table -> shared memory (one entry per thread); a specialised kernel reads its entries, whose
        # indices are constants there, straight from the parameters
        for i in range(0 if self.template else MAX_OPERANDS):
            pr, ptr, k, d = self.p(), self.rd(), self.r(), self.r()
            e("setp.eq.u32 %s, %s, %d;" % (pr, tx, i))
            e("ld.param.u64 %s, [VP+%d];" % (ptr, P_OPERAND + 16 * i))
            e("ld.param.u32 %s, [VP+%d];" % (k, P_OPERAND + 16 * i + 8))
            e("ld.param.u32 %s, [VP+%d];" % (d, P_OPERAND + 16 * i + 12))
            e("@%s st.shared.u64 [%%ub+%d], %s;" % (pr, OFF_OPB + 16 * i, ptr))
            e("@%s st.shared.v2.u32 [%%ub+%d], {%s, %s};" % (pr, OFF_OPB + 16 * i + 8, k, d))
        if not self.template:
            # decode the instruction stream: {case id, argument} per word
            ncode = self.param(P_NCODE, "s32")
            lp, ld_ = self.newlabel("dec"), self.newlabel("dec")
            i_, pr, ga, w, c, a, sa, code = self.r(), self.p(), self.rd(), self.r(), self.r(), self.r(), self.r(), self.param(P_CODE, "u64")
            e("mov.u32 %s, %s;" % (i_, tx))
            self.label(lp)
            e("setp.ge.s32 %s, %s, %s;" % (pr, i_, ncode))
            e("@%s bra %s;" % (pr, ld_))
            e("mul.wide.u32 %s, %s, 4;" % (ga, i_))
            e("add.u64 %s, %s, %s;" % (ga, ga, code))
            e("ld.global.nc.u32 %s, [%s];" % (w, ga))
            e("and.b32 %s, %s, 1023;" % (c, w))
            e("shr.u32 %s, %s, 14;" % (a, w))
            e("mov.u32 %s, dsm;" % sa)
            e("mad.lo.u32 %s, %s, 8, %s;" % (sa, i_, sa))
            e("st.shared.v2.u32 [%s], {%s, %s};" % (sa, c, a))
            e("add.u32 %s, %s, %d;" % (i_, i_, self.NT))
            e("bra %s;" % lp)
            self.label(ld_)
        e("bar.sync 0;")
        # per-CTA spill area: spill + cta * n_spill * TILE floats, this thread's 16 bytes
        t2, t3, cta = self.rd(), self.rd(), self.r()
        e("mov.u32 %s, %%ctaid.x;" % cta)
        e("mul.wide.u32 %s, %s, %d;" % (t2, cta, SLOT_BYTES))
        e("cvt.u64.u32 %s, %s;" % (t3, self.param(P_NSPILL)))
        e("mad.lo.u64 %%spb, %s, %s, %s;" % (t2, t3, self.param(P_SPILL, "u64")))
        e("mul.wide.u32 %s, %s, 16;" % (t2, tx))
        e("add.u64 %%spb, %%spb, %s;" % t2)
        for r_ in self.A + sum(self.R, []):
            e("mov.b64 %s, 0;" % r_)
        for r_ in self.S:
            e("mov.f32 %s, 0f00000000;" % r_)
        # CTA 0 clears the status word of the next run (the host alternates between two words)
        skip_c = self.newlabel("sc")
        pc, pz, sc_ptr, zero = self.p(), self.p(), self.param(P_STATUSCLEAR, "u64"), self.r()
        e("or.b32 %s, %s, %s;" % (zero, cta, tx))
        e("setp.ne.u32 %s, %s, 0;" % (pc, zero))
        e("setp.eq.u64 %s, %s, 0;" % (pz, sc_ptr))
        e("or.pred %s, %s, %s;" % (pc, pc, pz))
        e("@%s bra %s;" % (pc, skip_c))
        e("mov.u32 %s, 0;" % zero)
        e("st.global.u32 [%s], %s;" % (sc_ptr, zero))
        self.label(skip_c)
        e("mov.u32 %%tile, %s;" % cta)
        self.set_tile()

    def declarations(self):
        decl = []
        for kind, ty in (("f", ".f32"), ("r", ".b32"), ("rd", ".b64"), ("p", ".pred"), ("fd", ".f64"), ("h", ".b16")):
            if self.cnt[kind]:
                decl.append("\t.reg %s %%%s<%d>;" % (ty, kind, self.cnt[kind]))
        decl.append("\t.reg .b32 %pos0, %limit, %tnext, %tile, %ub, %sa, %ip, %case, %arg;")
        decl.append("\t.reg .b64 %tb4, %spb;")
        decl.append("\t.reg .pred %pfull;")
        decl.append("\t.local .align 8 .b8 PHBUF[96];")
        decl.append("\t.reg .b64 %s;" % ", ".join(self.PX + self.PR + self.PK))
        decl.append("\t.reg .b32 %phsite;")
        decl.append("\t.reg .f32 %s;" % ", ".join(self.S))
        decl.append("\t.reg .b64 %s;" % ", ".join(self.A + sum(self.R, [])))
        return decl

    def build(self):
        cases = self.cases()
        bad = "$BAD_%s" % self.name
        labels = [bad if c[0] == "bad" else "$C_%s_%d" % (self.name, i) for i, c in enumerate(cases)]
        body = self.lines
        e = self.e
        self.prologue()
        e("mov.u32 %ip, dsm;")
        self.fetch()
        e("JT_%s: .branchtargets %s;" % (self.name, ", ".join(labels)))
        self.label("$DISPATCH_%s" % self.name)
        e("brx.idx.uni %%case, JT_%s;" % self.name)
        # ---- leaves ----
        for lab, (kind, op, k) in zip(labels, cases):
            if kind == "bad":
                continue
            self.label(lab)
            self.own_brx = op in HOT
            if kind == "j":
                self.leaf_joint(op, k)
            else:
                self.leaf_plain(op)
            self.own_brx = False
        # a register slot this build does not have: report and stop (the host never emits one)
        self.label(bad)
        skip = self.newlabel("bad")
        v = self.r()
        e("@!%s bra %s;" % (self.tx_is_zero(), skip))
        e("mov.u32 %s, -7;" % v)
        e("st.global.u32 [%s], %s;" % (self.param(P_STATUS, "u64"), v))
        self.label(skip)
        e("exit;")
        self.lines.extend(self.cold)
        self.emit_general_reduction()
        # ---- assemble text ----
        head = []
        head.append(".const .align 8 .b64 KT_%s[%d] = {%s};" % (self.name, max(1, len(self.kt)), ", ".join("0x%016X" % w for w in self.kt) or "0"))
        head.append(".visible .entry %s(.param .align 8 .b8 VP[%d])" % (self.name, P_SIZE))
        head.append(".maxntid %d, 1, 1" % self.NT)
        head.append(".minnctapersm %d" % self.ctas)
        head.append("{")
        return "\n".join(head + self.declarations() + body + ["}"]) + "\n"

    def build_templates(self):
        """-> dict(head, prologue, leaves = {case id: (text, cold text, [site return labels])}, reduction):
        the pieces of a kernel that runs one instruction stream as straight-line code.  Placeholders:
        #I# (number of the instruction, makes labels unique), #NEXT# / #NEXTARG# (label and argument of the
        instruction that follows), #LOOP# / #LOOPARG# (of the first instruction of the per-tile body),
        #LITERAL# (the word behind a uconst), #SITEk# (number of the leaf's k-th sin/cos site among all
        sites of the kernel), #PHRET# (the return labels of all sites)."""
        assert self.template

        def capture(fn):
            self.lines, self.cold, self.leaf_sites = [], [], []
            fn()
            return "\n".join(self.lines) + "\n", "\n".join(self.cold) + ("\n" if self.cold else ""), list(self.leaf_sites)

        prologue = capture(self.prologue)[0].replace("#I#", "P")
        leaves = {}
        for i, (kind, op, k) in enumerate(self.cases()):
            if kind == "bad":
                continue
            leaves[i] = capture((lambda: self.leaf_joint(op, k)) if kind == "j" else (lambda: self.leaf_plain(op)))
        self.ph_sites = ["x"]
        reduction = capture(self.emit_general_reduction)[0].replace("#I#", "R")
        head = [".visible .entry #ENTRY#(.param .align 8 .b8 VP[%d])" % P_SIZE, ".maxntid %d, 1, 1" % self.NT,
                ".minnctapersm %d" % self.ctas, "{"] + self.declarations()
        assert not self.kt, "packed constants are immediates"
        return dict(head="\n".join(head) + "\n", prologue=prologue, leaves=leaves, reduction=reduction)


# name, register slots, CTAs per SM, threads per CTA.  The generator also takes 1024 threads (four elements per
# thread, 32 warps per SM with the wide build's slots); measured on the row DAGs that was 13 % slower than 512
# (the fixed cost of a dispatch is then spread over half the arithmetic), so no such kernel is built.  Loading the
# instruction pairs two leaves ahead (so that the indexed branch of a short leaf never waits for shared memory)
# was 4 % slower as well: the two register moves per dispatch cost more than the wait.
VARIANTS = [("dragon_vm_wide", 7, 1, 512), ("dragon_vm_dense", 3, 2, 512)]


MODULE_HEAD = [".version 8.8", ".target sm_100a", ".address_size 64", "", ".extern .shared .align 16 .b8 dsm[];",
               # 2/pi = 0x0.A2F9836E4E44... behind one word of zeros (its integer part), most significant word first
               ".const .align 4 .b32 TWO_OVER_PI[9] = {0x00000000, 0xA2F9836E, 0x4E441529, 0xFC2757D1, 0xF534DDC0, 0xDB629599, 0x3C439041, 0xFE5163AB, 0xDEBBC561};", ""]


def generate():
    out = list(MODULE_HEAD)
    for name, nr, ctas, threads in VARIANTS:
        out.append(Kernel(name, nr, ctas, threads).build())
    return "\n".join(out)


def specialise(template, code, loop_start, entry="dragon_vm_spec"):
    """Python twin of csrc/specialize.cpp (used by the tests to check the C++ stitcher and the templates):
    the PTX of the kernel that runs the instruction words ``code`` as straight-line code."""
    n = len(code)
    uconst = JOINT_STRIDE * len(JOINT) + PLAIN.index("uconst")
    body, cold, sites = [], [], []
    pc = 0

    def label(i):
        return "$I_%d" % i if i < n else "$I_END"

    while pc < n:
        case, arg = code[pc] & 1023, code[pc] >> 14
        text, cold_text, leaf_sites = template["leaves"][case]
        nxt = pc + 2 if case == uconst else pc + 1
        sub = {"I": str(pc), "NEXT": label(nxt), "NEXTARG": str(code[nxt] >> 14 if nxt < n else 0), "LOOP": label(loop_start),
               "LOOPARG": str(code[loop_start] >> 14), "LITERAL": str(code[pc + 1]) if case == uconst else "0"}
        for k in range(len(leaf_sites)):
            sub["SITE%d" % k] = str(len(sites) + k)

        def fill(t):
            parts = t.split("#")
            return "".join(p if i % 2 == 0 else sub[p] for i, p in enumerate(parts))

        sites += [fill(l) for l in leaf_sites]
        body.append(label(pc) + ":\n" + fill(text))
        cold.append(fill(cold_text))
        pc = nxt
    out = "\n".join(MODULE_HEAD) + "\n" + template["head"].replace("#ENTRY#", entry) + template["prologue"]
    out += "\tmov.u32 %%arg, %d;\n" % (code[0] >> 14) + "".join(body) + "$I_END:\n\texit;\n" + "".join(cold)
    if sites:
        out += template["reduction"].replace("#PHRET#", ", ".join(sites))
    return out + "}\n"


def templates_source():
    """C++ source of the leaf templates of both builds, compiled into the library for csrc/specialize.cpp."""
    out = ["// generated by vm_ptxgen.py: the leaves of the graph-VM kernel as PTX text with placeholders", "#include \"vm_templates.h\"", "",
           "namespace dragon {", "namespace vmt {", ""]

    def lit(text):
        # raw string literals in pieces: some compilers limit the length of one literal
        chunks, cur, size = [], [], 0
        for line in text.splitlines(True):
            cur.append(line)
            size += len(line)
            if size > 12000:
                chunks.append("".join(cur)); cur, size = [], 0
        if cur or not chunks:
            chunks.append("".join(cur))
        return "\n".join('R"PTX(%s)PTX"' % c for c in chunks)

    out.append("const char* const kModuleHead = %s;" % lit("\n".join(MODULE_HEAD) + "\n"))
    names = []
    for name, nr, ctas, threads in VARIANTS:
        t = Kernel(name, nr, ctas, threads, template=True).build_templates()
        n_cases = JOINT_STRIDE * len(JOINT) + len(PLAIN)
        tag = name.replace("dragon_vm_", "")
        out.append("static const Leaf kLeaves_%s[%d] = {" % (tag, n_cases))
        for i in range(n_cases):
            if i in t["leaves"]:
                text, cold, sites = t["leaves"][i]
                out.append("  {%s,\n   %s,\n   %d, \"%s\"}," % (lit(text), lit(cold), len(sites), ",".join(sites)))
            else:
                out.append("  {nullptr, nullptr, 0, nullptr},")
        out.append("};")
        names.append((tag, nr, n_cases, t))
    out.append("const Variant kVariants[%d] = {" % len(names))
    for tag, nr, n_cases, t in names:
        out.append("  {%d, %d, %s,\n   %s,\n   %s,\n   kLeaves_%s}," % (nr, n_cases, lit(t["head"]), lit(t["prologue"]), lit(t["reduction"]), tag))
    out.append("};")
    out.append("const int kNumVariants = %d;" % len(names))
    out += ["", "}  // namespace vmt", "}  // namespace dragon", ""]
    return "\n".join(out)




if __name__ == "__main__":
    text = templates_source() if "--templates" in sys.argv[1:] else generate()
    sys.argv = [a for a in sys.argv if a != "--templates"]
    if len(sys.argv) > 1:
        open(sys.argv[1], "w").write(text)
    else:
        sys.stdout.write(text)
