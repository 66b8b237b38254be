"""Generator of the graph-VM kernel, written directly in PTX for sm_100a.

The VM (csrc/vm_isa.h) is an accumulator machine whose instructions work on V-wide per-thread
values.  An interpreter spends its time in two places: the arithmetic of the instructions and the
dispatch between them.  Both are written out here instruction by instruction instead of leaving
them to a C++ compiler:

* dispatch is one 64-bit shared-memory load of the pre-decoded {case, argument} pair, a pointer
  increment and one uniform indexed branch (``brx.idx.uni``) over a table of leaf labels; the
  fetch of the next pair is issued at the top of a leaf, ahead of its arithmetic;
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

NT = 512            # threads per CTA
V = 8               # elements per thread
NP = V // 2         # packed pairs per value
TILE = NT * V       # 4096 elements
SLOT_BYTES = TILE * 4
HALF_BYTES = NT * 16
MAX_OPERANDS = 40
MAX_UNIFORMS = 512

# Params (csrc/vm_isa.h): byte offsets
P_CODE, P_NCODE, P_ROWMODE, P_N, P_COLS, P_NSPILL, P_SPILL, P_COLPART, P_SCALPART, P_STATUS, P_OPERAND = 0, 8, 12, 16, 24, 28, 32, 40, 48, 56, 64
P_SIZE = P_OPERAND + 16 * MAX_OPERANDS

JOINT = ["ldr", "str", "add", "sub", "rsub", "mul", "divp", "rdivp", "addto", "accum", "fmaur", "rtos", "stor", "spillr", "fillr"]
PLAIN = ["ldu", "addu", "subu", "rsubu", "mulu", "divpu", "rdivpu", "fmau", "lds", "sts", "adds", "subs", "rsubs", "muls", "divps",
         "rdivps", "sin", "cos", "sincos", "expc", "tanh", "sigmoid", "relu", "neg", "step", "clampmask", "onemsq", "yomy", "divpgb",
         "rbf16", "rowsum", "gld", "gst", "fill", "spill", "uload", "uconst", "loop_begin", "loop_end", "colout", "scalout", "end"]


def f32bits(x):
    return struct.unpack("<I", struct.pack("<f", x))[0]


def fc(x):
    return "0f%08X" % f32bits(x)


class Kernel:
    def __init__(self, name, nr, ctas_per_sm):
        self.name, self.nr, self.ctas = name, nr, ctas_per_sm
        self.lines = []
        self.cnt = {"f": 0, "r": 0, "rd": 0, "p": 0, "fd": 0, "h": 0}
        self.nlabel = 0
        self.kt = []          # packed constants (u64 words)
        self.A = ["%%A%d" % i for i in range(NP)]
        self.R = [["%%R%d_%d" % (k, i) for i in range(NP)] for k in range(nr)]

    # ---- plumbing -------------------------------------------------------------------------
    def e(self, s):
        self.lines.append("\t" + s)

    def label(self, s):
        self.lines.append(s + ":")

    def newlabel(self, stem="L"):
        self.nlabel += 1
        return "$%s_%s_%d" % (stem, self.name, self.nlabel)

    def t(self, kind):
        self.cnt[kind] += 1
        return "%%%s%d" % ({"f": "f", "r": "r", "rd": "rd", "p": "p", "fd": "fd", "h": "h"}[kind], self.cnt[kind] - 1)

    def f(self): return self.t("f")
    def r(self): return self.t("r")
    def rd(self): return self.t("rd")
    def p(self): return self.t("p")
    def fd(self): return self.t("fd")

    def K(self, x, y=None):
        """packed constant {x, y} (y defaults to x) loaded from the constant table"""
        w = f32bits(x) | (f32bits(x if y is None else y) << 32)
        if w not in self.kt:
            self.kt.append(w)
        d = self.rd()
        self.e("ld.const.b64 %s, [KT_%s+%d];" % (d, self.name, 8 * self.kt.index(w)))
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

    def add2(self, a, b, d=None):
        d = d or self.rd()
        self.e("add.rn.f32x2 %s, %s, %s;" % (d, a, b))
        return d

    def sub2(self, a, b, d=None):
        d = d or self.rd()
        self.e("sub.rn.f32x2 %s, %s, %s;" % (d, a, b))
        return d

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
        return [self.pack(sc[2 * i], sc[2 * i + 1], dst[i] if dst else None) for i in range(NP)]

    def rcp(self, x):
        d = self.f()
        self.e("rcp.approx.ftz.f32 %s, %s;" % (d, x))
        return d

    def rcp1pabs(self, x):
        """1 / (1 + |x|)"""
        a = self.f()
        self.e("abs.f32 %s, %s;" % (a, x))
        self.e("add.f32 %s, %s, 0f3F800000;" % (a, a))
        return self.rcp(a)

    # ---- dispatch ---------------------------------------------------------------------------
    def fetch(self):
        self.e("ld.shared.v2.u32 {%case, %arg}, [%ip];")
        self.e("add.u32 %ip, %ip, 8;")

    def jump(self):
        self.e("brx.idx.uni %%case, JT_%s;" % self.name)

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
        d = dst or [self.rd() for _ in range(NP)]
        self.e("ld.shared.v2.b64 {%s, %s}, [%s];" % (d[0], d[1], addr))
        self.e("ld.shared.v2.b64 {%s, %s}, [%s+%d];" % (d[2], d[3], addr, HALF_BYTES))
        return d

    def sts_v(self, addr, src):
        self.e("st.shared.v2.b64 [%s], {%s, %s};" % (addr, src[0], src[1]))
        self.e("st.shared.v2.b64 [%s+%d], {%s, %s};" % (addr, HALF_BYTES, src[2], src[3]))

    def ldg_v(self, addr, dst=None):
        d = dst or [self.rd() for _ in range(NP)]
        self.e("ld.global.v2.b64 {%s, %s}, [%s];" % (d[0], d[1], addr))
        self.e("ld.global.v2.b64 {%s, %s}, [%s+%d];" % (d[2], d[3], addr, HALF_BYTES))
        return d

    def stg_v(self, addr, src):
        self.e("st.global.v2.b64 [%s], {%s, %s};" % (addr, src[0], src[1]))
        self.e("st.global.v2.b64 [%s+%d], {%s, %s};" % (addr, HALF_BYTES, src[2], src[3]))

    def mov_v(self, dst, src):
        for i in range(NP):
            self.e("mov.b64 %s, %s;" % (dst[i], src[i]))

    # ---- elementary functions (csrc/vm_math.h, operation by operation) -----------------------
    def reduce_pio2(self, x):
        """x: packed pair -> (r packed, kb packed); the low bits of kb's lanes are the quadrant"""
        lo, hi = self.unpack(x)
        g = []
        for s in (lo, hi):   # beyond 6.5e6 (and for inf/NaN) the argument becomes x - x: 0, or NaN
            a, z, q, pr = self.f(), self.f(), self.f(), self.p()
            self.e("abs.f32 %s, %s;" % (a, s))
            self.e("setp.le.f32 %s, %s, %s;" % (pr, a, fc(6.5e6)))
            self.e("sub.f32 %s, %s, %s;" % (z, s, s))
            self.e("selp.f32 %s, %s, %s, %s;" % (q, s, z, pr))
            g.append(q)
        xg = self.pack(g[0], g[1])
        big = 12582912.0
        kb = self.fma2(xg, self.K(0.636619772367581343), self.K(big))
        k = self.add2(kb, self.K(-big))
        r = self.fma2(k, self.K(-1.57079637050628662109375), xg)
        r = self.fma2(k, self.K(4.371138828673793e-8), r)
        r = self.fma2(k, self.K(1.7151245100058819e-15), r)
        return r, kb

    def sin_poly(self, r, z):
        p = self.fma2(z, self.K(-1.9515285269243e-4), self.K(8.33216077944338e-3))
        p = self.fma2(z, p, self.K(-1.6666654609873324e-1))
        return self.fma2(self.mul2(r, z), p, r)

    def cos_poly(self, z):
        p = self.fma2(z, self.K(2.4433150705502356e-5), self.K(-1.3887316189460366e-3))
        p = self.fma2(z, p, self.K(4.1666645681363114e-2))
        return self.fma2(self.mul2(z, z), p, self.fma2(z, self.K(-0.5), self.K(1.0)))

    def sincos(self, xs, want_sin=True, want_cos=True):
        S, C = [], []
        for x in xs:
            r, kb = self.reduce_pio2(x)
            z = self.mul2(r, r)
            ps, pc = self.unpack(self.sin_poly(r, z)), self.unpack(self.cos_poly(z))
            q = [self.r(), self.r()]
            self.e("mov.b64 {%s, %s}, %s;" % (q[0], q[1], kb))
            so, co = [], []
            for j in range(2):
                b, pr = self.r(), self.p()
                self.e("and.b32 %s, %s, 1;" % (b, q[j]))
                self.e("setp.ne.u32 %s, %s, 0;" % (pr, b))
                if want_sin:
                    s, u = self.f(), self.r()
                    self.e("selp.f32 %s, %s, %s, %s;" % (s, pc[j], ps[j], pr))
                    self.e("shl.b32 %s, %s, 30;" % (u, q[j]))
                    self.e("and.b32 %s, %s, 0x80000000;" % (u, u))
                    self.e("xor.b32 %s, %s, %s;" % (s, s, u))
                    so.append(s)
                if want_cos:
                    c, v = self.f(), self.r()
                    self.e("selp.f32 %s, %s, %s, %s;" % (c, ps[j], pc[j], pr))
                    self.e("add.u32 %s, %s, 1;" % (v, q[j]))
                    self.e("shl.b32 %s, %s, 30;" % (v, v))
                    self.e("and.b32 %s, %s, 0x80000000;" % (v, v))
                    self.e("xor.b32 %s, %s, %s;" % (c, c, v))
                    co.append(c)
            if want_sin:
                S.append(self.pack(so[0], so[1]))
            if want_cos:
                C.append(self.pack(co[0], co[1]))
        return S, C

    def exp_core(self, x):
        """x packed, already clamped so that the result is a normal number: e^x = p * 2^n with the
        2^n applied by adding n to the exponent field of p (exact, as the multiplication is)"""
        big = 12582912.0
        nb = self.fma2(x, self.K(1.44269504088896341), self.K(big))
        n = self.add2(nb, self.K(-big))
        r = self.fma2(n, self.K(-0.693145751953125), x)
        r = self.fma2(n, self.K(-1.428606765330187e-6), r)
        e = self.fma2(r, self.K(1.3814663108745e-3), self.K(8.36871131029872e-3))
        e = self.fma2(r, e, self.K(4.16683865189979e-2))
        e = self.fma2(r, e, self.K(1.6666520673866728e-1))
        e = self.fma2(r, e, self.K(4.9999993454926206e-1))
        p = self.add2(self.fma2(self.mul2(r, r), e, r), self.K(1.0))
        pb, nbb = [self.r(), self.r()], [self.r(), self.r()]
        self.e("mov.b64 {%s, %s}, %s;" % (pb[0], pb[1], p))
        self.e("mov.b64 {%s, %s}, %s;" % (nbb[0], nbb[1], nb))
        for j in range(2):
            self.e("shl.b32 %s, %s, 23;" % (nbb[j], nbb[j]))
            self.e("add.u32 %s, %s, %s;" % (pb[j], pb[j], nbb[j]))
        return self.pack(pb[0], pb[1])

    def clamp(self, s, lo, hi):
        d = self.f()
        self.e("max.f32 %s, %s, %s;" % (d, s, fc(lo)))
        self.e("min.f32 %s, %s, %s;" % (d, d, fc(hi)))
        return d

    EXP_LO, EXP_HI = -86.0, 88.7   # e^x stays a normal fp32 number on this range

    def expc(self, xs):
        out = []
        for x in xs:
            lo, hi = self.unpack(x)
            out.append(self.exp_core(self.pack(self.clamp(lo, -10.0, 10.0), self.clamp(hi, -10.0, 10.0))))
        return out

    def sigmoid(self, xs):
        out = []
        for x in xs:
            lo, hi = self.unpack(self.mul2(x, self.K(-1.0)))
            e = self.exp_core(self.pack(self.clamp(lo, self.EXP_LO, self.EXP_HI), self.clamp(hi, self.EXP_LO, self.EXP_HI)))
            l2, h2 = self.unpack(self.add2(e, self.K(1.0)))
            out.append(self.pack(self.rcp(l2), self.rcp(h2)))
        return out

    def tanh(self, xs):
        out = []
        for x in xs:
            z = self.mul2(x, x)
            p = self.fma2(z, self.K(-5.89516999486988e-3), self.K(2.079598263424288e-2))
            p = self.fma2(z, p, self.K(-5.378383380013826e-2))
            p = self.fma2(z, p, self.K(1.333192417199396e-1))
            p = self.fma2(z, p, self.K(-3.3333298003965545e-1))
            small = self.unpack(self.fma2(self.mul2(x, z), p, x))
            xl = self.unpack(x)
            ax, am = [], []
            for s in xl:
                a, m = self.f(), self.f()
                self.e("abs.f32 %s, %s;" % (a, s))
                self.e("min.f32 %s, %s, 0f41A00000;" % (m, a))   # 20
                ax.append(a)
                am.append(m)
            e = self.exp_core(self.mul2(self.pack(am[0], am[1]), self.K(2.0)))
            e1 = self.unpack(self.add2(e, self.K(1.0)))
            big = self.unpack(self.fma2(self.pack(self.rcp(e1[0]), self.rcp(e1[1])), self.K(-2.0), self.K(1.0)))
            res = []
            for j in range(2):
                b, pr, d = self.f(), self.p(), self.f()
                self.e("copysign.f32 %s, %s, %s;" % (b, xl[j], big[j]))   # magnitude of big, sign of x
                self.e("setp.lt.f32 %s, %s, %s;" % (pr, ax[j], fc(0.6)))
                self.e("selp.f32 %s, %s, %s, %s;" % (d, small[j], b, pr))
                res.append(d)
            out.append(self.pack(res[0], res[1]))
        return out

    def divp(self, num, den, dst):
        """dst = num / (1 + |den|), packed lists"""
        for i in range(NP):
            lo, hi = self.unpack(den[i])
            self.mul2(num[i], self.pack(self.rcp1pabs(lo), self.rcp1pabs(hi)), dst[i])

    # ---- tile context -----------------------------------------------------------------------
    def set_tile(self):
        """from %tile: %tbase, %limit, %pfull, %pvec, %pfirst, %tnext, %pfast"""
        done, flat = self.newlabel("st"), self.newlabel("st")
        nt, t0 = self.rd(), self.rd()
        pr = self.p()
        self.e("add.s64 %s, %%tile, %%gs;" % nt)
        self.e("mov.s64 %tnext, 0;")
        self.e("@!%%prow bra.uni %s;" % flat)
        self.e("mul.lo.s64 %tbase, %tile, %cols64;")
        self.e("mov.s32 %limit, %cols;")
        t1 = self.r()
        self.e("and.b32 %s, %%cols, 3;" % t1)
        self.e("setp.eq.s32 %%pvec, %s, 0;" % t1)
        self.e("setp.lt.s64 %s, %s, %%ntiles;" % (pr, nt))
        self.e("@%s mul.lo.s64 %%tnext, %%gs, %%cols64;" % pr)
        self.e("bra.uni %s;" % done)
        self.label(flat)
        self.e("shl.b64 %%tbase, %%tile, %d;" % 12)
        self.e("sub.s64 %s, %%n, %%tbase;" % t0)
        self.e("min.s64 %s, %s, %d;" % (t0, t0, TILE))
        self.e("cvt.s32.s64 %%limit, %s;" % t0)
        self.e("setp.eq.s32 %pvec, %limit, %limit;")
        self.e("add.s64 %s, %s, 1;" % (nt, nt))
        self.e("shl.b64 %s, %s, 12;" % (nt, nt))
        self.e("setp.le.s64 %s, %s, %%n;" % (pr, nt))
        self.e("@%s shl.b64 %%tnext, %%gs, 12;" % pr)
        self.label(done)
        self.e("setp.eq.s32 %%pfull, %%limit, %d;" % TILE)
        self.e("setp.eq.s64 %pfirst, %tile, 0;")
        self.e("and.pred %pfast, %pfull, %pvec;")

    # position of element j of this thread inside the tile
    def lane_pos(self, j):
        d = self.r()
        self.e("add.u32 %s, %%pos0, %d;" % (d, (j >> 2) * NT * 4 + (j & 3)))
        return d

    def mask_tail(self, sc):
        """scalars with the lanes beyond %limit replaced by 0"""
        out = []
        for j, s in enumerate(sc):
            pr, d = self.p(), self.f()
            self.e("setp.lt.s32 %s, %s, %%limit;" % (pr, self.lane_pos(j)))
            self.e("selp.f32 %s, %s, 0f00000000, %s;" % (d, s, pr))
            out.append(d)
        return out

    # ---- global loads and stores of one operand ----------------------------------------------
    def operand(self):
        """-> (ptr u64, kind u32, dtype u32) of operand[%arg] from the shared-memory copy of the table"""
        a, ptr, kind, dt = self.r(), self.rd(), self.r(), self.r()
        self.e("shl.b32 %s, %%arg, 4;" % a)
        self.e("add.u32 %s, %s, %%opb;" % (a, a))
        self.e("ld.shared.u64 %s, [%s];" % (ptr, a))
        self.e("ld.shared.v2.u32 {%s, %s}, [%s+8];" % (kind, dt, a))
        return ptr, kind, dt

    def leaf_gld(self):
        ptr, kind, dt = self.operand()
        self.fetch()
        pfullk, pbf = self.p(), self.p()
        base = self.rd()
        self.e("setp.eq.u32 %s, %s, 0;" % (pfullk, kind))
        self.e("selp.b64 %s, %%tbase, 0, %s;" % (base, pfullk))
        self.e("setp.ne.u32 %s, %s, 0;" % (pbf, dt))
        lbf, ldone, lslow = self.newlabel("gld"), self.newlabel("gld"), self.newlabel("gld")
        self.e("@%s bra.uni %s;" % (pbf, lbf))
        # ---- fp32 ----
        adr = self.rd()
        self.e("add.s64 %s, %s, %%pos0_64;" % (adr, base))
        self.e("shl.b64 %s, %s, 2;" % (adr, adr))
        self.e("add.u64 %s, %s, %s;" % (adr, adr, ptr))
        self.prefetch(adr, pfullk, 4)
        self.e("@!%%pfast bra.uni %s;" % lslow)
        self.e("ld.global.nc.v2.b64 {%s, %s}, [%s];" % (self.A[0], self.A[1], adr))
        self.e("ld.global.nc.v2.b64 {%s, %s}, [%s+%d];" % (self.A[2], self.A[3], adr, HALF_BYTES))
        self.jump()
        self.label(lslow)
        for h in range(2):
            lv, ln = self.newlabel("gld"), self.newlabel("gld")
            pv, pos3 = self.p(), self.r()
            self.e("add.u32 %s, %%pos0, %d;" % (pos3, h * NT * 4 + 3))
            self.e("setp.lt.s32 %s, %s, %%limit;" % (pv, pos3))
            self.e("and.pred %s, %s, %%pvec;" % (pv, pv))
            self.e("@%s bra %s;" % (pv, lv))
            sc = []
            for e_ in range(4):
                pe, d = self.p(), self.f()
                self.e("setp.lt.s32 %s, %s, %%limit;" % (pe, self.lane_pos(4 * h + e_)))
                self.e("mov.f32 %s, 0f00000000;" % d)
                self.e("@%s ld.global.nc.f32 %s, [%s+%d];" % (pe, d, adr, h * HALF_BYTES + 4 * e_))
                sc.append(d)
            self.pack(sc[0], sc[1], self.A[2 * h])
            self.pack(sc[2], sc[3], self.A[2 * h + 1])
            self.e("bra %s;" % ln)
            self.label(lv)
            self.e("ld.global.nc.v2.b64 {%s, %s}, [%s+%d];" % (self.A[2 * h], self.A[2 * h + 1], adr, h * HALF_BYTES))
            self.label(ln)
        self.jump()
        # ---- bf16 ----
        self.label(lbf)
        adr = self.rd()
        self.e("add.s64 %s, %s, %%pos0_64;" % (adr, base))
        self.e("shl.b64 %s, %s, 1;" % (adr, adr))
        self.e("add.u64 %s, %s, %s;" % (adr, adr, ptr))
        self.prefetch(adr, pfullk, 2)
        for h in range(2):
            lv, ln = self.newlabel("gld"), self.newlabel("gld")
            pv, pos3 = self.p(), self.r()
            self.e("add.u32 %s, %%pos0, %d;" % (pos3, h * NT * 4 + 3))
            self.e("setp.lt.s32 %s, %s, %%limit;" % (pv, pos3))
            self.e("and.pred %s, %s, %%pvec;" % (pv, pv))
            self.e("@%s bra %s;" % (pv, lv))
            sc = []
            for e_ in range(4):
                pe, d, hh = self.p(), self.r(), self.t("h")
                self.e("setp.lt.s32 %s, %s, %%limit;" % (pe, self.lane_pos(4 * h + e_)))
                self.e("mov.b16 %s, 0;" % hh)
                self.e("@%s ld.global.nc.u16 %s, [%s+%d];" % (pe, hh, adr, h * NT * 8 + 2 * e_))
                self.e("cvt.u32.u16 %s, %s;" % (d, hh))
                self.e("shl.b32 %s, %s, 16;" % (d, d))
                sc.append(d)
            self.pack(sc[0], sc[1], self.A[2 * h])
            self.pack(sc[2], sc[3], self.A[2 * h + 1])
            self.e("bra %s;" % ln)
            self.label(lv)
            w0, w1 = self.r(), self.r()
            self.e("ld.global.nc.v2.u32 {%s, %s}, [%s+%d];" % (w0, w1, adr, h * NT * 8))
            for i, w in enumerate((w0, w1)):
                lo, hi = self.r(), self.r()
                self.e("shl.b32 %s, %s, 16;" % (lo, w))
                self.e("and.b32 %s, %s, 0xffff0000;" % (hi, w))
                self.pack(lo, hi, self.A[2 * h + i])
            self.label(ln)
        self.jump()

    def prefetch(self, adr, pfullk, esize):
        """pulls this CTA's next tile of a FULL operand into L2 while the current one is processed"""
        skip = self.newlabel("pf")
        pr, pa = self.p(), self.rd()
        self.e("setp.ne.s64 %s, %%tnext, 0;" % pr)
        self.e("and.pred %s, %s, %s;" % (pr, pr, pfullk))
        self.e("@!%s bra.uni %s;" % (pr, skip))
        self.e("mad.lo.s64 %s, %%tnext, %d, %s;" % (pa, esize, adr))
        for h in range(2):
            ph, ps = self.p(), self.r()
            self.e("add.u32 %s, %%pos0, %d;" % (ps, h * NT * 4))
            self.e("setp.lt.s32 %s, %s, %%limit;" % (ph, ps))
            self.e("@%s prefetch.global.L2 [%s+%d];" % (ph, pa, h * NT * 4 * esize))
        self.label(skip)

    def leaf_gst(self):
        ptr, kind, dt = self.operand()
        self.fetch()
        lout = self.newlabel("gst")
        pfullk, pscal, pbf, pr = self.p(), self.p(), self.p(), self.p()
        base = self.rd()
        self.e("setp.eq.u32 %s, %s, 0;" % (pfullk, kind))
        self.e("setp.eq.u32 %s, %s, 2;" % (pscal, kind))
        self.e("setp.ne.u32 %s, %s, 0;" % (pbf, dt))
        self.e("selp.b64 %s, %%tbase, 0, %s;" % (base, pfullk))
        # ROW and SCALAR shaped outputs are written by the first tile only
        self.e("or.pred %s, %s, %%pfirst;" % (pr, pfullk))
        self.e("@!%s bra.uni %s;" % (pr, lout))
        lscal, lbf, lslow = self.newlabel("gst"), self.newlabel("gst"), self.newlabel("gst")
        self.e("@%s bra.uni %s;" % (pscal, lscal))
        self.e("@%s bra.uni %s;" % (pbf, lbf))
        adr = self.rd()
        self.e("add.s64 %s, %s, %%pos0_64;" % (adr, base))
        self.e("shl.b64 %s, %s, 2;" % (adr, adr))
        self.e("add.u64 %s, %s, %s;" % (adr, adr, ptr))
        self.e("@!%%pfast bra.uni %s;" % lslow)
        self.stg_v(adr, self.A)
        self.jump()
        self.label(lslow)
        for h in range(2):
            lv, ln = self.newlabel("gst"), self.newlabel("gst")
            pv, pos3 = self.p(), self.r()
            self.e("add.u32 %s, %%pos0, %d;" % (pos3, h * NT * 4 + 3))
            self.e("setp.lt.s32 %s, %s, %%limit;" % (pv, pos3))
            self.e("and.pred %s, %s, %%pvec;" % (pv, pv))
            self.e("@%s bra %s;" % (pv, lv))
            sc = self.unpack(self.A[2 * h]) + self.unpack(self.A[2 * h + 1])
            for e_ in range(4):
                pe = self.p()
                self.e("setp.lt.s32 %s, %s, %%limit;" % (pe, self.lane_pos(4 * h + e_)))
                self.e("@%s st.global.f32 [%s+%d], %s;" % (pe, adr, h * HALF_BYTES + 4 * e_, sc[e_]))
            self.e("bra %s;" % ln)
            self.label(lv)
            self.e("st.global.v2.b64 [%s+%d], {%s, %s};" % (adr, h * HALF_BYTES, self.A[2 * h], self.A[2 * h + 1]))
            self.label(ln)
        self.jump()
        # bf16 tensors
        self.label(lbf)
        adr = self.rd()
        self.e("add.s64 %s, %s, %%pos0_64;" % (adr, base))
        self.e("shl.b64 %s, %s, 1;" % (adr, adr))
        self.e("add.u64 %s, %s, %s;" % (adr, adr, ptr))
        for h in range(2):
            lv, ln = self.newlabel("gst"), self.newlabel("gst")
            pv, pos3 = self.p(), self.r()
            sc = self.unpack(self.A[2 * h]) + self.unpack(self.A[2 * h + 1])
            w0, w1 = self.r(), self.r()
            self.e("cvt.rn.bf16x2.f32 %s, %s, %s;" % (w0, sc[1], sc[0]))
            self.e("cvt.rn.bf16x2.f32 %s, %s, %s;" % (w1, sc[3], sc[2]))
            self.e("add.u32 %s, %%pos0, %d;" % (pos3, h * NT * 4 + 3))
            self.e("setp.lt.s32 %s, %s, %%limit;" % (pv, pos3))
            self.e("and.pred %s, %s, %%pvec;" % (pv, pv))
            self.e("@%s bra %s;" % (pv, lv))
            for e_ in range(4):
                pe, hh, w = self.p(), self.t("h"), (w0, w1)[e_ >> 1]
                self.e("setp.lt.s32 %s, %s, %%limit;" % (pe, self.lane_pos(4 * h + e_)))
                if e_ & 1:
                    self.e("{ .reg .b16 %%lo; mov.b32 {%%lo, %s}, %s; }" % (hh, w))
                else:
                    self.e("{ .reg .b16 %%hi; mov.b32 {%s, %%hi}, %s; }" % (hh, w))
                self.e("@%s st.global.u16 [%s+%d], %s;" % (pe, adr, h * NT * 8 + 2 * e_, hh))
            self.e("bra %s;" % ln)
            self.label(lv)
            self.e("st.global.v2.u32 [%s+%d], {%s, %s};" % (adr, h * NT * 8, w0, w1))
            self.label(ln)
        self.jump()
        # one scalar, written by thread 0
        self.label(lscal)
        skip = self.newlabel("gst")
        p0 = self.p()
        self.e("setp.ne.u32 %s, %%tx, 0;" % p0)
        self.e("@%s bra %s;" % (p0, skip))
        a0, _ = self.unpack(self.A[0])
        sb = self.newlabel("gst")
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
        elif op == "fmaur":
            u = self.uniform()
            self.fetch()
            uu = self.splat(u)
            for i in range(NP):
                self.fma2(A[i], uu, R[i], A[i])
        else:
            self.fetch()
            if op == "ldr":
                self.mov_v(A, R)
            elif op == "str":
                self.mov_v(R, A)
            elif op == "add":
                for i in range(NP): self.add2(A[i], R[i], A[i])
            elif op == "sub":
                for i in range(NP): self.sub2(A[i], R[i], A[i])
            elif op == "rsub":
                for i in range(NP): self.sub2(R[i], A[i], A[i])
            elif op == "mul":
                for i in range(NP): self.mul2(A[i], R[i], A[i])
            elif op == "divp":
                self.divp(A, R, A)
            elif op == "rdivp":
                self.divp(R, A, A)
            elif op == "addto":
                for i in range(NP): self.add2(R[i], A[i], R[i])
            elif op == "accum":
                tail = self.newlabel("acc")
                self.e("@!%%pfull bra.uni %s;" % tail)
                for i in range(NP): self.add2(R[i], A[i], R[i])
                self.jump()
                self.label(tail)
                m = self.packs(self.mask_tail(self.scalars(A)))
                for i in range(NP): self.add2(R[i], m[i], R[i])
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
                self.divp([uu] * NP, A, A)
            for i in range(NP):
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
            for i in range(NP): self.fma2(A[i], uu, vv, A[i])
        elif op == "lds":
            a = self.slot_addr(); self.fetch(); self.lds_v(a, A)
        elif op == "sts":
            a = self.slot_addr(); self.fetch(); self.sts_v(a, A)
        elif op in ("adds", "subs", "rsubs", "muls", "divps", "rdivps"):
            a = self.slot_addr(); self.fetch()
            T = self.lds_v(a)
            for i in range(NP):
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
        elif op == "sincos":
            a = self.slot_addr(); self.fetch()
            S, C = self.sincos(A)
            self.sts_v(a, C)
            self.mov_v(A, S)
        elif op == "expc":
            self.fetch(); self.mov_v(A, self.expc(A))
        elif op == "tanh":
            self.fetch(); self.mov_v(A, self.tanh(A))
        elif op == "sigmoid":
            self.fetch(); self.mov_v(A, self.sigmoid(A))
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
                    self.e("mul.f32 %s, %s, %s;" % (g, g, rr))
                    self.e("mul.f32 %s, %s, %s;" % (d, g, rr))
                out.append(d)
            self.packs(out, A)
        elif op == "neg":
            self.fetch()
            m = self.K(-1.0)
            for i in range(NP): self.mul2(A[i], m, A[i])
        elif op == "onemsq":
            self.fetch()
            m, one = self.K(-1.0), self.K(1.0)
            for i in range(NP): self.fma2(self.mul2(A[i], m), A[i], one, A[i])
        elif op == "yomy":
            self.fetch()
            m, one = self.K(-1.0), self.K(1.0)
            for i in range(NP): self.mul2(A[i], self.fma2(A[i], m, one), A[i])
        elif op == "rbf16":
            self.fetch()
            for i in range(NP):
                lo, hi = self.unpack(A[i])
                w, l2, h2 = self.r(), self.r(), self.r()
                self.e("cvt.rn.bf16x2.f32 %s, %s, %s;" % (w, hi, lo))
                self.e("shl.b32 %s, %s, 16;" % (l2, w))
                self.e("and.b32 %s, %s, 0xffff0000;" % (h2, w))
                self.pack(l2, h2, A[i])
        elif op == "rowsum":
            self.fetch()
            self.leaf_rowsum()
        elif op == "gld":
            self.leaf_gld(); return
        elif op == "gst":
            self.leaf_gst(); return
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
            self.e("sub.u32 %loop_ip, %ip, 8;")   # entry of the first body instruction (just fetched)
        elif op == "loop_end":
            self.leaf_loop_end(); return
        elif op == "colout":
            self.leaf_colout()
        elif op == "scalout":
            self.leaf_scalout()
        elif op == "end":
            self.e("exit;")
            return
        else:
            raise ValueError(op)
        self.jump()

    def leaf_rowsum(self):
        A = self.A
        full, go = self.newlabel("rs"), self.newlabel("rs")
        s = self.f()
        sc = self.scalars(A)
        self.e("@%%pfull bra.uni %s;" % full)
        m = self.mask_tail(sc)
        self.e("mov.f32 %s, 0f00000000;" % s)
        for x in m: self.e("add.f32 %s, %s, %s;" % (s, s, x))
        self.e("bra.uni %s;" % go)
        self.label(full)
        self.e("mov.f32 %s, 0f00000000;" % s)
        for x in sc: self.e("add.f32 %s, %s, %s;" % (s, s, x))
        self.label(go)
        for o in (16, 8, 4, 2, 1):
            t = self.f()
            self.e("shfl.sync.bfly.b32 %s, %s, %d, 0x1f, 0xffffffff;" % (t, s, o))
            self.e("add.f32 %s, %s, %s;" % (s, s, t))
        pr, a = self.p(), self.r()
        self.e("setp.eq.u32 %s, %%lane, 0;" % pr)
        self.e("shl.b32 %s, %%warp, 2;" % a)
        self.e("add.u32 %s, %s, %%redb;" % (a, a))
        self.e("@%s st.shared.f32 [%s], %s;" % (pr, a, s))
        self.e("bar.sync 0;")
        tot = self.f()
        self.e("mov.f32 %s, 0f00000000;" % tot)
        for i in range(NT // 128):
            q = [self.f() for _ in range(4)]
            self.e("ld.shared.v4.f32 {%s, %s, %s, %s}, [%%redb+%d];" % (q[0], q[1], q[2], q[3], 16 * i))
            for x in q: self.e("add.f32 %s, %s, %s;" % (tot, tot, x))
        self.e("bar.sync 0;")
        tt = self.splat(tot)
        for i in range(NP): self.e("mov.b64 %s, %s;" % (A[i], tt))

    def leaf_uload(self):
        """U[arg & 511] = scalar operand[arg >> 9], by thread 0"""
        skip, lb = self.newlabel("ul"), self.newlabel("ul")
        ui, oi, a, ptr, dt, pr, pb, v = self.r(), self.r(), self.r(), self.rd(), self.r(), self.p(), self.p(), self.f()
        self.e("and.b32 %s, %%arg, 511;" % ui)
        self.e("shr.u32 %s, %%arg, 9;" % oi)
        self.fetch()
        self.e("setp.ne.u32 %s, %%tx, 0;" % pr)
        self.e("@%s bra %s;" % (pr, skip))
        self.e("shl.b32 %s, %s, 4;" % (a, oi))
        self.e("add.u32 %s, %s, %%opb;" % (a, a))
        self.e("ld.shared.u64 %s, [%s];" % (ptr, a))
        self.e("ld.shared.u32 %s, [%s+12];" % (dt, a))
        self.e("setp.ne.u32 %s, %s, 0;" % (pb, dt))
        self.e("@%s bra %s;" % (pb, lb))
        self.e("ld.global.nc.f32 %s, [%s];" % (v, ptr))
        self.e("bra %s;" % (skip + "_st"))
        self.label(lb)
        hh, w = self.t("h"), self.r()
        self.e("ld.global.nc.u16 %s, [%s];" % (hh, ptr))
        self.e("cvt.u32.u16 %s, %s;" % (w, hh))
        self.e("shl.b32 %s, %s, 16;" % (w, w))
        self.e("mov.b32 %s, %s;" % (v, w))
        self.label(skip + "_st")
        self.e("shl.b32 %s, %s, 2;" % (ui, ui))
        self.e("add.u32 %s, %s, %%ub;" % (ui, ui))
        self.e("st.shared.f32 [%s], %s;" % (ui, v))
        self.label(skip)

    def leaf_uconst(self):
        """U[arg] = the raw word that follows in the undecoded stream, by thread 0"""
        skip = self.newlabel("uc")
        ui, idx, pr, ga, w = self.r(), self.r(), self.p(), self.rd(), self.r()
        self.e("shl.b32 %s, %%arg, 2;" % ui)
        self.e("add.u32 %s, %s, %%ub;" % (ui, ui))
        self.e("sub.u32 %s, %%ip, %%codeb;" % idx)     # ip points at the literal's entry: 8 bytes per word
        self.e("shr.u32 %s, %s, 1;" % (idx, idx))          # -> byte offset in the 4-byte stream
        self.e("add.u32 %ip, %ip, 8;")
        self.fetch()
        self.e("setp.ne.u32 %s, %%tx, 0;" % pr)
        self.e("@%s bra %s;" % (pr, skip))
        self.e("cvt.u64.u32 %s, %s;" % (ga, idx))
        self.e("add.u64 %s, %s, %%code;" % (ga, ga))
        self.e("ld.global.nc.u32 %s, [%s];" % (w, ga))
        self.e("st.shared.u32 [%s], %s;" % (ui, w))
        self.label(skip)
        self.jump()

    def leaf_loop_end(self):
        out = self.newlabel("le")
        pr = self.p()
        self.e("add.s64 %tile, %tile, %gs;")
        self.e("setp.ge.s64 %s, %%tile, %%ntiles;" % pr)
        self.e("@%s bra.uni %s;" % (pr, out))
        self.set_tile()
        self.e("mov.u32 %ip, %loop_ip;")
        self.label(out)
        self.fetch()
        self.jump()

    def leaf_colout(self):
        """column partial sums: colpart[arg][cta][c] = acc"""
        A = self.A
        o, t = self.rd(), self.rd()
        self.e("mul.wide.u32 %s, %%arg, %%ncta;" % o)
        self.fetch()
        self.e("cvt.u64.u32 %s, %%cta;" % t)
        self.e("add.u64 %s, %s, %s;" % (o, o, t))
        self.e("mul.lo.u64 %s, %s, %%cols64;" % (o, o))
        self.e("add.u64 %s, %s, %%pos0_64;" % (o, o))
        self.e("shl.b64 %s, %s, 2;" % (o, o))
        self.e("add.u64 %s, %s, %%colpart;" % (o, o))
        sc = self.scalars(A)
        for j in range(V):
            pr = self.p()
            self.e("setp.lt.s32 %s, %s, %%cols;" % (pr, self.lane_pos(j)))
            self.e("@%s st.global.f32 [%s+%d], %s;" % (pr, o, ((j >> 2) * NT * 4 + (j & 3)) * 4, sc[j]))

    def leaf_scalout(self):
        """scalar partial sum: scalpart[arg][cta] = block sum of acc in fp64"""
        A = self.A
        o, t = self.rd(), self.rd()
        self.e("mul.wide.u32 %s, %%arg, %%ncta;" % o)
        self.fetch()
        self.e("cvt.u64.u32 %s, %%cta;" % t)
        self.e("add.u64 %s, %s, %s;" % (o, o, t))
        self.e("shl.b64 %s, %s, 3;" % (o, o))
        self.e("add.u64 %s, %s, %%scalpart;" % (o, o))
        s = self.fd()
        self.e("mov.f64 %s, 0d0000000000000000;" % s)
        for x in self.scalars(A):
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
        pr, a = self.p(), self.r()
        self.e("setp.eq.u32 %s, %%lane, 0;" % pr)
        self.e("shl.b32 %s, %%warp, 3;" % a)
        self.e("add.u32 %s, %s, %%redb;" % (a, a))
        self.e("@%s st.shared.f64 [%s], %s;" % (pr, a, s))
        self.e("bar.sync 0;")
        skip = self.newlabel("so")
        p0 = self.p()
        self.e("setp.ne.u32 %s, %%tx, 0;" % p0)
        self.e("@%s bra %s;" % (p0, skip))
        tot = self.fd()
        self.e("mov.f64 %s, 0d0000000000000000;" % tot)
        for i in range(NT // 32):
            d = self.fd()
            self.e("ld.shared.f64 %s, [%%redb+%d];" % (d, 8 * i))
            self.e("add.f64 %s, %s, %s;" % (tot, tot, d))
        self.e("st.global.f64 [%s], %s;" % (o, tot))
        self.label(skip)
        self.e("bar.sync 0;")

    # ---- the kernel ---------------------------------------------------------------------------
    def build(self):
        nr = self.nr
        cases = []
        for op in JOINT:
            for k in range(nr):
                cases.append(("j", op, k))
        for op in PLAIN:
            cases.append(("p", op, 0))
        labels = ["$C_%s_%d" % (self.name, i) for i in range(len(cases))]
        body = self.lines
        # ---- prologue ----
        e = self.e
        e("mov.u32 %tx, %tid.x;")
        e("mov.u32 %cta, %ctaid.x;")
        e("mov.u32 %ncta, %nctaid.x;")
        e("and.b32 %lane, %tx, 31;")
        e("shr.u32 %warp, %tx, 5;")
        e("shl.b32 %pos0, %tx, 2;")
        e("cvt.u64.u32 %pos0_64, %pos0;")
        e("ld.param.u64 %%code, [VP+%d];" % P_CODE)
        e("ld.param.s32 %%ncode, [VP+%d];" % P_NCODE)
        e("ld.param.s32 %%rowmode, [VP+%d];" % P_ROWMODE)
        e("ld.param.s64 %%n, [VP+%d];" % P_N)
        e("ld.param.s32 %%cols, [VP+%d];" % P_COLS)
        e("ld.param.s32 %%nspill, [VP+%d];" % P_NSPILL)
        e("ld.param.u64 %%spb, [VP+%d];" % P_SPILL)
        e("ld.param.u64 %%colpart, [VP+%d];" % P_COLPART)
        e("ld.param.u64 %%scalpart, [VP+%d];" % P_SCALPART)
        e("cvt.s64.s32 %cols64, %cols;")
        e("setp.ne.s32 %prow, %rowmode, 0;")
        e("cvt.u64.u32 %gs, %ncta;")
        # shared memory: code | uniforms | reduction scratch | operand table | slots
        e("mov.u32 %codeb, dsm;")
        t0 = self.r()
        e("add.s32 %s, %%ncode, 3;" % t0)
        e("and.b32 %s, %s, 0xfffffffc;" % (t0, t0))
        e("shl.b32 %s, %s, 3;" % (t0, t0))
        e("add.u32 %%ub, %%codeb, %s;" % t0)
        e("add.u32 %%redb, %%ub, %d;" % (MAX_UNIFORMS * 4))
        e("add.u32 %opb, %redb, 512;")
        e("add.u32 %%sa, %%opb, %d;" % (MAX_OPERANDS * 16))
        t1 = self.r()
        e("shl.b32 %s, %%tx, 4;" % t1)
        e("add.u32 %%sa, %%sa, %s;" % t1)
        # operand table -> shared memory (one entry per thread)
        for i in range(MAX_OPERANDS):
            pr, ptr, k, d = self.p(), self.rd(), self.r(), self.r()
            e("setp.eq.u32 %s, %%tx, %d;" % (pr, i))
            e("ld.param.u64 %s, [VP+%d];" % (ptr, P_OPERAND + 16 * i))
            e("ld.param.u32 %s, [VP+%d];" % (k, P_OPERAND + 16 * i + 8))
            e("ld.param.u32 %s, [VP+%d];" % (d, P_OPERAND + 16 * i + 12))
            e("@%s st.shared.u64 [%%opb+%d], %s;" % (pr, 16 * i, ptr))
            e("@%s st.shared.v2.u32 [%%opb+%d], {%s, %s};" % (pr, 16 * i + 8, k, d))
        # decode the instruction stream: {case id, argument} per word
        lp, ld_ = self.newlabel("dec"), self.newlabel("dec")
        i_, pr, ga, w, c, a, sa = self.r(), self.p(), self.rd(), self.r(), self.r(), self.r(), self.r()
        e("mov.u32 %s, %%tx;" % i_)
        self.label(lp)
        e("setp.ge.s32 %s, %s, %%ncode;" % (pr, i_))
        e("@%s bra %s;" % (pr, ld_))
        e("mul.wide.u32 %s, %s, 4;" % (ga, i_))
        e("add.u64 %s, %s, %%code;" % (ga, ga))
        e("ld.global.nc.u32 %s, [%s];" % (w, ga))
        e("and.b32 %s, %s, 1023;" % (c, w))
        e("shr.u32 %s, %s, 14;" % (a, w))
        e("shl.b32 %s, %s, 3;" % (sa, i_))
        e("add.u32 %s, %s, %%codeb;" % (sa, sa))
        e("st.shared.v2.u32 [%s], {%s, %s};" % (sa, c, a))
        e("add.u32 %s, %s, %d;" % (i_, i_, NT))
        e("bra %s;" % lp)
        self.label(ld_)
        e("bar.sync 0;")
        # per-CTA spill area: spill + cta * n_spill * TILE floats, this thread's 16 bytes
        t2, t3 = self.rd(), self.rd()
        e("mul.wide.u32 %s, %%cta, %d;" % (t2, SLOT_BYTES))
        e("cvt.s64.s32 %s, %%nspill;" % t3)
        e("mad.lo.u64 %%spb, %s, %s, %%spb;" % (t2, t3))
        e("mul.wide.u32 %s, %%tx, 16;" % t2)
        e("add.u64 %%spb, %%spb, %s;" % t2)
        for r_ in self.A + sum(self.R, []):
            e("mov.b64 %s, 0;" % r_)
        # tiles
        fl, dn = self.newlabel("nt"), self.newlabel("nt")
        e("@!%%prow bra.uni %s;" % fl)
        e("mov.s64 %ntiles, %n;")
        e("bra.uni %s;" % dn)
        self.label(fl)
        e("add.s64 %%ntiles, %%n, %d;" % (TILE - 1))
        e("shr.s64 %ntiles, %ntiles, 12;")
        self.label(dn)
        e("cvt.u64.u32 %tile, %cta;")
        self.set_tile()
        e("mov.u32 %ip, %codeb;")
        e("mov.u32 %loop_ip, %codeb;")
        self.fetch()
        e("JT_%s: .branchtargets %s;" % (self.name, ", ".join(labels)))
        self.jump()
        # ---- leaves ----
        for lab, (kind, op, k) in zip(labels, cases):
            self.label(lab)
            if kind == "j":
                self.leaf_joint(op, k)
            else:
                self.leaf_plain(op)
        # ---- assemble text ----
        head = []
        head.append(".const .align 8 .b64 KT_%s[%d] = {%s};" % (self.name, max(1, len(self.kt)), ", ".join("0x%016X" % w for w in self.kt) or "0"))
        head.append(".visible .entry %s(.param .align 8 .b8 VP[%d])" % (self.name, P_SIZE))
        head.append(".maxntid %d, 1, 1" % NT)
        head.append(".minnctapersm %d" % self.ctas)
        head.append("{")
        decl = []
        for kind, ty in (("f", ".f32"), ("r", ".b32"), ("rd", ".b64"), ("p", ".pred"), ("fd", ".f64"), ("h", ".b16")):
            if self.cnt[kind]:
                decl.append("\t.reg %s %%%s<%d>;" % (ty, {"f": "f", "r": "r", "rd": "rd", "p": "p", "fd": "fd", "h": "h"}[kind], self.cnt[kind]))
        decl.append("\t.reg .b32 %tx, %cta, %ncta, %lane, %warp, %pos0, %ncode, %rowmode, %cols, %nspill, %limit;")
        decl.append("\t.reg .b32 %codeb, %ub, %redb, %opb, %sa, %ip, %loop_ip, %case, %arg;")
        decl.append("\t.reg .b64 %pos0_64, %code, %n, %spb, %colpart, %scalpart, %cols64, %gs, %tile, %ntiles, %tbase, %tnext;")
        decl.append("\t.reg .pred %prow, %pfull, %pvec, %pfirst, %pfast;")
        decl.append("\t.reg .b64 %s;" % ", ".join(self.A + sum(self.R, [])))
        return "\n".join(head + decl + body + ["}"]) + "\n"


VARIANTS = [("dragon_vm_r7", 7, 1)]


def generate():
    out = [".version 8.8", ".target sm_100a", ".address_size 64", "", ".extern .shared .align 16 .b8 dsm[];", ""]
    for name, nr, ctas in VARIANTS:
        out.append(Kernel(name, nr, ctas).build())
    return "\n".join(out)


if __name__ == "__main__":
    text = generate()
    if len(sys.argv) > 1:
        open(sys.argv[1], "w").write(text)
    else:
        sys.stdout.write(text)
