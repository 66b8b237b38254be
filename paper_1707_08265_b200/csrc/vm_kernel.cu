// The graph-VM kernel: interprets the instruction stream of one fused segment (vm_isa.h).
//
// Geometry: 256 threads per CTA, one CTA per SM (the whole register file belongs to it), 16
// elements per thread held as four 128-bit vectors that are each contiguous across the warp,
// so a tile is 4096 elements.  Flat mode walks the element range tile by tile (grid-stride);
// row mode gives every tile one row of the [rows, cols] domain, which makes a row reduction a
// CTA-wide reduction and a column reduction a per-thread running sum.  The instruction stream
// and the uniforms sit in shared memory; the accumulator and the register slots are C arrays
// that are only ever indexed with compile-time constants (every register-operand instruction
// is its own switch case), so they live in registers.  One decoded instruction is amortised
// over 16 element operations per thread, and the next instruction word is fetched before the
// current one executes.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>
#include <mutex>
#include <string>
#include <type_traits>

#include "plan.h"
#include "vm_math.h"

namespace dragon {
namespace vm {

constexpr int NT = kVmThreads;
constexpr int V = kVmVec;
constexpr int NV4 = V / 4;
constexpr int NR = kVmRegs;
constexpr int TILE = kVmTile;
static_assert(V % 4 == 0 && NR >= 2 && NR <= 15, "register slot count out of range");

#define FORV _Pragma("unroll") for (int j = 0; j < V; ++j)

struct TileCtx {
  long long base;   // element offset of this tile for FULL operands
  int limit;        // valid elements in the tile (TILE when full)
  bool full;        // limit == TILE
  bool vec_ok;      // 4-element groups are 16-byte aligned
  bool first;       // tile 0 (stores of ROW / SCALAR shaped outputs happen here)
  long long next;   // element distance to this CTA's next tile, 0 when there is none (L2 prefetch)
};

__device__ __forceinline__ int lane_pos(int tid, int j) { return (j >> 2) * (NT * 4) + tid * 4 + (j & 3); }

__device__ __forceinline__ void load_operand(const Operand& o, const TileCtx& tc, int tid, float* t) {
  const long long base = o.kind == K_FULL ? tc.base : 0;
  if (o.dtype == DRAGON_F32) {
    const float* p = reinterpret_cast<const float*>(o.ptr) + base;
    if (o.kind == K_FULL && tc.next) {  // pull this CTA's next tile into L2 while the current one is processed
#pragma unroll
      for (int h = 0; h < NV4; ++h)
        if (h * NT * 4 + tid * 4 < tc.limit) asm volatile("prefetch.global.L2 [%0];" ::"l"(p + tc.next + h * NT * 4 + tid * 4));
    }
#pragma unroll
    for (int h = 0; h < NV4; ++h) {
      const int pos = h * NT * 4 + tid * 4;
      if (tc.vec_ok && pos + 3 < tc.limit) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(p + pos));
        t[4 * h + 0] = v.x; t[4 * h + 1] = v.y; t[4 * h + 2] = v.z; t[4 * h + 3] = v.w;
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) t[4 * h + e] = (pos + e < tc.limit) ? __ldg(p + pos + e) : 0.f;
      }
    }
  } else {
    const unsigned short* p = reinterpret_cast<const unsigned short*>(o.ptr) + base;
    if (o.kind == K_FULL && tc.next) {
#pragma unroll
      for (int h = 0; h < NV4; ++h)
        if (h * NT * 4 + tid * 4 < tc.limit) asm volatile("prefetch.global.L2 [%0];" ::"l"(p + tc.next + h * NT * 4 + tid * 4));
    }
#pragma unroll
    for (int h = 0; h < NV4; ++h) {
      const int pos = h * NT * 4 + tid * 4;
      if (tc.vec_ok && pos + 3 < tc.limit) {
        const uint2 v = __ldg(reinterpret_cast<const uint2*>(p + pos));
        t[4 * h + 0] = __uint_as_float(v.x << 16); t[4 * h + 1] = __uint_as_float(v.x & 0xffff0000u);
        t[4 * h + 2] = __uint_as_float(v.y << 16); t[4 * h + 3] = __uint_as_float(v.y & 0xffff0000u);
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e)
          t[4 * h + e] = (pos + e < tc.limit) ? __uint_as_float((unsigned)__ldg(p + pos + e) << 16) : 0.f;
      }
    }
  }
}

__device__ __forceinline__ void store_operand(const Operand& o, const TileCtx& tc, int tid, const float* t) {
  if (o.kind == K_SCALAR) {
    if (tc.first && tid == 0) {
      if (o.dtype == DRAGON_F32) *reinterpret_cast<float*>(o.ptr) = t[0];
      else *reinterpret_cast<unsigned short*>(o.ptr) = (unsigned short)vmmath::bf16_bits(t[0]);
    }
    return;
  }
  if (o.kind == K_ROW && !tc.first) return;
  const long long base = o.kind == K_FULL ? tc.base : 0;
  if (o.dtype == DRAGON_F32) {
    float* p = reinterpret_cast<float*>(o.ptr) + base;
#pragma unroll
    for (int h = 0; h < NV4; ++h) {
      const int pos = h * NT * 4 + tid * 4;
      if (tc.vec_ok && pos + 3 < tc.limit) {
        *reinterpret_cast<float4*>(p + pos) = make_float4(t[4 * h], t[4 * h + 1], t[4 * h + 2], t[4 * h + 3]);
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (pos + e < tc.limit) p[pos + e] = t[4 * h + e];
      }
    }
  } else {
    unsigned short* p = reinterpret_cast<unsigned short*>(o.ptr) + base;
#pragma unroll
    for (int h = 0; h < NV4; ++h) {
      const int pos = h * NT * 4 + tid * 4;
      if (tc.vec_ok && pos + 3 < tc.limit) {
        uint2 v;
        v.x = vmmath::bf16_bits(t[4 * h]) | (vmmath::bf16_bits(t[4 * h + 1]) << 16);
        v.y = vmmath::bf16_bits(t[4 * h + 2]) | (vmmath::bf16_bits(t[4 * h + 3]) << 16);
        *reinterpret_cast<uint2*>(p + pos) = v;
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (pos + e < tc.limit) p[pos + e] = (unsigned short)vmmath::bf16_bits(t[4 * h + e]);
      }
    }
  }
}

// a V-wide value <-> NV4 float4 cells spaced NT apart (one column per thread)
#define VEC_STORE(ptr, X) { float4* p_ = (ptr); _Pragma("unroll") for (int h = 0; h < NV4; ++h) p_[h * NT] = make_float4((X)[4 * h], (X)[4 * h + 1], (X)[4 * h + 2], (X)[4 * h + 3]); }
#define VEC_LOAD(X, ptr) { const float4* p_ = (ptr); _Pragma("unroll") for (int h = 0; h < NV4; ++h) { const float4 v_ = p_[h * NT]; (X)[4 * h] = v_.x; (X)[4 * h + 1] = v_.y; (X)[4 * h + 2] = v_.z; (X)[4 * h + 3] = v_.w; } }


// balanced binary search over [LO, HI): calls f(integral_constant<LEAF>, arg) for the leaf equal to cs
template <int LO, int HI, class F>
__device__ __forceinline__ void dispatch_tree(const int cs, const uint32_t arg, F& f) {
  if constexpr (HI - LO == 1) {
    f(std::integral_constant<int, LO>{}, arg);
  } else {
    constexpr int MID = (LO + HI) / 2;
    if (cs < MID) dispatch_tree<LO, MID>(cs, arg, f);
    else dispatch_tree<MID, HI>(cs, arg, f);
  }
}

__global__ void __launch_bounds__(NT, 1) vm_kernel(const __grid_constant__ Params p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // layout: code | uniforms | reduction scratch | V-wide slots
  uint2* code2 = reinterpret_cast<uint2*>(smem_raw);
  const int code_words = (p.n_code + 3) & ~3;
  float* U = reinterpret_cast<float*>(code2 + code_words);
  double* red = reinterpret_cast<double*>(U + kMaxUniforms);
  float4* slots = reinterpret_cast<float4*>(red + 64);                // [slot][NV4][NT]

  const int tid = threadIdx.x;
  for (int i = tid; i < p.n_code; i += NT) { const uint32_t cw = p.code[i]; code2[i] = make_uint2(cw & 1023u, cw >> 14); }
  __syncthreads();

  float acc[V], R[NR][V];
  FORV acc[j] = 0.f;
#pragma unroll
  for (int k = 0; k < NR; ++k) FORV R[k][j] = 0.f;

  const long long ntiles = p.row_mode ? p.n : (p.n + TILE - 1) / TILE;
  long long tile = blockIdx.x;
  TileCtx tc;
  const uint2* loop_ip = code2;
  const uint2* ip = code2;
  uint2 wn = make_uint2(0u, 0u);
  auto set_tile = [&]() {
    if (p.row_mode) {
      tc.base = tile * (long long)p.cols;
      tc.limit = p.cols;
      tc.vec_ok = (p.cols & 3) == 0;
    } else {
      tc.base = tile * (long long)TILE;
      const long long left = p.n - tc.base;
      tc.limit = left < TILE ? (int)left : TILE;
      tc.vec_ok = true;
    }
    tc.full = tc.limit == TILE;
    tc.first = tile == 0;
    // the whole next tile must exist for the prefetch addresses to stay inside the tensor
    const long long nt = tile + gridDim.x;
    tc.next = 0;
    if (p.row_mode) { if (nt < ntiles) tc.next = (long long)gridDim.x * p.cols; }
    else if ((nt + 1) * TILE <= p.n) tc.next = (long long)gridDim.x * TILE;
  };
  set_tile();
  float* spill = p.spill + (size_t)blockIdx.x * p.n_spill * TILE;

  // One instruction = one leaf of a balanced binary decision tree over the case id (the
  // compiler turns a switch of this size into a long compare chain, and indexed jumps are not
  // available from CUDA C); every leaf is compiled for its own constant case id, so register
  // slots are named statically.
  auto exec = [&](auto cs_tag, const uint32_t arg) {
    constexpr int CS = decltype(cs_tag)::value;
    asm volatile("// VMLEAF %0" ::"n"(CS));   // marks the leaf for the jump-table build step
    if constexpr (CS < kFirstPlain) {
      constexpr int J = CS / kJointStride, K = CS % kJointStride;
      if constexpr (J == J_LDR) { FORV acc[j] = R[K][j]; }
      else if constexpr (J == J_STR) { FORV R[K][j] = acc[j]; }
      else if constexpr (J == J_ADD) { FORV acc[j] = acc[j] + R[K][j]; }
      else if constexpr (J == J_SUB) { FORV acc[j] = acc[j] - R[K][j]; }
      else if constexpr (J == J_RSUB) { FORV acc[j] = R[K][j] - acc[j]; }
      else if constexpr (J == J_MUL) { FORV acc[j] = acc[j] * R[K][j]; }
      else if constexpr (J == J_DIVP) { FORV acc[j] = vmmath::divp_f(acc[j], R[K][j]); }
      else if constexpr (J == J_RDIVP) { FORV acc[j] = vmmath::divp_f(R[K][j], acc[j]); }
      else if constexpr (J == J_ADDTO) { FORV R[K][j] += acc[j]; }
      else if constexpr (J == J_ACCUM) {
        if (tc.full) { FORV R[K][j] += acc[j]; }
        else { FORV R[K][j] += (lane_pos(tid, j) < tc.limit) ? acc[j] : 0.f; }
      }
      else if constexpr (J == J_FMAUR) { const float u_ = U[arg]; FORV acc[j] = fmaf(acc[j], u_, R[K][j]); }
      else if constexpr (J == J_RTOS) { VEC_STORE(slots + (size_t)arg * NV4 * NT + tid, R[K]) }
      else if constexpr (J == J_STOR) { VEC_LOAD(R[K], slots + (size_t)arg * NV4 * NT + tid) }
      else if constexpr (J == J_SPILL) { VEC_STORE(reinterpret_cast<float4*>(spill + (size_t)arg * TILE) + tid, R[K]) }
      else if constexpr (J == J_FILL) { VEC_LOAD(R[K], reinterpret_cast<const float4*>(spill + (size_t)arg * TILE) + tid) }
    }
    else if constexpr (CS == P_LDU) { const float u = U[arg]; FORV acc[j] = u; }
    else if constexpr (CS == P_ADDU) { const float u = U[arg]; FORV acc[j] += u; }
    else if constexpr (CS == P_SUBU) { const float u = U[arg]; FORV acc[j] -= u; }
    else if constexpr (CS == P_RSUBU) { const float u = U[arg]; FORV acc[j] = u - acc[j]; }
    else if constexpr (CS == P_MULU) { const float u = U[arg]; FORV acc[j] *= u; }
    else if constexpr (CS == P_DIVPU) { const float u = vmmath::f_rcp(1.f + fabsf(U[arg])); FORV acc[j] *= u; }
    else if constexpr (CS == P_RDIVPU) { const float u = U[arg]; FORV acc[j] = vmmath::divp_f(u, acc[j]); }
    else if constexpr (CS == P_FMAU) { const float a = U[arg & 511u], b = U[arg >> 9]; FORV acc[j] = fmaf(acc[j], a, b); }
    else if constexpr (CS == P_LDS) { VEC_LOAD(acc, slots + (size_t)arg * NV4 * NT + tid) }
    else if constexpr (CS == P_STS) { VEC_STORE(slots + (size_t)arg * NV4 * NT + tid, acc) }
    else if constexpr (CS >= P_ADDS && CS <= P_RDIVPS) {
      float t[V];
      VEC_LOAD(t, slots + (size_t)arg * NV4 * NT + tid)
      if constexpr (CS == P_ADDS) { FORV acc[j] += t[j]; }
      else if constexpr (CS == P_SUBS) { FORV acc[j] -= t[j]; }
      else if constexpr (CS == P_RSUBS) { FORV acc[j] = t[j] - acc[j]; }
      else if constexpr (CS == P_MULS) { FORV acc[j] *= t[j]; }
      else if constexpr (CS == P_DIVPS) { FORV acc[j] = vmmath::divp_f(acc[j], t[j]); }
      else { FORV acc[j] = vmmath::divp_f(t[j], acc[j]); }
    }
    else if constexpr (CS == P_SIN) { FORV acc[j] = vmmath::sin_f(acc[j]); }
    else if constexpr (CS == P_COS) { FORV acc[j] = vmmath::cos_f(acc[j]); }
    else if constexpr (CS == P_SINCOS) {
      float t[V];
      FORV { float s_, c_; vmmath::sincos_f(acc[j], &s_, &c_); acc[j] = s_; t[j] = c_; }
      VEC_STORE(slots + (size_t)arg * NV4 * NT + tid, t)
    }
    else if constexpr (CS == P_EXPC) { FORV acc[j] = vmmath::exp_clamped10(acc[j]); }
    else if constexpr (CS == P_TANH) { FORV acc[j] = vmmath::tanh_f(acc[j]); }
    else if constexpr (CS == P_SIGMOID) { FORV acc[j] = vmmath::sigmoid_f(acc[j]); }
    else if constexpr (CS == P_RELU) { FORV acc[j] = fmaxf(acc[j], 0.f); }
    else if constexpr (CS == P_NEG) { FORV acc[j] = -acc[j]; }
    else if constexpr (CS == P_STEP) { FORV acc[j] = acc[j] > 0.f ? 1.f : 0.f; }
    else if constexpr (CS == P_CLAMPMASK) { FORV acc[j] = (acc[j] >= -10.f && acc[j] <= 10.f) ? 1.f : 0.f; }
    else if constexpr (CS == P_ONEMSQ) { FORV acc[j] = fmaf(-acc[j], acc[j], 1.f); }
    else if constexpr (CS == P_YOMY) { FORV acc[j] = acc[j] * (1.f - acc[j]); }
    else if constexpr (CS == P_DIVPGB) { FORV acc[j] = vmmath::divp_grad_b(acc[j]); }
    else if constexpr (CS == P_RBF16) { FORV acc[j] = vmmath::round_bf16(acc[j]); }
    else if constexpr (CS == P_ROWSUM) {
      float sum = 0.f;
      if (tc.full) { FORV sum += acc[j]; }
      else { FORV sum += (lane_pos(tid, j) < tc.limit) ? acc[j] : 0.f; }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      float* redf = reinterpret_cast<float*>(red);
      if ((tid & 31) == 0) redf[tid >> 5] = sum;
      __syncthreads();
      float tot = 0.f;
#pragma unroll
      for (int i = 0; i < NT / 32; ++i) tot += redf[i];
      __syncthreads();
      FORV acc[j] = tot;
    }
    else if constexpr (CS == P_GLD) { load_operand(p.operand[arg], tc, tid, acc); }
    else if constexpr (CS == P_GST) { store_operand(p.operand[arg], tc, tid, acc); }
    else if constexpr (CS == P_FILL) { VEC_LOAD(acc, reinterpret_cast<const float4*>(spill + (size_t)arg * TILE) + tid) }
    else if constexpr (CS == P_SPILL) { VEC_STORE(reinterpret_cast<float4*>(spill + (size_t)arg * TILE) + tid, acc) }
    // ---- control and once-per-CTA instructions ----
    else if constexpr (CS == P_ULOAD) {
      if (tid == 0) {
        const Operand& o = p.operand[arg >> 9];
        U[arg & 511u] = o.dtype == DRAGON_F32 ? __ldg(reinterpret_cast<const float*>(o.ptr))
                                              : __uint_as_float((unsigned)__ldg(reinterpret_cast<const unsigned short*>(o.ptr)) << 16);
      }
    }
    else if constexpr (CS == P_UCONST) {
      // the literal is the raw word that follows in the undecoded stream
      if (tid == 0) U[arg] = __uint_as_float(p.code[(int)(ip - code2) - 1]);
      wn = *ip;
      ++ip;
    }
    else if constexpr (CS == P_LOOP_BEGIN) {
      __syncthreads();    // uniforms written by thread 0 are visible from here on
      loop_ip = ip - 1;   // entry of the first body instruction (already in wn)
    }
    else if constexpr (CS == P_LOOP_END) {
      tile += gridDim.x;
      if (tile < ntiles) { set_tile(); wn = *loop_ip; ip = loop_ip + 1; }
    }
    else if constexpr (CS == P_COLOUT) {
      float* out = p.colpart + ((size_t)arg * gridDim.x + blockIdx.x) * p.cols;
      FORV { const int c = lane_pos(tid, j); if (c < p.cols) out[c] = acc[j]; }
    }
    else if constexpr (CS == P_SCALOUT) {
      double sum = 0.0;
      FORV sum += (double)acc[j];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      if ((tid & 31) == 0) red[tid >> 5] = sum;
      __syncthreads();
      if (tid == 0) {
        double tot = 0.0;
        for (int i = 0; i < NT / 32; ++i) tot += red[i];
        p.scalpart[(size_t)arg * gridDim.x + blockIdx.x] = tot;
      }
      __syncthreads();
    }
    else {  // P_END
      asm volatile("exit;");
    }
  };

  // Decoded instruction stream: one uint2 {case id, argument} per word, so that the decode of an
  // instruction is a single 64-bit shared-memory load.  `ip` points at the entry after `w`.
  ip = code2 + 1;
  uint2 w = code2[0];
  for (;;) {
    wn = *ip;   // fetched ahead of the dispatch below
    ++ip;
    const int cs = (int)w.x;                      // < P_COUNT_: launch_vm() validates the stream once
    asm volatile("// VMDISPATCH %0" ::"r"(cs));   // the build step puts an indexed jump here
    dispatch_tree<0, P_COUNT_>(cs, w.y, exec);
    w = wn;
  }
}

// ---- finishing reductions: per-CTA partials -> tensors (fixed order, fp64) ------------------

struct FinishParams {
  int n_jobs;
  struct Job {
    int kind;          // 0 column sums, 1 scalar
    const void* part;  // float [grid][cols] or double [grid]
    void* out;
    int dtype, cols, grid;
  } job[8];
};

__global__ void finish_kernel(const __grid_constant__ FinishParams fp) {
  const FinishParams::Job& jb = fp.job[blockIdx.y];
  if (jb.kind == 0) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= jb.cols) return;
    const float* part = reinterpret_cast<const float*>(jb.part);
    double s = 0.0;
    for (int g = 0; g < jb.grid; ++g) s += (double)part[(size_t)g * jb.cols + c];
    if (jb.dtype == DRAGON_F32) reinterpret_cast<float*>(jb.out)[c] = (float)s;
    else reinterpret_cast<unsigned short*>(jb.out)[c] = (unsigned short)vmmath::bf16_bits((float)s);
  } else if (blockIdx.x == 0 && threadIdx.x == 0) {
    const double* part = reinterpret_cast<const double*>(jb.part);
    double s = 0.0;
    for (int g = 0; g < jb.grid; ++g) s += part[g];
    if (jb.dtype == DRAGON_F32) *reinterpret_cast<float*>(jb.out) = (float)s;
    else *reinterpret_cast<unsigned short*>(jb.out) = (unsigned short)vmmath::bf16_bits((float)s);
  }
}

size_t vm_smem_bytes(int n_code, int n_smem_slots) {
  return (size_t)((n_code + 3) & ~3) * 8 + kMaxUniforms * 4 + 64 * 8 + kMaxOperands * 16 + (size_t)n_smem_slots * NV4 * NT * 16;
}

}  // namespace vm

}  // namespace dragon

// cubin of this same kernel with the dispatch tree replaced by one indexed jump (build step
// ptx_jumptable.py); size 0 when that step refused
extern "C" const unsigned long dragon_vm_jt_cubin_size;
extern "C" const unsigned char dragon_vm_jt_cubin[];
extern "C" const unsigned long dragon_vm_gen_cubin_size;
extern "C" const unsigned char dragon_vm_gen_cubin[];

namespace dragon {

// the kernel to launch: the jump-table build when it is there (and DRAGON_VM_DISPATCH != "tree"),
// else the compiled-in tree kernel
static const void* vm_entry() {
  static const void* entry = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    entry = reinterpret_cast<const void*>(vm::vm_kernel);
    const char* mode = std::getenv("DRAGON_VM_DISPATCH");
    if (mode && std::string(mode) == "gen") {
      cudaLibrary_t lib;
      cudaKernel_t k;
      if (cudaLibraryLoadData(&lib, dragon_vm_gen_cubin, nullptr, nullptr, 0, nullptr, nullptr, 0) == cudaSuccess &&
          cudaLibraryGetKernel(&k, lib, "dragon_vm_r7") == cudaSuccess) {
        entry = reinterpret_cast<const void*>(k);
        return;
      }
      cudaGetLastError();
    }
    if (dragon_vm_jt_cubin_size == 0 || (mode && std::string(mode) == "tree")) return;
    cudaLibrary_t lib;
    cudaKernel_t k;
    if (cudaLibraryLoadData(&lib, dragon_vm_jt_cubin, nullptr, nullptr, 0, nullptr, nullptr, 0) == cudaSuccess &&
        cudaLibraryGetKernel(&k, lib, "_ZN6dragon2vm9vm_kernelENS0_6ParamsE") == cudaSuccess) {
      entry = reinterpret_cast<const void*>(k);
    } else {
      cudaGetLastError();
    }
  });
  return entry;
}

// launch helpers used by api.cu
cudaError_t launch_vm(const vm::Params& p, int grid, int n_smem_slots, cudaStream_t st) {
  const size_t smem = vm::vm_smem_bytes(p.n_code, n_smem_slots);
  const void* entry = vm_entry();
  cudaError_t e = cudaFuncSetAttribute(entry, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e != cudaSuccess) return e;
  void* args[] = {const_cast<vm::Params*>(&p)};
  return cudaLaunchKernel(entry, dim3(grid), dim3(vm::NT), args, smem, st);
}

cudaError_t launch_finish(const VmSegment& sg, const std::vector<MemRef>& mems, void* const* mem_ptr, char* ws, cudaStream_t st) {
  if (sg.finish.empty()) return cudaSuccess;
  vm::FinishParams fp;
  fp.n_jobs = (int)sg.finish.size();
  int max_cols = 1;
  for (int i = 0; i < fp.n_jobs; ++i) {
    const FinishJob& j = sg.finish[i];
    auto& o = fp.job[i];
    o.kind = j.kind;
    o.grid = sg.grid;
    o.cols = sg.cols;
    o.dtype = mems[j.mem].dtype;
    o.out = mem_ptr[j.mem];
    if (j.kind == 0) { o.part = ws + sg.colpart_off + (size_t)j.acc * sg.grid * sg.cols * sizeof(float); max_cols = std::max(max_cols, sg.cols); }
    else o.part = ws + sg.scalpart_off + (size_t)j.acc * sg.grid * sizeof(double);
  }
  dim3 grid((max_cols + 127) / 128, fp.n_jobs);
  vm::finish_kernel<<<grid, 128, 0, st>>>(fp);
  return cudaGetLastError();
}

}  // namespace dragon
