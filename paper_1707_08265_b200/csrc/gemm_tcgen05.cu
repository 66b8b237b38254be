// InnerProduct contraction C[M,N] = A[M,K] * B[N,K]^T: bf16 operands, fp32 accumulation in
// tensor memory, fp32 or bf16 output.  Hand-written for sm_100a:
//   - operands are staged by TMA (cp.async.bulk.tensor, 128-byte swizzle; every CTA loads its own
//     tiles) into a ring of shared-memory stages guarded by full/empty mbarriers;
//   - one elected thread issues tcgen05.mma (kind::f16; cta_group::1 with 128 x 256 x 16, or, in the
//     pair kernel, cta_group::2 with 256 x 256 x 16 over the two CTAs of a cluster) with the
//     accumulator in TMEM; tcgen05.commit releases stages and signals the epilogue;
//   - four epilogue warps read their 32-lane TMEM quadrants with tcgen05.ld and write C;
//   - CTAs are persistent (one per SM) and walk the 128 x 256 output tiles in an L2-friendly
//     order; two TMEM accumulators alternate, so the epilogue of one tile overlaps the main loop
//     of the next.
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer,
// warps 2..5 = epilogue.  Every mbarrier wait is bounded by a clock budget; when it runs out
// the kernel records DRAGON_ERR_TIMEOUT in the status word, stops issuing work, frees its TMEM
// and returns.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstdlib>
#include <mutex>

#include "plan.h"
#include "vm_math.h"

namespace dragon {
namespace {

constexpr int kTileM = 128;
constexpr int kTileN = 256;
constexpr int kTileK = 64;          // one 128-byte swizzle row of bf16
constexpr int kStages = 4;
constexpr int kUmmaK = 16;
constexpr int kAccBufs = 2;         // double-buffered accumulators: 2 x 256 TMEM columns
constexpr int kGemmThreads = 192;
constexpr uint32_t kStageBytesA = kTileM * kTileK * 2;
constexpr uint32_t kStageBytesB = kTileN * kTileK * 2;
constexpr uint32_t kStageBytes = kStageBytesA + kStageBytesB;
constexpr size_t kGemmSmem = 1024 /*alignment slack*/ + (size_t)kStages * kStageBytes + 256 /*barriers*/;
constexpr long long kWaitBudgetCycles = 4000000000LL;   // about two seconds

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// bounded wait: false when the clock budget ran out (the caller records the failure and unwinds)
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long budget = kWaitBudgetCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > budget) return false;
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

// shared-memory matrix descriptor: K-major tile, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);          // start address
  d |= (uint64_t)1 << 16;                            // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset
  d |= (uint64_t)1 << 46;                            // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                            // SWIZZLE_128B
  return d;
}
// the same for an MN-major operand (the memory matrix is [K, MN] row-major): the tile is stored as
// chunks of 64 MN-elements; inside a chunk every K-row is one 128-byte swizzle row, 8 K-rows form a
// 1024-byte group (stride byte offset) and chunks are 8192 bytes apart (leading byte offset)
__device__ __forceinline__ uint64_t make_smem_desc_mn(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);
  d |= (uint64_t)(8192 >> 4) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// instruction descriptor: D = f32, A = B = bf16, M x N; bits 15 / 16 select MN-major A / B
constexpr uint32_t make_idesc(int m, int n, bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
}

// ---- helpers of the pair kernel (two CTAs of a cluster on one tile) --------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// the shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrival on an mbarrier of another CTA of the cluster (bar: a shared::cluster address)
__device__ __forceinline__ void mbar_arrive_remote(uint32_t bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}
// TMA copy of one CTA of a pair into its own shared memory; the bytes are counted on the mbarrier `bar` (a
// shared::cluster address: the first CTA's); each CTA copies only what it reads itself
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void umma_f16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// the MMAs issued so far are done: one arrival on the mbarrier at this address in both CTAs of the pair
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((unsigned short)3) : "memory");
}

struct EpiArg {
  int opc, operand, dtype;   // EpiOpc, EpiOperand, type of the memory operand
  float c;                   // EO_CONST
  const void* ptr;           // EO_SCALAR: one element; EO_ROW: N elements; EO_FULL: [M, N] row-major
};

struct GemmArgs {
  void* C;
  int c_dtype;
  int M, N, K;
  int tiles_m, tiles_n;
  int* status;
  // epilogue: C = act(acc + bias[col]); bias is a row vector of N elements (null: none)
  const void* bias;
  int bias_dtype;
  int relu;
  // then multiplied by step(mask[row, col]) (1 where the bf16 mask element is > 0, else 0); null: none
  const unsigned short* mask;
  // clock budget of the pipeline waits (the waits that let in-flight work finish during an unwind keep the
  // full budget), and the failure-detection test's hook: the producer leaves out the loads of its first
  // stage, so that the consumer's first wait is for a signal that nothing sends
  long long wait_budget;
  int drop_first_load;
  // and then the epilogue program: n_epi operations on every element, in order (plan.h: EpiSpec)
  int n_epi;
  EpiArg epi[kMaxEpiOps];
  // partial column sums of the values that are written (before their rounding to C's type), one row of N floats
  // per 32 output rows: colpart[(row / 32)][col]; null: none.  A finishing kernel adds the rows in a fixed order.
  float* colpart;
};

__device__ __forceinline__ float epi_load(const void* p, int dtype, size_t i) {
  return dtype == DRAGON_F32 ? __ldg(reinterpret_cast<const float*>(p) + i)
                             : __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p) + i) << 16);
}

// one operation of the epilogue program on the 32 accumulator values of this thread (row `row`, columns col0..col0+31);
// the elementary functions are those of the VM's leaves
__device__ __forceinline__ void epi_apply(const EpiArg& e, uint32_t* v, int row, int col0, int M, int N) {
  float x[32];
  if (e.operand == EO_CONST || e.operand == EO_SCALAR) {
    const float c = e.operand == EO_CONST ? e.c : epi_load(e.ptr, e.dtype, 0);
#pragma unroll
    for (int j = 0; j < 32; ++j) x[j] = c;
  } else if (e.operand == EO_ROW || e.operand == EO_FULL) {
    const size_t base = (e.operand == EO_FULL ? (size_t)(row < M ? row : 0) * N : 0) + col0;
    const bool aligned = (N & 7) == 0 && col0 + 32 <= N && (reinterpret_cast<uintptr_t>(e.ptr) & 15) == 0;
    if (aligned && e.dtype == DRAGON_F32) {
      const float4* p4 = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(e.ptr) + base);
#pragma unroll
      for (int j = 0; j < 8; ++j) { const float4 t = __ldg(p4 + j); x[4 * j] = t.x; x[4 * j + 1] = t.y; x[4 * j + 2] = t.z; x[4 * j + 3] = t.w; }
    } else if (aligned) {
      const uint4* p8 = reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned short*>(e.ptr) + base);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint4 t = __ldg(p8 + j);
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) { x[8 * j + 2 * k] = __uint_as_float(w[k] << 16); x[8 * j + 2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u); }
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) x[j] = col0 + j < N ? epi_load(e.ptr, e.dtype, base + j) : 0.f;
    }
  }
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    float a = __uint_as_float(v[j]);
    switch (e.opc) {
      case E_ADD: a = a + x[j]; break;
      case E_SUB: a = a - x[j]; break;
      case E_RSUB: a = x[j] - a; break;
      case E_MUL: a = a * x[j]; break;
      case E_RELU: a = fmaxf(a, 0.f); break;
      case E_TANH: a = vmmath::tanh_f(a); break;
      case E_SIGMOID: a = vmmath::sigmoid_f(a); break;
      case E_EXPC: a = vmmath::exp_clamped10(a); break;
      case E_SIN: a = vmmath::sin_f(a); break;
      case E_NEG: a = -a; break;
      case E_SQRT: a = vmmath::sqrt_f(a); break;
      case E_RCP: a = vmmath::f_rcp(a); break;
      default: a = vmmath::round_bf16(a); break;    // E_RBF16
    }
    v[j] = __float_as_uint(a);
  }
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// tile order: groups of 8 row-blocks share their column sweep, so that the B tiles of a sweep
// and the 8 A row-blocks stay in L2 while they are reused
__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int* tm, int* tn) {
  const int group = 8 * tiles_n;
  const int g0 = (t / group) * 8;
  const int rows = min(8, tiles_m - g0);
  const int r = t % group;
  *tm = g0 + r % rows;
  *tn = r / rows;
}

template <bool kAMn, bool kBMn, bool kPair>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_bf16_tcgen05(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const GemmArgs g) {
  // kPair: two CTAs of a cluster work on one 256 x 256 tile (tcgen05.mma.cta_group::2): CTA r of the pair holds rows
  // r*128.. of the A tile and of the accumulator and rows r*128.. of the B tile (half of the N extent), each loads
  // its own halves with its own TMA copies, and the pair's first CTA issues the MMAs for both.  Per stage a CTA
  // then stages 16 KB of B instead of 32 KB (six stages instead of four) and its tensor unit reads half the B bytes.
  constexpr int kSt = kPair ? 6 : kStages;
  constexpr uint32_t kSBB = kPair ? kStageBytesB / 2 : kStageBytesB;
  constexpr uint32_t kSB = kStageBytesA + kSBB;
  static_assert((size_t)kSt * kSB == (size_t)kStages * kStageBytes, "same shared-memory footprint");
  extern __shared__ unsigned char gemm_smem_raw[];
  const uint32_t raw = smem_u32(gemm_smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;                 // 1024-byte aligned operand stages
  unsigned char* tiles_ptr = gemm_smem_raw + (tiles - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles_ptr + (size_t)kSt * kSB);
  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * kSt;
  const uint32_t bar_acc_full = bar_empty + 8 * kSt, bar_acc_empty = bar_acc_full + 8 * kAccBufs;
  const uint32_t bar_drain = bar_acc_empty + 8 * kAccBufs;     // used by an unwind only: "every MMA issued so far is done"
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kSt + 2 * kAccBufs + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int k_tiles = (g.K + kTileK - 1) / kTileK;
  const int n_tiles = g.tiles_m * g.tiles_n;
  // who walks the tiles: every CTA on its own, or every pair (tiles are then 256 rows high, 128 per CTA)
  const uint32_t rank = kPair ? cluster_ctarank() : 0u;
  const int unit = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int n_units = kPair ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  constexpr int kRowsPerTile = kPair ? 2 * kTileM : kTileM;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kSt; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    for (int b = 0; b < kAccBufs; ++b) { mbar_init(bar_acc_full + 8 * b, 1); mbar_init(bar_acc_empty + 8 * b, kPair ? 8 : 4); }
    mbar_init(bar_drain, 1);
    abort_flag[0] = 0;
    abort_flag[1] = 0;   // a flag nobody sets, for waits that must not be cut short
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // TMEM: two accumulators of kTileN fp32 columns x 128 lanes
    if (kPair) {   // the same warp of both CTAs, the same shared-memory location
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)(kAccBufs * kTileN)) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)(kAccBufs * kTileN)) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  if (kPair) cluster_sync_all();   // nobody signals a barrier of the other CTA before it is initialised
  const uint32_t bar_full_first = kPair ? map_to_cta(bar_full, 0) : bar_full;   // the pair counts its copies on the first CTA's barriers

  int issued = 0;          // thread 0 (the producer): stages handed to the TMA engine so far
  int first_issued = 0;    // ... of which the first few may have been left out by the test hook
  if (warp == 0) {
    if (lane == 0) {  // TMA producer: one running stage counter across all tiles of this CTA
      bool ok = true;
      for (int t = unit; t < n_tiles && ok; t += n_units) {
        int tm, tn;
        tile_coords(t, g.tiles_m, g.tiles_n, &tm, &tn);
        for (int kt = 0; kt < k_tiles; ++kt, ++issued) {
          const int s = issued % kSt, it = issued / kSt;
          if (!mbar_wait(bar_empty + 8 * s, (it & 1) ^ 1, abort_flag, g.wait_budget)) { *abort_flag = 1; atomicExch(g.status, DRAGON_ERR_TIMEOUT); ok = false; break; }
          if (g.drop_first_load && issued == 0) { first_issued = 1; continue; }     // failure-detection test: this stage's signal never comes
          const uint32_t dst = tiles + (uint32_t)s * kSB;
          if (kPair) {   // both CTAs copy their halves; the first CTA's barrier expects the bytes of both
            if (rank == 0) mbar_expect_tx(bar_full + 8 * s, 2 * kSB);
            const int a0 = tm * kRowsPerTile + (int)rank * kTileM, b0 = tn * kTileN + (int)rank * (kTileN / 2);
            if (!kAMn) {
              tma_load_2d_pair(dst, &tmap_a, kt * kTileK, a0, bar_full_first + 8 * s);
            } else {
#pragma unroll
              for (int c = 0; c < kTileM / 64; ++c) tma_load_2d_pair(dst + c * 8192, &tmap_a, a0 + c * 64, kt * kTileK, bar_full_first + 8 * s);
            }
            if (!kBMn) {
              tma_load_2d_pair(dst + kStageBytesA, &tmap_b, kt * kTileK, b0, bar_full_first + 8 * s);
            } else {
#pragma unroll
              for (int c = 0; c < kTileN / 128; ++c) tma_load_2d_pair(dst + kStageBytesA + c * 8192, &tmap_b, b0 + c * 64, kt * kTileK, bar_full_first + 8 * s);
            }
            continue;
          }
          mbar_expect_tx(bar_full + 8 * s, kStageBytes);
          if (!kAMn) {
            tma_load_2d(dst, &tmap_a, kt * kTileK, tm * kTileM, bar_full + 8 * s);
          } else {  // boxes of 64 MN-elements x 64 K-rows, one per chunk
#pragma unroll
            for (int c = 0; c < kTileM / 64; ++c) tma_load_2d(dst + c * 8192, &tmap_a, tm * kTileM + c * 64, kt * kTileK, bar_full + 8 * s);
          }
          if (!kBMn) {
            tma_load_2d(dst + kStageBytesA, &tmap_b, kt * kTileK, tn * kTileN, bar_full + 8 * s);
          } else {
#pragma unroll
            for (int c = 0; c < kTileN / 64; ++c) tma_load_2d(dst + kStageBytesA + c * 8192, &tmap_b, tn * kTileN + c * 64, kt * kTileK, bar_full + 8 * s);
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {  // MMA issuer (of a pair: the first CTA's)
      constexpr uint32_t idesc = make_idesc(kRowsPerTile, kTileN, kAMn, kBMn);
      int consumed = 0, local = 0;
      bool ok = true;
      for (int t = unit; t < n_tiles && ok; t += n_units, ++local) {
        const int buf = local % kAccBufs, use = local / kAccBufs;
        // the epilogue must have drained this accumulator (first use passes at once)
        if (!mbar_wait(bar_acc_empty + 8 * buf, (use & 1) ^ 1, abort_flag, g.wait_budget)) { *abort_flag = 1; atomicExch(g.status, DRAGON_ERR_TIMEOUT); break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * kTileN);
        for (int kt = 0; kt < k_tiles; ++kt, ++consumed) {
          const int s = consumed % kSt, it = consumed / kSt;
          if (!mbar_wait(bar_full + 8 * s, it & 1, abort_flag, g.wait_budget)) { *abort_flag = 1; atomicExch(g.status, DRAGON_ERR_TIMEOUT); ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = tiles + (uint32_t)s * kSB, b_addr = a_addr + kStageBytesA;
          const uint64_t a_desc = kAMn ? make_smem_desc_mn(a_addr) : make_smem_desc(a_addr);
          const uint64_t b_desc = kBMn ? make_smem_desc_mn(b_addr) : make_smem_desc(b_addr);
#pragma unroll
          for (int k = 0; k < kTileK / kUmmaK; ++k) {
            // 16 elements along K: K-major = 32 bytes inside the swizzle row (2 descriptor units),
            // MN-major = two 8-row groups = 2048 bytes (128 units)
            if (kPair) umma_f16_pair(d_tmem, a_desc + (kAMn ? 128 : 2) * k, b_desc + (kBMn ? 128 : 2) * k, idesc, (kt > 0 || k > 0) ? 1u : 0u);
            else umma_f16(d_tmem, a_desc + (kAMn ? 128 : 2) * k, b_desc + (kBMn ? 128 : 2) * k, idesc, (kt > 0 || k > 0) ? 1u : 0u);
          }
          if (kPair) umma_commit_pair(bar_empty + 8 * s);   // the stage is free in both CTAs once these MMAs have read it
          else umma_commit(bar_empty + 8 * s);
        }
        if (ok) { if (kPair) umma_commit_pair(bar_acc_full + 8 * buf); else umma_commit(bar_acc_full + 8 * buf); }   // accumulator complete
      }
      if (*abort_flag) {   // unwinding: every MMA issued so far must be done before its operands and the TMEM go away
        if (kPair) umma_commit_pair(bar_drain); else umma_commit(bar_drain);
        mbar_wait(bar_drain, 0, abort_flag + 1);
      }
    }
  } else {
    // epilogue: warp w owns TMEM lanes 32*(w%4) .. +31, i.e. rows 32*(w%4) + lane of the tile
    const int q = warp & 3;
    int local = 0;
    for (int t = unit; t < n_tiles; t += n_units, ++local) {
      const int buf = local % kAccBufs, use = local / kAccBufs;
      int tm, tn;
      tile_coords(t, g.tiles_m, g.tiles_n, &tm, &tn);
      const bool ok = mbar_wait(bar_acc_full + 8 * buf, use & 1, abort_flag, g.wait_budget);
      if (!ok) { if (lane == 0) { *abort_flag = 1; atomicExch(g.status, DRAGON_ERR_TIMEOUT); } break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int row = tm * kRowsPerTile + (int)rank * kTileM + q * 32 + lane;
#pragma unroll 1
      for (int c = 0; c < kTileN; c += 32) {
        uint32_t v[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * kTileN + c), v);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        const int col0 = tn * kTileN + c;
        if (g.bias != nullptr && col0 < g.N) {
          // every lane of the warp reads the same 32 bias values (broadcast loads)
          if (col0 + 32 <= g.N && (g.N & 7) == 0 && (reinterpret_cast<uintptr_t>(g.bias) & 15) == 0) {
            if (g.bias_dtype == DRAGON_F32) {
              const float4* b4 = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(g.bias) + col0);
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const float4 b = __ldg(b4 + j);
                v[4 * j] = __float_as_uint(__uint_as_float(v[4 * j]) + b.x);
                v[4 * j + 1] = __float_as_uint(__uint_as_float(v[4 * j + 1]) + b.y);
                v[4 * j + 2] = __float_as_uint(__uint_as_float(v[4 * j + 2]) + b.z);
                v[4 * j + 3] = __float_as_uint(__uint_as_float(v[4 * j + 3]) + b.w);
              }
            } else {
              const uint4* b8 = reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned short*>(g.bias) + col0);
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const uint4 b = __ldg(b8 + j);
                const uint32_t w[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                  v[8 * j + 2 * k] = __float_as_uint(__uint_as_float(v[8 * j + 2 * k]) + __uint_as_float(w[k] << 16));
                  v[8 * j + 2 * k + 1] = __float_as_uint(__uint_as_float(v[8 * j + 2 * k + 1]) + __uint_as_float(w[k] & 0xffff0000u));
                }
              }
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (col0 + j < g.N) {
                const float b = g.bias_dtype == DRAGON_F32
                                    ? __ldg(reinterpret_cast<const float*>(g.bias) + col0 + j)
                                    : __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(g.bias) + col0 + j) << 16);
                v[j] = __float_as_uint(__uint_as_float(v[j]) + b);
              }
          }
        }
        if (g.relu) {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(fmaxf(__uint_as_float(v[j]), 0.f));
        }
        if (g.mask != nullptr && row < g.M && col0 < g.N) {
          const unsigned short* mrow = g.mask + (size_t)row * g.N + col0;
          if ((g.N & 7) == 0 && col0 + 32 <= g.N && (reinterpret_cast<uintptr_t>(g.mask) & 15) == 0) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint4 m = *reinterpret_cast<const uint4*>(mrow + 8 * j);
              const uint32_t w[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                v[8 * j + 2 * k] = __float_as_uint(__uint_as_float(v[8 * j + 2 * k]) * (__uint_as_float(w[k] << 16) > 0.f ? 1.f : 0.f));
                v[8 * j + 2 * k + 1] = __float_as_uint(__uint_as_float(v[8 * j + 2 * k + 1]) * (__uint_as_float(w[k] & 0xffff0000u) > 0.f ? 1.f : 0.f));
              }
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (col0 + j < g.N) v[j] = __float_as_uint(__uint_as_float(v[j]) * (__uint_as_float((uint32_t)mrow[j] << 16) > 0.f ? 1.f : 0.f));
          }
        }
        if (col0 < g.N)
          for (int e = 0; e < g.n_epi; ++e) epi_apply(g.epi[e], v, row, col0, g.M, g.N);
        if (g.colpart != nullptr && col0 < g.N) {
          // sum over the 32 rows that this warp holds, for each of its 32 columns: a transposing butterfly (at
          // every step a lane keeps one half of its values and receives the other lanes' share of that half):
          // 31 shuffles, after which lane c holds the sum of column col0 + c
          float t[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) t[j] = row < g.M ? __uint_as_float(v[j]) : 0.f;
#pragma unroll
          for (int sft = 16; sft >= 1; sft >>= 1) {
            const bool upper = (lane & sft) != 0;
#pragma unroll
            for (int j = 0; j < sft; ++j) {
              const float send = upper ? t[j] : t[j + sft], keep = upper ? t[j + sft] : t[j];
              t[j] = keep + __shfl_xor_sync(0xffffffffu, send, sft);
            }
          }
          if (col0 + lane < g.N) g.colpart[(size_t)(tm * (kRowsPerTile / 32) + (int)rank * 4 + q) * g.N + col0 + lane] = t[0];
        }
        if (row < g.M && col0 < g.N) {
          if (g.c_dtype == DRAGON_F32) {
            float* out = reinterpret_cast<float*>(g.C) + (size_t)row * g.N + col0;
            if ((g.N & 3) == 0 && col0 + 32 <= g.N) {
#pragma unroll
              for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<float4*>(out + j) = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + j < g.N) out[j] = __uint_as_float(v[j]);
            }
          } else {
            unsigned short* out = reinterpret_cast<unsigned short*>(g.C) + (size_t)row * g.N + col0;
            if ((g.N & 7) == 0 && col0 + 32 <= g.N) {
#pragma unroll
              for (int j = 0; j < 32; j += 8) {
                uint4 pk;
                pk.x = vmmath::bf16_bits(__uint_as_float(v[j])) | (vmmath::bf16_bits(__uint_as_float(v[j + 1])) << 16);
                pk.y = vmmath::bf16_bits(__uint_as_float(v[j + 2])) | (vmmath::bf16_bits(__uint_as_float(v[j + 3])) << 16);
                pk.z = vmmath::bf16_bits(__uint_as_float(v[j + 4])) | (vmmath::bf16_bits(__uint_as_float(v[j + 5])) << 16);
                pk.w = vmmath::bf16_bits(__uint_as_float(v[j + 6])) | (vmmath::bf16_bits(__uint_as_float(v[j + 7])) << 16);
                *reinterpret_cast<uint4*>(out + j) = pk;
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + j < g.N) out[j] = (unsigned short)vmmath::bf16_bits(__uint_as_float(v[j]));
            }
          }
        }
      }
      // this warp is done reading the accumulator: hand it back to the MMA issuer
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        if (kPair && rank != 0) mbar_arrive_remote(map_to_cta(bar_acc_empty + 8 * buf, 0));
        else mbar_arrive(bar_acc_empty + 8 * buf);
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (*abort_flag) {
    // an unwind: every role has stopped (barrier above).  The copies that the producer has handed to the TMA
    // engine and that nobody consumed must land before the CTA's shared memory goes away; this wait keeps the
    // full budget whatever the pipeline's budget is.
    if (threadIdx.x == 0) {
      if (kPair) {   // the copies are counted on the first CTA's barriers: give them time instead (they take microseconds)
        const long long t0 = clock64();
        while (clock64() - t0 < 20000000LL) { }
      } else {
        for (int i = std::max(first_issued, issued > kSt ? issued - kSt : 0); i < issued; ++i)
          mbar_wait(bar_full + 8 * (i % kSt), (i / kSt) & 1, abort_flag + 1);
      }
    }
    __syncthreads();
  }
  if (kPair) cluster_sync_all();   // neither CTA leaves while the other may still signal its barriers or read its tiles
  if (warp == 1) {
    if (kPair) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)(kAccBufs * kTileN)) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)(kAccBufs * kTileN)) : "memory");
  }
}

// ---- host side ---------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// row-major bf16 [rows, cols] viewed as a 2-D tensor map with boxes of box_rows x 64 elements
// (K-major operand: rows = M or N, cols = K, box_rows = tile height; MN-major operand: rows = K,
// cols = M or N, box_rows = 64)
bool make_tmap(CUtensorMap* map, const void* ptr, int rows, int cols, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The encoding of a tensor map depends only on the pointer and the extents; a function runs with the same
// workspace and, usually, the same feed pointers step after step, so the last few encodings are kept.
bool cached_tmap(CUtensorMap* map, const void* ptr, int rows, int cols, int box_rows) {
  struct Entry { const void* ptr; int rows, cols, box; CUtensorMap map; };
  static std::mutex mu;
  static Entry cache[64];
  static int used = 0, next = 0;
  std::lock_guard<std::mutex> lock(mu);
  for (int i = 0; i < used; ++i)
    if (cache[i].ptr == ptr && cache[i].rows == rows && cache[i].cols == cols && cache[i].box == box_rows) { *map = cache[i].map; return true; }
  if (!make_tmap(map, ptr, rows, cols, box_rows)) return false;
  cache[next] = Entry{ptr, rows, cols, box_rows, *map};
  next = (next + 1) % 64;
  used = std::min(used + 1, 64);
  return true;
}

}  // namespace

// C[M,N] = opA * opB^T with K the contraction length.  a_mn / b_mn: the operand is given as the
// row-major matrix [K, M] (resp. [K, N]) instead of [M, K] (resp. [N, K]).
// epi: the operations that follow on every element, in order (operands by memory id, pointers in mem_ptr).
// bias (may be null): row vector of N elements of type bias_dtype (fp32 or bf16), added to every
// row of the product; relu: max(., 0) applied after it; mask (may be null): bf16 [M, N], the result is
// multiplied by 1 where the mask element is > 0 and by 0 elsewhere; all before the rounding to C's type.
int launch_gemm_bf16(const void* A, const void* B, void* C, int c_dtype, int M, int N, int K, bool a_mn, bool b_mn, int* status,
                     cudaStream_t st, const void* bias, int bias_dtype, bool relu, const void* mask,
                     const std::vector<EpiSpec>& epi, const std::vector<MemRef>& mems, void* const* mem_ptr, float* colpart) {
  const int a_inner = a_mn ? M : K, b_inner = b_mn ? N : K;
  if (M <= 0 || N <= 0 || K <= 0 || (a_inner & 7) || (b_inner & 7) || ((uintptr_t)A & 15) || ((uintptr_t)B & 15) || ((uintptr_t)C & 15)) {
    set_error("InnerProduct: the contiguous extent of every operand must be a multiple of 8 and all pointers 16-byte aligned (M=%d N=%d K=%d)", M, N, K);
    return DRAGON_ERR_UNSUPPORTED;
  }
  // Two CTAs per 256 x 256 tile wherever the product has more than one block of 128 rows (measured 8-9 % faster on
  // the 8192 x 4096 x 4096 products: the tensor units read half the B bytes from shared memory);
  // DRAGON_GEMM_PAIR=0 / 1 forces one CTA per 128 x 256 tile / the pair kernel.
  bool pair = M > kTileM;
  if (const char* e = std::getenv("DRAGON_GEMM_PAIR")) pair = e[0] == '1';
  CUtensorMap ta, tb;
  const bool ok_a = a_mn ? cached_tmap(&ta, A, K, M, 64) : cached_tmap(&ta, A, M, K, kTileM);
  const bool ok_b = b_mn ? cached_tmap(&tb, B, K, N, 64) : cached_tmap(&tb, B, N, K, pair ? kTileN / 2 : kTileN);
  if (!ok_a || !ok_b) {
    set_error("InnerProduct: cannot encode the TMA descriptors (no CUDA driver?)");
    return DRAGON_ERR_CUDA;
  }
  auto kern = pair ? (a_mn ? gemm_bf16_tcgen05<true, true, true> : (b_mn ? gemm_bf16_tcgen05<false, true, true> : gemm_bf16_tcgen05<false, false, true>))
                   : (a_mn ? gemm_bf16_tcgen05<true, true, false> : (b_mn ? gemm_bf16_tcgen05<false, true, false> : gemm_bf16_tcgen05<false, false, false>));
  if (a_mn && !b_mn) { set_error("InnerProduct: this operand layout combination is not built"); return DRAGON_ERR_UNSUPPORTED; }
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { set_error("InnerProduct: no current device"); return DRAGON_ERR_CUDA; }
  // once per device and kernel variant: the shared-memory attribute and the SM count
  static std::mutex mu;
  static bool attr_set[64][6] = {};
  static int sm_counts[64] = {};
  const int variant = (a_mn ? 2 : (b_mn ? 1 : 0)) + (pair ? 3 : 0);
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!attr_set[dev][variant]) {
      cudaError_t attr_err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGemmSmem);
      if (attr_err != cudaSuccess) { set_error("InnerProduct: %s", cudaGetErrorString(attr_err)); return DRAGON_ERR_CUDA; }
      attr_set[dev][variant] = true;
    }
    if (!sm_counts[dev] && (cudaDeviceGetAttribute(&sm_counts[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_counts[dev] <= 0))
      sm_counts[dev] = kDefaultSmCount;
  }
  const int sm_count = sm_counts[dev];
  const int tile_rows = pair ? 2 * kTileM : kTileM;
  const int tiles_m = (M + tile_rows - 1) / tile_rows, tiles_n = (N + kTileN - 1) / kTileN;
  GemmArgs g{C, c_dtype, M, N, K, tiles_m, tiles_n, status, bias, bias_dtype, relu ? 1 : 0, reinterpret_cast<const unsigned short*>(mask),
             kWaitBudgetCycles, 0, 0, {}, colpart};
  if ((int)epi.size() > kMaxEpiOps) { set_error("InnerProduct: epilogue program too long"); return DRAGON_ERR_UNSUPPORTED; }
  for (const EpiSpec& e : epi) {
    EpiArg& a = g.epi[g.n_epi++];
    a.opc = e.opc; a.operand = e.operand; a.c = e.c;
    a.dtype = e.mem >= 0 ? mems[e.mem].dtype : DRAGON_F32;
    a.ptr = e.mem >= 0 ? mem_ptr[e.mem] : nullptr;
    if (e.operand != EO_NONE && e.operand != EO_CONST && !a.ptr) { set_error("InnerProduct: epilogue operand has no memory"); return DRAGON_ERR_INVALID_ARG; }
  }
  // failure-detection test only: DRAGON_GEMM_WAIT_BUDGET=<clock cycles> shortens the pipeline waits and
  // DRAGON_GEMM_DROP_FIRST_LOAD=1 makes the first of them wait for a signal that nothing sends
  if (const char* e = std::getenv("DRAGON_GEMM_WAIT_BUDGET")) { const long long b = std::atoll(e); if (b > 0) g.wait_budget = std::min(b, kWaitBudgetCycles); }
  if (const char* e = std::getenv("DRAGON_GEMM_DROP_FIRST_LOAD")) g.drop_first_load = e[0] == '1';
  cudaError_t e;
  if (pair) {   // clusters of two CTAs, one CTA per SM
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * std::min(tiles_m * tiles_n, sm_count / 2));
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = kGemmSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kern, ta, tb, g);
  } else {
    const int grid = std::min(tiles_m * tiles_n, sm_count);   // persistent CTAs, one per SM
    kern<<<grid, kGemmThreads, kGemmSmem, st>>>(ta, tb, g);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) { set_error("InnerProduct: launch failed: %s", cudaGetErrorString(e)); return DRAGON_ERR_CUDA; }
  return DRAGON_OK;
}

}  // namespace dragon
