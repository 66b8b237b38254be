// Launch side of the graph VM.  The interpreter kernel itself is written in PTX by
// vm_ptxgen.py (two builds: "wide" and "dense", see vm_isa.h); its cubin is embedded in the
// library by the build and loaded here.  This file also holds the small finishing kernel that
// turns per-CTA partial sums into tensors.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>
#include <mutex>

#include "plan.h"
#include "vm_math.h"

// cubin assembled from the generated PTX (build.py)
extern "C" const unsigned long dragon_vm_gen_cubin_size;
extern "C" const unsigned char dragon_vm_gen_cubin[];

namespace dragon {
namespace vm {

// ---- finishing reductions: per-CTA partials -> tensors (fixed order, fp64) ------------------

// a segment reduces at most kVmScalarAccs sums in scalar accumulators, kVmRegsWide - 2 in pinned register
// slots and kVmSmemSlots - 2 in pinned shared-memory slots
constexpr int kMaxFinishJobs = kVmScalarAccs + kVmRegsWide - 2 + kVmSmemSlots - 2;

struct FinishParams {
  int n_jobs;
  struct Job {
    int kind;          // 0 column sums, 1 scalar
    const void* part;  // float [grid][cols] or double [grid]
    void* out;
    int dtype, cols, grid;
    int chunks, chunk_stride;              // scalar partials of a chunked run: one [accumulator][grid] set per chunk
  } job[kMaxFinishJobs];
};
static_assert(kMaxFinishJobs >= kVmScalarAccs + kVmRegsDense - 2 + kVmSmemSlotsDense - 2 && sizeof(FinishParams) <= 4096,
              "every build's reductions fit one finishing launch");

constexpr int kFinishThreads = 256;

__global__ void finish_kernel(const __grid_constant__ FinishParams fp) {
  // launched as a programmatic dependent of the VM kernel: its blocks may be resident before that
  // kernel ends, and wait here until its partial sums are complete and visible
  cudaGridDependencySynchronize();
  const FinishParams::Job& jb = fp.job[blockIdx.y];
  __shared__ double sh[kFinishThreads];
  if (jb.kind == 0) {
    // a block owns 32 columns; its 8 warps each sum every 8th partial row (coalesced 128-byte
    // reads), then warp 0 adds the 8 slices in order: the same order on every run
    const int lane = threadIdx.x & 31, slice = threadIdx.x >> 5, c = blockIdx.x * 32 + lane;
    const float* part = reinterpret_cast<const float*>(jb.part);
    double s = 0.0;
    if (c < jb.cols) {
      // four partial rows in flight per warp (independent running sums, added in a fixed order afterwards)
      constexpr int kStep = kFinishThreads / 32;
      double s1 = 0.0, s2 = 0.0, s3 = 0.0;
      int g = slice;
      for (; g + 3 * kStep < jb.grid; g += 4 * kStep) {
        const float a0 = part[(size_t)g * jb.cols + c], a1 = part[(size_t)(g + kStep) * jb.cols + c];
        const float a2 = part[(size_t)(g + 2 * kStep) * jb.cols + c], a3 = part[(size_t)(g + 3 * kStep) * jb.cols + c];
        s += (double)a0; s1 += (double)a1; s2 += (double)a2; s3 += (double)a3;
      }
      for (; g < jb.grid; g += kStep) s += (double)part[(size_t)g * jb.cols + c];
      s = (s + s1) + (s2 + s3);
    }
    sh[threadIdx.x] = s;
    __syncthreads();
    if (slice == 0 && c < jb.cols) {
      for (int k = 1; k < kFinishThreads / 32; ++k) s += sh[k * 32 + lane];
      if (jb.dtype == DRAGON_F32) reinterpret_cast<float*>(jb.out)[c] = (float)s;
      else reinterpret_cast<unsigned short*>(jb.out)[c] = (unsigned short)vmmath::bf16_bits((float)s);
    }
  } else if (blockIdx.x == 0) {
    // one block per scalar: strided partial sums, then a tree in shared memory; the order is
    // fixed by the thread count, so the result is the same on every run
    const double* part = reinterpret_cast<const double*>(jb.part);
    double s = 0.0;
    for (int c = 0; c < jb.chunks; ++c)
      for (int g = threadIdx.x; g < jb.grid; g += kFinishThreads) s += part[(size_t)c * jb.chunk_stride + g];
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int w = kFinishThreads / 2; w > 0; w >>= 1) {
      if ((int)threadIdx.x < w) sh[threadIdx.x] += sh[threadIdx.x + w];
      __syncthreads();
    }
    if (threadIdx.x == 0) {
      if (jb.dtype == DRAGON_F32) *reinterpret_cast<float*>(jb.out) = (float)sh[0];
      else *reinterpret_cast<unsigned short*>(jb.out) = (unsigned short)vmmath::bf16_bits((float)sh[0]);
    }
  }
}

// shared memory of one CTA: decoded instruction stream | uniforms | reduction scratch | operand table | slots
size_t vm_smem_bytes(int n_code, int n_smem_slots) {
  return (size_t)((n_code + 3) & ~3) * 8 + kMaxUniforms * 4 + kVmReduceBytes + kMaxOperands * 16 + (size_t)n_smem_slots * kVmTile * 4;
}

}  // namespace vm

struct VmKernels {
  cudaError_t err = cudaErrorUnknown;
  cudaKernel_t wide = nullptr, dense = nullptr;
};

// loads the embedded cubin once per process (kernels of a cudaLibrary_t are usable on every device)
static const VmKernels& vm_kernels() {
  static VmKernels k;
  static std::once_flag once;
  std::call_once(once, [] {
    cudaLibrary_t lib;
    k.err = cudaLibraryLoadData(&lib, dragon_vm_gen_cubin, nullptr, nullptr, 0, nullptr, nullptr, 0);
    if (k.err == cudaSuccess) k.err = cudaLibraryGetKernel(&k.wide, lib, "dragon_vm_wide");
    if (k.err == cudaSuccess) k.err = cudaLibraryGetKernel(&k.dense, lib, "dragon_vm_dense");
    if (k.err == cudaSuccess) k.err = cudaFuncSetAttribute(k.wide, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (k.err == cudaSuccess) k.err = cudaFuncSetAttribute(k.dense, cudaFuncAttributeMaxDynamicSharedMemorySize, 113 * 1024);
  });
  return k;
}

// spec_kernel: the kernel specialised for this program (same parameters, same launch shape), or nullptr for the interpreter
cudaError_t launch_vm(const vm::Params& p, int grid, int n_smem_slots, bool dense, cudaStream_t st, void* spec_kernel) {
  const void* fn = spec_kernel;
  if (!fn) {
    const VmKernels& k = vm_kernels();
    if (k.err != cudaSuccess) return k.err;
    fn = reinterpret_cast<const void*>(dense ? k.dense : k.wide);
  }
  const size_t smem = vm::vm_smem_bytes(p.n_code, n_smem_slots);
  if (smem > (size_t)(dense ? 113 : 227) * 1024) return cudaErrorInvalidConfiguration;
  void* args[] = {const_cast<vm::Params*>(&p)};
  return cudaLaunchKernel(fn, dim3(grid), dim3(kVmThreads), args, smem, st);
}

// Hands the PTX of a specialised kernel to the driver's assembler and fetches the kernel.  On failure the
// assembler's messages (or the runtime's error) are left in sg->spec_log and the interpreter keeps the program.
void load_specialized(VmSegment* sg) {
  static const char* kEntry = "dragon_vm_spec";
  sg->spec_state = -1;
  // test hook: behave as if the driver had no assembler, so that the fall-back to the interpreter can be exercised
  if (const char* off = std::getenv("DRAGON_VM_NO_ASSEMBLER")) {
    if (off[0] == '1') { sg->spec_log = "no assembler (DRAGON_VM_NO_ASSEMBLER=1)"; return; }
  }
  std::string ptx;
  if (specialize_ptx(*sg, kEntry, &ptx) != DRAGON_OK) { sg->spec_log = last_error(); return; }
  char log[4096] = "";
  cudaJitOption opt[] = {cudaJitErrorLogBuffer, cudaJitErrorLogBufferSizeBytes};
  void* val[] = {log, reinterpret_cast<void*>(sizeof(log))};
  cudaLibrary_t lib = nullptr;
  cudaKernel_t kernel = nullptr;
  cudaError_t e = cudaLibraryLoadData(&lib, ptx.c_str(), opt, val, 2, nullptr, nullptr, 0);
  if (e == cudaSuccess) e = cudaLibraryGetKernel(&kernel, lib, kEntry);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (sg->dense ? 113 : 227) * 1024);
  if (e != cudaSuccess) {
    sg->spec_log = std::string(cudaGetErrorString(e)) + (log[0] ? std::string(": ") + log : std::string());
    cudaGetLastError();
    if (lib) cudaLibraryUnload(lib);
    return;
  }
  sg->spec_lib = lib;
  sg->spec_kernel = kernel;
  sg->spec_state = 1;
}

void unload_specialized(VmSegment* sg) {
  if (sg->spec_lib) cudaLibraryUnload(reinterpret_cast<cudaLibrary_t>(sg->spec_lib));
  sg->spec_lib = sg->spec_kernel = nullptr;
  sg->spec_state = 0;
}

cudaError_t launch_finish(const VmSegment& sg, const std::vector<MemRef>& mems, void* const* mem_ptr, char* ws, cudaStream_t st, int chunks) {
  if (sg.finish.empty()) return cudaSuccess;
  if ((int)sg.finish.size() > vm::kMaxFinishJobs) return cudaErrorInvalidValue;   // the code generator never emits more
  vm::FinishParams fp;
  fp.n_jobs = (int)sg.finish.size();
  int max_cols = 1;
  for (int i = 0; i < fp.n_jobs; ++i) {
    const FinishJob& j = sg.finish[i];
    auto& o = fp.job[i];
    o.kind = j.kind;
    o.grid = sg.grid;
    o.cols = sg.cols;
    o.chunks = chunks;
    o.chunk_stride = sg.n_scalacc * sg.grid;
    o.dtype = mems[j.mem].dtype;
    o.out = mem_ptr[j.mem];
    if (j.kind == 0) { o.part = ws + sg.colpart_off + (size_t)j.acc * sg.grid * sg.cols * sizeof(float); max_cols = std::max(max_cols, sg.cols); }
    else o.part = ws + sg.scalpart_off + (size_t)j.acc * sg.grid * sizeof(double);
  }
  dim3 grid((max_cols + 31) / 32, fp.n_jobs);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(vm::kFinishThreads);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, vm::finish_kernel, fp);
}

// column sums of n_part partial rows (float [n_part][cols]) -> out[cols], fp64, fixed order
cudaError_t launch_colsum_finish(const float* part, int n_part, int cols, void* out, int dtype, cudaStream_t st) {
  vm::FinishParams fp;
  fp.n_jobs = 1;
  fp.job[0].kind = 0;
  fp.job[0].part = part;
  fp.job[0].out = out;
  fp.job[0].dtype = dtype;
  fp.job[0].cols = cols;
  fp.job[0].grid = n_part;
  fp.job[0].chunks = 1;
  fp.job[0].chunk_stride = 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((cols + 31) / 32, 1);
  cfg.blockDim = dim3(vm::kFinishThreads);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, vm::finish_kernel, fp);
}

}  // namespace dragon
