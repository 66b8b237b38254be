// Row kernels around the contraction: SoftmaxCrossEntropy forward / gradient (one CTA per
// row: warp-shuffle + shared-memory reductions), the mean of the per-row losses, and the bf16
// transpose that feeds K-major operands to the tensor-core GEMM.
#include <cuda_runtime.h>

#include "plan.h"
#include "vm_math.h"

namespace dragon {
namespace {

constexpr int kRowThreads = 256;

__device__ __forceinline__ float load_logit(const void* z, int dtype, size_t i) {
  return dtype == DRAGON_F32 ? __ldg(reinterpret_cast<const float*>(z) + i)
                             : __uint_as_float((unsigned)__ldg(reinterpret_cast<const unsigned short*>(z) + i) << 16);
}

template <bool kMax>
__device__ __forceinline__ float block_reduce(float v, float* sh) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float w = __shfl_xor_sync(0xffffffffu, v, o);
    v = kMax ? fmaxf(v, w) : v + w;
  }
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = sh[0];
#pragma unroll
  for (int i = 1; i < kRowThreads / 32; ++i) r = kMax ? fmaxf(r, sh[i]) : r + sh[i];
  __syncthreads();
  return r;
}

// eight consecutive logits at element index i (a multiple of 8) as floats
__device__ __forceinline__ void load8(const void* z, int dtype, size_t i, float* v) {
  if (dtype == DRAGON_F32) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(z) + i));
    const float4 b = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(z) + i) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  } else {
    const uint4 u = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned short*>(z) + i));
    v[0] = __uint_as_float(u.x << 16); v[1] = __uint_as_float(u.x & 0xffff0000u);
    v[2] = __uint_as_float(u.y << 16); v[3] = __uint_as_float(u.y & 0xffff0000u);
    v[4] = __uint_as_float(u.z << 16); v[5] = __uint_as_float(u.z & 0xffff0000u);
    v[6] = __uint_as_float(u.w << 16); v[7] = __uint_as_float(u.w & 0xffff0000u);
  }
}
__device__ __forceinline__ void store8(void* z, int dtype, size_t i, const float* v) {
  if (dtype == DRAGON_F32) {
    float4* p = reinterpret_cast<float4*>(reinterpret_cast<float*>(z) + i);
    p[0] = make_float4(v[0], v[1], v[2], v[3]);
    p[1] = make_float4(v[4], v[5], v[6], v[7]);
  } else {
    uint4 u;
    u.x = vmmath::bf16_bits(v[0]) | (vmmath::bf16_bits(v[1]) << 16);
    u.y = vmmath::bf16_bits(v[2]) | (vmmath::bf16_bits(v[3]) << 16);
    u.z = vmmath::bf16_bits(v[4]) | (vmmath::bf16_bits(v[5]) << 16);
    u.w = vmmath::bf16_bits(v[6]) | (vmmath::bf16_bits(v[7]) << 16);
    *reinterpret_cast<uint4*>(reinterpret_cast<unsigned short*>(z) + i) = u;
  }
}

// mode 0: rowloss[m] = logsumexp(z[m,:]) - z[m,label];  mode 1: dz[m,j] = dL/M * (softmax - onehot);
// mode 2: both in one pass over the logits.
// Rows whose length is a multiple of 8 are read and written 8 elements (16 or 32 bytes) per thread.
template <int kMode>
__global__ void __launch_bounds__(kRowThreads) sce_kernel(const void* z, int zdtype, const int* labels, int rows, int cols,
                                                          float* rowloss, void* dz, int dzdtype, const float* dl_ptr,
                                                          float dl_imm, int* status) {
  __shared__ float sh[kRowThreads / 32];
  const int m = blockIdx.x;
  const size_t off = (size_t)m * cols;
  const bool vec = (cols & 7) == 0;
  float mx = -INFINITY;
  if (vec) {
    for (int j = threadIdx.x * 8; j < cols; j += kRowThreads * 8) {
      float v[8];
      load8(z, zdtype, off + j, v);
#pragma unroll
      for (int e = 0; e < 8; ++e) mx = fmaxf(mx, v[e]);
    }
  } else {
    for (int j = threadIdx.x; j < cols; j += kRowThreads) mx = fmaxf(mx, load_logit(z, zdtype, off + j));
  }
  mx = block_reduce<true>(mx, sh);
  float se = 0.f;
  if (vec) {
    for (int j = threadIdx.x * 8; j < cols; j += kRowThreads * 8) {
      float v[8];
      load8(z, zdtype, off + j, v);
#pragma unroll
      for (int e = 0; e < 8; ++e) se += vmmath::exp_wide(v[e] - mx);
    }
  } else {
    for (int j = threadIdx.x; j < cols; j += kRowThreads) se += vmmath::exp_wide(load_logit(z, zdtype, off + j) - mx);
  }
  se = block_reduce<false>(se, sh);
  const int lab = __ldg(labels + m);
  const bool ok = lab >= 0 && lab < cols;
  if (!ok && threadIdx.x == 0) atomicExch(status, DRAGON_ERR_INVALID_ARG);
  if (kMode != 1) {
    if (threadIdx.x == 0) rowloss[m] = ok ? (logf(se) + mx - load_logit(z, zdtype, off + lab)) : 0.f;
  }
  if (kMode != 0) {
    const float dl = dl_ptr ? __ldg(dl_ptr) : dl_imm;
    const float sc = dl / (float)rows, inv = 1.f / se;
    if (vec) {
      for (int j = threadIdx.x * 8; j < cols; j += kRowThreads * 8) {
        float v[8];
        load8(z, zdtype, off + j, v);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          float g = vmmath::exp_wide(v[e] - mx) * inv;
          if (j + e == lab) g -= 1.f;
          v[e] = ok ? g * sc : 0.f;
        }
        store8(dz, dzdtype, off + j, v);
      }
    } else {
      for (int j = threadIdx.x; j < cols; j += kRowThreads) {
        float g = vmmath::exp_wide(load_logit(z, zdtype, off + j) - mx) * inv;
        if (ok && j == lab) g -= 1.f;
        g = ok ? g * sc : 0.f;
        if (dzdtype == DRAGON_F32) reinterpret_cast<float*>(dz)[off + j] = g;
        else reinterpret_cast<unsigned short*>(dz)[off + j] = (unsigned short)vmmath::bf16_bits(g);
      }
    }
  }
}

// The same for rows that fit the CTA's registers (cols <= kChunks * 2048, a multiple of 8): the row
// is read from memory once, the exponentials are computed once and kept.  Every thread owns the
// same elements and adds them in the same order as in sce_kernel, so the results are identical.
// colpart (may be null): the CTAs then walk the rows with the grid's stride, every thread keeps running sums of
// the gradient values of its own columns (as computed, before their rounding to dz's type) and writes them to
// colpart[blockIdx.x][.] at the end: partial column sums for the bias gradient behind the logits.
template <int kMode, int kChunks>
__global__ void __launch_bounds__(kRowThreads) sce_row_kernel(const void* z, int zdtype, const int* labels, int rows, int cols,
                                                              float* rowloss, void* dz, int dzdtype, const float* dl_ptr,
                                                              float dl_imm, int* status, float* colpart) {
  __shared__ float sh[kRowThreads / 32];
  float cs[kChunks][8];
#pragma unroll
  for (int c = 0; c < kChunks; ++c)
#pragma unroll
    for (int e = 0; e < 8; ++e) cs[c][e] = 0.f;
  for (int m = blockIdx.x; m < rows; m += gridDim.x) {
  const size_t off = (size_t)m * cols;
  float v[kChunks][8];
  float mx = -INFINITY;
#pragma unroll
  for (int c = 0; c < kChunks; ++c) {
    const int j = (c * kRowThreads + threadIdx.x) * 8;
    if (j < cols) {
      load8(z, zdtype, off + j, v[c]);
#pragma unroll
      for (int e = 0; e < 8; ++e) mx = fmaxf(mx, v[c][e]);
    }
  }
  mx = block_reduce<true>(mx, sh);
  float se = 0.f;
#pragma unroll
  for (int c = 0; c < kChunks; ++c) {
    const int j = (c * kRowThreads + threadIdx.x) * 8;
    if (j < cols) {
#pragma unroll
      for (int e = 0; e < 8; ++e) { v[c][e] = vmmath::exp_wide(v[c][e] - mx); se += v[c][e]; }
    }
  }
  se = block_reduce<false>(se, sh);
  const int lab = __ldg(labels + m);
  const bool ok = lab >= 0 && lab < cols;
  if (!ok && threadIdx.x == 0) atomicExch(status, DRAGON_ERR_INVALID_ARG);
  if (kMode != 1) {
    if (threadIdx.x == 0) rowloss[m] = ok ? (logf(se) + mx - load_logit(z, zdtype, off + lab)) : 0.f;
  }
  if (kMode != 0) {
    const float dl = dl_ptr ? __ldg(dl_ptr) : dl_imm;
    const float sc = dl / (float)rows, inv = 1.f / se;
#pragma unroll
    for (int c = 0; c < kChunks; ++c) {
      const int j = (c * kRowThreads + threadIdx.x) * 8;
      if (j < cols) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          float g = v[c][e] * inv;
          if (j + e == lab) g -= 1.f;
          v[c][e] = ok ? g * sc : 0.f;
          cs[c][e] += v[c][e];
        }
        store8(dz, dzdtype, off + j, v[c]);
      }
    }
  }
  }
  if (kMode != 0 && colpart != nullptr) {
#pragma unroll
    for (int c = 0; c < kChunks; ++c) {
      const int j = (c * kRowThreads + threadIdx.x) * 8;
      if (j < cols) {
        float4* p = reinterpret_cast<float4*>(colpart + (size_t)blockIdx.x * cols + j);
        p[0] = make_float4(cs[c][0], cs[c][1], cs[c][2], cs[c][3]);
        p[1] = make_float4(cs[c][4], cs[c][5], cs[c][6], cs[c][7]);
      }
    }
  }
}

__global__ void __launch_bounds__(kRowThreads) mean_kernel(const float* v, int n, float* out) {
  __shared__ double sh[kRowThreads];
  double s = 0.0;
  for (int i = threadIdx.x; i < n; i += kRowThreads) s += (double)v[i];
  sh[threadIdx.x] = s;
  __syncthreads();
  for (int o = kRowThreads / 2; o > 0; o >>= 1) {
    if (threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *out = (float)(sh[0] / (double)n);
}

// out[c, r] = in[r, c], 16-bit elements, 64x64 tiles through shared memory
__global__ void __launch_bounds__(256) transpose16_kernel(const unsigned short* __restrict__ in, unsigned short* __restrict__ out,
                                                           int rows, int cols) {
  __shared__ unsigned short tile[64][64 + 2];
  const int r0 = blockIdx.y * 64, c0 = blockIdx.x * 64;
  const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;
  for (int i = ty; i < 64; i += 4) {
    const int r = r0 + i, c = c0 + tx;
    tile[i][tx] = (r < rows && c < cols) ? in[(size_t)r * cols + c] : (unsigned short)0;
  }
  __syncthreads();
  for (int i = ty; i < 64; i += 4) {
    const int c = c0 + i, r = r0 + tx;
    if (c < cols && r < rows) out[(size_t)c * rows + r] = tile[tx][i];
  }
}

}  // namespace

// colpart / n_colpart (dz given, rows that fit the registers only): partial column sums of dz, n_colpart rows of cols floats
cudaError_t launch_sce_fwd(const void* z, int zdtype, const int* labels, int rows, int cols, float* rowloss, float* out,
                           int* status, cudaStream_t st, void* dz, int dzdtype, float dl_imm, float* colpart, int n_colpart) {
  const bool in_regs = (cols & 7) == 0 && cols <= 2 * kRowThreads * 8;
  if (colpart && !(dz && in_regs && n_colpart > 0 && n_colpart <= rows)) return cudaErrorInvalidValue;
  if (dz) {   // the gradient with respect to the logits in the same pass (dL is a constant)
    if (in_regs) sce_row_kernel<2, 2><<<colpart ? n_colpart : rows, kRowThreads, 0, st>>>(z, zdtype, labels, rows, cols, rowloss, dz, dzdtype, nullptr, dl_imm, status, colpart);
    else sce_kernel<2><<<rows, kRowThreads, 0, st>>>(z, zdtype, labels, rows, cols, rowloss, dz, dzdtype, nullptr, dl_imm, status);
  } else if (in_regs)
    sce_row_kernel<0, 2><<<rows, kRowThreads, 0, st>>>(z, zdtype, labels, rows, cols, rowloss, nullptr, 0, nullptr, 0.f, status, nullptr);
  else
    sce_kernel<0><<<rows, kRowThreads, 0, st>>>(z, zdtype, labels, rows, cols, rowloss, nullptr, 0, nullptr, 0.f, status);
  mean_kernel<<<1, kRowThreads, 0, st>>>(rowloss, rows, out);
  return cudaGetLastError();
}

cudaError_t launch_sce_bwd(const void* z, int zdtype, const int* labels, int rows, int cols, void* dz, int dzdtype,
                           const float* dl_ptr, float dl_imm, int* status, cudaStream_t st, float* colpart, int n_colpart) {
  const bool in_regs = (cols & 7) == 0 && cols <= 2 * kRowThreads * 8;
  if (colpart && !(in_regs && n_colpart > 0 && n_colpart <= rows)) return cudaErrorInvalidValue;
  if (in_regs)
    sce_row_kernel<1, 2><<<colpart ? n_colpart : rows, kRowThreads, 0, st>>>(z, zdtype, labels, rows, cols, nullptr, dz, dzdtype, dl_ptr, dl_imm, status, colpart);
  else
    sce_kernel<1><<<rows, kRowThreads, 0, st>>>(z, zdtype, labels, rows, cols, nullptr, dz, dzdtype, dl_ptr, dl_imm, status);
  return cudaGetLastError();
}

cudaError_t launch_transpose16(const void* in, void* out, int rows, int cols, cudaStream_t st) {
  dim3 grid((cols + 63) / 64, (rows + 63) / 64);
  transpose16_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const unsigned short*>(in), reinterpret_cast<unsigned short*>(out), rows, cols);
  return cudaGetLastError();
}

// ---- allocation-free loss ------------------------------------------------------------------------

// Scratch of dragon_softmax_ce_loss_static(): one partial loss per row plus a status word.  It is
// part of the library image, so every GPU that loads the library holds these 257 KiB until exit.
constexpr int kStaticMaxRows = 65536;
static __device__ __align__(256) float g_static_rowloss[kStaticMaxRows + 64];

namespace {
// device address of the scratch array, looked up once per device (index = CUDA device ordinal)
float* static_scratch_for_current_device(int* err) {
  // Filled without a lock: two threads that race here look up the same symbol on the same device and
  // store the same address, so whichever write lands last changes nothing.  The address belongs to
  // the device's primary context; it is not looked up again after a cudaDeviceReset().
  static float* cache[64] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { *err = DRAGON_ERR_CUDA; return nullptr; }
  if (!cache[dev]) {
    // in host code the array's name is only a handle; the kernels need the address on this device
    float* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_rowloss);
    if (e != cudaSuccess || !ptr) {
      set_error("dragon_softmax_ce_loss_static: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
      *err = DRAGON_ERR_CUDA;
      return nullptr;
    }
    cache[dev] = ptr;
  }
  return cache[dev];
}
}  // namespace

}  // namespace dragon

extern "C" int dragon_softmax_ce_loss_static(const void* logits, int dtype, const int32_t* labels, int rows, int cols,
                                             float* loss_out, void* cuda_stream) {
  using namespace dragon;
  if (!logits || !labels || !loss_out || rows <= 0 || cols <= 0 || (dtype != DRAGON_F32 && dtype != DRAGON_BF16)) {
    set_error("dragon_softmax_ce_loss_static: bad argument");
    return DRAGON_ERR_INVALID_ARG;
  }
  // the row kernels read the logits with 16-byte vector loads: a misaligned pointer must be an error code, not a fault
  if (((uintptr_t)logits & 15) || ((uintptr_t)labels & 3) || ((uintptr_t)loss_out & 3)) {
    set_error("dragon_softmax_ce_loss_static: logits must be 16-byte aligned, labels and loss_out 4-byte aligned");
    return DRAGON_ERR_INVALID_ARG;
  }
  if (rows > kStaticMaxRows) {
    set_error("dragon_softmax_ce_loss_static: %d rows exceed the built-in scratch (at most %d rows)", rows, kStaticMaxRows);
    return DRAGON_ERR_WORKSPACE;
  }
  int err = DRAGON_OK;
  float* scratch = static_scratch_for_current_device(&err);
  if (!scratch) return err;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  int* status = reinterpret_cast<int*>(scratch + kStaticMaxRows);
  // the status word must start at zero; the per-row losses are overwritten in full by every call
  cudaError_t e = cudaMemsetAsync(status, 0, sizeof(int), st);
  if (e == cudaSuccess) e = launch_sce_fwd(logits, dtype, labels, rows, cols, scratch, loss_out, status, st, nullptr, 0, 0.f, nullptr, 0);
  if (e != cudaSuccess) {
    set_error("dragon_softmax_ce_loss_static: CUDA error: %s", cudaGetErrorString(e));
    return DRAGON_ERR_CUDA;
  }
  return DRAGON_OK;
}
