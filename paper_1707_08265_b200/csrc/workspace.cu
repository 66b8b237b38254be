// The workspace of Sec. 3.1: it owns named tensors in device memory, any of them can be fed or fetched
// by name at any time, and functions run against it by name, so that state (the weights and moments of
// an updater, Sec. 3.2) stays on the device between runs.  Host code only: no kernel lives here.
#include <cuda_runtime.h>

#include <cstring>
#include <map>
#include <new>
#include <string>

#include "plan.h"

using dragon::set_error;

namespace {

struct Entry {
  int dtype = DRAGON_F32;
  dragon::Shape shape;
  size_t bytes = 0;
  void* ptr = nullptr;    // current contents
  void* spare = nullptr;  // second buffer of a tensor that a function overwrites but cannot update in place
};

size_t dtype_bytes(int dtype) { return dtype == DRAGON_BF16 ? 2 : 4; }

}  // namespace

struct dragon_workspace {
  std::map<std::string, Entry> tensors;
  std::map<const dragon_function_t*, std::pair<void*, size_t>> scratch;  // function -> its scratch area
  size_t bytes = 0;
};

namespace {

int device_alloc(dragon_workspace* w, size_t bytes, void** out, cudaStream_t st, bool zero) {
  void* p = nullptr;
  const size_t padded = (bytes + 255) / 256 * 256;
  if (cudaMalloc(&p, padded ? padded : 256) != cudaSuccess) {
    set_error("workspace: cannot allocate %zu bytes of device memory: %s", padded, cudaGetErrorString(cudaGetLastError()));
    return DRAGON_ERR_CUDA;
  }
  if (zero && cudaMemsetAsync(p, 0, padded ? padded : 256, st) != cudaSuccess) {
    set_error("workspace: cannot clear a new tensor: %s", cudaGetErrorString(cudaGetLastError()));
    cudaFree(p);
    return DRAGON_ERR_CUDA;
  }
  w->bytes += padded ? padded : 256;
  *out = p;
  return DRAGON_OK;
}

int find_or_create(dragon_workspace* w, const char* what, const std::string& name, int dtype, const dragon::Shape& shape,
                   cudaStream_t st, Entry** out) {
  auto it = w->tensors.find(name);
  if (it != w->tensors.end()) {
    if (it->second.dtype != dtype) { set_error("%s: tensor '%s' of the workspace has another type", what, name.c_str()); return DRAGON_ERR_DTYPE; }
    if (it->second.shape != shape) { set_error("%s: tensor '%s' of the workspace has another shape", what, name.c_str()); return DRAGON_ERR_SHAPE; }
    *out = &it->second;
    return DRAGON_OK;
  }
  Entry e;
  e.dtype = dtype;
  e.shape = shape;
  e.bytes = (size_t)shape.numel() * dtype_bytes(dtype);
  const int rc = device_alloc(w, e.bytes, &e.ptr, st, true);
  if (rc != DRAGON_OK) return rc;
  *out = &w->tensors.emplace(name, e).first->second;
  return DRAGON_OK;
}

}  // namespace

extern "C" {

dragon_workspace_t* dragon_workspace_create(void) { return new (std::nothrow) dragon_workspace(); }

void dragon_workspace_destroy(dragon_workspace_t* w) {
  if (!w) return;
  for (auto& kv : w->tensors) {
    if (kv.second.ptr) cudaFree(kv.second.ptr);
    if (kv.second.spare) cudaFree(kv.second.spare);
  }
  for (auto& kv : w->scratch)
    if (kv.second.first) cudaFree(kv.second.first);
  delete w;
}

size_t dragon_workspace_bytes(const dragon_workspace_t* w) { return w ? w->bytes : 0; }

int dragon_workspace_feed(dragon_workspace_t* w, const char* name, int dtype, int rank, const int64_t* shape, const void* src,
                          void* cuda_stream) {
  if (!w || !name || rank < 0 || rank > 2 || (rank > 0 && !shape)) { set_error("dragon_workspace_feed: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  if (dtype != DRAGON_F32 && dtype != DRAGON_BF16 && dtype != DRAGON_I32) { set_error("dragon_workspace_feed: unknown type %d", dtype); return DRAGON_ERR_DTYPE; }
  dragon::Shape s;
  s.rank = rank;
  for (int i = 0; i < rank; ++i) {
    if (shape[i] <= 0) { set_error("dragon_workspace_feed: extent %d of '%s' is not positive", i, name); return DRAGON_ERR_SHAPE; }
    s.d[i] = shape[i];
  }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  Entry* e = nullptr;
  const int rc = find_or_create(w, "dragon_workspace_feed", name, dtype, s, st, &e);
  if (rc != DRAGON_OK) return rc;
  if (src && cudaMemcpyAsync(e->ptr, src, e->bytes, cudaMemcpyDefault, st) != cudaSuccess) {
    set_error("dragon_workspace_feed: copy of '%s' failed: %s", name, cudaGetErrorString(cudaGetLastError()));
    return DRAGON_ERR_CUDA;
  }
  return DRAGON_OK;
}

int dragon_workspace_fetch(dragon_workspace_t* w, const char* name, void* dst, size_t bytes, void* cuda_stream) {
  if (!w || !name || !dst) { set_error("dragon_workspace_fetch: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  auto it = w->tensors.find(name);
  if (it == w->tensors.end()) { set_error("dragon_workspace_fetch: the workspace has no tensor '%s'", name); return DRAGON_ERR_MISSING_INPUT; }
  if (bytes != it->second.bytes) { set_error("dragon_workspace_fetch: '%s' holds %zu bytes, not %zu", name, it->second.bytes, bytes); return DRAGON_ERR_SHAPE; }
  if (cudaMemcpyAsync(dst, it->second.ptr, bytes, cudaMemcpyDefault, reinterpret_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
    set_error("dragon_workspace_fetch: copy of '%s' failed: %s", name, cudaGetErrorString(cudaGetLastError()));
    return DRAGON_ERR_CUDA;
  }
  return DRAGON_OK;
}

void* dragon_workspace_tensor(dragon_workspace_t* w, const char* name, int* dtype, int* rank, int64_t* shape) {
  if (!w || !name) { set_error("dragon_workspace_tensor: bad argument"); return nullptr; }
  auto it = w->tensors.find(name);
  if (it == w->tensors.end()) { set_error("dragon_workspace_tensor: the workspace has no tensor '%s'", name); return nullptr; }
  if (dtype) *dtype = it->second.dtype;
  if (rank) *rank = it->second.shape.rank;
  if (shape)
    for (int i = 0; i < it->second.shape.rank; ++i) shape[i] = it->second.shape.d[i];
  return it->second.ptr;
}

int dragon_workspace_run(dragon_workspace_t* w, dragon_function_t* f, const char* const* output_names, void* cuda_stream) {
  if (!w || !f) { set_error("dragon_workspace_run: bad argument"); return DRAGON_ERR_INVALID_ARG; }
  if (!f->not_executable.empty()) { set_error("dragon_workspace_run: %s", f->not_executable.c_str()); return DRAGON_ERR_UNSUPPORTED; }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  std::vector<const void*> feeds(f->n_in, nullptr);
  std::vector<void*> fetches(f->n_out, nullptr);
  std::vector<Entry*> in_entry(f->n_in, nullptr);
  for (int j = 0; j < f->n_in; ++j) {
    if (!f->prune.used_inputs[j]) continue;  // a pruned input need not exist (the redundant b of Sec. 2.2)
    const dragon::TensorInfo& t = f->in_info[j];
    auto it = w->tensors.find(t.name);
    if (it == w->tensors.end()) { set_error("dragon_workspace_run: input '%s' has not been fed", t.name.c_str()); return DRAGON_ERR_MISSING_INPUT; }
    if (it->second.dtype != t.dtype) { set_error("dragon_workspace_run: tensor '%s' of the workspace has another type than the function's input", t.name.c_str()); return DRAGON_ERR_DTYPE; }
    if (it->second.shape != t.shape) { set_error("dragon_workspace_run: tensor '%s' of the workspace has another shape than the function's input", t.name.c_str()); return DRAGON_ERR_SHAPE; }
    in_entry[j] = &it->second;
    feeds[j] = it->second.ptr;
  }
  std::vector<Entry*> out_entry(f->n_out, nullptr);
  std::vector<uint8_t> to_spare(f->n_out, 0);
  for (int j = 0; j < f->n_out; ++j) {
    const dragon::TensorInfo& t = f->out_info[j];
    const std::string name = output_names && output_names[j] ? output_names[j] : t.name;
    Entry* e = nullptr;
    const int rc = find_or_create(w, "dragon_workspace_run", name, t.dtype, t.shape, st, &e);
    if (rc != DRAGON_OK) return rc;
    for (int q = 0; q < j; ++q)
      if (out_entry[q] == e) { set_error("dragon_workspace_run: two outputs are bound to '%s'", name.c_str()); return DRAGON_ERR_INVALID_ARG; }
    out_entry[j] = e;
    fetches[j] = e->ptr;
    // the tensor is also read by this run: overwrite it in place where every thread only overwrites what it
    // has read (dragon_function_can_alias), otherwise write a second buffer and let the name point to it afterwards
    for (int i = 0; i < f->n_in; ++i) {
      if (in_entry[i] != e) continue;
      if (dragon_function_can_alias(f, i, j) == 1) break;
      if (!e->spare) {
        const int rc2 = device_alloc(w, e->bytes, &e->spare, st, false);
        if (rc2 != DRAGON_OK) return rc2;
      }
      fetches[j] = e->spare;
      to_spare[j] = 1;
      break;
    }
  }
  if (!f->workspace) {  // the function's scratch area lives in the workspace too
    auto& sc = w->scratch[f];
    const size_t need = dragon_function_workspace_bytes(f);
    if (sc.second < need) {
      if (sc.first) { cudaFree(sc.first); w->bytes -= sc.second; }
      sc = {nullptr, 0};
      const int rc = device_alloc(w, need, &sc.first, st, false);
      if (rc != DRAGON_OK) return rc;
      sc.second = need;
    }
    const int rc = dragon_function_set_workspace(f, sc.first, sc.second);
    if (rc != DRAGON_OK) return rc;
  }
  const int rc = dragon_run(f, feeds.data(), fetches.data(), cuda_stream);
  if (rc != DRAGON_OK) return rc;
  for (int j = 0; j < f->n_out; ++j)
    if (to_spare[j]) std::swap(out_entry[j]->ptr, out_entry[j]->spare);
  return DRAGON_OK;
}

}  // extern "C"
