// Library-wide pieces of the C ABI: status strings, launch accounting, device queries and the
// whole-step entry point that moves a step's inputs and results across PCIe around the two
// kernels (Alg. 1, blocks "Sparse Attention Mask Creation" and "Verification with Sparse
// Attention").
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>
#include <new>

#include "specattn.h"
#include "nvtx_range.h"

namespace specattn {

std::atomic<long long> g_launch_count{0};

// Number of SMs of the current device (cached per device ordinal); <= 0 on failure.
int device_sm_count() {
  static std::mutex mu;
  static int cache[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  if (dev < 0 || dev >= 64) return -1;
  std::lock_guard<std::mutex> lock(mu);
  if (cache[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
      cudaGetLastError();
      return -1;
    }
    cache[dev] = n;
  }
  return cache[dev];
}

}  // namespace specattn

extern "C" const char* specattn_status_string(int code) {
  switch (code) {
    case SPECATTN_OK: return "ok";
    case SPECATTN_ERR_NULL: return "a required pointer is NULL";
    case SPECATTN_ERR_STRUCT_SIZE: return "struct_size does not match this library";
    case SPECATTN_ERR_RANGE: return "a scalar argument is out of range";
    case SPECATTN_ERR_ALIGN: return "a pointer or stride breaks the 16-byte alignment rules";
    case SPECATTN_ERR_WORKSPACE: return "workspace missing or too small";
    case SPECATTN_ERR_UNSUPPORTED: return "shape outside what the kernels support";
    case SPECATTN_ERR_CUDA: return "the CUDA runtime reported an error";
    case SPECATTN_ERR_STATIC_SCRATCH:
      return "the shape needs more scratch than the library's built-in static buffer holds";
    default: return "unknown status code";
  }
}

extern "C" int64_t specattn_kernel_launch_count(void) {
  return static_cast<int64_t>(specattn::g_launch_count.load(std::memory_order_relaxed));
}

namespace specattn {
namespace {

// Copy streams and events of the whole-step call, created on first use per device and kept
// until the process exits.  One call at a time per device enqueues through them (the mutex is
// held while enqueueing, which never blocks on the GPU).
struct HostPipe {
  cudaStream_t h2d = nullptr, d2h = nullptr;
  cudaEvent_t start = nullptr, q_in = nullptr, done = nullptr;
  cudaEvent_t layer_in[SPECATTN_MAX_DRAFT_LAYERS] = {nullptr};
  cudaEvent_t* layer_out = nullptr;  // one per target layer
  int n_layer_out = 0;
  std::mutex mu;
};
HostPipe g_pipe[64];

bool make_event(cudaEvent_t* e) {
  if (*e != nullptr) return true;
  if (cudaEventCreateWithFlags(e, cudaEventDisableTiming) != cudaSuccess) {
    cudaGetLastError();
    *e = nullptr;
    return false;
  }
  return true;
}

// Called with pipe.mu held.
bool prepare_pipe(HostPipe& pipe, int n_target_layers) {
  if (pipe.h2d == nullptr && cudaStreamCreateWithFlags(&pipe.h2d, cudaStreamNonBlocking) != cudaSuccess) {
    cudaGetLastError();
    pipe.h2d = nullptr;
    return false;
  }
  if (pipe.d2h == nullptr && cudaStreamCreateWithFlags(&pipe.d2h, cudaStreamNonBlocking) != cudaSuccess) {
    cudaGetLastError();
    pipe.d2h = nullptr;
    return false;
  }
  if (!make_event(&pipe.start) || !make_event(&pipe.q_in) || !make_event(&pipe.done)) return false;
  for (int u = 0; u < SPECATTN_MAX_DRAFT_LAYERS; ++u)
    if (!make_event(&pipe.layer_in[u])) return false;
  if (pipe.n_layer_out < n_target_layers) {
    cudaEvent_t* grown = new (std::nothrow) cudaEvent_t[n_target_layers];
    if (grown == nullptr) return false;
    for (int j = 0; j < n_target_layers; ++j) grown[j] = (j < pipe.n_layer_out) ? pipe.layer_out[j] : nullptr;
    delete[] pipe.layer_out;
    pipe.layer_out = grown;
    const int old = pipe.n_layer_out;
    pipe.n_layer_out = n_target_layers;
    for (int j = old; j < n_target_layers; ++j)
      if (!make_event(&pipe.layer_out[j])) return false;
  }
  return true;
}

}  // namespace
}  // namespace specattn

// The step as a three-lane pipeline.  Lane "in" (a copy stream) uploads all query blocks, then
// the draft rows one mapped draft layer at a time; the caller's stream runs the selection of a
// draft layer as soon as its rows have landed and then the verify launches of the target layers
// mapped to it, while the next draft layer is still crossing PCIe; lane "out" (a second copy
// stream) downloads a layer's results while later layers compute and later inputs upload.  The
// call returns with everything enqueued; the caller's stream has been made to wait for the last
// download, so stream order is what it would be had everything run on that stream.
extern "C" int specattn_verify_step_host(const specattn_step_host_args* args, void* cuda_stream) {
  specattn::NvtxRange nvtx_range("specattn_verify_step_host");
  if (args == nullptr) return SPECATTN_ERR_NULL;
  if (args->struct_size != sizeof(specattn_step_host_args)) return SPECATTN_ERR_STRUCT_SIZE;
  const specattn_step_host_args& S = *args;
  if (!S.select || !S.draft_probs_host || S.n_target_layers < 0) return SPECATTN_ERR_NULL;
  if (S.n_target_layers > 0 && (!S.verify || !S.q_host || !S.out_host || !S.lse_host)) return SPECATTN_ERR_NULL;
  const specattn_select_args& sel = *S.select;
  if (sel.struct_size != sizeof(specattn_select_args)) return SPECATTN_ERR_STRUCT_SIZE;
  if (!sel.draft_probs || !sel.layer_map) return SPECATTN_ERR_NULL;
  if (sel.n_draft_layers < 1 || sel.n_draft_layers > SPECATTN_MAX_DRAFT_LAYERS) return SPECATTN_ERR_RANGE;
  if (sel.n_target_layers != S.n_target_layers) return SPECATTN_ERR_RANGE;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

  bool used[SPECATTN_MAX_DRAFT_LAYERS] = {false};
  for (int j = 0; j < sel.n_target_layers; ++j) {
    const int u = sel.layer_map[j];
    if (u < -1 || u >= sel.n_draft_layers) return SPECATTN_ERR_RANGE;
    if (u >= 0) used[u] = true;
  }
  for (int u = 0; u < sel.n_draft_layers; ++u)
    if (used[u] && (!S.draft_probs_host[u] || !sel.draft_probs[u])) return SPECATTN_ERR_NULL;
  for (int j = 0; j < S.n_target_layers; ++j) {
    const specattn_verify_args& v = S.verify[j];
    if (v.struct_size != sizeof(specattn_verify_args)) return SPECATTN_ERR_STRUCT_SIZE;
    if (!S.q_host[j] || !S.out_host[j] || !S.lse_host[j] || !v.q || !v.out || !v.lse) return SPECATTN_ERR_NULL;
  }

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return SPECATTN_ERR_CUDA;
  }
  specattn::HostPipe& pipe = specattn::g_pipe[dev];
  std::lock_guard<std::mutex> lock(pipe.mu);
  if (!specattn::prepare_pipe(pipe, S.n_target_layers)) return SPECATTN_ERR_CUDA;
  auto ok = [](cudaError_t e) {
    if (e == cudaSuccess) return true;
    cudaGetLastError();
    return false;
  };

  // the copy lanes start after whatever the caller's stream already holds
  if (!ok(cudaEventRecord(pipe.start, stream)) || !ok(cudaStreamWaitEvent(pipe.h2d, pipe.start, 0)) ||
      !ok(cudaStreamWaitEvent(pipe.d2h, pipe.start, 0)))
    return SPECATTN_ERR_CUDA;

  // lane "in": query blocks first (small), then the draft rows in the order the layers need them
  for (int j = 0; j < S.n_target_layers; ++j) {
    const specattn_verify_args& v = S.verify[j];
    const size_t rows = static_cast<size_t>(v.batch) * v.n_q * v.n_q_heads;
    if (!ok(cudaMemcpyAsync(const_cast<void*>(v.q), S.q_host[j], rows * v.head_dim * 2, cudaMemcpyHostToDevice,
                            pipe.h2d)))
      return SPECATTN_ERR_CUDA;
  }
  if (!ok(cudaEventRecord(pipe.q_in, pipe.h2d))) return SPECATTN_ERR_CUDA;
  const size_t layer_bytes = static_cast<size_t>(sel.batch) * sel.n_draft_heads * sel.gamma *
                             static_cast<size_t>(sel.L_stride) * sizeof(float);
  bool uploaded[SPECATTN_MAX_DRAFT_LAYERS] = {false};
  auto upload = [&](int u) {
    if (uploaded[u]) return true;
    uploaded[u] = true;
    return ok(cudaMemcpyAsync(const_cast<float*>(sel.draft_probs[u]), S.draft_probs_host[u], layer_bytes,
                              cudaMemcpyHostToDevice, pipe.h2d)) &&
           ok(cudaEventRecord(pipe.layer_in[u], pipe.h2d));
  };
  for (int j = 0; j < S.n_target_layers; ++j)
    if (sel.layer_map[j] >= 0 && !upload(sel.layer_map[j])) return SPECATTN_ERR_CUDA;

  // the caller's stream: selection per draft layer when first needed, then the verify launches
  if (!ok(cudaStreamWaitEvent(stream, pipe.q_in, 0))) return SPECATTN_ERR_CUDA;
  bool selected[SPECATTN_MAX_DRAFT_LAYERS] = {false};
  const void* planned[SPECATTN_MAX_DRAFT_LAYERS + 1];
  int n_planned = 0;
  // A verify launch may skip its wait for the preceding kernel (SPECATTN_VERIFY_LISTS_STABLE)
  // only when that kernel is another verify launch: the first one after a selection or a plan
  // launch enqueued here reads what those kernels wrote, so the flag is dropped for it.
  bool fresh = true;
  for (int j = 0; j < S.n_target_layers; ++j) {
    const int u = sel.layer_map[j];
    if (u >= 0 && !selected[u]) {
      selected[u] = true;
      fresh = true;
      if (!ok(cudaStreamWaitEvent(stream, pipe.layer_in[u], 0))) return SPECATTN_ERR_CUDA;
      specattn_select_args one = sel;  // the lists of draft layer u only
      const int32_t only = u;
      one.n_target_layers = 1;
      one.layer_map = &only;
      const int rc = specattn_select_topp(&one, cuda_stream);
      if (rc != SPECATTN_OK) return rc;
    }
    const specattn_verify_args& v = S.verify[j];
    // a work partition that several layers share is computed before its first user
    if (v.plan != nullptr) {
      bool done = false;
      for (int k = 0; k < n_planned && !done; ++k) done = planned[k] == v.plan;
      if (!done) {
        const int prc = specattn_verify_plan(&v, const_cast<void*>(v.plan), specattn_verify_plan_bytes(&v), cuda_stream);
        if (prc != SPECATTN_OK) return prc;
        if (n_planned < SPECATTN_MAX_DRAFT_LAYERS + 1) planned[n_planned++] = v.plan;
        fresh = true;
      }
    }
    specattn_verify_args call = v;
    if (fresh) call.flags &= ~SPECATTN_VERIFY_LISTS_STABLE;
    fresh = false;
    const int rc = specattn_sparse_verify(&call, cuda_stream);
    if (rc != SPECATTN_OK) return rc;
    // lane "out"
    const size_t rows = static_cast<size_t>(v.batch) * v.n_q * v.n_q_heads;
    if (!ok(cudaEventRecord(pipe.layer_out[j], stream)) || !ok(cudaStreamWaitEvent(pipe.d2h, pipe.layer_out[j], 0)) ||
        !ok(cudaMemcpyAsync(S.out_host[j], v.out, rows * v.head_dim * sizeof(float), cudaMemcpyDeviceToHost,
                            pipe.d2h)) ||
        !ok(cudaMemcpyAsync(S.lse_host[j], v.lse, rows * sizeof(float), cudaMemcpyDeviceToHost, pipe.d2h)))
      return SPECATTN_ERR_CUDA;
  }
  // join: later work on the caller's stream sees the inputs consumed and the results delivered
  if (!ok(cudaEventRecord(pipe.done, pipe.d2h)) || !ok(cudaStreamWaitEvent(stream, pipe.done, 0)))
    return SPECATTN_ERR_CUDA;
  if (!ok(cudaEventRecord(pipe.done, pipe.h2d)) || !ok(cudaStreamWaitEvent(stream, pipe.done, 0)))
    return SPECATTN_ERR_CUDA;
  return SPECATTN_OK;
}
