// Library-wide pieces of the C ABI: status strings, launch accounting, device queries and the
// whole-step entry point that moves a step's inputs and results across PCIe around the two
// kernels (Alg. 1, blocks "Sparse Attention Mask Creation" and "Verification with Sparse
// Attention").
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>

#include "specattn.h"

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

extern "C" int specattn_verify_step_host(const specattn_step_host_args* args, void* cuda_stream) {
  if (args == nullptr) return SPECATTN_ERR_NULL;
  if (args->struct_size != sizeof(specattn_step_host_args)) return SPECATTN_ERR_STRUCT_SIZE;
  const specattn_step_host_args& S = *args;
  if (!S.select || !S.draft_probs_host || S.n_target_layers < 0) return SPECATTN_ERR_NULL;
  if (S.n_target_layers > 0 && (!S.verify || !S.q_host || !S.out_host || !S.lse_host)) return SPECATTN_ERR_NULL;
  const specattn_select_args& sel = *S.select;
  if (sel.struct_size != sizeof(specattn_select_args)) return SPECATTN_ERR_STRUCT_SIZE;
  if (!sel.draft_probs || !sel.layer_map) return SPECATTN_ERR_NULL;
  if (sel.n_draft_layers < 1 || sel.n_draft_layers > SPECATTN_MAX_DRAFT_LAYERS) return SPECATTN_ERR_RANGE;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

  bool used[SPECATTN_MAX_DRAFT_LAYERS] = {false};
  for (int j = 0; j < sel.n_target_layers; ++j) {
    const int u = sel.layer_map[j];
    if (u < -1 || u >= sel.n_draft_layers) return SPECATTN_ERR_RANGE;
    if (u >= 0) used[u] = true;
  }
  const size_t layer_bytes = static_cast<size_t>(sel.batch) * sel.n_draft_heads * sel.gamma *
                             static_cast<size_t>(sel.L_stride) * sizeof(float);
  for (int u = 0; u < sel.n_draft_layers; ++u) {
    if (!used[u]) continue;
    if (!S.draft_probs_host[u] || !sel.draft_probs[u]) return SPECATTN_ERR_NULL;
    if (cudaMemcpyAsync(const_cast<float*>(sel.draft_probs[u]), S.draft_probs_host[u], layer_bytes,
                        cudaMemcpyHostToDevice, stream) != cudaSuccess) {
      cudaGetLastError();
      return SPECATTN_ERR_CUDA;
    }
  }
  int rc = specattn_select_topp(&sel, cuda_stream);
  if (rc != SPECATTN_OK) return rc;
  for (int j = 0; j < S.n_target_layers; ++j) {
    const specattn_verify_args& v = S.verify[j];
    if (v.struct_size != sizeof(specattn_verify_args)) return SPECATTN_ERR_STRUCT_SIZE;
    if (!S.q_host[j] || !S.out_host[j] || !S.lse_host[j] || !v.q || !v.out || !v.lse) return SPECATTN_ERR_NULL;
    const size_t rows = static_cast<size_t>(v.batch) * v.n_q * v.n_q_heads;
    if (cudaMemcpyAsync(const_cast<void*>(v.q), S.q_host[j], rows * v.head_dim * 2, cudaMemcpyHostToDevice,
                        stream) != cudaSuccess) {
      cudaGetLastError();
      return SPECATTN_ERR_CUDA;
    }
    rc = specattn_sparse_verify(&v, cuda_stream);
    if (rc != SPECATTN_OK) return rc;
    if (cudaMemcpyAsync(S.out_host[j], v.out, rows * v.head_dim * sizeof(float), cudaMemcpyDeviceToHost,
                        stream) != cudaSuccess ||
        cudaMemcpyAsync(S.lse_host[j], v.lse, rows * sizeof(float), cudaMemcpyDeviceToHost, stream) !=
            cudaSuccess) {
      cudaGetLastError();
      return SPECATTN_ERR_CUDA;
    }
  }
  return SPECATTN_OK;
}
