// m2rnn_bwd for callers that cannot allocate device memory: the scratch the backward pass needs
// lives in a fixed array that is part of the library's device image.
#include <cuda_runtime.h>

#include <mutex>

#include "m2rnn.h"

namespace {

// Every GPU that loads the library holds this array until the process exits.  All calls share it.
static __device__ __align__(256) unsigned char g_static_scratch[M2RNN_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void *g_scratch_addr[kMaxDevices];  // device address of g_static_scratch, per device; null = not looked up yet
std::mutex g_scratch_mutex;

// In host code `g_static_scratch` only names the symbol; the device address has to be asked for,
// once per device, with that device current.
int scratch_address(void **out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return M2RNN_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
      (void)cudaGetLastError();
      return M2RNN_ERR_CUDA;
    }
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return M2RNN_OK;
}

}  // namespace

extern "C" int m2rnn_bwd_static_scratch(const m2rnn_params *params, const void *q, const void *k,
                                        const void *v, const float *gate, const void *W,
                                        const float *h0, const float *alpha, const float *beta,
                                        const void *w_r, const float *ckpt, const void *dy,
                                        const float *d_hT, void *dq, void *dk, void *dv,
                                        float *dgate, float *dW, float *dh0, int32_t *dev_status,
                                        void *stream) {
  if (!params) return M2RNN_ERR_NULL;
  // size check first: a problem that does not fit is refused before the device is touched
  const size_t need = m2rnn_bwd_workspace_bytes(params, ckpt != nullptr);
  if (need > (size_t)M2RNN_STATIC_SCRATCH_BYTES) return M2RNN_ERR_WORKSPACE;
  void *scratch = nullptr;
  const int rc = scratch_address(&scratch);
  if (rc != M2RNN_OK) return rc;
  // every word of the scratch that the backward kernels read is written earlier in the same call,
  // so what an earlier call left behind never needs clearing
  return m2rnn_bwd(params, q, k, v, gate, W, h0, alpha, beta, w_r, ckpt, dy, d_hT, dq, dk, dv, dgate,
                   dW, dh0, scratch, (size_t)M2RNN_STATIC_SCRATCH_BYTES, dev_status, stream);
}
