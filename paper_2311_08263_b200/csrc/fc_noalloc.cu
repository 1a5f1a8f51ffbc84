// Window attention for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside a host process whose device
// memory is owned and budgeted entirely by another component (an inference server's arena, a
// real-time loop that must never enter the allocator), or in code that runs after start-up when
// allocation would stall or fragment the pool.  fc_op_window_attention needs scratch for its
// per-split partial results; here that scratch is a fixed array compiled into the library, so the
// caller passes only inputs and outputs.
//
// The array below is a device symbol.  Inside host code its name is only a host-side handle, not a
// device address, so it must never be handed to a kernel directly: the real address is looked up once
// per device with cudaGetSymbolAddress and that pointer is what the kernels get.
#include <cstdio>
#include <mutex>

#include "fc_internal.h"

namespace {

// Every GPU that loads the library holds this much memory until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[FC_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void *g_scratch_addr[kMaxDevices] = {nullptr};
std::mutex g_scratch_mutex;

// Device address of the scratch array on the current device (looked up on first use per device).
int scratch_for_current_device(void **out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FC_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void *p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess || !p) {
      fprintf(stderr, "fc_op_window_attention_noalloc: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(e));
      return FC_ERR_CUDA;
    }
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return FC_OK;
}

}  // namespace

extern "C" int fc_op_window_attention_noalloc(const void *q, const void *kcache, const void *vcache,
                                              const int32_t *kv_len, float *out, int32_t batch, int32_t c,
                                              int32_t n_heads, int32_t n_kv_heads, int32_t head_dim,
                                              int32_t max_seq, int32_t max_len, int32_t dtype, void *cuda_stream) {
  const size_t need = fc::window_attention_scratch_bytes(batch, c, n_heads, n_kv_heads, head_dim, max_len, dtype);
  if (need == 0) return FC_ERR_ARG;
  if (need > (size_t)FC_NOALLOC_SCRATCH_BYTES) {
    fprintf(stderr,
            "fc_op_window_attention_noalloc: this problem needs %zu bytes of scratch but the built-in array holds "
            "%zu; use fc_op_window_attention with caller-provided scratch\n",
            need, (size_t)FC_NOALLOC_SCRATCH_BYTES);
    return FC_ERR_CAPACITY;
  }
  void *scratch = nullptr;
  int rc = scratch_for_current_device(&scratch);
  if (rc != FC_OK) return rc;
  // run_window_attention clears the arrival counters (the only part of the scratch that must start at
  // zero) on the stream before the kernel; whatever an earlier call left elsewhere is overwritten.
  return fc::run_window_attention(q, kcache, vcache, kv_len, out, batch, c, n_heads, n_kv_heads, head_dim, max_seq,
                                  max_len, dtype, scratch, need, (cudaStream_t)cuda_stream);
}
