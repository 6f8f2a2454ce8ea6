// pc_parallel_attn_static: pc_parallel_attn for callers that cannot hand over a workspace
// because they are not allowed to allocate device memory at the point of the call
// (a serving loop that fixed its memory plan at start-up, a plug-in running inside
// somebody else's allocator, code between a framework's "no allocation" markers).
// The scratch of the attention (work counter, window cos/sin tables, rotated queries or per-split
// partial outputs) lives in one array that is part of the library image instead.
//
// The array's name is only a handle on the host: its device address is asked for once
// per device with cudaGetSymbolAddress and that address is what the kernels get.
#include "../../include/pc.h"

#include <cuda_runtime.h>

#include <mutex>

// Scratch shared by every call on a device.  Resident on each GPU that loads the library
// until the process exits.
static __device__ __align__(256) unsigned char pc_static_scratch[PC_STATIC_SCRATCH_BYTES];

namespace {

constexpr int MAX_DEVICES = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[MAX_DEVICES] = {};   // device address of pc_static_scratch, per device ordinal

// Device address of the scratch array on the current device (looked up on first use there).
cudaError_t scratch_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, pc_static_scratch);
    if (e != cudaSuccess) return e;
    if (p == nullptr) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" {

size_t pc_parallel_attn_static_scratch_bytes(void) { return static_cast<size_t>(PC_STATIC_SCRATCH_BYTES); }

int32_t pc_parallel_attn_static(int32_t B, int32_t w, int32_t Hq, int32_t Hkv, int32_t d, int32_t Nk,
                                const void* q_win, int32_t q_pos0, float rope_theta, float softmax_scale,
                                const void* k_cache, const void* v_cache, const void* k_win, const void* v_win,
                                void* out, float* lse_out, int32_t* status_word, void* stream) {
  // Size check first, on the host: the plan (number of key splits) depends on the shape
  // and on the SM count of the current device, exactly as in pc_parallel_attn.
  const size_t need = pc_parallel_attn_workspace_bytes(B, w, Hq, Hkv, d, Nk);
  if (need == 0) {
    // let the regular entry point name the argument error (nothing is launched for one)
    return pc_parallel_attn(B, w, Hq, Hkv, d, Nk, q_win, q_pos0, rope_theta, softmax_scale, k_cache, v_cache, k_win,
                            v_win, out, lse_out, status_word, nullptr, 0, stream);
  }
  if (need > static_cast<size_t>(PC_STATIC_SCRATCH_BYTES)) return PC_ERR_SCRATCH_LIMIT;
  void* scratch = nullptr;
  if (scratch_address(&scratch) != cudaSuccess) return PC_ERR_CUDA;
  // The work counter at the head of the scratch is cleared on the stream by the call
  // below; nothing else in the scratch is read before it is written.
  return pc_parallel_attn(B, w, Hq, Hkv, d, Nk, q_win, q_pos0, rope_theta, softmax_scale, k_cache, v_cache, k_win,
                          v_win, out, lse_out, status_word, scratch, static_cast<size_t>(PC_STATIC_SCRATCH_BYTES),
                          stream);
}

}  // extern "C"
