// delta_attn_decode_step_noalloc -- the decode step for callers that cannot give the library
// any workspace and cannot allocate one themselves.
//
// The regular decode step keeps its split-KV partial results and arrival tickets in the
// caller's workspace.  Some callers have no way to provide that: code that runs inside an
// application whose memory manager has already claimed the whole device (a cudaMalloc there
// fails, or is forbidden by the host application's rules), latency-critical loops that must
// not hit the implicit device-wide synchronisation of cudaMalloc/cudaFree, and plug-ins that
// only ever see the raw input and output pointers.  For them the scratch lives in a
// fixed-size array that is part of the library image itself.
//
// The array below is reserved on every GPU that loads this library, from load until the
// process exits.  All calls on a device share it, and it keeps whatever the previous call left
// there: the part that must start at zero (arrival tickets, counters) is cleared on the stream
// at the start of every call.  Two calls whose kernels can overlap on the same GPU (different
// streams, or different host threads) would race on it; callers must serialise them.
#include <mutex>

#include "delta_internal.cuh"

namespace delta {
namespace {

constexpr size_t kTicketBytes = 4096;                 // 1024 (batch x KV head) tickets
constexpr size_t kCounterBytes = 4096;                // counter slots (only CNT_SLOTS * 8 used)
constexpr size_t kPartialBytes = 8u << 20;            // split-KV partial outputs
constexpr size_t kScratchBytes = kTicketBytes + kCounterBytes + kPartialBytes;
constexpr int kMaxDevices = 64;

// Host code must never hand this name to a kernel: on the host it is only a stand-in for the
// symbol.  The device address is looked up once per device (below) and passed as a pointer.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device; resolved on first use.
cudaError_t scratch_on_current_device(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress((void**)&p, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = p;
  }
  *out = static_cast<unsigned char*>(g_scratch_addr[dev]);
  return cudaSuccess;
}

}  // namespace
}  // namespace delta

using namespace delta;

extern "C" delta_status_t delta_attn_decode_step_noalloc(
    const void* q_new, const void* k_new, const void* v_new, void* k_cache, void* v_cache, void* out,
    const float* qhat_in, float* qhat_out, float* R, int32_t n, int32_t B, int32_t H, int32_t H_kv,
    int32_t d, int32_t T_max, delta_dtype_t dtype, float theta, int32_t window, void* stream) {
  if (!q_new || !k_new || !v_new || !k_cache || !v_cache || !out || !qhat_in || !qhat_out || !R)
    return DELTA_ERR_INVALID_ARG;
  if (qhat_in == qhat_out) return DELTA_ERR_INVALID_ARG;   // other CTAs still read the old reference
  // cache tiles are staged with bulk copies and rows are read as 16-byte vectors
  if ((((uintptr_t)q_new | (uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)k_cache | (uintptr_t)v_cache |
        (uintptr_t)out | (uintptr_t)qhat_in | (uintptr_t)qhat_out | (uintptr_t)R) & 15u) != 0)
    return DELTA_ERR_INVALID_ARG;
  if (B < 1 || H < 1 || H_kv < 1 || T_max < 1 || H % H_kv != 0) return DELTA_ERR_INVALID_ARG;
  if (dtype != DELTA_F32 && dtype != DELTA_BF16) return DELTA_ERR_INVALID_ARG;
  if (!(theta >= 0.0f) || !(theta <= 3.0e38f) || window < 0) return DELTA_ERR_INVALID_ARG;
  if (d != 64 && d != 128) return DELTA_ERR_UNSUPPORTED;
  const int g = H / H_kv;
  if (g != 1 && g != 2 && g != 4 && g != 8) return DELTA_ERR_UNSUPPORTED;
  if (T_max > kMaxDecodeSplits * kDecodeChunkMax) return DELTA_ERR_UNSUPPORTED;
  if (n < 1) return DELTA_ERR_STATE;
  if (n >= T_max) return DELTA_ERR_CAPACITY;
  // the built-in scratch has a fixed size: refuse anything that would not fit
  const size_t bkv = (size_t)B * H_kv;
  const size_t partial_need = bkv * kMaxDecodeSplits * g * (size_t)(d + 2) * sizeof(float);
  if (bkv * sizeof(uint32_t) > kTicketBytes || partial_need > kPartialBytes)
    return DELTA_ERR_SCRATCH_LIMIT;

  unsigned char* base = nullptr;
  cudaError_t e = scratch_on_current_device(&base);
  if (e != cudaSuccess) return cuda_fail(e);
  cudaStream_t cs = (cudaStream_t)stream;
  // tickets and the counters in front of the status word must start at zero; the partial
  // results are fully rewritten.  The status word (counter slot CNT_STATUS) is left alone: a
  // time-out recorded by an earlier step stays there until delta_noalloc_device_status reads it.
  if ((e = cudaMemsetAsync(base, 0, kTicketBytes + CNT_STATUS * sizeof(unsigned long long), cs)) != cudaSuccess)
    return cuda_fail(e);

  Workspace w{};
  w.qhat[0] = const_cast<float*>(qhat_in);
  w.qhat[1] = qhat_out;
  w.R = R;
  w.dec_ticket = reinterpret_cast<uint32_t*>(base);
  w.counters = reinterpret_cast<unsigned long long*>(base + kTicketBytes);
  w.dec_partial = reinterpret_cast<float*>(base + kTicketBytes + kCounterBytes);
  const Shape s{B, H, H_kv, d, T_max, (T_max + DELTA_TILE_ROWS - 1) / DELTA_TILE_ROWS};
  e = launch_decode_step(s, w, q_new, k_new, v_new, k_cache, v_cache, out, n, theta, window,
                         (int)dtype, /*qhat_sel=*/0, cs);
  return e == cudaSuccess ? DELTA_OK : cuda_fail(e);
}

extern "C" delta_status_t delta_noalloc_device_status(uint32_t* host_status, void* stream) {
  if (!host_status) return DELTA_ERR_INVALID_ARG;
  unsigned char* base = nullptr;
  cudaError_t e = scratch_on_current_device(&base);
  if (e != cudaSuccess) return cuda_fail(e);
  cudaStream_t cs = (cudaStream_t)stream;
  unsigned long long* word = reinterpret_cast<unsigned long long*>(base + kTicketBytes) + CNT_STATUS;
  unsigned long long v = 0;
  if ((e = cudaMemcpyAsync(&v, word, sizeof(v), cudaMemcpyDeviceToHost, cs)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemsetAsync(word, 0, sizeof(v), cs)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaStreamSynchronize(cs)) != cudaSuccess) return cuda_fail(e);
  *host_status = (uint32_t)v;
  return v == 0 ? DELTA_OK : (delta_status_t)(uint32_t)v;
}
