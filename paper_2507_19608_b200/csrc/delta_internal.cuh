// Internal declarations shared by the translation units of the delta-attention library.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "../../include/delta_attn.h"

namespace delta {

// Device counters (uint64) in the workspace.
enum CounterSlot {
  CNT_PREFILL_NNZ = 0, CNT_PREFILL_ELEMS, CNT_PREFILL_MACS_DONE, CNT_PREFILL_MACS_DENSE,
  CNT_DECODE_NNZ, CNT_DECODE_ELEMS, CNT_DECODE_MACS_DONE, CNT_DECODE_MACS_DENSE,
  CNT_STATUS,  // low 32 bits: device status word (0 = ok)
  CNT_SLOTS = 16,
  // the prefill counters are kept in CNT_SHARDS shards of 4 (nnz, elements, done, dense) behind
  // the plain slots, so that thousands of CTAs do not queue on four addresses; the host adds them
  CNT_SHARDS = 32,
  CNT_SHARD_BASE = CNT_SLOTS,
  CNT_TOTAL = CNT_SLOTS + 4 * CNT_SHARDS
};

constexpr int DELTA_CKPT_ROWS = 8;     // the chain kernel leaves its reference every 8 rows
constexpr int kMaxDecodeSplits = 64;   // split-KV partials per (batch, KV head)
constexpr int kDecodeChunkMax = 1024;  // keys per decode CTA (scores live in shared memory)

// Device pointers carved from the caller's workspace.
struct Workspace {
  float* dq;            // [B,H,T_max,d]
  uint32_t* mask;       // [B,H,T_max,d/32]
  uint16_t* row_nnz;    // [B,H,T_max]
  uint32_t* tile_nnz;   // [B,H,n_tiles]
  uint8_t* idx;         // [B,H,T_max,d]
  float* qhat_tile;     // [B,H,n_tiles,d]
  float* ckpt;          // [B,H,ceil(T_max/8),d] reference in front of every 8-row block (query deltas)
  float* qhat[2];       // [B,H,d] ping-pong (decode reads one, writes the other)
  float* R;             // [B,H,T_max]
  unsigned long long* counters;  // [CNT_TOTAL]
  float* dec_partial;   // [B,H_kv,kMaxDecodeSplits,g,(d+2)]
  uint32_t* dec_ticket; // [B,H_kv]
  float* kt;            // [B,H_kv,d,round_up(T_max,4)] channel-major fp32 keys (tensor-core prefill only)
  __nv_bfloat16* qhat_rows;  // [B,H,T_max,d] reference state after every row (telescoped prefill only)
  // compressed key-delta cache (key deltas, bf16): values, segment offsets, segment bases, pool
  // fill per KV head, and its own 32-row-aligned copies of the mask words and fired counts
  uint16_t* kp_vals;    // [B,H_kv,capacity]
  uint32_t* kp_segoff;  // [B,H_kv,segments+1]
  uint16_t* kp_base;    // [B,H_kv,segments,d]
  uint32_t* kp_used;    // [B,H_kv]
  uint32_t* kp_mask;    // [B,H_kv,segments*32,d/32]
  uint16_t* kp_nnz;     // [B,H_kv,segments*32]
  size_t zero_bytes;    // leading span of the workspace that a reset clears (q_hat, counters, tickets)
  size_t total_bytes;
};

struct Shape {
  int B, H, H_kv, d, T_max, n_tiles;
  int g() const { return H / H_kv; }
  int n_ckpt() const { return (T_max + DELTA_CKPT_ROWS - 1) / DELTA_CKPT_ROWS; }
};

void count_launch(int n = 1);
// Records the text of a failed CUDA runtime call for delta_last_cuda_error; returns DELTA_ERR_CUDA.
delta_status_t cuda_fail(cudaError_t e);

// K1a: token-sequential delta chain (Eq. 2-3): the reference in front of every 8-row block and
// every 64-row tile, and the final reference.
// key_stream: the stream is K in the KV-cache layout, one chain set per KV head (strategy 3).
// reverse: rows are taken from T-1 down to 0 (strategy 2; query stream only).
// zero_ptr, zero_bytes: a span (16-byte aligned, a multiple of 16 bytes) that the kernel's first
// CTA clears before anything else: the deferred clearing of a state reset (none if null).
cudaError_t launch_delta_chain(const Shape& s, const Workspace& w, const void* q, int T, float theta, int dtype,
                               int init, bool key_stream, bool reverse, void* zero_ptr, size_t zero_bytes,
                               cudaStream_t st);
// K1b: row-parallel finish: delta values, mask words and (key stream) reference rows from the
// 8-row checkpoints; counts, compacted indices, Eq. 6 counters, the decode hand-off row
// R(T-1)[j] = q_hat . k_j and (want_kt) the channel-major fp32 key copy.
// SMs of the current device (queried once per device).
int device_sm_count();
// programmatic: 1 = launched with programmatic stream serialisation (its launch overlaps the end
// of the kernel in front; the kernel waits for that kernel's completion itself); 2 = the same, but
// the kernel does not wait: the kernel in front releases it once the chain kernel's results are
// complete (query deltas behind the telescoped attention kernel); 0 = an ordinary launch.
cudaError_t launch_delta_finish(const Shape& s, const Workspace& w, const void* q, const void* k, int T,
                                float theta, int window, int shape, int dtype, int init, bool want_kt,
                                bool key_stream, bool reverse, int programmatic, cudaStream_t st);
// K2 (generic): fused hybrid attention on CUDA cores, any supported dtype.
cudaError_t launch_hybrid_attn_generic(const Shape& s, const Workspace& w, const void* q,
                                       const void* k, const void* v, void* out, int T, int window,
                                       int shape, int dtype, cudaStream_t st);
// K3: one decode step.
cudaError_t launch_decode_step(const Shape& s, const Workspace& w, const void* q_new,
                               const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                               void* out, int n, float theta, int window, int dtype, int qhat_sel,
                               cudaStream_t st);

// K3 (key deltas): one decode step of strategy (3); bf16 only, needs w.qhat_rows (reference-key cache).
// K3 with the score products on the tensor cores (bf16, d = 64): same step, same state.
// Host-side cache of the key cache's tensor map (encoded once per cache pointer, not per step).
struct DecodeTmapCache {
  const void* ptr = nullptr;
  alignas(64) unsigned char map[128];
};
// Does the step at position n take this kernel?  (bf16, d = 64, and a cache short enough for 64
// slices of nine tiles.)  n < 0: shape and type only.
bool decode_tc_applies(const Shape& s, int dtype, int n);
cudaError_t launch_decode_step_tc(const Shape& s, const Workspace& w, const void* q_new, const void* k_new,
                                  const void* v_new, void* k_cache, void* v_cache, void* out, int n, float theta,
                                  int window, int qhat_sel, DecodeTmapCache* cache, cudaStream_t st);
// The same for key deltas: tiles come from the reference-key cache or, inside the window, the key cache.
cudaError_t launch_decode_step_key_tc(const Shape& s, const Workspace& w, const void* q_new, const void* k_new,
                                      const void* v_new, void* k_cache, void* v_cache, void* out, int n,
                                      float theta, int window, int qhat_sel, DecodeTmapCache* cache_k,
                                      DecodeTmapCache* cache_h, cudaStream_t st);
// K3 (key deltas) from the compressed key-delta cache, the kernel that builds that cache behind a
// prefill, and its geometry (values per KV head at most, 32-row segments).
size_t keypack_capacity(int T_max, int d);
int keypack_segments(int T_max);
cudaError_t launch_pack_keys(const Shape& s, const Workspace& w, const void* k, int T, cudaStream_t st);
cudaError_t launch_decode_step_keypacked(const Shape& s, const Workspace& w, const void* q_new, const void* k_new,
                                         const void* v_new, void* k_cache, void* v_cache, void* out, int n,
                                         float theta, int window, int qhat_sel, cudaStream_t st);
cudaError_t launch_decode_step_key(const Shape& s, const Workspace& w, const void* q_new,
                                   const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                   void* out, int n, float theta, int window, int qhat_sel,
                                   cudaStream_t st);

// ---- bounds-checking build ------------------------------------------------------------
// DELTA_IN(index, extent, counters) guards a global access whose index a kernel computed by
// hand: true in the regular build (the guard compiles away); in a -DDELTA_DEBUG_BOUNDS build
// false for an index outside [0, extent), with DELTA_ERR_BOUNDS recorded in the status word, so
// the access is skipped instead of made (no trap, no assert: the context stays usable).
#ifdef DELTA_DEBUG_BOUNDS
__device__ __forceinline__ bool delta_in_bounds(size_t idx, size_t extent, unsigned long long* counters) {
  if (idx < extent) return true;
  atomicMax(&counters[CNT_STATUS], (unsigned long long)DELTA_ERR_BOUNDS);
  return false;
}
#define DELTA_IN(idx, extent, counters) delta_in_bounds((size_t)(idx), (size_t)(extent), (counters))
#else
#define DELTA_IN(idx, extent, counters) true
#endif

// ---- small device helpers -------------------------------------------------------------
__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) {
  return __float2bfloat16_rn(x);
}

// Is the causal pair (i, j <= i) inside the exact window?  shape: 0 block, 1 sliding.
__host__ __device__ __forceinline__ bool in_window(int i, int j, int W, int shape) {
  if (W <= 0) return false;
  return shape == 0 ? (i / W) == (j / W) : (i - j) < W;
}
// Number of in-window keys of query row i.
__host__ __device__ __forceinline__ int in_window_count(int i, int W, int shape) {
  if (W <= 0) return 0;
  return shape == 0 ? (i % W) + 1 : (i + 1 < W ? i + 1 : W);
}

// Number of queries i in [j, T) whose pair (i, j) is inside the exact window (key j's column).
__host__ __device__ __forceinline__ int in_window_col_count(int j, int T, int W, int shape) {
  if (W <= 0) return 0;
  const int last = shape == 0 ? (j / W + 1) * W : j + W;   // first query past the window
  return (last < T ? last : T) - j;
}

}  // namespace delta
