// C ABI of the delta-attention library: argument checks, workspace carving, launch order.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "delta_internal.cuh"
#include "k2_tc.cuh"

namespace delta {
static std::atomic<unsigned long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }
static thread_local char g_cuda_err[256] = "";
delta_status_t cuda_fail(cudaError_t e) {
  snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
  return DELTA_ERR_CUDA;
}
}  // namespace delta

using namespace delta;

// NVTX range over an entry point (shows up in a timeline profiler; free when none is attached).
namespace {
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
};
}  // namespace

struct delta_state {
  delta_config_t cfg;
  Shape shape;
  Workspace ws;
  void* base;
  size_t bytes;
  int n;         // tokens seen (of the longest sequence, after a prefill over sequences of different lengths)
  std::vector<int> n_b;   // tokens seen per batch element
  bool ragged = false;    // the batch elements stand at different positions
  std::vector<DecodeTmapCache> dec_tmap_b, dec_tmap_h_b;   // per batch element, for ragged decoding
  int qhat_sel;  // which q_hat buffer is current
  int forced_kernel;  // -1 auto, 0 generic, 1 tensor-core
  // Eq. 6 bookkeeping that needs no device work: sum of window lengths and sequence lengths
  double win_sum[2], len_sum[2];
  DecodeTmapCache dec_tmap;   // tensor map of the key cache the decode steps read
  DecodeTmapCache dec_tmap_h; // and of the reference-key cache (key deltas)
  int forced_decode_kernel = -1;   // -1: chosen per step
  bool key_cache_packed = false;   // key deltas: decode from the compressed key-delta cache
  // optional per-kernel timing of prefill (host-side event objects)
  bool profiling = false, profiled = false;
  // a reset has been asked for and the chain kernel of the next prefill does the clearing (no
  // launch of its own: a memset in front of the chain kernel costs 2 us of a 38 us step)
  bool zero_pending = false;
  cudaEvent_t ev[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
};

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static delta_status_t check_config(const delta_config_t* c) {
  if (!c) return DELTA_ERR_INVALID_ARG;
  if (c->B < 1 || c->H < 1 || c->H_kv < 1 || c->T_max < 1) return DELTA_ERR_INVALID_ARG;
  if (c->H % c->H_kv != 0) return DELTA_ERR_INVALID_ARG;
  if (c->dtype != DELTA_F32 && c->dtype != DELTA_BF16) return DELTA_ERR_INVALID_ARG;
  if (c->prefill_window != DELTA_WIN_BLOCK && c->prefill_window != DELTA_WIN_SLIDING)
    return DELTA_ERR_INVALID_ARG;
  if (c->init != DELTA_INIT_BASIS_EXACT && c->init != DELTA_INIT_ZERO_STATE)
    return DELTA_ERR_INVALID_ARG;
  if (c->source != DELTA_SRC_QUERY && c->source != DELTA_SRC_KEY && c->source != DELTA_SRC_QUERY_BOTTOM_UP)
    return DELTA_ERR_INVALID_ARG;
  if (c->d != 64 && c->d != 128) return DELTA_ERR_UNSUPPORTED;
  // key deltas (strategy 3) are served by the telescoped tensor-core kernel only
  // and so are bottom-up query deltas (strategy 2)
  if (c->source != DELTA_SRC_QUERY && !(c->dtype == DELTA_BF16 && tcq_kernel_shape(c->d)))
    return DELTA_ERR_UNSUPPORTED;
  const int g = c->H / c->H_kv;
  if (g != 1 && g != 2 && g != 4 && g != 8) return DELTA_ERR_UNSUPPORTED;
  if (c->T_max > kMaxDecodeSplits * kDecodeChunkMax) return DELTA_ERR_UNSUPPORTED;
  if ((long long)c->B * c->H > 65535) return DELTA_ERR_UNSUPPORTED;
  return DELTA_OK;
}

// Carve the workspace; base may be null (size query).
static void carve(const delta_config_t& c, char* base, Workspace* w) {
  const size_t BH = (size_t)c.B * c.H, BKV = (size_t)c.B * c.H_kv;
  const size_t nt = (c.T_max + DELTA_TILE_ROWS - 1) / DELTA_TILE_ROWS;
  const size_t g = c.H / c.H_kv;
  size_t off = 0;
  auto take = [&](size_t bytes) { char* p = base ? base + off : nullptr; off += align_up(bytes, 256); return p; };
  // what a reset has to zero comes first, as one contiguous span: the two reference buffers
  // (Eq. 3: the reference starts at 0), the counters and the decode tickets.  The score row R
  // needs no zeroing: prefill writes entries 0..T-1 and a decode step reads only entries below
  // its position.
  w->qhat[0] = (float*)take(BH * c.d * 4);
  w->qhat[1] = (float*)take(BH * c.d * 4);
  w->counters = (unsigned long long*)take(CNT_TOTAL * 8);
  w->dec_ticket = (uint32_t*)take(BKV * 4);
  w->zero_bytes = off;
  w->dq = (float*)take(BH * c.T_max * c.d * 4);
  w->mask = (uint32_t*)take(BH * c.T_max * (c.d / 32) * 4);
  w->row_nnz = (uint16_t*)take(BH * c.T_max * 2);
  w->tile_nnz = (uint32_t*)take(BH * nt * 4);
  w->idx = (uint8_t*)take(BH * c.T_max * c.d);
  w->qhat_tile = (float*)take(BH * nt * c.d * 4);
  w->ckpt = (float*)take(BH * (((size_t)c.T_max + DELTA_CKPT_ROWS - 1) / DELTA_CKPT_ROWS) * c.d * 4);
  w->R = (float*)take(BH * c.T_max * 4);
  w->dec_partial = (float*)take(BKV * kMaxDecodeSplits * g * (c.d + 2) * 4);
  w->kt = (c.dtype == DELTA_BF16 && tc_kernel_shape(c.d))
              ? (float*)take(BKV * c.d * (((size_t)c.T_max + 3) / 4 * 4) * 4) : nullptr;
  w->qhat_rows = (c.dtype == DELTA_BF16 && tcq_kernel_shape(c.d))
                     ? (__nv_bfloat16*)take(BH * c.T_max * c.d * 2) : nullptr;
  if (c.source == DELTA_SRC_KEY && c.dtype == DELTA_BF16) {
    // compressed key-delta cache: sized for the worst case (every element fires)
    const size_t nseg = (size_t)keypack_segments(c.T_max);
    w->kp_vals = (uint16_t*)take(BKV * keypack_capacity(c.T_max, c.d) * 2);
    w->kp_segoff = (uint32_t*)take(BKV * (nseg + 1) * 4);
    w->kp_base = (uint16_t*)take(BKV * nseg * c.d * 2);
    w->kp_used = (uint32_t*)take(BKV * 4);
    w->kp_mask = (uint32_t*)take(BKV * nseg * 32 * (c.d / 32) * 4);
    w->kp_nnz = (uint16_t*)take(BKV * nseg * 32 * 2);
  } else {
    w->kp_vals = nullptr; w->kp_segoff = nullptr; w->kp_base = nullptr; w->kp_used = nullptr;
    w->kp_mask = nullptr; w->kp_nnz = nullptr;
  }
  w->total_bytes = off;
}

extern "C" {

delta_status_t delta_state_workspace_bytes(const delta_config_t* cfg, size_t* bytes) {
  if (!bytes) return DELTA_ERR_INVALID_ARG;
  delta_status_t s = check_config(cfg);
  if (s != DELTA_OK) return s;
  Workspace w;
  carve(*cfg, nullptr, &w);
  *bytes = w.total_bytes;
  return DELTA_OK;
}

// defer: leave the clearing of the device span to the next prefill (see zero_pending)
static delta_status_t zero_state(delta_state* st, cudaStream_t stream, bool defer) {
  if (defer) {
    st->zero_pending = true;
  } else {
    // one memset: the span carve() put at the front of the workspace
    cudaError_t e = cudaMemsetAsync(st->base, 0, st->ws.zero_bytes, stream);
    if (e != cudaSuccess) return cuda_fail(e);
    st->zero_pending = false;
  }
  st->n = 0;
  st->n_b.assign((size_t)st->cfg.B, 0);
  st->ragged = false;
  st->qhat_sel = 0;
  st->win_sum[0] = st->win_sum[1] = st->len_sum[0] = st->len_sum[1] = 0.0;
  return DELTA_OK;
}

delta_status_t delta_state_init(const delta_config_t* cfg, void* workspace, size_t workspace_bytes,
                                void* stream, delta_state_t** out) {
  if (!out) return DELTA_ERR_INVALID_ARG;
  *out = nullptr;
  delta_status_t s = check_config(cfg);
  if (s != DELTA_OK) return s;
  if (!workspace) return DELTA_ERR_INVALID_ARG;
  if (((uintptr_t)workspace & 255u) != 0) return DELTA_ERR_WORKSPACE;
  Workspace w;
  carve(*cfg, (char*)workspace, &w);
  if (workspace_bytes < w.total_bytes) return DELTA_ERR_WORKSPACE;
  delta_state* st = new (std::nothrow) delta_state();
  if (!st) return DELTA_ERR_INVALID_ARG;
  st->cfg = *cfg;
  st->shape = Shape{cfg->B, cfg->H, cfg->H_kv, cfg->d, cfg->T_max,
                    (cfg->T_max + DELTA_TILE_ROWS - 1) / DELTA_TILE_ROWS};
  st->ws = w;
  st->base = workspace;
  st->bytes = workspace_bytes;
  st->forced_kernel = -1;
  s = zero_state(st, (cudaStream_t)stream, /*defer=*/false);
  if (s != DELTA_OK) { delete st; return s; }
  *out = st;
  return DELTA_OK;
}

delta_status_t delta_state_reset(delta_state_t* st, void* stream) {
  if (!st) return DELTA_ERR_INVALID_ARG;
  return zero_state(st, (cudaStream_t)stream, /*defer=*/true);
}

delta_status_t delta_state_destroy(delta_state_t* st) {
  if (!st) return DELTA_ERR_INVALID_ARG;
  for (auto& ev : st->ev)
    if (ev) cudaEventDestroy(ev);
  delete st;
  return DELTA_OK;
}

delta_status_t delta_state_enable_profiling(delta_state_t* st, int32_t enable) {
  if (!st) return DELTA_ERR_INVALID_ARG;
  if (enable) {
    for (auto& ev : st->ev)
      if (!ev) {
        cudaError_t e = cudaEventCreate(&ev);
        if (e != cudaSuccess) return cuda_fail(e);
      }
  }
  st->profiling = enable != 0;
  st->profiled = false;
  return DELTA_OK;
}

delta_status_t delta_state_prefill_kernel_ms(delta_state_t* st, float* ms) {
  if (!st || !ms) return DELTA_ERR_INVALID_ARG;
  if (!st->profiling || !st->profiled) return DELTA_ERR_STATE;
  cudaError_t e = cudaEventSynchronize(st->ev[4]);
  if (e != cudaSuccess) return cuda_fail(e);
  for (int i = 0; i < 4; ++i)
    if ((e = cudaEventElapsedTime(&ms[i], st->ev[i], st->ev[i + 1])) != cudaSuccess) return cuda_fail(e);
  return DELTA_OK;
}

int32_t delta_state_position(const delta_state_t* st) { return st ? st->n : -1; }

int32_t delta_state_sequence_position(const delta_state_t* st, int32_t b) {
  return (st && b >= 0 && b < st->cfg.B) ? st->n_b[(size_t)b] : -1;
}

// Can prefill kernel `which` (1 or 2) serve this state?
static bool tc_eligible(const delta_state* st, int which) {
  if (st->cfg.dtype != DELTA_BF16 || !tc_kernel_available(64)) return false;
  if (st->cfg.source != DELTA_SRC_QUERY && which != 2 && which != 3 && which != 4 && which != 5) return false;
  if ((which == 4 || which == 5) && (st->cfg.d != 64 || (st->shape.g() % 2) != 0)) return false;
  return which == 1 ? tc_kernel_shape(st->cfg.d) : tcq_kernel_shape(st->cfg.d);
}

int32_t delta_state_prefill_kernel(const delta_state_t* st) {
  if (!st) return -1;
  if (st->forced_kernel >= 0) return st->forced_kernel;
  return tc_eligible(st, 2) ? 2 : 0;   // the telescoped tensor-core kernel is the fastest where it applies
}

// Can the tensor-core decode kernel serve this state at all (whatever the slice length)?
static bool decode_tc_possible(const delta_state* st) {
  return st->cfg.source != DELTA_SRC_QUERY_BOTTOM_UP && decode_tc_applies(st->shape, st->cfg.dtype, -1);
}

int32_t delta_state_decode_kernel(const delta_state_t* st) {
  if (!st) return -1;
  if (!decode_tc_possible(st)) return 0;
  if (st->forced_decode_kernel >= 0) return st->forced_decode_kernel;
  return decode_tc_applies(st->shape, st->cfg.dtype, st->n) ? 1 : 0;
}

delta_status_t delta_state_set_decode_kernel(delta_state_t* st, int32_t which) {
  if (!st || which < -1 || which > 1) return DELTA_ERR_INVALID_ARG;
  if (which == 1 && !decode_tc_possible(st)) return DELTA_ERR_UNSUPPORTED;
  st->forced_decode_kernel = which;
  return DELTA_OK;
}

delta_status_t delta_state_set_key_cache(delta_state_t* st, int32_t packed) {
  if (!st || packed < 0 || packed > 1) return DELTA_ERR_INVALID_ARG;
  if (st->cfg.source != DELTA_SRC_KEY || !st->ws.kp_vals) return DELTA_ERR_UNSUPPORTED;
  if (st->n != 0) return DELTA_ERR_STATE;      // the encoding is built by the prefill
  st->key_cache_packed = packed != 0;
  return DELTA_OK;
}

delta_status_t delta_key_cache_bytes(const delta_state_t* st, uint64_t* packed_bytes, uint64_t* dense_bytes,
                                     void* stream) {
  if (!st || !packed_bytes || !dense_bytes) return DELTA_ERR_INVALID_ARG;
  const delta_config_t& c = st->cfg;
  if (c.source != DELTA_SRC_KEY || !st->ws.kp_vals || !st->key_cache_packed) return DELTA_ERR_UNSUPPORTED;
  const size_t bkv = (size_t)c.B * c.H_kv;
  std::vector<uint32_t> used(bkv);
  cudaError_t e = cudaMemcpyAsync(used.data(), st->ws.kp_used, bkv * 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e);
  if ((e = cudaStreamSynchronize((cudaStream_t)stream)) != cudaSuccess) return cuda_fail(e);
  uint64_t packed = 0, dense = 0;
  for (int b = 0; b < c.B; ++b) {
    const uint64_t rows = (uint64_t)st->n_b[(size_t)b], segs = (rows + 31) / 32;
    for (int h = 0; h < c.H_kv; ++h)
      packed += 2ull * used[(size_t)b * c.H_kv + h]            // values (with the segments' padding)
                + rows * (uint64_t)(c.d / 8)                    // mask words
                + rows * 2                                      // fired counts
                + segs * (uint64_t)c.d * 2 + (segs + 1) * 4;    // segment bases and offsets
    dense += (uint64_t)c.H_kv * rows * (uint64_t)c.d * 2;
  }
  *packed_bytes = packed;
  *dense_bytes = dense;
  return DELTA_OK;
}

delta_status_t delta_state_set_prefill_kernel(delta_state_t* st, int32_t which) {
  if (!st || which < -1 || which > 5) return DELTA_ERR_INVALID_ARG;
  if (which >= 1 && !tc_eligible(st, which)) return DELTA_ERR_UNSUPPORTED;
  if (which == 0 && st->cfg.source != DELTA_SRC_QUERY) return DELTA_ERR_UNSUPPORTED;
  st->forced_kernel = which;
  return DELTA_OK;
}

static delta_status_t check_theta_window(float theta, int32_t window) {
  if (!(theta >= 0.0f) || !std::isfinite(theta)) return DELTA_ERR_INVALID_ARG;
  if (window < 0) return DELTA_ERR_INVALID_ARG;
  return DELTA_OK;
}

}  // extern "C"

// The state's workspace and shape as one batch element sees them (every array is laid out batch
// element by batch element; the counters are shared).
static void view_of(const delta_state* st, int b, Shape* sh, Workspace* w) {
  const delta_config_t& c = st->cfg;
  *sh = st->shape;
  sh->B = 1;
  *w = st->ws;
  const size_t Hs = (c.source == DELTA_SRC_KEY) ? c.H_kv : c.H;      // heads of the delta stream
  const size_t nt = st->shape.n_tiles, nck = st->shape.n_ckpt(), g = c.H / c.H_kv;
  const size_t ub = (size_t)b;
  w->dq += ub * Hs * c.T_max * c.d;
  w->mask += ub * Hs * c.T_max * (c.d / 32);
  w->row_nnz += ub * Hs * c.T_max;
  w->tile_nnz += ub * Hs * nt;
  w->idx += ub * Hs * c.T_max * c.d;
  w->qhat_tile += ub * Hs * nt * c.d;
  w->ckpt += ub * Hs * nck * c.d;
  w->qhat[0] += ub * Hs * c.d;
  w->qhat[1] += ub * Hs * c.d;
  w->R += ub * c.H * c.T_max;
  w->dec_partial += ub * c.H_kv * kMaxDecodeSplits * g * (c.d + 2);
  w->dec_ticket += ub * c.H_kv;
  if (w->kt) w->kt += ub * c.H_kv * c.d * (((size_t)c.T_max + 3) / 4 * 4);
  if (w->qhat_rows) w->qhat_rows += ub * Hs * c.T_max * c.d;
  if (w->kp_vals) {
    const size_t nseg = (size_t)keypack_segments(c.T_max);
    w->kp_vals += ub * c.H_kv * keypack_capacity(c.T_max, c.d);
    w->kp_segoff += ub * c.H_kv * (nseg + 1);
    w->kp_base += ub * c.H_kv * nseg * c.d;
    w->kp_used += ub * c.H_kv;
    w->kp_mask += ub * c.H_kv * nseg * 32 * (c.d / 32);
    w->kp_nnz += ub * c.H_kv * nseg * 32;
  }
}

// The three kernels of a prefill over one view (the whole batch, or one batch element).
static delta_status_t prefill_launch(delta_state* st, const Shape& shape, const Workspace& ws, const void* q,
                                     const void* k, const void* v, void* out, int32_t T, float theta,
                                     int32_t window, cudaStream_t cs, bool prof) {
  const delta_config_t& c = st->cfg;
  cudaError_t e;
  // a pending reset: the chain kernel clears the span, less the front of qhat[0] that the chain
  // kernels of this prefill fill themselves (one reference per head of the delta stream)
  void* zero_ptr = nullptr;
  size_t zero_bytes = 0;
  if (st->zero_pending) {
    const size_t skip = (size_t)c.B * (c.source == DELTA_SRC_KEY ? c.H_kv : c.H) * c.d * sizeof(float);
    zero_ptr = (char*)st->base + skip;
    zero_bytes = st->ws.zero_bytes - skip;
    st->zero_pending = false;
  }
#define MARK(i) do { if (prof && (e = cudaEventRecord(st->ev[i], cs)) != cudaSuccess) return cuda_fail(e); } while (0)
  const int which = delta_state_prefill_kernel(st);
  const bool use_tc = which == 1;
  const bool key = c.source == DELTA_SRC_KEY;
  const bool rev = c.source == DELTA_SRC_QUERY_BOTTOM_UP;
  const bool tcq = which >= 2 && which <= 5;
  if ((key || rev) && !tcq) return DELTA_ERR_UNSUPPORTED;   // no tensor-core kernel on this device
  // The telescoped attention kernel reads nothing the finish kernel writes (delta values,
  // mask words, counts, indices, counters, hand-off row), so it runs directly behind the chain
  // kernel and the finish kernel comes last.  Both are launched with programmatic stream
  // serialisation: the attention CTAs are resident and set up by the time the chain ends, and
  // the finish kernel's launch overlaps the end of the attention kernel.  With per-kernel
  // timing on, the kernels run in their natural order with events between them.
  const bool chained = tcq && !prof;
  MARK(0);
  // the delta stream: the queries (strategy 1) or the keys, per KV head (strategy 3)
  if ((e = launch_delta_chain(shape, ws, key ? k : q, T, theta, c.dtype, c.init, key, rev, zero_ptr, zero_bytes, cs)) != cudaSuccess)
    return cuda_fail(e);
  auto attention = [&]() -> cudaError_t {
    if (use_tc) return launch_hybrid_attn_tc(shape, ws, q, k, v, out, T, window, c.prefill_window, cs);
    if (tcq)
      return launch_hybrid_attn_tcq(shape, ws, q, k, v, out, T, theta, c.init, window, c.prefill_window, key,
                                    rev, /*form=*/which == 3 ? 1 : which == 4 ? 2 : which == 5 ? 3 : 0, cs);
    return launch_hybrid_attn_generic(shape, ws, q, k, v, out, T, window, c.prefill_window, c.dtype, cs);
  };
  if (chained && !key) {
    if ((e = attention()) != cudaSuccess) return cuda_fail(e);
    // (released by the attention CTAs once the chain is complete: it runs beside their last wave)
    if ((e = launch_delta_finish(shape, ws, q, k, T, theta, window, c.prefill_window, c.dtype, c.init,
                                 use_tc, key, rev, 2, cs)) != cudaSuccess)
      return cuda_fail(e);
  } else if (chained) {
    // key deltas: the finish kernel writes the reference-key rows the attention kernel streams,
    // so it comes first (both programmatically serialised behind the kernel in front)
    if ((e = launch_delta_finish(shape, ws, q, k, T, theta, window, c.prefill_window, c.dtype, c.init,
                                 use_tc, key, rev, 1, cs)) != cudaSuccess)
      return cuda_fail(e);
    if ((e = attention()) != cudaSuccess) return cuda_fail(e);
  } else {
    MARK(1);
    if ((e = launch_delta_finish(shape, ws, q, k, T, theta, window, c.prefill_window, c.dtype, c.init,
                                 use_tc, key, rev, 0, cs)) != cudaSuccess)
      return cuda_fail(e);
    MARK(2);
    if ((e = attention()) != cudaSuccess) return cuda_fail(e);
  }
  MARK(3);
  // key deltas with the compressed cache: encode the key stream behind everything it is built from
  if (key && st->key_cache_packed && (e = launch_pack_keys(shape, ws, k, T, cs)) != cudaSuccess) return cuda_fail(e);
  MARK(4);
#undef MARK
  return DELTA_OK;
}

extern "C" {

delta_status_t delta_attn_prefill(delta_state_t* st, const void* q, const void* k, const void* v,
                                  void* out, int32_t T, int32_t H, int32_t H_kv, int32_t d,
                                  float theta, int32_t window, void* stream) {
  NvtxRange range("delta_attn_prefill");
  if (!st || !q || !k || !v || !out) return DELTA_ERR_INVALID_ARG;
  if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15u) != 0) return DELTA_ERR_INVALID_ARG;
  const delta_config_t& c = st->cfg;
  if (H != c.H || H_kv != c.H_kv || d != c.d) return DELTA_ERR_INVALID_ARG;
  delta_status_t s = check_theta_window(theta, window);
  if (s != DELTA_OK) return s;
  if (T < 1) return DELTA_ERR_INVALID_ARG;
  if (T > c.T_max) return DELTA_ERR_CAPACITY;
  if (st->n != 0) return DELTA_ERR_STATE;
  const bool prof = st->profiling;
  s = prefill_launch(st, st->shape, st->ws, q, k, v, out, T, theta, window, (cudaStream_t)stream, prof);
  if (s != DELTA_OK) return s;
  st->profiled = prof;
  st->n = T;
  st->n_b.assign((size_t)c.B, T);
  st->ragged = false;
  st->qhat_sel = 0;
  st->win_sum[0] += (double)c.B * (double)(window < T ? window : T);
  st->len_sum[0] += (double)c.B * (double)T;
  return DELTA_OK;
}

delta_status_t delta_attn_prefill_varlen(delta_state_t* st, const void* q, const void* k, const void* v,
                                         void* out, const int32_t* seq_lens, const int32_t* windows,
                                         float theta, void* stream) {
  NvtxRange range("delta_attn_prefill_varlen");
  if (!st || !q || !k || !v || !out || !seq_lens || !windows) return DELTA_ERR_INVALID_ARG;
  if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15u) != 0) return DELTA_ERR_INVALID_ARG;
  const delta_config_t& c = st->cfg;
  if (!(theta >= 0.0f) || !std::isfinite(theta)) return DELTA_ERR_INVALID_ARG;
  for (int b = 0; b < c.B; ++b) {
    if (seq_lens[b] < 1 || windows[b] < 0) return DELTA_ERR_INVALID_ARG;
    if (seq_lens[b] > c.T_max) return DELTA_ERR_CAPACITY;
  }
  if (st->n != 0) return DELTA_ERR_STATE;
  const size_t es = c.dtype == DELTA_F32 ? 4 : 2;
  size_t q_off = 0;     // elements in front of sequence b in the packed query / output arrays
  int t_longest = 0;
  bool same = true;
  for (int b = 0; b < c.B; ++b) {
    Shape sh;
    Workspace ws;
    view_of(st, b, &sh, &ws);
    const int T = seq_lens[b];
    const size_t kv_off = (size_t)b * c.H_kv * c.T_max * c.d * es;
    delta_status_t s = prefill_launch(st, sh, ws, (const char*)q + q_off * es, (const char*)k + kv_off,
                                      (const char*)v + kv_off, (char*)out + q_off * es, T, theta, windows[b],
                                      (cudaStream_t)stream, false);
    if (s != DELTA_OK) return s;
    q_off += (size_t)c.H * T * c.d;
    st->n_b[(size_t)b] = T;
    st->win_sum[0] += (double)(windows[b] < T ? windows[b] : T);
    st->len_sum[0] += (double)T;
    t_longest = T > t_longest ? T : t_longest;
    same = same && T == seq_lens[0];
  }
  st->profiled = false;
  st->n = t_longest;
  st->ragged = !same;
  st->qhat_sel = 0;
  return DELTA_OK;
}

delta_status_t delta_prefill_staging_bytes(const delta_config_t* cfg, int32_t T, size_t* bytes) {
  if (!bytes) return DELTA_ERR_INVALID_ARG;
  delta_status_t s = check_config(cfg);
  if (s != DELTA_OK) return s;
  if (T < 1 || T > cfg->T_max) return DELTA_ERR_INVALID_ARG;
  const size_t es = cfg->dtype == DELTA_F32 ? 4 : 2;
  const size_t qb = align_up((size_t)cfg->B * cfg->H * T * cfg->d * es, 256);
  const size_t kb = align_up((size_t)cfg->B * cfg->H_kv * cfg->T_max * cfg->d * es, 256);
  *bytes = 2 * qb + 2 * kb;
  return DELTA_OK;
}

delta_status_t delta_attn_prefill_host(delta_state_t* st, const void* q_host, const void* k_host,
                                       const void* v_host, void* out_host, void* staging,
                                       size_t staging_bytes, int32_t T, float theta,
                                       int32_t window, void* stream) {
  if (!st || !q_host || !k_host || !v_host || !out_host || !staging) return DELTA_ERR_INVALID_ARG;
  const delta_config_t& c = st->cfg;
  size_t need = 0;
  delta_status_t s = delta_prefill_staging_bytes(&c, T, &need);
  if (s != DELTA_OK) return s;
  if (staging_bytes < need || ((uintptr_t)staging & 255u)) return DELTA_ERR_WORKSPACE;
  if (st->n != 0) return DELTA_ERR_STATE;
  s = check_theta_window(theta, window);
  if (s != DELTA_OK) return s;
  const size_t es = c.dtype == DELTA_F32 ? 4 : 2;
  const size_t q_bytes = (size_t)c.B * c.H * T * c.d * es;
  const size_t qb = align_up(q_bytes, 256);
  const size_t kb = align_up((size_t)c.B * c.H_kv * c.T_max * c.d * es, 256);
  char* dq_ = (char*)staging;
  char* dout = dq_ + qb;
  char* dk = dout + qb;
  char* dv = dk + kb;
  cudaStream_t cs = (cudaStream_t)stream;
  cudaError_t e;
  if ((e = cudaMemcpyAsync(dq_, q_host, q_bytes, cudaMemcpyHostToDevice, cs)) != cudaSuccess) return cuda_fail(e);
  // host K/V hold T rows per head; the device copy uses the cache layout with T_max rows
  const size_t row = (size_t)c.d * es;
  const size_t units = (size_t)c.B * c.H_kv;
  if (T == c.T_max) {      // the two layouts coincide: one contiguous copy each
    if ((e = cudaMemcpyAsync(dk, k_host, units * T * row, cudaMemcpyHostToDevice, cs)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(dv, v_host, units * T * row, cudaMemcpyHostToDevice, cs)) != cudaSuccess) return cuda_fail(e);
  } else {
    if ((e = cudaMemcpy2DAsync(dk, (size_t)c.T_max * row, k_host, (size_t)T * row, (size_t)T * row, units,
                               cudaMemcpyHostToDevice, cs)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpy2DAsync(dv, (size_t)c.T_max * row, v_host, (size_t)T * row, (size_t)T * row, units,
                               cudaMemcpyHostToDevice, cs)) != cudaSuccess) return cuda_fail(e);
  }
  s = delta_attn_prefill(st, dq_, dk, dv, dout, T, c.H, c.H_kv, c.d, theta, window, stream);
  if (s != DELTA_OK) return s;
  if ((e = cudaMemcpyAsync(out_host, dout, q_bytes, cudaMemcpyDeviceToHost, cs)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaStreamSynchronize(cs)) != cudaSuccess) return cuda_fail(e);
  return DELTA_OK;
}

}  // extern "C"

// One decode-step launch over a view (the whole batch, or one batch element) at position n.
static cudaError_t decode_launch(delta_state* st, const Shape& shape, const Workspace& ws, const void* q_new,
                                 const void* k_new, const void* v_new, void* k_cache, void* v_cache, void* out,
                                 int n, float theta, int32_t window, DecodeTmapCache* tmap, DecodeTmapCache* tmap_h,
                                 cudaStream_t cs) {
  const bool tcs = decode_tc_possible(st) &&
                   (st->forced_decode_kernel >= 0 ? st->forced_decode_kernel == 1
                                                  : decode_tc_applies(shape, st->cfg.dtype, n));
  if (st->cfg.source == DELTA_SRC_KEY && st->key_cache_packed)
    return launch_decode_step_keypacked(shape, ws, q_new, k_new, v_new, k_cache, v_cache, out, n, theta, window,
                                        st->qhat_sel, cs);
  if (st->cfg.source == DELTA_SRC_KEY)
    return tcs ? launch_decode_step_key_tc(shape, ws, q_new, k_new, v_new, k_cache, v_cache, out, n, theta, window,
                                           st->qhat_sel, tmap, tmap_h, cs)
               : launch_decode_step_key(shape, ws, q_new, k_new, v_new, k_cache, v_cache, out, n, theta, window,
                                        st->qhat_sel, cs);
  return tcs ? launch_decode_step_tc(shape, ws, q_new, k_new, v_new, k_cache, v_cache, out, n, theta, window,
                                     st->qhat_sel, tmap, cs)
             : launch_decode_step(shape, ws, q_new, k_new, v_new, k_cache, v_cache, out, n, theta, window,
                                  st->cfg.dtype, st->qhat_sel, cs);
}

extern "C" {

delta_status_t delta_attn_decode_step(delta_state_t* st, const void* q_new, const void* k_new,
                                      const void* v_new, void* k_cache, void* v_cache, void* out,
                                      float theta, int32_t window, void* stream) {
  NvtxRange range("delta_attn_decode_step");
  if (!st || !q_new || !k_new || !v_new || !k_cache || !v_cache || !out) return DELTA_ERR_INVALID_ARG;
  // every decode kernel stages cache tiles with bulk copies and reads rows as 16-byte vectors
  if ((((uintptr_t)q_new | (uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)k_cache | (uintptr_t)v_cache |
        (uintptr_t)out) & 15u) != 0)
    return DELTA_ERR_INVALID_ARG;
  delta_status_t s = check_theta_window(theta, window);
  if (s != DELTA_OK) return s;
  const delta_config_t& c = st->cfg;
  if (c.source == DELTA_SRC_QUERY_BOTTOM_UP) return DELTA_ERR_UNSUPPORTED;   // strategy (2) has no decode
  if (st->n < 1) return DELTA_ERR_STATE;
  if (st->n >= c.T_max) return DELTA_ERR_CAPACITY;      // (the longest sequence decides)
  cudaStream_t cs = (cudaStream_t)stream;
  cudaError_t e = cudaSuccess;
  if (!st->ragged) {
    e = decode_launch(st, st->shape, st->ws, q_new, k_new, v_new, k_cache, v_cache, out, st->n, theta, window,
                      &st->dec_tmap, &st->dec_tmap_h, cs);
    if (e != cudaSuccess) return cuda_fail(e);
    const int L = st->n + 1;
    st->win_sum[1] += (double)c.B * (double)(window < L ? window : L);
    st->len_sum[1] += (double)c.B * (double)L;
  } else {
    // the batch elements stand at different positions: one launch per element over its view
    const size_t es = c.dtype == DELTA_F32 ? 4 : 2;
    if (st->dec_tmap_b.size() != (size_t)c.B) { st->dec_tmap_b.resize((size_t)c.B); st->dec_tmap_h_b.resize((size_t)c.B); }
    for (int b = 0; b < c.B; ++b) {
      Shape sh;
      Workspace ws;
      view_of(st, b, &sh, &ws);
      const size_t qo = (size_t)b * c.H * c.d * es, ko = (size_t)b * c.H_kv * c.d * es;
      const size_t co = (size_t)b * c.H_kv * c.T_max * c.d * es;
      e = decode_launch(st, sh, ws, (const char*)q_new + qo, (const char*)k_new + ko, (const char*)v_new + ko,
                        (char*)k_cache + co, (char*)v_cache + co, (char*)out + qo, st->n_b[(size_t)b], theta, window,
                        &st->dec_tmap_b[(size_t)b], &st->dec_tmap_h_b[(size_t)b], cs);
      if (e != cudaSuccess) return cuda_fail(e);
      const int L = st->n_b[(size_t)b] + 1;
      st->win_sum[1] += (double)(window < L ? window : L);
      st->len_sum[1] += (double)L;
    }
  }
  for (auto& nb : st->n_b) nb += 1;
  st->qhat_sel ^= 1;
  st->n += 1;
  return DELTA_OK;
}

static void finish_stage(delta_stage_stats_t* o, const unsigned long long* c, double win, double len) {
  o->nnz = c[0]; o->elements = c[1]; o->macs_done = c[2]; o->macs_dense = c[3];
  o->S_m = o->elements ? 1.0 - (double)o->nnz / (double)o->elements : 0.0;
  o->S_c_eq6 = len > 0.0 ? o->S_m * (1.0 - win / len) : 0.0;
  o->S_c_exact = o->macs_dense ? 1.0 - (double)o->macs_done / (double)o->macs_dense : 0.0;
}

delta_status_t delta_sparsity_stats(const delta_state_t* st, delta_stats_t* host_out, void* stream) {
  NvtxRange range("delta_sparsity_stats");
  if (!st || !host_out) return DELTA_ERR_INVALID_ARG;
  unsigned long long c[CNT_TOTAL] = {};
  if (!st->zero_pending) {      // (after a reset the counters are zero, whatever the device still holds)
    cudaError_t e = cudaMemcpyAsync(c, st->ws.counters, sizeof(c), cudaMemcpyDeviceToHost,
                                    (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e);
    if ((e = cudaStreamSynchronize((cudaStream_t)stream)) != cudaSuccess) return cuda_fail(e);
  }
  memset(host_out, 0, sizeof(*host_out));
  for (int sh = 0; sh < CNT_SHARDS; ++sh)          // prefill counters are sharded on the device
    for (int i = 0; i < 4; ++i) c[CNT_PREFILL_NNZ + i] += c[CNT_SHARD_BASE + 4 * sh + i];
  finish_stage(&host_out->prefill, c + CNT_PREFILL_NNZ, st->win_sum[0], st->len_sum[0]);
  finish_stage(&host_out->decode, c + CNT_DECODE_NNZ, st->win_sum[1], st->len_sum[1]);
  unsigned long long sum[4];
  for (int i = 0; i < 4; ++i) sum[i] = c[CNT_PREFILL_NNZ + i] + c[CNT_DECODE_NNZ + i];
  finish_stage(&host_out->combined, sum, 0.0, 0.0);
  // combined Eq. 6 value: the stages' Eq. 6 values weighted by their dense multiply-adds
  const double dp = (double)host_out->prefill.macs_dense, dd = (double)host_out->decode.macs_dense;
  host_out->combined.S_c_eq6 =
      (dp + dd) > 0.0 ? (host_out->prefill.S_c_eq6 * dp + host_out->decode.S_c_eq6 * dd) / (dp + dd) : 0.0;
  host_out->n = st->n;
  host_out->device_status = (uint32_t)c[CNT_STATUS];
  return host_out->device_status == 0 ? DELTA_OK : (delta_status_t)host_out->device_status;
}

int32_t delta_window_from_gamma(int32_t n, double gamma, int32_t w_max) {
  if (n < 0 || !(gamma >= 0.0)) return 0;
  const double w = std::floor(gamma * (double)n);
  const double m = w < (double)w_max ? w : (double)w_max;
  return m < 0.0 ? 0 : (int32_t)m;
}

delta_status_t delta_state_view(const delta_state_t* st, int32_t what, const void** dev_ptr,
                                size_t* bytes) {
  if (!st || !dev_ptr || !bytes) return DELTA_ERR_INVALID_ARG;
  const delta_config_t& c = st->cfg;
  const size_t BH = (size_t)c.B * c.H;
  const size_t nt = st->shape.n_tiles;
  switch (what) {
    case DELTA_VIEW_DQ: *dev_ptr = st->ws.dq; *bytes = BH * c.T_max * c.d * 4; break;
    case DELTA_VIEW_MASK: *dev_ptr = st->ws.mask; *bytes = BH * c.T_max * (c.d / 32) * 4; break;
    case DELTA_VIEW_ROW_NNZ: *dev_ptr = st->ws.row_nnz; *bytes = BH * c.T_max * 2; break;
    case DELTA_VIEW_TILE_NNZ: *dev_ptr = st->ws.tile_nnz; *bytes = BH * nt * 4; break;
    case DELTA_VIEW_IDX: *dev_ptr = st->ws.idx; *bytes = BH * c.T_max * c.d; break;
    case DELTA_VIEW_QHAT_TILE: *dev_ptr = st->ws.qhat_tile; *bytes = BH * nt * c.d * 4; break;
    case DELTA_VIEW_QHAT: *dev_ptr = st->ws.qhat[st->qhat_sel]; *bytes = BH * c.d * 4; break;
    case DELTA_VIEW_R: *dev_ptr = st->ws.R; *bytes = BH * c.T_max * 4; break;
    case DELTA_VIEW_COUNTERS: *dev_ptr = st->ws.counters; *bytes = (size_t)CNT_TOTAL * 8; break;
    default: return DELTA_ERR_INVALID_ARG;
  }
  return DELTA_OK;
}

int32_t delta_debug_bounds_build(void) {
#ifdef DELTA_DEBUG_BOUNDS
  return 1;
#else
  return 0;
#endif
}

uint64_t delta_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* delta_status_string(delta_status_t s) {
  switch (s) {
    case DELTA_OK: return "ok";
    case DELTA_ERR_INVALID_ARG: return "invalid argument";
    case DELTA_ERR_UNSUPPORTED: return "unsupported configuration";
    case DELTA_ERR_WORKSPACE: return "workspace too small or misaligned";
    case DELTA_ERR_CAPACITY: return "sequence capacity T_max exceeded";
    case DELTA_ERR_STATE: return "call order: state not in the required condition";
    case DELTA_ERR_CUDA: return "CUDA runtime error";
    case DELTA_ERR_TIMEOUT: return "bounded device-side wait ran out";
    case DELTA_ERR_BOUNDS: return "index out of range in a kernel (bounds-checking build)";
    case DELTA_ERR_SCRATCH_LIMIT:
      return "problem larger than the built-in scratch of delta_attn_decode_step_noalloc";
  }
  return "unknown status";
}

const char* delta_last_cuda_error(void) { return g_cuda_err; }

}  // extern "C"
