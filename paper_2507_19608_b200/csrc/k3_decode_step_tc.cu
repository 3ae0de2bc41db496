// K3 (tensor-core scores) -- one decode step of strategy (1) for bf16 caches with d = 64
// (Section III-A "Decoding Stage Considerations", Section III-B "Decoding Stage").
//
// Eq. 4's running sum telescopes: R(n)[j] = (sum of all Delta q so far) . k_j = q_hat(n) . k_j,
// and for bf16 inputs every element of q_hat is a copy of an input element, so the whole score
// row of a step is two small dense products per cached key: q_hat . k_j (outside the window) and
// q . k_j (the W_d most recent keys).  Both come from ONE tensor-core product per 128-key tile,
//   S[128 keys][16] = K_tile[128][64] . Qcat[16][64]^T,
// where the rows of Qcat are the G new reference vectors, the G new query vectors and zeros.
// The score row R is no longer read; it is written (R[j] = q_hat . k_j) because it is part of
// the carried state.  The FP32 pipes keep what is not a contraction of useful shape: the
// threshold step (Eq. 2-3), the softmax and P.V (G rows of P against the value tile).
//
// Grid = (key slices, batch x KV heads); a CTA serves the G query heads of one KV head.
//   1. threshold q_new against the carried reference, build Qcat in the operand layout;
//   2. warp 0 streams the slice's key tiles with TMA (128-byte swizzle, five stages) and issues
//      the products; all score tiles of the slice stay in tensor memory (16 columns per tile);
//   3. one softmax over the slice: every thread reads its keys' scores (lane = key), hybrid
//      select, scale, R written; maximum and sum reduced once per slice, not per tile;
//   4. P.V with the value tiles streamed by bulk copies through the same five stages once the
//      products are done, the warps releasing stages through mbarriers (no block-wide barrier
//      per tile);
//   5. the slice result is stored and the last CTA of the (batch, KV head) merges the slices.
// The key and value that arrive with this step are scored on the FP32 pipes by the CTA that
// owns their slice (their cache row is written by this very kernel).
// Every wait is bounded; after a time-out the kernel still runs to its end and the status word
// records DELTA_ERR_TIMEOUT.
//
// KEY = true is the same step for key deltas (strategy 3): the score of key j is q_new . k_j for
// the W_d most recent keys and q_new . k_hat(j) for the older ones (the column recursion of
// Eq. 4, telescoped; k_hat(j) is the reference key after row j, kept in the library's
// reference-key cache).  Qcat holds the G query rows only, and the tile a product reads is a
// tile of the reference-key cache (keys older than the window), of the key cache (keys inside
// it) or -- the one tile the window's edge falls into -- a reference-key tile whose window rows
// warp 0 replaces in shared memory by the original keys.  The threshold step runs over k_new
// (one vector per KV head), nothing like R is carried, and the CTA that owns the new key's
// slice appends k_new, v_new and k_hat(n) to their caches.
#include <cuda.h>

#include "decode_common.cuh"
#include "k2_tc.cuh"
#include "tc_common.cuh"

namespace delta {

namespace {

constexpr int TCD = 64;                // head dimension
constexpr int TK = 128;                // keys per tile
constexpr int MAXT = 9;                // tiles per slice at most (1152 keys)
constexpr int SCOL = 16;               // tensor-memory columns per tile (N of the product)
constexpr uint32_t DEC_TMEM_COLS = 256;
// CTAs the key slices aim for.  Measured at batch 16, 2049 keys: 256 CTAs 24.5 us per step, 384 CTAs
// 30.3, 512 CTAs 29.2, 768 CTAs 31.6 (a CTA's fixed cost outweighs the better balance).
constexpr int kTcTargetCtas = 296;

// One ring of five 16 KiB stages serves both streams: all five carry key tiles while the score
// products run and value tiles afterwards.  Measured at batch 16 (warm L2 / L2 flushed before every
// step, us per step): 2 key + 3 value stages 19.0 / 30.9, 3 + 2: 18.6 / 29.8, 4 + 1: 18.4 / 29.2,
// all five shared: 18.3 / 28.8.
constexpr int NKS = 5;                 // key-ring stages
constexpr int NVS_OWN = 0;             // value-ring stages of its own
constexpr int NVS = NVS_OWN + NKS;     // plus the key stages once the score products are done
enum { BAR_K0 = 0, BAR_KFREE0 = BAR_K0 + NKS, BAR_S = BAR_KFREE0 + NKS, BAR_V0, BAR_VFREE0 = BAR_V0 + NVS, DEC_NUM_BARS = BAR_VFREE0 + NVS };


// The G probabilities of one key (contiguous, 16-byte aligned for G >= 4).
template <int G> __device__ __forceinline__ void load_probs(const float* p, float (&pr)[G]) {
  if constexpr (G % 4 == 0) {
#pragma unroll
    for (int i = 0; i < G; i += 4) {
      const float4 v = *reinterpret_cast<const float4*>(p + i);
      pr[i] = v.x; pr[i + 1] = v.y; pr[i + 2] = v.z; pr[i + 3] = v.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < G; ++i) pr[i] = p[i];
  }
}

}  // namespace

template <int G, bool KEY>
__global__ void __launch_bounds__(DNT, 2) decode_step_tc_kernel(
    const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_h,
    const __nv_bfloat16* __restrict__ q_new,
    const __nv_bfloat16* __restrict__ k_new, const __nv_bfloat16* __restrict__ v_new,
    __nv_bfloat16* __restrict__ k_cache, __nv_bfloat16* __restrict__ v_cache,
    __nv_bfloat16* __restrict__ khat_cache, uint16_t* __restrict__ row_nnz,
    __nv_bfloat16* __restrict__ out, const float* __restrict__ qhat_in, float* __restrict__ qhat_out,
    float* __restrict__ R, float* __restrict__ partial, uint32_t* __restrict__ ticket,
    unsigned long long* __restrict__ counters, int n, int T_max, int H, int chunk, int nsplit,
    float theta, int W, float scale_log2e) {
  using TC = __nv_bfloat16;
  constexpr int D = TCD;
  constexpr int LPK = D / 8, KPW = 32 / LPK;
  extern __shared__ unsigned char dsm_raw0[];
  const uint32_t raw = smem_u32(dsm_raw0);
  const uint32_t base = (raw + 1023u) & ~1023u;          // swizzled operand tiles want 1 KiB alignment
  unsigned char* sm = dsm_raw0 + (base - raw);
  constexpr uint32_t OFF_K = 0;                          // [2][128][64] bf16, 128-byte swizzle
  constexpr uint32_t OFF_V = OFF_K + NKS * TILE_BYTES;     // [NVS_OWN][128][64] bf16, plain rows
  constexpr uint32_t OFF_QC = OFF_V + NVS_OWN * TILE_BYTES;  // Qcat [16][64] bf16, 128-byte swizzle
  constexpr uint32_t OFF_F = OFF_QC + 2048;              // floats from here on
  float* q_s = reinterpret_cast<float*>(sm + OFF_F);     // [G][D]
  float* qh_s = q_s + G * D;                             // [G][D]
  float* red = reinterpret_cast<float*>(sm + OFF_K);     // [DNW][G][D]: the key ring is free by then
  float* wgt = qh_s + G * D;                             // [G * kMaxDecodeSplits] (merge) / [DNW][2G] (reductions)
  float* p_s = wgt + G * kMaxDecodeSplits;               // [MAXT * TK + 1][G] probabilities
  float* st_s = p_s + (MAXT * TK + 1) * G;               // [24]
  __shared__ __align__(8) unsigned long long bars[DEC_NUM_BARS];
  __shared__ uint32_t s_tmem;
  __shared__ int s_last, s_fail;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.x, bkv = blockIdx.y;
  const int H_kv = H / G;
  const int b = bkv / H_kv, kvh = bkv - b * H_kv;
  const int L = n + 1;
  const int j0 = split * chunk;
  const int len = max(0, min(chunk, L - j0));            // keys of the slice, the new one included
  const int cached = max(0, min(len, n - j0));           // of which already in the cache
  const int n_tiles = (cached + TK - 1) / TK;            // tiles that go through the tensor cores
  const bool has_new = (n >= j0) && (n < j0 + len);
  const int wl = n - W + 1;                              // first key inside the decode window
  // key deltas: where tile t's rows come from -- 0 reference-key cache, 1 key cache, 2 mixed
  auto tile_kind = [&](int t) -> int {
    const int a0 = j0 + t * TK, a1 = a0 + min(TK, cached - t * TK) - 1;     // cached keys of the tile
    if (a1 < wl) return 0;
    if (a0 >= wl) return 1;
    return 2;
  };
  const uint32_t bar0 = smem_u32(&bars[0]);
#define DBAR(i) (bar0 + 8u * (uint32_t)(i))

  // Decode steps follow one another in a stream: launched with programmatic stream
  // serialisation, the next step's CTAs may become resident as soon as all of this step's have
  // started; whatever touches global memory waits for the step in front below.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)),
                 "r"(DEC_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  const TC* vc = v_cache + (size_t)bkv * T_max * D;
  auto v_rows = [&](int t) { return min(TK, cached - t * TK); };
  // value stage s: three of its own, then the two key stages (free once all score products are done)
  auto v_stage_off = [&](int s2) -> uint32_t {
    return s2 < NVS_OWN ? OFF_V + (uint32_t)s2 * TILE_BYTES : OFF_K + (uint32_t)(s2 - NVS_OWN) * TILE_BYTES;
  };
  auto issue_v = [&](int t) {
    const uint32_t bytes = (uint32_t)v_rows(t) * D * 2u;
    const uint32_t bar = DBAR(BAR_V0 + (t % NVS));
    tc::mbar_expect_tx(bar, bytes);
    bulk_load(base + v_stage_off(t % NVS), vc + (size_t)(j0 + t * TK) * D, bytes, bar);
  };

  auto issue_k = [&](int t) {
    tc::mbar_expect_tx(DBAR(BAR_K0 + (t % NKS)), TILE_BYTES);
    const CUtensorMap* src = (KEY && tile_kind(t) != 1) ? &tm_h : &tm_k;
    tc::tma_load_3d(base + OFF_K + (t % NKS) * TILE_BYTES, src, DBAR(BAR_K0 + (t % NKS)), 0, j0 + t * TK, bkv);
  };
  // the step in front (or the prefill) has written the carried reference, the cache rows and
  // the slice tickets this step reads
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (tid == 0) {
    for (int i = 0; i < DEC_NUM_BARS; ++i) tc::mbar_init(DBAR(i), i >= BAR_VFREE0 ? (uint32_t)DNW : 1u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    tc::fence_proxy_async();
    s_fail = 0;
    // the first key and value tiles are on their way while the threshold step below runs
    if (n_tiles > 0) issue_k(0);
    for (int t = 1; t < NKS && t < n_tiles; ++t) issue_k(t);
    for (int t = 0; t < NVS_OWN && t < n_tiles; ++t) issue_v(t);
  }

  // ---- 1. threshold step (Eq. 2-3) and Qcat
  // operand row r, channel c of Qcat (128-byte swizzle)
  auto qc_off = [&](int r, int c) -> uint32_t {
    return (uint32_t)r * 128u + ((((uint32_t)c >> 3) ^ ((uint32_t)r & 7u)) << 4) + ((uint32_t)c & 7u) * 2u;
  };
  constexpr int QROWS = KEY ? G : 2 * G;     // operand rows in use
  int fired_total = 0;
  if constexpr (!KEY) {
    // the new query rows against the carried reference queries
    for (int e0 = 0; e0 < G * D; e0 += DNT) {
      const int e = e0 + tid;
      bool fire = false;
      if (e < G * D) {
        const int hh = e / D, c = e - hh * D;
        const size_t o = ((size_t)b * H + kvh * G + hh) * D + c;
        const TC xb = q_new[o];
        const float x = to_f32(xb);
        const float old = qhat_in[o];
        fire = fabsf(__fsub_rn(x, old)) > theta;
        const float nq = fire ? x : old;
        q_s[e] = x;
        qh_s[e] = nq;
        if (split == 0) qhat_out[o] = nq;
        // operand rows: hh = new reference (exactly bf16), G + hh = new query
        *reinterpret_cast<uint16_t*>(sm + OFF_QC + qc_off(hh, c)) = (uint16_t)(__float_as_uint(nq) >> 16);
        *reinterpret_cast<TC*>(sm + OFF_QC + qc_off(G + hh, c)) = xb;
      }
      fired_total += __syncthreads_count(fire);
    }
    if (split == 0 && tid == 0) {
      const int n_in = min(L, max(W, 0));
      const int n_out = L - n_in;
      atomicAdd(&counters[CNT_DECODE_NNZ], (unsigned long long)fired_total);
      atomicAdd(&counters[CNT_DECODE_ELEMS], (unsigned long long)G * D);
      atomicAdd(&counters[CNT_DECODE_MACS_DONE],
                (unsigned long long)n_in * D * G + (unsigned long long)n_out * fired_total);
      atomicAdd(&counters[CNT_DECODE_MACS_DENSE], (unsigned long long)L * D * G);
    }
  } else {
    // the new key against the carried reference key (qh_s[0..D) = k_hat(n)); the query rows are
    // the operand
    bool fire = false;
    if (tid < D) {
      const size_t o = (size_t)bkv * D + tid;
      const float x = to_f32(k_new[o]);
      const float old = qhat_in[o];
      fire = fabsf(__fsub_rn(x, old)) > theta;
      const float nk = fire ? x : old;
      qh_s[tid] = nk;                        // exactly bf16: a copy of an input element (or 0)
      if (split == 0) qhat_out[o] = nk;
    }
    for (int e = tid; e < G * D; e += DNT) {
      const int hh = e / D, c = e - hh * D;
      const TC xb = q_new[((size_t)b * H + kvh * G + hh) * D + c];
      q_s[e] = to_f32(xb);
      *reinterpret_cast<TC*>(sm + OFF_QC + qc_off(hh, c)) = xb;
    }
    fired_total = __syncthreads_count(fire);
    // multiply-adds of this step for the slice's keys: d inside the window, nnz(Delta k_j) outside
    {
      unsigned long long done = 0;
      for (int jj = tid; jj < len; jj += DNT) {
        const int j = j0 + jj;
        const int nz = (j == n) ? fired_total : (int)row_nnz[(size_t)bkv * T_max + j];
        done += (n - j < W) ? (unsigned long long)D : (unsigned long long)nz;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) done += __shfl_down_sync(0xffffffffu, done, o);
      if (lane == 0 && done) atomicAdd(&counters[CNT_DECODE_MACS_DONE], done * G);
    }
    if (split == 0 && tid == 0) {
      atomicAdd(&counters[CNT_DECODE_NNZ], (unsigned long long)fired_total);
      atomicAdd(&counters[CNT_DECODE_ELEMS], (unsigned long long)D);
      atomicAdd(&counters[CNT_DECODE_MACS_DENSE], (unsigned long long)L * D * G);
    }
  }
  for (int e = tid; e < (16 - QROWS) * D; e += DNT) {       // unused operand rows: zeros
    const int r = QROWS + e / D, c = e % D;
    *reinterpret_cast<uint16_t*>(sm + OFF_QC + qc_off(r, c)) = 0;
  }
  if (tid < 8) { st_s[tid] = -INFINITY; st_s[8 + tid] = 0.0f; }
  tc::fence_proxy_async();           // Qcat was written through the generic proxy
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem = s_tmem;

  // ---- 2. key tiles through the tensor cores (warp 0: lane 0 issues the copies and products)
  if (warp == 0 && n_tiles > 0) {
    const uint32_t IDESC = tc::make_idesc(SCOL, 0);
    const TC* kc = k_cache + (size_t)bkv * T_max * D;
    for (int t = 0; t < n_tiles; ++t) {
      if (!mbar_wait(DBAR(BAR_K0 + (t % NKS)), (t / NKS) & 1)) s_fail = 1;
      const uint32_t kb = base + OFF_K + (t % NKS) * TILE_BYTES;
      if (KEY && tile_kind(t) == 2) {
        // the window's edge falls into this tile: its window rows become the original keys
        const int r0 = wl - (j0 + t * TK), r1 = min(TK, cached - t * TK);
        for (int e = lane; e < (r1 - r0) * 8; e += 32) {
          const int r = r0 + (e >> 3), ch = e & 7;
          *reinterpret_cast<uint4*>(sm + OFF_K + (t % NKS) * TILE_BYTES + (uint32_t)r * 128u +
                                    (((uint32_t)ch ^ ((uint32_t)r & 7u)) << 4)) =
              *reinterpret_cast<const uint4*>(kc + (size_t)(j0 + t * TK + r) * D + ch * 8);
        }
        tc::fence_proxy_async();
      }
      __syncwarp();
      if (lane == 0) {
        tc::tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc::tc_mma(tmem + SCOL * t, tc::make_desc(kb + ks * 32, 16, 1024),
                     tc::make_desc(base + OFF_QC + ks * 32, 16, 1024), IDESC, ks > 0 ? 1u : 0u);
        if (t + NKS < n_tiles) {
          // the stage is free once these products are done: then refill it
          tc::tc_commit(DBAR(BAR_KFREE0 + (t % NKS)));
          if (!mbar_wait(DBAR(BAR_KFREE0 + (t % NKS)), (t / NKS) & 1)) s_fail = 1;
          issue_k(t + NKS);
        }
      }
      __syncwarp();
    }
    if (lane == 0) {
      tc::tc_commit(DBAR(BAR_S));
      // the key stages turn into value stages as soon as the last product has read them
      if (n_tiles > NVS_OWN) {
        if (!mbar_wait(DBAR(BAR_S), 0)) s_fail = 1;
        for (int t = NVS_OWN; t < NVS && t < n_tiles; ++t) issue_v(t);
      }
    }
    __syncwarp();
  }

  // the key and value that arrive with this step: into the cache, scored on the FP32 pipes
  // (warp 0; results in p_s row MAXT*TK below)
  float new_s[G];         // scaled hybrid score of the new key, per head (warp 0, all lanes)
#pragma unroll
  for (int hh = 0; hh < G; ++hh) new_s[hh] = -INFINITY;
  if (has_new && DELTA_IN(n, T_max, counters)) {
    for (int e = tid; e < D; e += DNT) {
      k_cache[((size_t)bkv * T_max + n) * D + e] = k_new[(size_t)bkv * D + e];
      v_cache[((size_t)bkv * T_max + n) * D + e] = v_new[(size_t)bkv * D + e];
      if constexpr (KEY)      // k_hat(n): exactly bf16
        reinterpret_cast<uint16_t*>(khat_cache)[((size_t)bkv * T_max + n) * D + e] =
            (uint16_t)(__float_as_uint(qh_s[e]) >> 16);
    }
    if (KEY && tid == 0) row_nnz[(size_t)bkv * T_max + n] = (uint16_t)fired_total;
    if (warp == 0) {
      const float k0 = to_f32(k_new[(size_t)bkv * D + lane]), k1 = to_f32(k_new[(size_t)bkv * D + 32 + lane]);
      if constexpr (!KEY) {
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
          float pr = fmaf(qh_s[hh * D + lane], k0, qh_s[hh * D + 32 + lane] * k1);
          float pq = fmaf(q_s[hh * D + lane], k0, q_s[hh * D + 32 + lane] * k1);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            pr += __shfl_xor_sync(0xffffffffu, pr, o);
            pq += __shfl_xor_sync(0xffffffffu, pq, o);
          }
          if (lane == 0) R[((size_t)b * H + kvh * G + hh) * T_max + n] = pr;     // R[n] = q_hat . k_new
          new_s[hh] = ((W > 0) ? pq : pr) * scale_log2e;                          // the new key is inside any window
        }
      } else {
        // the new key is inside any window W_d >= 1; with W_d = 0 even it is scored by its reference
        const float r0 = (W > 0) ? k0 : qh_s[lane], r1 = (W > 0) ? k1 : qh_s[32 + lane];
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
          float pq = fmaf(q_s[hh * D + lane], r0, q_s[hh * D + 32 + lane] * r1);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) pq += __shfl_xor_sync(0xffffffffu, pq, o);
          new_s[hh] = pq * scale_log2e;
        }
      }
    }
  }

  // ---- 3. one softmax over the slice.  Warp w reads tensor-memory lanes 32 (w % 4) ..; warps
  // 0..3 take the even tiles, warps 4..7 the odd ones.
  if (n_tiles > 0) {
    if (!mbar_wait(DBAR(BAR_S), 0)) s_fail = 1;
    tc::tc_fence_after();
  }
  constexpr int TPW = (MAXT + 1) / 2;     // tiles per warp at most
  float sv[TPW][G];                       // scaled hybrid scores of this thread's keys
  float mx[G];
#pragma unroll
  for (int hh = 0; hh < G; ++hh) mx[hh] = new_s[hh];
  const uint32_t lane_sel = (uint32_t)(32 * (warp & 3)) << 16;
  float* Rg = KEY ? nullptr : R + ((size_t)b * H + kvh * G) * T_max;
#pragma unroll
  for (int u = 0; u < TPW; ++u) {
    const int t = 2 * u + (warp >> 2);
#pragma unroll
    for (int hh = 0; hh < G; ++hh) sv[u][hh] = -INFINITY;
    if (t < n_tiles) {                    // warp-uniform
      float v[16];
      tc::tc_ld16(tmem + SCOL * t + lane_sel, v);
      const int jj = t * TK + 32 * (warp & 3) + lane;       // key within the slice
      const int j = j0 + jj;
      if (jj < cached) {
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
          float s;
          if constexpr (KEY) {
            s = v[hh] * scale_log2e;                          // the tile's rows already are the hybrid keys
          } else {
            if (DELTA_IN(j, T_max, counters)) Rg[(size_t)hh * T_max + j] = v[hh];   // R[j] = q_hat . k_j
            s = ((n - j < W) ? v[G + hh] : v[hh]) * scale_log2e;
          }
          sv[u][hh] = s;
          mx[hh] = fmaxf(mx[hh], s);
        }
      }
    }
  }
  tc::tc_fence_before();
#pragma unroll
  for (int hh = 0; hh < G; ++hh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], o));
    if (lane == 0) wgt[warp * 2 * G + hh] = mx[hh];
  }
  __syncthreads();
  float sum[G];
#pragma unroll
  for (int hh = 0; hh < G; ++hh) {
    float m = wgt[hh];
#pragma unroll
    for (int w2 = 1; w2 < DNW; ++w2) m = fmaxf(m, wgt[w2 * 2 * G + hh]);
    mx[hh] = m;                           // the slice's maximum (never -inf: the slice has a key)
    sum[hh] = 0.0f;
  }
#pragma unroll
  for (int u = 0; u < TPW; ++u) {
    const int t = 2 * u + (warp >> 2);
    if (t < n_tiles) {
      const int jj = t * TK + 32 * (warp & 3) + lane;
#pragma unroll
      for (int hh = 0; hh < G; ++hh) {
        const float p = exp2f(sv[u][hh] - mx[hh]);          // 0 for keys past the cached rows
        sum[hh] += p;
        p_s[(size_t)jj * G + hh] = p;
      }
    }
  }
  if (warp == 0 && has_new) {
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
      const float p = exp2f(new_s[hh] - mx[hh]);
      if (lane == 0) { sum[hh] += p; p_s[(size_t)(MAXT * TK) * G + hh] = p; }
    }
  }
#pragma unroll
  for (int hh = 0; hh < G; ++hh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum[hh] += __shfl_xor_sync(0xffffffffu, sum[hh], o);
    if (lane == 0) wgt[warp * 2 * G + G + hh] = sum[hh];
  }
  __syncthreads();
  if (tid < G) {
    float s = 0.0f;
    for (int w2 = 0; w2 < DNW; ++w2) s += wgt[w2 * 2 * G + G + tid];
    st_s[tid] = mx[tid];
    st_s[8 + tid] = s;
  }

  // ---- 4. P.V: value tiles through a two-stage ring; lane (l % 8) holds 8 channels, l / 8 the key
  const int sub = lane / LPK;
  const int c0 = (lane % LPK) * 8;
  float acc[G][8];
#pragma unroll
  for (int hh = 0; hh < G; ++hh)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[hh][e] = 0.0f;
  for (int t = 0; t < n_tiles; ++t) {
    const int stg = t % NVS;
    const uint32_t par = (uint32_t)(t / NVS) & 1u;
    if (!mbar_wait(DBAR(BAR_V0 + stg), par)) s_fail = 1;
    const TC* vt = reinterpret_cast<const TC*>(sm + v_stage_off(stg));
    const int rows = v_rows(t);
    for (int jb = warp * KPW; jb < rows; jb += DNW * KPW) {
      const int jj = jb + sub;
      if (jj < rows) {
        float vv[8];
        load8(vt + (size_t)jj * D + c0, vv);
        float pr[G];
        load_probs<G>(p_s + (size_t)(t * TK + jj) * G, pr);
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
          const float2 p2 = make_float2(pr[hh], pr[hh]);
#pragma unroll
          for (int e = 0; e < 8; e += 2) {
            const float2 a = tc::ffma2(p2, make_float2(vv[e], vv[e + 1]), make_float2(acc[hh][e], acc[hh][e + 1]));
            acc[hh][e] = a.x;
            acc[hh][e + 1] = a.y;
          }
        }
      }
    }
    // the warps run through the ring at their own pace: a stage is refilled (by the last warp)
    // once all of them have released it
    __syncwarp();
    if (lane == 0) tc::mbar_arrive(DBAR(BAR_VFREE0 + stg));
    if (warp == DNW - 1 && t + NVS < n_tiles) {
      // the whole warp waits (a lone lane polling beside its working warp would make the warp
      // run both paths in turns)
      if (!mbar_wait(DBAR(BAR_VFREE0 + stg), par)) s_fail = 1;
      if (lane == 0) issue_v(t + NVS);
      __syncwarp();
    }
  }
  if (has_new && warp == 0 && sub == 0) {
    float vv[8];
    load8(v_new + (size_t)bkv * D + c0, vv);
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
      const float p = p_s[(size_t)(MAXT * TK) * G + hh];
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[hh][e] = fmaf(p, vv[e], acc[hh][e]);
    }
  }
  __syncthreads();
  if (warp == 0) {
    tc::tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(DEC_TMEM_COLS) : "memory");
  }
#undef DBAR
  decode_merge_slices<TC, D, G>(acc, red, wgt, st_s, &s_last, s_fail, partial, ticket, counters, out, split, bkv,
                                nsplit, b, H, kvh);
}

// Slice geometry of a step at position n: one wave of two CTAs per SM, no slice shorter than a
// tile or longer than MAXT tiles.
static void decode_tc_slices(const Shape& s, int n, int* nsplit_out, int* chunk_out) {
  const int L = n + 1;
  const int bkv = s.B * s.H_kv;
  int nsplit = kTcTargetCtas / bkv;
  if (nsplit > kMaxDecodeSplits) nsplit = kMaxDecodeSplits;
  const int max_by_len = (L + TK - 1) / TK;    // no slice shorter than a tile (batch 1, 2049 keys: 8.9 us per
                                               // step with 128-key slices, 9.4 with 256, 10.4 with 64)
  if (nsplit > max_by_len) nsplit = max_by_len;
  const int min_by_len = (L + MAXT * TK - 1) / (MAXT * TK);
  if (nsplit < min_by_len) nsplit = min_by_len;
  if (nsplit < 1) nsplit = 1;
  int chunk = (L + nsplit - 1) / nsplit;
  chunk = (chunk + 31) / 32 * 32;
  *nsplit_out = (L + chunk - 1) / chunk;
  *chunk_out = chunk;
}

bool decode_tc_applies(const Shape& s, int dtype, int n) {
  if (s.d != TCD || dtype != DELTA_BF16 || tc::encode_fn() == nullptr) return false;
  if (n < 0) return true;      // shape and type only
  int nsplit, chunk;
  decode_tc_slices(s, n, &nsplit, &chunk);
  return chunk <= MAXT * TK && nsplit <= kMaxDecodeSplits;
}

// The tensor map of a [B*H_kv, T_max, 64] bf16 cache, encoded once per cache pointer.
static const CUtensorMap* cached_map(DecodeTmapCache* cache, const void* ptr, const Shape& s) {
  static_assert(sizeof(CUtensorMap) <= sizeof(cache->map), "tensor-map cache");
  CUtensorMap* m = reinterpret_cast<CUtensorMap*>(cache->map);
  if (cache->ptr != ptr) {
    if (!tc::encode3(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, ptr, TCD, (uint64_t)s.T_max, (uint64_t)s.B * s.H_kv,
                     TCD * 2, (uint64_t)s.T_max * TCD * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B))
      return nullptr;
    cache->ptr = ptr;
  }
  return m;
}

template <bool KEY>
static cudaError_t launch_tc(const Shape& s, const Workspace& w, const void* q_new, const void* k_new,
                             const void* v_new, void* k_cache, void* v_cache, void* out, int n, float theta,
                             int window, int qhat_sel, DecodeTmapCache* cache_k, DecodeTmapCache* cache_h,
                             cudaStream_t st) {
  const int bkv = s.B * s.H_kv;
  int nsplit, chunk;
  decode_tc_slices(s, n, &nsplit, &chunk);
  if (nsplit > kMaxDecodeSplits || chunk > MAXT * TK) return cudaErrorInvalidValue;
  const CUtensorMap* tkp = cached_map(cache_k, k_cache, s);
  const CUtensorMap* thp = KEY ? cached_map(cache_h, w.qhat_rows, s) : tkp;
  if (!tkp || !thp) return cudaErrorInvalidValue;
  const CUtensorMap& tk = *tkp;
  const CUtensorMap& th = *thp;
  const float scale_log2e = 1.4426950408889634f / sqrtf((float)s.d);
  const int G = s.g();
  const dim3 grid(nsplit, bkv);
  const size_t smem = 1024 + (size_t)(NKS + NVS_OWN) * TILE_BYTES + 2048 +
                      ((size_t)2 * G * TCD + (size_t)G * kMaxDecodeSplits + (size_t)(MAXT * TK + 1) * G + 24) * 4;
  cudaError_t err = cudaSuccess;
  using TC = __nv_bfloat16;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(DNT);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
#define LAUNCH(GG)                                                                               \
  do {                                                                                           \
    auto kern = decode_step_tc_kernel<GG, KEY>;                                                  \
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);    \
    if (err != cudaSuccess) return err;                                                          \
    /* two CTAs per SM need the largest shared-memory carve-out */                               \
    err = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout,             \
                               (int)cudaSharedmemCarveoutMaxShared);                             \
    if (err != cudaSuccess) return err;                                                          \
    err = cudaLaunchKernelEx(&cfg, kern, tk, th, (const TC*)q_new, (const TC*)k_new, (const TC*)v_new,     \
                             (TC*)k_cache, (TC*)v_cache, w.qhat_rows, w.row_nnz, (TC*)out,                 \
                             (const float*)w.qhat[qhat_sel], w.qhat[qhat_sel ^ 1], w.R, w.dec_partial,     \
                             w.dec_ticket, w.counters, n, s.T_max, s.H, chunk, nsplit, theta, window,      \
                             scale_log2e);                                                                 \
  } while (0)
  switch (G) {
    case 1: LAUNCH(1); break;
    case 2: LAUNCH(2); break;
    case 4: LAUNCH(4); break;
    case 8: LAUNCH(8); break;
    default: return cudaErrorInvalidValue;
  }
#undef LAUNCH
  count_launch();
  return err != cudaSuccess ? err : cudaGetLastError();
}

cudaError_t launch_decode_step_tc(const Shape& s, const Workspace& w, const void* q_new, const void* k_new,
                                  const void* v_new, void* k_cache, void* v_cache, void* out, int n, float theta,
                                  int window, int qhat_sel, DecodeTmapCache* cache, cudaStream_t st) {
  return launch_tc<false>(s, w, q_new, k_new, v_new, k_cache, v_cache, out, n, theta, window, qhat_sel, cache,
                          nullptr, st);
}

cudaError_t launch_decode_step_key_tc(const Shape& s, const Workspace& w, const void* q_new, const void* k_new,
                                      const void* v_new, void* k_cache, void* v_cache, void* out, int n,
                                      float theta, int window, int qhat_sel, DecodeTmapCache* cache_k,
                                      DecodeTmapCache* cache_h, cudaStream_t st) {
  if (!w.qhat_rows) return cudaErrorNotSupported;
  return launch_tc<true>(s, w, q_new, k_new, v_new, k_cache, v_cache, out, n, theta, window, qhat_sel, cache_k,
                         cache_h, st);
}

}  // namespace delta
