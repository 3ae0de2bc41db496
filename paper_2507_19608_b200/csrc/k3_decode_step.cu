// K3 -- one decode step of strategy (1) carried past prefill (Section III-A "Decoding Stage
// Considerations", Section III-B "Decoding Stage", Section III-C).  HBM-bound: one streaming
// pass over the K and V cache plus a read-modify-write of the carried score row R.
//
// Grid = (key splits, batch x KV heads).  A CTA serves the G query heads that share one KV
// head, so every cached key and value row is read once for the group, and walks its slice of
// the cache in tiles of 16 KiB of keys (and as much of values).  Tiles are contiguous in the
// cache, so one bulk asynchronous copy per tile and tensor brings them into a two-stage ring
// in shared memory while the previous tile is processed; the R entries of the tile are
// fetched with coalesced loads ahead of their use.  Per tile:
//   1. dot products of every key with the G delta vectors (Eq. 4), with the G query vectors
//      for the W_d most recent keys, and with the new references for the key that arrives now;
//   2. R[j] += dq.k_j written back coalesced (R[n] = q_hat.k_new for the new key), the
//      hybrid select, the scale;
//   3. online softmax over the tile (one warp per head);
//   4. P.V accumulated in registers.
// In front of the tiles the CTA thresholds q_new against the carried reference (Eq. 2-3) for
// its G heads; at the end it stores (max, sum, partial output) and the last CTA of a
// (batch, KV head) to finish merges the slices and writes the output rows.
#include "decode_common.cuh"

namespace delta {

template <typename TC, int D, int G>
__global__ void __launch_bounds__(DNT) decode_step_kernel(
    const TC* __restrict__ q_new, const TC* __restrict__ k_new, const TC* __restrict__ v_new,
    TC* __restrict__ k_cache, TC* __restrict__ v_cache, TC* __restrict__ out,
    const float* __restrict__ qhat_in, float* __restrict__ qhat_out, float* __restrict__ R,
    float* __restrict__ partial, uint32_t* __restrict__ ticket,
    unsigned long long* __restrict__ counters, int n, int T_max, int H, int chunk, int nsplit,
    float theta, int W, float scale_log2e) {
  constexpr int LPK = D / 8;     // lanes per key row (8 elements each)
  constexpr int KPW = 32 / LPK;  // key rows per warp iteration
  constexpr int ROWB = D * (int)sizeof(TC);
  constexpr int TK = TILE_BYTES / ROWB;              // keys per tile (128 for bf16 d=64)
  constexpr int RPT = (TK + 31) / 32;                // R entries per lane and tile (one head per warp)
  extern __shared__ __align__(128) unsigned char dsm_raw[];
  TC* sK = reinterpret_cast<TC*>(dsm_raw);                         // [2][TK][D]
  TC* sV = reinterpret_cast<TC*>(dsm_raw + 2 * TILE_BYTES);        // [2][TK][D]
  float* q_s = reinterpret_cast<float*>(dsm_raw + 4 * TILE_BYTES); // [G][D]
  float* dq_s = q_s + G * D;     // [G][D]
  float* qh_s = dq_s + G * D;    // [G][D]
  float* red = qh_s + G * D;     // [DNW][G][D]
  float* spd = red + DNW * G * D;  // [G][TK] delta dot products (new reference . k_new for the new key)
  float* spq = spd + G * TK;     // [G][TK] exact dot products (window only)
  float* sc = spq + G * TK;      // [G][TK] scaled scores, then probabilities
  float* st_s = sc + G * TK;     // [3][8]: running max, running sum, rescale of this tile
  __shared__ __align__(8) unsigned long long bars[2];
  __shared__ int s_last, s_fail;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.x, bkv = blockIdx.y;
  const int H_kv = H / G;
  const int b = bkv / H_kv, kvh = bkv - b * H_kv;
  const int L = n + 1;  // keys after this step
  const int j0 = split * chunk;
  const int len = max(0, min(chunk, L - j0));
  const int n_tiles = (len + TK - 1) / TK;
  const TC* kc = k_cache + (size_t)bkv * T_max * D;
  const TC* vc = v_cache + (size_t)bkv * T_max * D;
  const uint32_t bar0 = smem_u32(&bars[0]);

  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar0), "r"(1) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar0 + 8), "r"(1) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_fail = 0;
  }
  if (tid < 8) { st_s[tid] = -INFINITY; st_s[8 + tid] = 0.0f; st_s[16 + tid] = 1.0f; }
  __syncthreads();

  // cached rows of tile t (the row that arrives with this step is not in the cache yet)
  auto tile_cached_rows = [&](int t) { return max(0, min(min(TK, len - t * TK), n - (j0 + t * TK))); };
  auto issue_tile = [&](int t) {
    const int rows = tile_cached_rows(t);
    const uint32_t bar = bar0 + 8 * (t & 1);
    const uint32_t bytes = (uint32_t)rows * ROWB;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(2 * bytes) : "memory");
    if (bytes) {
      bulk_load(smem_u32(sK) + (t & 1) * TILE_BYTES, kc + (size_t)(j0 + t * TK) * D, bytes, bar);
      bulk_load(smem_u32(sV) + (t & 1) * TILE_BYTES, vc + (size_t)(j0 + t * TK) * D, bytes, bar);
    }
  };
  if (tid == 0) {
    if (n_tiles > 0) issue_tile(0);
    if (n_tiles > 1) issue_tile(1);
  }

  // ---- 0. delta of the new query rows against the carried reference (Eq. 2-3)
  int fired_total = 0;
  for (int e0 = 0; e0 < G * D; e0 += DNT) {
    const int e = e0 + tid;
    bool fire = false;
    if (e < G * D) {
      const int hh = e / D, c = e - hh * D;
      const size_t o = ((size_t)b * H + kvh * G + hh) * D + c;
      const float x = to_f32(q_new[o]);
      const float old = qhat_in[o];
      const float diff = __fsub_rn(x, old);
      fire = fabsf(diff) > theta;
      q_s[e] = x;
      dq_s[e] = fire ? diff : 0.0f;
      const float nq = fire ? x : old;
      qh_s[e] = nq;
      if (split == 0) qhat_out[o] = nq;
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

  const int sub = lane / LPK;       // which key row of the warp iteration
  const int c0 = (lane % LPK) * 8;  // first of this lane's 8 channels
  float acc[G][8], dqr[G][8];   // partial outputs; this lane's 8 channels of the G delta vectors
#pragma unroll
  for (int hh = 0; hh < G; ++hh)
#pragma unroll
    for (int e = 0; e < 8; ++e) { acc[hh][e] = 0.0f; dqr[hh][e] = dq_s[hh * D + c0 + e]; }
  float* Rg = R + ((size_t)b * H + kvh * G) * T_max;   // R rows of the group's heads

  for (int t = 0; t < n_tiles; ++t) {
    const int tj0 = j0 + t * TK;
    const int rows = min(TK, len - t * TK);           // keys of this tile, the new one included
    const TC* kt = sK + (size_t)(t & 1) * TK * D;
    const TC* vt = sV + (size_t)(t & 1) * TK * D;
    const bool has_new = (n >= tj0) && (n < tj0 + rows);
    const bool any_win = (n - (tj0 + rows - 1)) < W;   // some key of the tile is inside the window

    // R entries of the tile (warp hh < G holds head hh's, lane-strided): coalesced, in flight
    // while the tile's copies land
    float r_old[RPT];
#pragma unroll
    for (int u = 0; u < RPT; ++u) {
      const int jj = lane + 32 * u;
      r_old[u] = (warp < G && jj < rows && tj0 + jj < n) ? Rg[(size_t)warp * T_max + tj0 + jj] : 0.0f;
    }
    if (!mbar_wait(bar0 + 8 * (t & 1), (t >> 1) & 1)) s_fail = 1;
    if (has_new) {
      // the key and value that arrive with this step: into the tile and into the cache
      const int jn = n - tj0;
      for (int e = tid; e < D; e += DNT) {
        const TC kv = k_new[(size_t)bkv * D + e], vv = v_new[(size_t)bkv * D + e];
        const_cast<TC*>(kt)[jn * D + e] = kv;
        const_cast<TC*>(vt)[jn * D + e] = vv;
        k_cache[((size_t)bkv * T_max + n) * D + e] = kv;
        v_cache[((size_t)bkv * T_max + n) * D + e] = vv;
      }
      __syncthreads();
    }

    // ---- 1. dot products of this tile
    for (int jb = warp * KPW; jb < rows; jb += DNW * KPW) {
      const int jj = jb + sub;
      const bool valid = jj < rows;
      const bool warp_has_new = has_new && (tj0 + jb <= n) && (n < tj0 + jb + KPW);
      const bool warp_in_win = any_win && (n - (tj0 + jb + KPW - 1)) < W;
      float kv[8];
      if (valid) load8(kt + (size_t)jj * D + c0, kv);
      else {
#pragma unroll
        for (int e = 0; e < 8; ++e) kv[e] = 0.0f;
      }
      float pd[G];
#pragma unroll
      for (int hh = 0; hh < G; ++hh) {
        pd[hh] = 0.0f;
#pragma unroll
        for (int e = 0; e < 8; ++e) pd[hh] = fmaf(dqr[hh][e], kv[e], pd[hh]);
      }
      if constexpr (G == 4) {
        // four heads reduced over the key's lanes together: the value set halves as the lane
        // distance halves; lane (l & 6) of the key group ends with head ((l >> 2) & 1) * 2 + ((l >> 1) & 1)
        const int kl = lane % LPK;
        if constexpr (LPK == 16) {
#pragma unroll
          for (int hh = 0; hh < G; ++hh) pd[hh] += __shfl_xor_sync(0xffffffffu, pd[hh], 8);
        }
        const bool h4 = kl & 4, h2 = kl & 2;
        const float a0 = (h4 ? pd[2] : pd[0]) + __shfl_xor_sync(0xffffffffu, h4 ? pd[0] : pd[2], 4);
        const float a1 = (h4 ? pd[3] : pd[1]) + __shfl_xor_sync(0xffffffffu, h4 ? pd[1] : pd[3], 4);
        float z = (h2 ? a1 : a0) + __shfl_xor_sync(0xffffffffu, h2 ? a0 : a1, 2);
        z += __shfl_xor_sync(0xffffffffu, z, 1);
        if (valid && (kl & 1) == 0 && kl < 8) spd[((h4 ? 2 : 0) + (h2 ? 1 : 0)) * TK + jj] = z;
      } else {
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
#pragma unroll
          for (int o = LPK / 2; o > 0; o >>= 1) pd[hh] += __shfl_xor_sync(0xffffffffu, pd[hh], o);
          if (valid && (lane % LPK) == 0) spd[hh * TK + jj] = pd[hh];
        }
      }
      // rare paths: exact scores of the W_d most recent keys, new reference . new key
      if (warp_in_win || warp_has_new) {
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
          float pq = 0.0f, pr = 0.0f;
          const float* qh = q_s + hh * D + c0;
          const float* rh = qh_s + hh * D + c0;
#pragma unroll
          for (int e = 0; e < 8; ++e) { pq = fmaf(qh[e], kv[e], pq); pr = fmaf(rh[e], kv[e], pr); }
#pragma unroll
          for (int o = LPK / 2; o > 0; o >>= 1) {
            pq += __shfl_xor_sync(0xffffffffu, pq, o);
            pr += __shfl_xor_sync(0xffffffffu, pr, o);
          }
          if (valid && (lane % LPK) == 0) {
            spq[hh * TK + jj] = pq;
            if (tj0 + jj == n) spd[hh * TK + jj] = pr;
          }
        }
      }
    }
    __syncthreads();

    // ---- 2+3. warp hh serves head hh: R update (coalesced), hybrid select, scale, online softmax
    if (warp < G) {
      float* s = sc + warp * TK;
      float* Rh = Rg + (size_t)warp * T_max + tj0;
      float mx = -INFINITY;
#pragma unroll
      for (int u = 0; u < RPT; ++u) {
        const int jj = lane + 32 * u;
        if (jj < rows) {
          const int j = tj0 + jj;
          const float Rn = r_old[u] + spd[warp * TK + jj];     // r_old is 0 for the key that arrives now
          Rh[jj] = Rn;
          const float v = ((n - j < W) ? spq[warp * TK + jj] : Rn) * scale_log2e;
          s[jj] = v;
          mx = fmaxf(mx, v);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_old = st_s[warp];
      const float m_new = fmaxf(m_old, mx);
      float sum = 0.0f;
      for (int jj = lane; jj < rows; jj += 32) {
        const float p = exp2f(s[jj] - m_new);
        s[jj] = p;
        sum += p;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      if (lane == 0) {
        const float al = exp2f(m_old - m_new);
        st_s[warp] = m_new;
        st_s[8 + warp] = fmaf(st_s[8 + warp], al, sum);
        st_s[16 + warp] = al;
      }
    }
    __syncthreads();

    // ---- 4. P.V over the tile
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
      const float al = st_s[16 + hh];
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[hh][e] *= al;
    }
    for (int jb = warp * KPW; jb < rows; jb += DNW * KPW) {
      const int jj = jb + sub;
      if (jj < rows) {
        float vv[8];
        load8(vt + (size_t)jj * D + c0, vv);
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
          const float p = sc[hh * TK + jj];
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[hh][e] = fmaf(p, vv[e], acc[hh][e]);
        }
      }
    }
    __syncthreads();   // the tile's buffers and score arrays are free
    if (tid == 0 && t + 2 < n_tiles) issue_tile(t + 2);
  }

  decode_merge_slices<TC, D, G>(acc, red, spd, st_s, &s_last, s_fail, partial, ticket, counters, out,
                                split, bkv, nsplit, b, H, kvh);
}

cudaError_t launch_decode_step(const Shape& s, const Workspace& w, const void* q_new,
                               const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                               void* out, int n, float theta, int window, int dtype, int qhat_sel,
                               cudaStream_t st) {
  const int L = n + 1;
  const int bkv = s.B * s.H_kv;
  const int es = dtype == DELTA_F32 ? 4 : 2;
  const int TK = TILE_BYTES / (s.d * es);
  // one wave of two CTAs per SM (the ring holds 64 KiB), no slice shorter than a quarter tile
  int nsplit = kDecodeTargetCtas / bkv;
  if (nsplit > kMaxDecodeSplits) nsplit = kMaxDecodeSplits;
  const int max_by_len = (L + TK / 4 - 1) / (TK / 4);
  if (nsplit > max_by_len) nsplit = max_by_len;
  if (nsplit < 1) nsplit = 1;
  int chunk = (L + nsplit - 1) / nsplit;
  chunk = (chunk + 31) / 32 * 32;
  nsplit = (L + chunk - 1) / chunk;
  if (nsplit > kMaxDecodeSplits) return cudaErrorInvalidValue;
  const float scale_log2e = 1.4426950408889634f / sqrtf((float)s.d);
  const int G = s.g();
  const dim3 grid(nsplit, bkv);
  const size_t smem = (size_t)4 * TILE_BYTES +
                      ((size_t)3 * G * s.d + (size_t)DNW * G * s.d + (size_t)3 * G * TK + 24) * 4;
  cudaError_t err = cudaSuccess;
#define LAUNCH(TC, DD, GG)                                                                       \
  do {                                                                                           \
    auto kern = decode_step_kernel<TC, DD, GG>;                                                  \
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);    \
    if (err != cudaSuccess) return err;                                                          \
    kern<<<grid, DNT, smem, st>>>((const TC*)q_new, (const TC*)k_new, (const TC*)v_new,          \
                                  (TC*)k_cache, (TC*)v_cache, (TC*)out, w.qhat[qhat_sel],        \
                                  w.qhat[qhat_sel ^ 1], w.R, w.dec_partial, w.dec_ticket,        \
                                  w.counters, n, s.T_max, s.H, chunk, nsplit, theta, window,     \
                                  scale_log2e);                                                  \
  } while (0)
#define LAUNCH_G(TC, DD)                                         \
  switch (G) {                                                   \
    case 1: LAUNCH(TC, DD, 1); break;                            \
    case 2: LAUNCH(TC, DD, 2); break;                            \
    case 4: LAUNCH(TC, DD, 4); break;                            \
    case 8: LAUNCH(TC, DD, 8); break;                            \
    default: return cudaErrorInvalidValue;                       \
  }
  if (dtype == DELTA_F32) {
    if (s.d == 64) { LAUNCH_G(float, 64) } else { LAUNCH_G(float, 128) }
  } else {
    if (s.d == 64) { LAUNCH_G(__nv_bfloat16, 64) } else { LAUNCH_G(__nv_bfloat16, 128) }
  }
#undef LAUNCH_G
#undef LAUNCH
  count_launch();
  return cudaGetLastError();
}

}  // namespace delta
