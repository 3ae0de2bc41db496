// K3 (key deltas) -- one decode step of strategy (3) (Section III-A, adopted by the paper;
// Section III-B "Decoding Stage", Section III-C).  The carried state is the reference key of
// every KV head; the library keeps, next to the caller's K cache, a cache of reference-key rows
// k_hat(j) = sum over s <= j of Delta k(s) (Eq. 3, telescoped Eq. 4).  A step
//   0. thresholds k_new against the carried reference key (Eq. 2-3), appends k_new / v_new to
//      the caller's caches and k_hat(n) to the reference-key cache,
//   1. scores every key j <= n for the g query heads of the KV head: q_new.k_j for the W_d most
//      recent keys, q_new.k_hat(j) for the older ones,
//   2. online softmax and P.V exactly as in the query-delta step.
// Same grid, tiling, bulk-copy ring and slice merge as decode_step_kernel; the tile streamed
// through the ring is the reference-key cache, and the rows of the window are replaced in
// shared memory by the original keys.
#include "decode_common.cuh"

namespace delta {

template <int D, int G>
__global__ void __launch_bounds__(DNT) decode_step_key_kernel(
    const __nv_bfloat16* __restrict__ q_new, const __nv_bfloat16* __restrict__ k_new,
    const __nv_bfloat16* __restrict__ v_new, __nv_bfloat16* __restrict__ k_cache,
    __nv_bfloat16* __restrict__ v_cache, __nv_bfloat16* __restrict__ khat_cache,
    __nv_bfloat16* __restrict__ out, const float* __restrict__ khat_in, float* __restrict__ khat_out,
    uint16_t* __restrict__ row_nnz, float* __restrict__ partial, uint32_t* __restrict__ ticket,
    unsigned long long* __restrict__ counters, int n, int T_max, int H, int chunk, int nsplit,
    float theta, int W, float scale_log2e) {
  using TC = __nv_bfloat16;
  constexpr int LPK = D / 8;
  constexpr int KPW = 32 / LPK;
  constexpr int ROWB = D * (int)sizeof(TC);
  constexpr int TK = TILE_BYTES / ROWB;
  extern __shared__ __align__(128) unsigned char dsm_raw[];
  TC* sK = reinterpret_cast<TC*>(dsm_raw);                         // [2][TK][D]
  TC* sV = reinterpret_cast<TC*>(dsm_raw + 2 * TILE_BYTES);        // [2][TK][D]
  float* q_s = reinterpret_cast<float*>(dsm_raw + 4 * TILE_BYTES); // [G][D]
  float* red = q_s + G * D;      // [DNW][G][D]
  float* sc = red + DNW * G * D; // [G][max(TK, kMaxDecodeSplits)] scaled scores, then probabilities
  constexpr int SC_LD = TK > kMaxDecodeSplits ? TK : kMaxDecodeSplits;
  float* st_s = sc + G * SC_LD;  // [3][8]
  TC* khat_new_s = reinterpret_cast<TC*>(st_s + 24);   // [D] reference-key row of this step
  __shared__ __align__(8) unsigned long long bars[2];
  __shared__ int s_last, s_fail;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.x, bkv = blockIdx.y;
  const int H_kv = H / G;
  const int b = bkv / H_kv, kvh = bkv - b * H_kv;
  const int L = n + 1;
  const int j0 = split * chunk;
  const int len = max(0, min(chunk, L - j0));
  const int n_tiles = (len + TK - 1) / TK;
  const TC* hc = khat_cache + (size_t)bkv * T_max * D;
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

  auto tile_cached_rows = [&](int t) { return max(0, min(min(TK, len - t * TK), n - (j0 + t * TK))); };
  auto issue_tile = [&](int t) {
    const int rows = tile_cached_rows(t);
    const uint32_t bar = bar0 + 8 * (t & 1);
    const uint32_t bytes = (uint32_t)rows * ROWB;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(2 * bytes) : "memory");
    if (bytes) {
      bulk_load(smem_u32(sK) + (t & 1) * TILE_BYTES, hc + (size_t)(j0 + t * TK) * D, bytes, bar);
      bulk_load(smem_u32(sV) + (t & 1) * TILE_BYTES, vc + (size_t)(j0 + t * TK) * D, bytes, bar);
    }
  };
  if (tid == 0) {
    if (n_tiles > 0) issue_tile(0);
    if (n_tiles > 1) issue_tile(1);
  }

  // ---- 0. delta of the new key against the carried reference key (Eq. 2-3); query rows
  bool fire = false;
  if (tid < D) {
    const size_t o = (size_t)bkv * D + tid;
    const float x = to_f32(k_new[o]);
    const float old = khat_in[o];
    fire = fabsf(__fsub_rn(x, old)) > theta;
    const float nk = fire ? x : old;
    khat_new_s[tid] = __float2bfloat16_rn(nk);       // exact: a copy of a bf16 input element (or 0)
    if (split == 0) khat_out[o] = nk;
  }
  for (int e = tid; e < G * D; e += DNT) {
    const int hh = e / D, c = e - hh * D;
    q_s[e] = to_f32(q_new[((size_t)b * H + kvh * G + hh) * D + c]);
  }
  const int fired_total = __syncthreads_count(fire);

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

  const int sub = lane / LPK;
  const int c0 = (lane % LPK) * 8;
  float acc[G][8], qr[G][8];
#pragma unroll
  for (int hh = 0; hh < G; ++hh)
#pragma unroll
    for (int e = 0; e < 8; ++e) { acc[hh][e] = 0.0f; qr[hh][e] = q_s[hh * D + c0 + e]; }

  for (int t = 0; t < n_tiles; ++t) {
    const int tj0 = j0 + t * TK;
    const int rows = min(TK, len - t * TK);
    TC* kt = sK + (size_t)(t & 1) * TK * D;
    TC* vt = sV + (size_t)(t & 1) * TK * D;
    const bool has_new = (n >= tj0) && (n < tj0 + rows);
    const int w_lo = max(tj0, n - W + 1);            // first key of the window inside this tile
    const int w_hi = min(tj0 + rows, n);             // cached window keys: [w_lo, w_hi)
    if (!mbar_wait(bar0 + 8 * (t & 1), (t >> 1) & 1)) s_fail = 1;
    if (has_new || w_lo < w_hi) {
      // original keys of the window replace the reference rows of the tile
      for (int e = tid; e < (w_hi - w_lo) * (D / 8); e += DNT) {
        const int r = e / (D / 8), cq = (e - r * (D / 8)) * 8;
        *reinterpret_cast<uint4*>(kt + (size_t)(w_lo - tj0 + r) * D + cq) =
            *reinterpret_cast<const uint4*>(kc + (size_t)(w_lo + r) * D + cq);
      }
      if (has_new) {
        const int jn = n - tj0;
        for (int e = tid; e < D; e += DNT) {
          const TC kv = k_new[(size_t)bkv * D + e], vv = v_new[(size_t)bkv * D + e];
          kt[jn * D + e] = (W > 0) ? kv : khat_new_s[e];     // the new key is inside any window W_d >= 1
          vt[jn * D + e] = vv;
          k_cache[((size_t)bkv * T_max + n) * D + e] = kv;
          v_cache[((size_t)bkv * T_max + n) * D + e] = vv;
          khat_cache[((size_t)bkv * T_max + n) * D + e] = khat_new_s[e];
        }
        if (tid == 0) row_nnz[(size_t)bkv * T_max + n] = (uint16_t)fired_total;
      }
      __syncthreads();
    }

    // ---- 1. scaled scores of this tile
    for (int jb = warp * KPW; jb < rows; jb += DNW * KPW) {
      const int jj = jb + sub;
      const bool valid = jj < rows;
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
        for (int e = 0; e < 8; ++e) pd[hh] = fmaf(qr[hh][e], kv[e], pd[hh]);
      }
#pragma unroll
      for (int hh = 0; hh < G; ++hh) {
#pragma unroll
        for (int o = LPK / 2; o > 0; o >>= 1) pd[hh] += __shfl_xor_sync(0xffffffffu, pd[hh], o);
        if (valid && (lane % LPK) == 0) sc[hh * SC_LD + jj] = pd[hh] * scale_log2e;
      }
    }
    __syncthreads();

    // ---- 2. online softmax over the tile (warp hh serves head hh)
    if (warp < G) {
      float* s = sc + warp * SC_LD;
      float mx = -INFINITY;
      for (int jj = lane; jj < rows; jj += 32) mx = fmaxf(mx, s[jj]);
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

    // ---- 3. P.V over the tile
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
          const float p = sc[hh * SC_LD + jj];
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[hh][e] = fmaf(p, vv[e], acc[hh][e]);
        }
      }
    }
    __syncthreads();
    if (tid == 0 && t + 2 < n_tiles) issue_tile(t + 2);
  }

  decode_merge_slices<TC, D, G>(acc, red, sc, st_s, &s_last, s_fail, partial, ticket, counters, out,
                                split, bkv, nsplit, b, H, kvh);
}

cudaError_t launch_decode_step_key(const Shape& s, const Workspace& w, const void* q_new,
                                   const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                   void* out, int n, float theta, int window, int qhat_sel,
                                   cudaStream_t st) {
  using TC = __nv_bfloat16;
  if (!w.qhat_rows) return cudaErrorNotSupported;
  const int L = n + 1;
  const int bkv = s.B * s.H_kv;
  const int TK = TILE_BYTES / (s.d * 2);
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
  const int sc_ld = TK > kMaxDecodeSplits ? TK : kMaxDecodeSplits;
  const dim3 grid(nsplit, bkv);
  const size_t smem = (size_t)4 * TILE_BYTES +
                      ((size_t)G * s.d + (size_t)DNW * G * s.d + (size_t)G * sc_ld + 24) * 4 + (size_t)s.d * 2;
  cudaError_t err = cudaSuccess;
#define LAUNCH(DD, GG)                                                                           \
  do {                                                                                           \
    auto kern = decode_step_key_kernel<DD, GG>;                                                  \
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);    \
    if (err != cudaSuccess) return err;                                                          \
    kern<<<grid, DNT, smem, st>>>((const TC*)q_new, (const TC*)k_new, (const TC*)v_new,          \
                                  (TC*)k_cache, (TC*)v_cache, w.qhat_rows, (TC*)out,             \
                                  w.qhat[qhat_sel], w.qhat[qhat_sel ^ 1], w.row_nnz,             \
                                  w.dec_partial, w.dec_ticket, w.counters, n, s.T_max, s.H,      \
                                  chunk, nsplit, theta, window, scale_log2e);                    \
  } while (0)
#define LAUNCH_G(DD)                                             \
  switch (G) {                                                   \
    case 1: LAUNCH(DD, 1); break;                                \
    case 2: LAUNCH(DD, 2); break;                                \
    case 4: LAUNCH(DD, 4); break;                                \
    case 8: LAUNCH(DD, 8); break;                                \
    default: return cudaErrorInvalidValue;                       \
  }
  if (s.d == 64) { LAUNCH_G(64) } else if (s.d == 128) { LAUNCH_G(128) } else return cudaErrorNotSupported;
#undef LAUNCH_G
#undef LAUNCH
  count_launch();
  return cudaGetLastError();
}

}  // namespace delta
