// K3 (key deltas, compressed key-delta cache) -- Section III-A "Decoding Stage Considerations"
// and Section III-C: what decoding keeps of the keys is the delta stream, not the keys.
//
// Encoding.  Per KV head the thresholded key stream (Eq. 2-3) is kept as
//   mask    one bit per (row, channel): the element fired                     d / 8 bytes per row
//   values  for every fired element the key value that became the reference (= reference before
//           + Delta k; bf16, so the reference rows it reproduces are exact), row after row,
//           channels ascending                                                2 nnz(row) bytes
//   base    the reference key in front of every 32-row segment                2 d bytes per 32 rows
//   offset  position of every segment's first value in the pool (segments start on multiples of
//           8 values so that a tile's values are one 16-byte aligned bulk copy)
// At the delta sparsity the method reaches (about 0.6) that is roughly 46 % of the bytes of the
// dense reference-key rows the other key-delta decode kernels stream.  The last W_d original
// keys are read from the key cache rows inside the decode window.
//
// pack_keys_kernel builds the encoding behind a prefill (from the mask words and counts the
// finish kernel wrote, the keys and the reference-key rows).  decode_step_keypacked_kernel is
// decode_step_key_kernel with one change: a tile of reference-key rows is not copied from a
// dense cache but rebuilt in shared memory, thread (channel, 32-row segment) walking its rows
// from the segment's base; the step also appends the new row to the encoding.
#include "decode_common.cuh"

namespace delta {

namespace {
constexpr int SEG = 32;     // rows per segment of the encoding
__host__ __device__ inline uint32_t round8(uint32_t x) { return (x + 7u) & ~7u; }
}  // namespace

template <int D>
__global__ void __launch_bounds__(256) pack_keys_kernel(
    const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ khat_rows,
    const uint32_t* __restrict__ mask, const uint16_t* __restrict__ row_nnz, uint16_t* __restrict__ vals,
    uint32_t* __restrict__ seg_off, uint16_t* __restrict__ base, uint32_t* __restrict__ used,
    uint32_t* __restrict__ kp_mask, uint16_t* __restrict__ kp_nnz, int T, int T_max, size_t cap, int nseg_max,
    unsigned long long* __restrict__ counters) {
  constexpr int NW = D / 32;
  extern __shared__ uint32_t s_off[];          // [nseg + 1]
  const int bkv = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nseg = (T + SEG - 1) / SEG;
  const uint16_t* nz = row_nnz + (size_t)bkv * T_max;
  // segment sizes (padded to 8 values), then their running sum
  for (int s = tid; s < nseg; s += 256) {
    uint32_t sum = 0;
    for (int r = 0; r < SEG && s * SEG + r < T; ++r) sum += nz[s * SEG + r];
    s_off[s + 1] = sum;
  }
  __syncthreads();
  if (tid == 0) {
    uint32_t run = 0;
    s_off[0] = 0;
    for (int s = 0; s < nseg; ++s) {
      const uint32_t sz = s_off[s + 1];
      s_off[s + 1] = run + sz;                  // exact end of segment s
      // the next segment starts on a multiple of 8; the last one leaves the exact end
      if (s + 1 < nseg) { run = round8(run + sz); }
      else run += sz;
    }
    used[bkv] = run;
  }
  __syncthreads();
  uint32_t* so = seg_off + (size_t)bkv * (nseg_max + 1);
  // start of segment s: the exact end of s-1 rounded up
  for (int s = tid; s <= nseg; s += 256) so[s] = (s == 0) ? 0u : (s < nseg ? round8(s_off[s]) : s_off[s]);
  const __nv_bfloat16* kp = k + (size_t)bkv * T_max * D;
  const uint32_t* mk = mask + (size_t)bkv * T_max * NW;
  // the encoding's own copy of mask words and counts: per-head stride a multiple of 32 rows, so
  // that every tile of it starts on a 16-byte boundary (bulk copies)
  for (int e = tid; e < T * NW; e += 256) kp_mask[(size_t)bkv * nseg_max * SEG * NW + e] = mk[e];
  for (int e = tid; e < T; e += 256) kp_nnz[(size_t)bkv * nseg_max * SEG + e] = nz[e];
  uint16_t* vp = vals + (size_t)bkv * cap;
  for (int s = warp; s < nseg; s += 8) {
    // reference in front of the segment
    for (int c = lane; c < D; c += 32)
      base[((size_t)bkv * nseg_max + s) * D + c] =
          (s == 0) ? (uint16_t)0
                   : reinterpret_cast<const uint16_t*>(khat_rows)[((size_t)bkv * T_max + s * SEG - 1) * D + c];
    uint32_t off = (s == 0) ? 0u : round8(s_off[s]);
    for (int r = 0; r < SEG && s * SEG + r < T; ++r) {
      const int row = s * SEG + r;
      uint32_t below = 0;
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        const uint32_t word = mk[(size_t)row * NW + w];
        if (((word >> lane) & 1u) && DELTA_IN(off + below + __popc(word & ((1u << lane) - 1u)), cap, counters))
          vp[off + below + __popc(word & ((1u << lane) - 1u))] =
              reinterpret_cast<const uint16_t*>(kp)[(size_t)row * D + w * 32 + lane];
        below += __popc(word);
      }
      off += below;
    }
  }
}

template <int D, int G>
__global__ void __launch_bounds__(DNT) decode_step_keypacked_kernel(
    const __nv_bfloat16* __restrict__ q_new, const __nv_bfloat16* __restrict__ k_new,
    const __nv_bfloat16* __restrict__ v_new, __nv_bfloat16* __restrict__ k_cache,
    __nv_bfloat16* __restrict__ v_cache, __nv_bfloat16* __restrict__ out, const float* __restrict__ khat_in,
    float* __restrict__ khat_out, uint16_t* __restrict__ row_nnz, uint32_t* __restrict__ mask,
    uint32_t* __restrict__ kp_mask, uint16_t* __restrict__ kp_nnz, uint16_t* __restrict__ vals, uint32_t* __restrict__ seg_off, uint16_t* __restrict__ base_snap,
    uint32_t* __restrict__ used, float* __restrict__ partial, uint32_t* __restrict__ ticket,
    unsigned long long* __restrict__ counters, int n, int T_max, int H, int chunk, int nsplit, float theta, int W,
    float scale_log2e, size_t cap, int nseg_max) {
  using TC = __nv_bfloat16;
  constexpr int LPK = D / 8;
  constexpr int KPW = 32 / LPK;
  constexpr int ROWB = D * (int)sizeof(TC);
  constexpr int TK = TILE_BYTES / ROWB;          // 128 rows (d = 64), 64 rows (d = 128)
  constexpr int NW = D / 32;
  constexpr int SPT = TK / SEG;                  // segments per tile; D * SPT == DNT threads rebuild a tile
  static_assert(D * SPT == DNT, "one thread per (channel, segment) of a tile");
  constexpr int VAL_BYTES = TILE_BYTES + 64;     // a tile's values: at most TK * D, plus segment padding
  constexpr int MASK_BYTES = TK * NW * 4, NNZ_BYTES = TK * 2, BASE_BYTES = SPT * D * 2;
  constexpr int STAGE_BYTES = TILE_BYTES + VAL_BYTES + MASK_BYTES + NNZ_BYTES + BASE_BYTES;
  extern __shared__ __align__(128) unsigned char dsm_raw[];
  TC* sK = reinterpret_cast<TC*>(dsm_raw);                         // [2][TK][D]   rebuilt reference-key tiles
  unsigned char* sStage = dsm_raw + 2 * TILE_BYTES;                // [2] { values, masks, counts, bases, V tile }
  float* q_s = reinterpret_cast<float*>(sStage + 2 * STAGE_BYTES); // [G][D]
  float* red = q_s + G * D;      // [DNW][G][D]
  float* sc = red + DNW * G * D; // [G][max(TK, kMaxDecodeSplits)] scaled scores, then probabilities
  constexpr int SC_LD = TK > kMaxDecodeSplits ? TK : kMaxDecodeSplits;
  float* st_s = sc + G * SC_LD;  // [3][8]
  TC* khat_new_s = reinterpret_cast<TC*>(st_s + 24);   // [D] reference-key row of this step
  uint32_t* so_s = reinterpret_cast<uint32_t*>(khat_new_s + D);   // [chunk / 32 + 2] segment offsets of the slice
  __shared__ __align__(8) unsigned long long bars[2];
  __shared__ int s_last, s_fail;
  __shared__ uint32_t s_words[4];
  __shared__ uint32_t s_pool;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.x, bkv = blockIdx.y;
  const int H_kv = H / G;
  const int b = bkv / H_kv, kvh = bkv - b * H_kv;
  const int L = n + 1;
  const int j0 = split * chunk;
  const int len = max(0, min(chunk, L - j0));
  const int n_tiles = (len + TK - 1) / TK;
  const bool has_new = (n >= j0) && (n < j0 + len);
  const TC* kc = k_cache + (size_t)bkv * T_max * D;
  const TC* vc = v_cache + (size_t)bkv * T_max * D;
  uint32_t* so_g = seg_off + (size_t)bkv * (nseg_max + 1);
  uint16_t* vals_g = vals + (size_t)bkv * cap;
  const uint32_t bar0 = smem_u32(&bars[0]);

  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar0), "r"(1) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar0 + 8), "r"(1) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_fail = 0;
  }
  if (tid < 8) { st_s[tid] = -INFINITY; st_s[8 + tid] = 0.0f; st_s[16 + tid] = 1.0f; }

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
  if (warp < NW) {
    const uint32_t word = __ballot_sync(0xffffffffu, fire);
    if (lane == 0) s_words[warp] = word;
  }
  for (int e = tid; e < G * D; e += DNT) {
    const int hh = e / D, c = e - hh * D;
    q_s[e] = to_f32(q_new[((size_t)b * H + kvh * G + hh) * D + c]);
  }
  if (tid == 0) s_pool = used[bkv];
  const int fired_total = __syncthreads_count(fire);

  // ---- the new row joins the encoding (the CTA that owns the new key's slice)
  const int seg_n = n / SEG;
  if (has_new) {
    const uint32_t pool = s_pool;
    const bool opens = (n % SEG) == 0;
    const uint32_t pos = opens ? round8(pool) : pool;
    if (tid < D) {
      if (opens) base_snap[((size_t)bkv * nseg_max + seg_n) * D + tid] =
          (uint16_t)(__float_as_uint(khat_in[(size_t)bkv * D + tid]) >> 16);      // exactly bf16
      if (fire) {
        uint32_t rank = __popc(s_words[tid >> 5] & ((1u << (tid & 31)) - 1u));
        for (int w = 0; w < (tid >> 5); ++w) rank += __popc(s_words[w]);
        if (DELTA_IN(pos + rank, cap, counters))
          vals_g[pos + rank] = reinterpret_cast<const uint16_t*>(k_new)[(size_t)bkv * D + tid];
      }
      if (tid < NW) {
        mask[((size_t)bkv * T_max + n) * NW + tid] = s_words[tid];
        kp_mask[((size_t)bkv * nseg_max * SEG + n) * NW + tid] = s_words[tid];
      }
    }
    if (tid == 0 && DELTA_IN(seg_n + 1, nseg_max + 1, counters)) {
      if (opens) so_g[seg_n] = pos;
      so_g[seg_n + 1] = pos + (uint32_t)fired_total;
      used[bkv] = pos + (uint32_t)fired_total;
      row_nnz[(size_t)bkv * T_max + n] = (uint16_t)fired_total;
      kp_nnz[(size_t)bkv * nseg_max * SEG + n] = (uint16_t)fired_total;
    }
  }
  // segment offsets of the slice (the cached rows; the new row is scored from registers)
  const int seg0 = j0 / SEG;
  const int nseg_slice = (min(len, max(0, n - j0)) + SEG - 1) / SEG;
  // (the entry behind the last cached segment is being rewritten by this step where the new row
  // extends or follows that segment: the old and the new value both bound its cached values)
  for (int s = tid; s <= nseg_slice; s += DNT) so_s[s] = so_g[seg0 + s];
  __syncthreads();

  auto tile_cached_rows = [&](int t) { return max(0, min(min(TK, len - t * TK), n - (j0 + t * TK))); };
  auto issue_tile = [&](int t) {
    const int rows = tile_cached_rows(t);
    const uint32_t bar = bar0 + 8 * (t & 1);
    unsigned char* stg = sStage + (size_t)(t & 1) * STAGE_BYTES;
    const int s0 = t * SPT, s1 = s0 + (rows + SEG - 1) / SEG;       // segments of the tile, slice-relative
    const uint32_t v0 = so_s[s0], v1 = rows ? so_s[s1] : v0;
    const uint32_t val_bytes = round8(v1 - v0) * 2u;
    const uint32_t mask_bytes = ((uint32_t)rows * NW * 4u + 15u) & ~15u, nnz_bytes = ((uint32_t)rows * 2u + 15u) & ~15u;
    const uint32_t base_bytes = (uint32_t)(s1 - s0) * D * 2u, v_bytes = (uint32_t)rows * ROWB;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar),
                 "r"(val_bytes + mask_bytes + nnz_bytes + base_bytes + v_bytes)
                 : "memory");
    if (rows) {
      const int tj0 = j0 + t * TK;
      if (val_bytes) bulk_load(smem_u32(stg), vals_g + v0, val_bytes, bar);
      bulk_load(smem_u32(stg + VAL_BYTES), kp_mask + ((size_t)bkv * nseg_max * SEG + tj0) * NW, mask_bytes, bar);
      bulk_load(smem_u32(stg + VAL_BYTES + MASK_BYTES), kp_nnz + (size_t)bkv * nseg_max * SEG + tj0, nnz_bytes, bar);
      bulk_load(smem_u32(stg + VAL_BYTES + MASK_BYTES + NNZ_BYTES),
                base_snap + ((size_t)bkv * nseg_max + seg0 + s0) * D, base_bytes, bar);
      bulk_load(smem_u32(stg + VAL_BYTES + MASK_BYTES + NNZ_BYTES + BASE_BYTES), vc + (size_t)tj0 * D, v_bytes, bar);
    }
  };
  if (tid == 0) {
    if (n_tiles > 0) issue_tile(0);
    if (n_tiles > 1) issue_tile(1);
  }

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
    unsigned char* stg = sStage + (size_t)(t & 1) * STAGE_BYTES;
    TC* vt = reinterpret_cast<TC*>(stg + VAL_BYTES + MASK_BYTES + NNZ_BYTES + BASE_BYTES);
    const bool tile_new = (n >= tj0) && (n < tj0 + rows);
    const int w_lo = max(tj0, n - W + 1);            // first key of the window inside this tile
    const int w_hi = min(tj0 + rows, n);             // cached window keys: [w_lo, w_hi)
    if (!mbar_wait(bar0 + 8 * (t & 1), (t >> 1) & 1)) s_fail = 1;
    // ---- rebuild the tile's reference-key rows: thread = (channel, segment), rows in order
    {
      const int cached = tile_cached_rows(t);
      const int c = tid % D, sg = tid / D;
      const uint16_t* sv = reinterpret_cast<const uint16_t*>(stg);
      const uint32_t* sm = reinterpret_cast<const uint32_t*>(stg + VAL_BYTES);
      const uint16_t* sn = reinterpret_cast<const uint16_t*>(stg + VAL_BYTES + MASK_BYTES);
      const uint16_t* sb = reinterpret_cast<const uint16_t*>(stg + VAL_BYTES + MASK_BYTES + NNZ_BYTES);
      if (sg * SEG < cached) {
        uint16_t kh = sb[sg * D + c];
        uint32_t off = so_s[t * SPT + sg] - so_s[t * SPT];
        const int r_end = min(SEG, cached - sg * SEG);
        for (int r = 0; r < r_end; ++r) {
          const int row = sg * SEG + r;
          const uint32_t word = sm[row * NW + (c >> 5)];
          if ((word >> (c & 31)) & 1u) {
            uint32_t rank = __popc(word & ((1u << (c & 31)) - 1u));
            for (int w = 0; w < (c >> 5); ++w) rank += __popc(sm[row * NW + w]);
            kh = sv[off + rank];
          }
          reinterpret_cast<uint16_t*>(kt)[row * D + c] = kh;
          off += sn[row];
        }
      }
    }
    __syncthreads();
    if (tile_new || w_lo < w_hi) {
      // original keys of the window replace the reference rows of the tile
      for (int e = tid; e < (w_hi - w_lo) * (D / 8); e += DNT) {
        const int r = e / (D / 8), cq = (e - r * (D / 8)) * 8;
        *reinterpret_cast<uint4*>(kt + (size_t)(w_lo - tj0 + r) * D + cq) =
            *reinterpret_cast<const uint4*>(kc + (size_t)(w_lo + r) * D + cq);
      }
      if (tile_new) {
        const int jn = n - tj0;
        for (int e = tid; e < D; e += DNT) {
          const TC kv = k_new[(size_t)bkv * D + e], vv = v_new[(size_t)bkv * D + e];
          kt[jn * D + e] = (W > 0) ? kv : khat_new_s[e];     // the new key is inside any window W_d >= 1
          vt[jn * D + e] = vv;
          k_cache[((size_t)bkv * T_max + n) * D + e] = kv;
          v_cache[((size_t)bkv * T_max + n) * D + e] = vv;
        }
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

// Pool capacity per KV head, in values: every element fired, plus the padding of the segments.
size_t keypack_capacity(int T_max, int d) { return (size_t)T_max * d + 8u * ((size_t)T_max / SEG + 2); }
int keypack_segments(int T_max) { return (T_max + SEG - 1) / SEG; }

cudaError_t launch_pack_keys(const Shape& s, const Workspace& w, const void* k, int T, cudaStream_t st) {
  if (!w.kp_vals || !w.qhat_rows) return cudaErrorNotSupported;
  const int bkv = s.B * s.H_kv;
  const int nseg_max = keypack_segments(s.T_max);
  const size_t cap = keypack_capacity(s.T_max, s.d);
  const size_t smem = ((size_t)(T + SEG - 1) / SEG + 2) * 4;
  using TC = __nv_bfloat16;
  if (s.d == 64)
    pack_keys_kernel<64><<<bkv, 256, smem, st>>>((const TC*)k, w.qhat_rows, w.mask, w.row_nnz, w.kp_vals, w.kp_segoff,
                                                 w.kp_base, w.kp_used, w.kp_mask, w.kp_nnz, T, s.T_max, cap, nseg_max,
                                                 w.counters);
  else if (s.d == 128)
    pack_keys_kernel<128><<<bkv, 256, smem, st>>>((const TC*)k, w.qhat_rows, w.mask, w.row_nnz, w.kp_vals,
                                                  w.kp_segoff, w.kp_base, w.kp_used, w.kp_mask, w.kp_nnz, T, s.T_max, cap,
                                                  nseg_max, w.counters);
  else return cudaErrorNotSupported;
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_decode_step_keypacked(const Shape& s, const Workspace& w, const void* q_new, const void* k_new,
                                         const void* v_new, void* k_cache, void* v_cache, void* out, int n,
                                         float theta, int window, int qhat_sel, cudaStream_t st) {
  using TC = __nv_bfloat16;
  if (!w.kp_vals) return cudaErrorNotSupported;
  const int L = n + 1;
  const int bkv = s.B * s.H_kv;
  const int TK = TILE_BYTES / (s.d * 2);
  int nsplit = kDecodeTargetCtas / bkv;
  if (nsplit > kMaxDecodeSplits) nsplit = kMaxDecodeSplits;
  const int max_by_len = (L + TK - 1) / TK;
  if (nsplit > max_by_len) nsplit = max_by_len;
  const int min_by_len = (L + kDecodeChunkMax - 1) / kDecodeChunkMax;     // no slice longer than the chunk limit
  if (nsplit < min_by_len) nsplit = min_by_len;
  if (nsplit < 1) nsplit = 1;
  int chunk = (L + nsplit - 1) / nsplit;
  chunk = (chunk + TK - 1) / TK * TK;          // slices start on tile (and segment) boundaries
  nsplit = (L + chunk - 1) / chunk;
  if (nsplit > kMaxDecodeSplits || chunk > kDecodeChunkMax) return cudaErrorInvalidValue;
  const float scale_log2e = 1.4426950408889634f / sqrtf((float)s.d);
  const int G = s.g();
  const int sc_ld = TK > kMaxDecodeSplits ? TK : kMaxDecodeSplits;
  const int nseg_max = keypack_segments(s.T_max);
  const size_t cap = keypack_capacity(s.T_max, s.d);
  const size_t stage = (size_t)TILE_BYTES + (TILE_BYTES + 64) + (size_t)TK * (s.d / 32) * 4 + (size_t)TK * 2 +
                       (size_t)(TK / SEG) * s.d * 2;
  const size_t smem = (size_t)2 * TILE_BYTES + 2 * stage +
                      ((size_t)G * s.d + (size_t)DNW * G * s.d + (size_t)G * sc_ld + 24) * 4 + (size_t)s.d * 2 +
                      ((size_t)kDecodeChunkMax / SEG + 2) * 4;
  const dim3 grid(nsplit, bkv);
  cudaError_t err = cudaSuccess;
#define LAUNCH(DD, GG)                                                                           \
  do {                                                                                           \
    auto kern = decode_step_keypacked_kernel<DD, GG>;                                            \
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);    \
    if (err != cudaSuccess) return err;                                                          \
    kern<<<grid, DNT, smem, st>>>((const TC*)q_new, (const TC*)k_new, (const TC*)v_new, (TC*)k_cache,      \
                                  (TC*)v_cache, (TC*)out, w.qhat[qhat_sel], w.qhat[qhat_sel ^ 1], w.row_nnz, \
                                  w.mask, w.kp_mask, w.kp_nnz, w.kp_vals, w.kp_segoff, w.kp_base, w.kp_used, w.dec_partial, \
                                  w.dec_ticket, w.counters, n, s.T_max, s.H, chunk, nsplit, theta, window, \
                                  scale_log2e, cap, nseg_max);                                             \
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
