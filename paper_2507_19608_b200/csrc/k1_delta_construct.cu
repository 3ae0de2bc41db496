// K1 -- delta construction over the query stream (Section II-C, Eq. 2-3; Section III-A
// strategy (1)), in two kernels.
//
// delta_chain_kernel: the token-sequential part.  Eq. 3 makes every channel a chain along the
// tokens (the reference is the last value that fired), so the only parallelism is across
// channels: one thread per channel, one warp per 32 channels (= one mask word), one CTA per
// (batch, head).  The chain itself is three dependent FP32 operations per token; everything
// else is kept off it: a producer warp streams the head's query rows into a ring of
// shared-memory stages with bulk asynchronous copies (the rows do not depend on the carried
// state), delta values leave with one coalesced store per row, every thread collects its
// channel's fire bits of 32 rows in one register and a 32 x 32 bit transpose across the warp
// (five shuffles) turns them into the 32 rows' mask words.
//
// delta_finish_kernel: everything that is parallel over rows once the mask exists -- the delta
// values themselves (query deltas), per-row and per-tile non-zero counts, the compacted channel
// indices, the counters behind Eq. 6 --
// plus two passes over the keys that prefill needs anyway: the hand-off row
// R(T-1)[j] = q_hat(T-1).k_j for decode and, for the tensor-core attention kernel, the
// channel-major fp32 copy of the keys.
#include "delta_internal.cuh"

namespace delta {

namespace {

constexpr int RC = 32;       // rows per ring stage (one mask flush per stage)
constexpr int NS = 8;        // ring stages

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait (about a second of SM clock); false if it ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > 2000000000ll) return false;
  }
  return true;
}

}  // namespace

// EMIT: also store the delta values and the reference rows (key deltas); without it the chain
// leaves mask words and per-tile references only (query deltas: the rest is rebuilt row-parallel).
template <typename TIn, int D, bool EMIT>
__global__ void __launch_bounds__(D + 32) delta_chain_kernel(
    const TIn* __restrict__ q, float* __restrict__ dq, uint32_t* __restrict__ mask,
    float* __restrict__ qhat_tile, float* __restrict__ qhat_out,
    __nv_bfloat16* __restrict__ qhat_rows, unsigned long long* __restrict__ counters, int T,
    int T_max, int n_tiles, float theta, int basis_exact, int src_rows) {
  // q: the stream that becomes the delta matrix, [heads][src_rows][D] with rows 0..T-1 read
  // (queries: src_rows = T; keys in the KV-cache layout: src_rows = T_max)
  constexpr int NW = D / 32;                       // chain warps = mask words per row
  constexpr uint32_t ROW_BYTES = D * sizeof(TIn);
  constexpr uint32_t STAGE_BYTES = RC * ROW_BYTES;
  extern __shared__ __align__(128) unsigned char ring[];   // [NS][RC][D] of TIn
  __shared__ __align__(8) unsigned long long bars[2 * NS];   // full[NS], empty[NS]
  __shared__ int s_fail;

  const int bh = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[NS]);
  const int n_chunks = (T + RC - 1) / RC;

  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full0 + 8 * s), "r"(1) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty0 + 8 * s), "r"(NW) : "memory");
    }
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == NW) {
    // ---- producer: keeps up to NS stages of query rows in flight
    if (lane == 0) {
      const unsigned char* src = reinterpret_cast<const unsigned char*>(q) + (size_t)bh * src_rows * ROW_BYTES;
      const uint32_t ring0 = smem_u32(ring);
      for (int i = 0; i < n_chunks; ++i) {
        const int s = i % NS;
        if (i >= NS && !mbar_wait(empty0 + 8 * s, ((i / NS) - 1) & 1)) { s_fail = 1; break; }
        const int rows = min(RC, T - i * RC);
        const uint32_t bytes = (uint32_t)rows * ROW_BYTES;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full0 + 8 * s),
                     "r"(bytes)
                     : "memory");
        asm volatile(
            "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                ring0 + s * STAGE_BYTES),
            "l"(src + (size_t)i * STAGE_BYTES), "r"(bytes), "r"(full0 + 8 * s)
            : "memory");
      }
    }
  } else {
    // ---- chain warps: thread c owns channel c
    const int c = tid;
    float* dqp = dq ? dq + (size_t)bh * T_max * D + c : nullptr;   // null: values left to the finish kernel
    __nv_bfloat16* qrp = qhat_rows ? qhat_rows + (size_t)bh * T_max * D + c : nullptr;
    uint32_t* maskp = mask + (size_t)bh * T_max * NW + warp;
    float qh = 0.0f;          // reference state, starts at zero (Eq. 3)
    bool failed = false;
    for (int i = 0; i < n_chunks; ++i) {
      const int s = i % NS;
      const int t0 = i * RC;
      if ((t0 % DELTA_TILE_ROWS) == 0)
        qhat_tile[((size_t)bh * n_tiles + t0 / DELTA_TILE_ROWS) * D + c] = qh;
      if (!mbar_wait(full0 + 8 * s, (i / NS) & 1)) { failed = true; break; }
      const TIn* rows = reinterpret_cast<const TIn*>(ring + (size_t)s * STAGE_BYTES) + c;
      const int nrows = min(RC, T - t0);
      // bit r of `bits`: did this thread's channel fire in row t0 + r
      uint32_t bits = 0;
      if (nrows == RC && !(t0 == 0 && basis_exact)) {
        // full stage, no basis row: all loads first, then nothing but the dependent chain,
        // its store and one bit per row
        float x[RC];
#pragma unroll
        for (int r = 0; r < RC; ++r) x[r] = to_f32(rows[r * D]);
#pragma unroll
        for (int r = 0; r < RC; ++r) {
          const float diff = __fsub_rn(x[r], qh);      // one IEEE subtraction
          const bool fire = fabsf(diff) > theta;       // strict; NaN compares false
          qh = fire ? x[r] : qh;
          if (EMIT) {
            dqp[(size_t)(t0 + r) * D] = fire ? diff : 0.0f;
            if (qrp) qrp[(size_t)(t0 + r) * D] = __float2bfloat16_rn(qh);
          }
          bits |= fire ? (1u << r) : 0u;
        }
      } else {
        for (int r = 0; r < nrows; ++r) {
          const float x = to_f32(rows[r * D]);
          bool fire;
          float delta;
          if (t0 + r == 0 && basis_exact) {
            fire = true;                                 // the basis vector is kept whole
            delta = x;
          } else {
            const float diff = __fsub_rn(x, qh);
            fire = fabsf(diff) > theta;
            delta = fire ? diff : 0.0f;
          }
          qh = fire ? x : qh;
          if (EMIT) {
            dqp[(size_t)(t0 + r) * D] = delta;
            if (qrp) qrp[(size_t)(t0 + r) * D] = __float2bfloat16_rn(qh);
          }
          bits |= fire ? (1u << r) : 0u;
        }
      }
      // 32 x 32 bit transpose across the warp: lane r ends up with the mask word of row t0 + r
      uint32_t mymask = bits;
#pragma unroll
      for (int j = 16; j > 0; j >>= 1) {
        const uint32_t km = (j == 16) ? 0x0000FFFFu : (j == 8) ? 0x00FF00FFu : (j == 4) ? 0x0F0F0F0Fu
                          : (j == 2) ? 0x33333333u : 0x55555555u;
        const uint32_t other = __shfl_xor_sync(0xffffffffu, mymask, j);
        mymask = (lane & j) ? (((other >> j) & km) | (mymask & ~km))
                            : ((mymask & km) | ((other & km) << j));
      }
      if (lane < nrows) maskp[(size_t)(t0 + lane) * NW] = mymask;
      __syncwarp();
      if (lane == 0)
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty0 + 8 * s) : "memory");
    }
    if (!failed) qhat_out[(size_t)bh * D + c] = qh;
    if (failed) s_fail = 1;
  }
  __syncthreads();
  if (tid == 0 && s_fail) atomicMax(&counters[CNT_STATUS], (unsigned long long)DELTA_ERR_TIMEOUT);
}

cudaError_t launch_delta_chain(const Shape& s, const Workspace& w, const void* q, int T,
                               float theta, int dtype, int init, bool want_qhat_rows, bool key_stream,
                               cudaStream_t st) {
  __nv_bfloat16* qrows = want_qhat_rows ? w.qhat_rows : nullptr;
  // query deltas: the chain leaves mask words and per-tile references only; delta values are
  // recomputed row-parallel by the finish kernel.  Key deltas: the chain stores them itself.
  float* dq_out = key_stream ? w.dq : nullptr;
  const int grid = s.B * (key_stream ? s.H_kv : s.H);
  const int src_rows = key_stream ? s.T_max : T;
  const int basis = (init == DELTA_INIT_BASIS_EXACT) ? 1 : 0;
  cudaError_t err = cudaSuccess;
#define LAUNCH(TIN, DD)                                                                          \
  do {                                                                                           \
    auto kern = key_stream ? delta_chain_kernel<TIN, DD, true> : delta_chain_kernel<TIN, DD, false>; \
    const size_t smem = (size_t)NS * RC * DD * sizeof(TIN);                                      \
    if (smem > 48 * 1024) {                                                                      \
      err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);  \
      if (err != cudaSuccess) return err;                                                        \
    }                                                                                            \
    kern<<<grid, DD + 32, smem, st>>>((const TIN*)q, dq_out, w.mask, w.qhat_tile, w.qhat[0], qrows, \
                                      w.counters, T, s.T_max, s.n_tiles, theta, basis, src_rows); \
  } while (0)
  if (dtype == DELTA_F32) {
    if (s.d == 64) LAUNCH(float, 64); else LAUNCH(float, 128);
  } else {
    if (s.d == 64) LAUNCH(__nv_bfloat16, 64); else LAUNCH(__nv_bfloat16, 128);
  }
#undef LAUNCH
  count_launch();
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// delta_finish_kernel: block roles by blockIdx.x.
//   [0, n_idx_blocks): one block per (batch, head, 64-row tile): row/tile counts, compacted
//       indices, counters of Eq. 6 (d multiply-adds per in-window causal pair,
//       nnz(Delta q_i) per out-of-window pair, against d per causal pair of dense attention).
//   [n_idx_blocks, ...): one block per (batch, KV head, 64 keys): hand-off row
//       R(T-1)[j] = q_hat(T-1).k_j for the heads of the group, and the channel-major fp32 key
//       copy when kt != nullptr.
template <typename TIn, int D>
__global__ void __launch_bounds__(256, 4) delta_finish_kernel(
    const uint32_t* __restrict__ mask, uint16_t* __restrict__ row_nnz,
    uint32_t* __restrict__ tile_nnz, uint8_t* __restrict__ idx,
    unsigned long long* __restrict__ counters, const TIn* __restrict__ k,
    const float* __restrict__ qhat, float* __restrict__ R, float* __restrict__ kt, int T,
    int T_max, int n_tiles, int BH, int H, int g, int W, int shape, int n_idx_blocks, int kt_ld,
    int key_stream, const TIn* __restrict__ q, float* __restrict__ dq,
    const float* __restrict__ qhat_tile, int basis_exact) {
  constexpr int NW = D / 32;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if ((int)blockIdx.x < n_idx_blocks) {
    // ---- one block per (batch, head, 64-row tile); warp w serves rows 8w .. 8w+7
    __shared__ unsigned long long s_red[3][8];
    const int tiles_used = (T + DELTA_TILE_ROWS - 1) / DELTA_TILE_ROWS;
    const int bh = blockIdx.x / tiles_used, tile = blockIdx.x - bh * tiles_used;
    const int t0 = tile * DELTA_TILE_ROWS;
    const int rows = min(DELTA_TILE_ROWS, T - t0);
    const int r_mine = warp * 8 + (lane & 7);        // lanes 0..7 hold one row each
    uint32_t mw[NW];
#pragma unroll
    for (int w2 = 0; w2 < NW; ++w2)
      mw[w2] = (r_mine < rows) ? mask[((size_t)bh * T_max + t0 + r_mine) * NW + w2] : 0u;
    unsigned long long done = 0, dense = 0, tsum = 0;
    if (lane < 8 && r_mine < rows) {
      int nnz = 0;
#pragma unroll
      for (int w2 = 0; w2 < NW; ++w2) nnz += __popc(mw[w2]);
      row_nnz[(size_t)bh * T_max + t0 + r_mine] = (uint16_t)nnz;
      tsum = (unsigned long long)nnz;
      const int i = t0 + r_mine;
      if (!key_stream) {
        // query deltas: row i meets i + 1 keys, nnz multiply-adds per out-of-window key
        const int n_in = in_window_count(i, W, shape);
        done = (unsigned long long)n_in * D + (unsigned long long)(i + 1 - n_in) * nnz;
        dense = (unsigned long long)(i + 1) * D;
      } else {
        // key deltas: key i meets the T - i queries behind it, for each of the g query heads
        const int n_q = T - i;
        const int n_in = in_window_col_count(i, T, W, shape);
        done = (unsigned long long)g * ((unsigned long long)n_in * D + (unsigned long long)(n_q - n_in) * nnz);
        dense = (unsigned long long)g * n_q * D;
      }
    }
    for (int o = 4; o > 0; o >>= 1) {
      tsum += __shfl_down_sync(0xffffffffu, tsum, o);
      done += __shfl_down_sync(0xffffffffu, done, o);
      dense += __shfl_down_sync(0xffffffffu, dense, o);
    }
    if (lane == 0) { s_red[0][warp] = tsum; s_red[1][warp] = done; s_red[2][warp] = dense; }
    // compacted indices: lane = channel within each mask word; the warp's 8 rows are assembled
    // in shared memory and leave as 16-byte stores (8 consecutive rows are contiguous)
    __shared__ __align__(16) uint8_t s_idx[8][8 * D];
    uint8_t* srow = s_idx[warp];
    const int my_rows = min(8, rows - warp * 8);
    for (int r = 0; r < my_rows; ++r) {
      uint32_t m[NW];
      int nnz = 0;
#pragma unroll
      for (int w2 = 0; w2 < NW; ++w2) {
        m[w2] = __shfl_sync(0xffffffffu, mw[w2], r);
        nnz += __popc(m[w2]);
      }
      int basep = 0;
#pragma unroll
      for (int w2 = 0; w2 < NW; ++w2) {
        if ((m[w2] >> lane) & 1u)
          srow[r * D + basep + __popc(m[w2] & ((1u << lane) - 1u))] = (uint8_t)(w2 * 32 + lane);
        basep += __popc(m[w2]);
      }
#pragma unroll
      for (int pp = lane; pp < D; pp += 32)
        if (pp >= nnz) srow[r * D + pp] = 0xFF;
    }
    __syncwarp();
    {
      uint4* dst = reinterpret_cast<uint4*>(idx + ((size_t)bh * T_max + t0 + warp * 8) * D);
      const uint4* src = reinterpret_cast<const uint4*>(srow);
      for (int e = lane; e < my_rows * D / 16; e += 32) dst[e] = src[e];
    }
    // delta values of the tile (query deltas; with key deltas the chain kernel stores them).
    // With the mask known the reference in front of a row is the last fired row below it, so a
    // 64-row tile splits into row segments: thread (channel, segment) finds its segment's last
    // fired value, takes the nearest earlier one (or the reference in front of the tile) as
    // carry-in and walks its rows with one select per row.
    if (dq != nullptr) {
      constexpr int NSEG = 256 / D, SEG = DELTA_TILE_ROWS / NSEG;   // 4 x 16 rows (d=64), 2 x 32 (d=128)
      __shared__ uint32_t s_mask[DELTA_TILE_ROWS][NW];
      __shared__ float s_lastx[NSEG][D];
      __shared__ uint8_t s_has[NSEG][D];
      for (int e = tid; e < DELTA_TILE_ROWS * NW; e += 256) {
        const int r = e / NW;
        s_mask[r][e - r * NW] = (r < rows) ? mask[((size_t)bh * T_max + t0 + r) * NW + (e - r * NW)] : 0u;
      }
      const int c = tid % D, seg = tid / D;
      const TIn* qp0 = q + ((size_t)bh * T + t0 + seg * SEG) * D + c;
      float x[SEG];
#pragma unroll
      for (int r = 0; r < SEG; ++r) x[r] = (seg * SEG + r < rows) ? to_f32(qp0[(size_t)r * D]) : 0.0f;
      __syncthreads();
      uint32_t bits = 0;      // bit r: channel c fired in row seg*SEG + r
#pragma unroll
      for (int r = 0; r < SEG; ++r) bits |= ((s_mask[seg * SEG + r][c >> 5] >> (c & 31)) & 1u) << r;
      float lastx = 0.0f;
#pragma unroll
      for (int r = 0; r < SEG; ++r) lastx = ((bits >> r) & 1u) ? x[r] : lastx;
      s_lastx[seg][c] = lastx;
      s_has[seg][c] = bits != 0u;
      __syncthreads();
      float ref = qhat_tile[((size_t)bh * n_tiles + tile) * D + c];   // reference in front of the tile
      for (int s2 = 0; s2 < seg; ++s2) ref = s_has[s2][c] ? s_lastx[s2][c] : ref;
      float* dqp = dq + ((size_t)bh * T_max + t0 + seg * SEG) * D + c;
#pragma unroll
      for (int r = 0; r < SEG; ++r) {
        if (seg * SEG + r < rows) {
          const bool fire = (bits >> r) & 1u;
          const float diff = (t0 + seg * SEG + r == 0 && basis_exact) ? x[r] : __fsub_rn(x[r], ref);
          dqp[(size_t)r * D] = fire ? diff : 0.0f;
          ref = fire ? x[r] : ref;
        }
      }
    }
    __syncthreads();
    if (tid == 0) {
      unsigned long long a = 0, b2 = 0, c2 = 0;
      for (int w2 = 0; w2 < 8; ++w2) { a += s_red[0][w2]; b2 += s_red[1][w2]; c2 += s_red[2][w2]; }
      tile_nnz[(size_t)bh * n_tiles + tile] = (uint32_t)a;
      unsigned long long* cs = counters + CNT_SHARD_BASE + 4 * (blockIdx.x % CNT_SHARDS);
      atomicAdd(&cs[0], a);
      atomicAdd(&cs[1], (unsigned long long)rows * D);
      atomicAdd(&cs[2], b2);
      atomicAdd(&cs[3], c2);
    }
    return;
  }

  // ---- key pass: 64 keys of one (batch, KV head)
  __shared__ float tile[D][65];
  __shared__ float qh[8][D];
  const int kblocks = (T + 63) / 64;
  const int item = (int)blockIdx.x - n_idx_blocks;
  const int bkv = item / kblocks, j0 = (item - bkv * kblocks) * 64;
  const int H_kv = H / g;
  const int b = bkv / H_kv, kvh = bkv - b * H_kv;
  const TIn* kp = k + (size_t)bkv * T_max * D;
  {
    constexpr int VEC = 16 / sizeof(TIn);            // elements per 16-byte load
    constexpr int CPR = D / VEC;                     // 16-byte chunks per key row
    for (int e = tid; e < 64 * CPR; e += 256) {
      const int j = e / CPR, c = (e - j * CPR) * VEC;
      TIn vals[VEC];
      if (j0 + j < T) {
        *reinterpret_cast<uint4*>(vals) = *reinterpret_cast<const uint4*>(kp + (size_t)(j0 + j) * D + c);
#pragma unroll
        for (int i = 0; i < VEC; ++i) tile[c + i][j] = to_f32(vals[i]);
      } else {
#pragma unroll
        for (int i = 0; i < VEC; ++i) tile[c + i][j] = 0.0f;
      }
    }
  }
  for (int e = tid; e < g * D; e += 256) {
    const int hh = e / D, c = e - hh * D;
    qh[hh][c] = qhat[((size_t)b * H + kvh * g + hh) * D + c];
  }
  __syncthreads();
  if (kt != nullptr) {
    float* op = kt + (size_t)bkv * D * kt_ld;
    for (int e = tid; e < 64 * D; e += 256) {
      const int c = e >> 6, j = e & 63;
      if (j0 + j < kt_ld) op[(size_t)c * kt_ld + j0 + j] = tile[c][j];
    }
  }
  {
    const int j = tid & 63;
    for (int hh = tid >> 6; hh < g; hh += 4) {
      float acc = 0.0f;
#pragma unroll 8
      for (int c = 0; c < D; ++c) acc = fmaf(qh[hh][c], tile[c][j], acc);
      if (j0 + j < T) R[((size_t)b * H + kvh * g + hh) * T_max + j0 + j] = acc;
    }
  }
}

cudaError_t launch_delta_finish(const Shape& s, const Workspace& w, const void* q, const void* k, int T,
                                int window, int shape, int dtype, int init, bool want_kt, bool key_stream,
                                cudaStream_t st) {
  // key deltas: the index/counter pass runs over the KV heads and there is no hand-off row
  const int BH = s.B * (key_stream ? s.H_kv : s.H);
  const int tiles_used = (T + DELTA_TILE_ROWS - 1) / DELTA_TILE_ROWS;
  const int n_idx_blocks = BH * tiles_used;
  const int n_key_blocks = key_stream ? 0 : s.B * s.H_kv * ((T + 63) / 64);
  const int kt_ld = (s.T_max + 3) / 4 * 4;
  float* kt = (want_kt && w.kt) ? w.kt : nullptr;
#define LAUNCH(TIN, DD)                                                                          \
  delta_finish_kernel<TIN, DD><<<n_idx_blocks + n_key_blocks, 256, 0, st>>>(                     \
      w.mask, w.row_nnz, w.tile_nnz, w.idx, w.counters, (const TIN*)k, w.qhat[0], w.R, kt, T,    \
      s.T_max, s.n_tiles, BH, s.H, s.g(), window, shape, n_idx_blocks, kt_ld, key_stream ? 1 : 0,   \
      key_stream ? nullptr : (const TIN*)q, key_stream ? nullptr : w.dq, w.qhat_tile,                \
      init == DELTA_INIT_BASIS_EXACT ? 1 : 0)
  if (dtype == DELTA_F32) {
    if (s.d == 64) LAUNCH(float, 64); else LAUNCH(float, 128);
  } else {
    if (s.d == 64) LAUNCH(__nv_bfloat16, 64); else LAUNCH(__nv_bfloat16, 128);
  }
#undef LAUNCH
  count_launch();
  return cudaGetLastError();
}

}  // namespace delta
