// K1 -- delta construction over the query stream (Section II-C, Eq. 2-3; Section III-A
// strategy (1)).  One thread owns one channel chain and walks the tokens in order; a warp
// owns 32 adjacent channels, so every row is one coalesced load and one coalesced store and
// the row's mask word is a single ballot.  Loads do not depend on the carried state, so they
// are issued one batch of rows ahead of the compare/select chain.
//
// Outputs per (batch, head): delta values (fp32, +0 where not fired), bit mask, per-row and
// per-tile non-zero counts, compacted channel indices, the reference state in front of every
// 64-row tile, and the final reference state.
#include "delta_internal.cuh"

namespace delta {

constexpr int kBatchRows = 16;  // rows loaded ahead of the dependent chain

template <typename TIn, int D>
__global__ void __launch_bounds__(D) delta_construct_kernel(
    const TIn* __restrict__ q, float* __restrict__ dq, uint32_t* __restrict__ mask,
    uint16_t* __restrict__ row_nnz, uint32_t* __restrict__ tile_nnz, uint8_t* __restrict__ idx,
    float* __restrict__ qhat_tile, __nv_bfloat16* __restrict__ qhat_tile_bf16,
    float* __restrict__ qhat_out, unsigned long long* __restrict__ counters, int T, int T_max,
    int n_tiles, float theta, int basis_exact) {
  constexpr int NW = D / 32;
  const int bh = blockIdx.x;
  const int c = threadIdx.x;
  const int lane = c & 31, warp = c >> 5;
  const TIn* qp = q + (size_t)bh * T * D + c;
  float* dqp = dq + (size_t)bh * T_max * D + c;
  uint32_t* maskp = mask + (size_t)bh * T_max * NW;
  uint16_t* nnzp = row_nnz + (size_t)bh * T_max;
  uint8_t* idxp = idx + (size_t)bh * T_max * D;

  __shared__ uint32_t smask[DELTA_TILE_ROWS][NW];
  __shared__ uint32_t s_tile_sum;
  __shared__ unsigned long long s_total;
  if (c == 0) { s_tile_sum = 0; s_total = 0; }

  float qh = 0.0f;  // reference state, starts at zero (Eq. 3)
  float cur[kBatchRows], nxt[kBatchRows];
  const int n_batches = (T + kBatchRows - 1) / kBatchRows;
#pragma unroll
  for (int r = 0; r < kBatchRows; ++r) cur[r] = (r < T) ? to_f32(qp[(size_t)r * D]) : 0.0f;

  for (int b = 0; b < n_batches; ++b) {
    const int t0 = b * kBatchRows;
    // rows of the next batch: in flight while this batch's chain runs
    {
      const int t1 = t0 + kBatchRows;
#pragma unroll
      for (int r = 0; r < kBatchRows; ++r)
        nxt[r] = (t1 + r < T) ? to_f32(qp[(size_t)(t1 + r) * D]) : 0.0f;
    }
    if ((t0 % DELTA_TILE_ROWS) == 0) {
      const size_t o = ((size_t)bh * n_tiles + t0 / DELTA_TILE_ROWS) * D + c;
      qhat_tile[o] = qh;
      if (qhat_tile_bf16) qhat_tile_bf16[o] = __float2bfloat16_rn(qh);
    }
#pragma unroll
    for (int r = 0; r < kBatchRows; ++r) {
      const int t = t0 + r;
      if (t < T) {  // uniform across the block
        const float x = cur[r];
        bool fire;
        float delta;
        if (t == 0 && basis_exact) {
          fire = true;           // the basis vector is kept whole
          delta = x;
        } else {
          const float diff = __fsub_rn(x, qh);   // one IEEE subtraction
          fire = fabsf(diff) > theta;            // strict; NaN compares false
          delta = fire ? diff : 0.0f;
        }
        qh = fire ? x : qh;
        dqp[(size_t)t * D] = delta;
        const uint32_t m = __ballot_sync(0xffffffffu, fire);
        if (lane == 0) smask[t % DELTA_TILE_ROWS][warp] = m;
      }
    }
#pragma unroll
    for (int r = 0; r < kBatchRows; ++r) cur[r] = nxt[r];

    // end of a 64-row tile (or of the stream): emit mask words, counts and compacted indices
    const int t_end = min(t0 + kBatchRows, T);
    if ((t_end % DELTA_TILE_ROWS) == 0 || t_end == T) {
      __syncthreads();
      const int tile = (t_end - 1) / DELTA_TILE_ROWS;
      const int tile_t0 = tile * DELTA_TILE_ROWS;
      const int rows = t_end - tile_t0;
      uint32_t my_sum = 0;
      for (int r = warp; r < rows; r += NW) {
        const int t = tile_t0 + r;
        uint32_t m[NW];
        int nnz = 0;
#pragma unroll
        for (int w = 0; w < NW; ++w) { m[w] = smask[r][w]; nnz += __popc(m[w]); }
        int base = 0;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
          if ((m[w] >> lane) & 1u) {
            const int pos = base + __popc(m[w] & ((1u << lane) - 1u));
            idxp[(size_t)t * D + pos] = (uint8_t)(w * 32 + lane);
          }
          base += __popc(m[w]);
        }
#pragma unroll
        for (int p = lane; p < D; p += 32)
          if (p >= nnz) idxp[(size_t)t * D + p] = 0xFF;
        if (lane < NW) maskp[(size_t)t * NW + lane] = smask[r][lane];
        if (lane == 0) { nnzp[t] = (uint16_t)nnz; my_sum += nnz; }
      }
      if (lane == 0 && my_sum) atomicAdd(&s_tile_sum, my_sum);
      __syncthreads();
      if (c == 0) {
        tile_nnz[(size_t)bh * n_tiles + tile] = s_tile_sum;
        s_total += s_tile_sum;
        s_tile_sum = 0;
      }
      // smask and s_tile_sum are reused by the next tile only after the next __syncthreads
      // pair above, and lane 0 of each warp writes smask rows of the next tile only after
      // every warp has passed the second barrier.
    }
  }
  qhat_out[(size_t)bh * D + c] = qh;
  __syncthreads();
  if (c == 0) {
    atomicAdd(&counters[CNT_PREFILL_NNZ], s_total);
    atomicAdd(&counters[CNT_PREFILL_ELEMS], (unsigned long long)T * D);
  }
}

cudaError_t launch_delta_construct(const Shape& s, const Workspace& w, const void* q, int T,
                                   float theta, int dtype, int init, cudaStream_t st) {
  const int grid = s.B * s.H;
  const int basis = (init == DELTA_INIT_BASIS_EXACT) ? 1 : 0;
#define LAUNCH(TIN, DD)                                                                          \
  delta_construct_kernel<TIN, DD><<<grid, DD, 0, st>>>(                                          \
      (const TIN*)q, w.dq, w.mask, w.row_nnz, w.tile_nnz, w.idx, w.qhat_tile, w.qhat_tile_bf16,  \
      w.qhat[0], w.counters, T, s.T_max, s.n_tiles, theta, basis)
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
// K4 -- counters behind Eq. 6 for the prefill stage: multiply-adds actually needed for the
// score matrix (d per in-window causal pair, nnz(Delta q_i) per out-of-window pair) against
// d per causal pair of dense attention.
__global__ void __launch_bounds__(256) prefill_stats_kernel(
    const uint16_t* __restrict__ row_nnz, unsigned long long* __restrict__ counters, int T,
    int T_max, int d, int W, int shape, int total_rows) {
  unsigned long long done = 0, dense = 0;
  for (int r = blockIdx.x * blockDim.x + threadIdx.x; r < total_rows; r += gridDim.x * blockDim.x) {
    const int bh = r / T, i = r - bh * T;
    const unsigned nnz = row_nnz[(size_t)bh * T_max + i];
    const int n_in = in_window_count(i, W, shape);
    const int n_out = (i + 1) - n_in;
    done += (unsigned long long)n_in * d + (unsigned long long)n_out * nnz;
    dense += (unsigned long long)(i + 1) * d;
  }
  for (int o = 16; o > 0; o >>= 1) {
    done += __shfl_down_sync(0xffffffffu, done, o);
    dense += __shfl_down_sync(0xffffffffu, dense, o);
  }
  __shared__ unsigned long long s_done[8], s_dense[8];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { s_done[warp] = done; s_dense[warp] = dense; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w2 = 1; w2 < 8; ++w2) { done += s_done[w2]; dense += s_dense[w2]; }
    atomicAdd(&counters[CNT_PREFILL_MACS_DONE], done);
    atomicAdd(&counters[CNT_PREFILL_MACS_DENSE], dense);
  }
}

cudaError_t launch_prefill_stats(const Shape& s, const Workspace& w, int T, int window, int shape,
                                 cudaStream_t st) {
  const int total = s.B * s.H * T;
  int grid = (total + 255) / 256;
  if (grid > 296) grid = 296;
  prefill_stats_kernel<<<grid, 256, 0, st>>>(w.row_nnz, w.counters, T, s.T_max, s.d, window, shape,
                                             total);
  count_launch();
  return cudaGetLastError();
}

}  // namespace delta
