// K2 (generic) -- fused hybrid delta attention on the plain FP32 pipes (Section III-B; Eq. 1, 4).
// Serves every supported element type; it is the production path for fp32 inputs and the
// fall-back for bf16 shapes the tensor-core kernel does not take.
//
// One CTA owns 64 query rows of one head and walks the key tiles up to the diagonal:
//   * tiles that touch the window get the exact 64x64xd product;
//   * tiles with out-of-window pairs get the running delta sums of Eq. 4:
//       R(i)[j] = seed[j] + sum_{s = i0..i} sum_{c fired in row s} dq[s][c] * k_j[c],
//     seed[j] = q_hat(i0 - 1) . k_j (the reference in front of the tile telescopes every
//     earlier row of the recursion).  A warp owns 8 consecutive rows and all 64 keys, walks its
//     rows in order with the compacted channel lists, and skips everything that did not fire;
//   * scale, causal mask, online softmax, P.V accumulate in registers.
#include "delta_internal.cuh"

namespace delta {

namespace {
constexpr int BM = 64, BN = 64, NT = 256, NWARP = NT / 32;

template <int D> struct GenSmem {
  static constexpr int KS_LD = BN + 1;
  static constexpr int QS_LD = D + 4;
  static constexpr int SS_LD = BN + 1;
  static constexpr size_t floats = (size_t)D * KS_LD      // Ks  [D][BN+1]  channel-major keys
                                   + (size_t)BN * D       // Vs  [BN][D]
                                   + (size_t)BM * QS_LD   // Qs  [BM][D+4]
                                   + (size_t)BM * D       // dQs [BM][D]
                                   + (size_t)BM * SS_LD   // Ss  [BM][BN+1]
                                   + (size_t)NWARP * BN   // seedp
                                   + (size_t)NWARP * BN   // tot
                                   + D                    // qhat
                                   + 3 * BM;              // m, l, alpha
  static constexpr size_t bytes = floats * 4 + (size_t)BM * D /*idx*/ + BM * 4 /*nnz*/;
};
}  // namespace

template <typename TIn, int D>
__global__ void __launch_bounds__(NT, (D == 64 ? 2 : 1)) hybrid_attn_generic_kernel(
    const TIn* __restrict__ q, const TIn* __restrict__ k, const TIn* __restrict__ v,
    TIn* __restrict__ out, const float* __restrict__ dq, const uint16_t* __restrict__ row_nnz,
    const uint8_t* __restrict__ idx, const float* __restrict__ qhat_tile, int T, int T_max,
    int n_tiles, int H, int g, int W, int shape, float scale_log2e) {
  using SM = GenSmem<D>;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* Ks = reinterpret_cast<float*>(smem_raw);
  float* Vs = Ks + (size_t)D * SM::KS_LD;
  float* Qs = Vs + (size_t)BN * D;
  float* dQs = Qs + (size_t)BM * SM::QS_LD;
  float* Ss = dQs + (size_t)BM * D;
  float* seedp = Ss + (size_t)BM * SM::SS_LD;
  float* tot = seedp + NWARP * BN;
  float* qhat_s = tot + NWARP * BN;
  float* m_s = qhat_s + D;
  float* l_s = m_s + BM;
  float* alpha_s = l_s + BM;
  uint8_t* idxs = reinterpret_cast<uint8_t*>(alpha_s + BM);
  int* nnz_s = reinterpret_cast<int*>(idxs + (size_t)BM * D);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;  // heaviest query tiles first
  const int bh = blockIdx.y;
  const int b = bh / H, h = bh - b * H;
  const int kvh = h / g, H_kv = H / g;
  const int i0 = qt * BM;

  const TIn* qp = q + ((size_t)bh * T + i0) * D;
  const float* dqp = dq + ((size_t)bh * T_max + i0) * D;
  const uint8_t* idxp = idx + ((size_t)bh * T_max + i0) * D;
  const uint16_t* nnzp = row_nnz + (size_t)bh * T_max + i0;
  const TIn* kp = k + ((size_t)b * H_kv + kvh) * (size_t)T_max * D;
  const TIn* vp = v + ((size_t)b * H_kv + kvh) * (size_t)T_max * D;
  const int rows_valid = min(BM, T - i0);

  // ---- stage the query tile: exact rows, delta rows, compacted indices, counts, reference
  for (int e = tid; e < BM * D; e += NT) {
    const int r = e / D, c = e - r * D;
    const bool ok = r < rows_valid;
    Qs[r * SM::QS_LD + c] = ok ? to_f32(qp[(size_t)r * D + c]) : 0.0f;
    dQs[r * D + c] = ok ? dqp[(size_t)r * D + c] : 0.0f;
    idxs[r * D + c] = ok ? idxp[(size_t)r * D + c] : (uint8_t)0xFF;
  }
  if (tid < BM) {
    nnz_s[tid] = tid < rows_valid ? (int)nnzp[tid] : 0;
    m_s[tid] = -INFINITY;
    l_s[tid] = 0.0f;
  }
  if (tid < D) qhat_s[tid] = qhat_tile[((size_t)bh * n_tiles + qt) * D + tid];

  const int ty = tid >> 4, tx = tid & 15;  // 16 x 16 micro-tile grid for the dense products
  constexpr int EV = D / 16;
  float O[4][EV];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int e = 0; e < EV; ++e) O[r][e] = 0.0f;

  const int i1 = i0 + rows_valid - 1;  // last valid row of the tile
  for (int jt = 0; jt <= qt; ++jt) {
    const int j0 = jt * BN;
    const int j1 = min(j0 + BN, T) - 1;
    // conservative tile classification (the per-element predicate decides in the end)
    bool need_exact, all_in;
    if (W <= 0) { need_exact = false; all_in = false; }
    else if (shape == 0) {
      need_exact = (i0 / W <= j1 / W) && (j0 / W <= i1 / W);
      all_in = (i0 / W == i1 / W) && (j0 / W == j1 / W) && (i0 / W == j0 / W);
    } else {
      need_exact = max(0, i0 - j1) < W;
      all_in = (i1 - j0) < W;
    }
    const bool need_delta = !all_in;

    __syncthreads();  // previous tile's consumers are done with Ks / Vs / Ss
    for (int e = tid; e < BN * D; e += NT) {
      const int j = e / D, c = e - j * D;
      const bool ok = (j0 + j) < T;
      Ks[c * SM::KS_LD + j] = ok ? to_f32(kp[(size_t)(j0 + j) * D + c]) : 0.0f;
      Vs[j * D + c] = ok ? to_f32(vp[(size_t)(j0 + j) * D + c]) : 0.0f;
    }
    __syncthreads();

    if (need_exact) {
      float acc[4][4];
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[r][e] = 0.0f;
#pragma unroll 4
      for (int c = 0; c < D; ++c) {
        float a[4], bb[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) a[r] = Qs[(4 * ty + r) * SM::QS_LD + c];
#pragma unroll
        for (int e = 0; e < 4; ++e) bb[e] = Ks[c * SM::KS_LD + tx + 16 * e];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[r][e] = fmaf(a[r], bb[e], acc[r][e]);
      }
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int e = 0; e < 4; ++e) Ss[(4 * ty + r) * SM::SS_LD + tx + 16 * e] = acc[r][e];
      __syncwarp();  // rows 8*warp .. 8*warp+7 are written and read by this warp only
    }

    if (need_delta) {
      // seed partial: this warp's slice of q_hat . k_j
      {
        constexpr int CS = D / NWARP;
        float s0 = 0.0f, s1 = 0.0f;
#pragma unroll
        for (int cc = 0; cc < CS; ++cc) {
          const int c = warp * CS + cc;
          const float x = qhat_s[c];
          s0 = fmaf(x, Ks[c * SM::KS_LD + lane], s0);
          s1 = fmaf(x, Ks[c * SM::KS_LD + lane + 32], s1);
        }
        seedp[warp * BN + lane] = s0;
        seedp[warp * BN + lane + 32] = s1;
      }
      float acc0 = 0.0f, acc1 = 0.0f;
      for (int r = 0; r < 8; ++r) {
        const int row = warp * 8 + r;
        const int nz = nnz_s[row];
        const uint8_t* ip = idxs + row * D;
        const float* xp = dQs + row * D;
        for (int p = 0; p < nz; ++p) {      // only fired channels; zero rows cost nothing
          const int c = ip[p];
          const float x = xp[c];
          acc0 = fmaf(x, Ks[c * SM::KS_LD + lane], acc0);
          acc1 = fmaf(x, Ks[c * SM::KS_LD + lane + 32], acc1);
        }
        const int i = i0 + row;
        if (!in_window(i, j0 + lane, W, shape)) Ss[row * SM::SS_LD + lane] = acc0;
        if (!in_window(i, j0 + lane + 32, W, shape)) Ss[row * SM::SS_LD + lane + 32] = acc1;
      }
      tot[warp * BN + lane] = acc0;
      tot[warp * BN + lane + 32] = acc1;
    }
    __syncthreads();

    // ---- scale, causal mask, online softmax (warp = 8 rows, lane = 2 columns)
    {
      float pre0 = 0.0f, pre1 = 0.0f;
      if (need_delta) {
#pragma unroll
        for (int w2 = 0; w2 < NWARP; ++w2) {
          pre0 += seedp[w2 * BN + lane];
          pre1 += seedp[w2 * BN + lane + 32];
        }
        for (int w2 = 0; w2 < warp; ++w2) {
          pre0 += tot[w2 * BN + lane];
          pre1 += tot[w2 * BN + lane + 32];
        }
      }
      for (int r = 0; r < 8; ++r) {
        const int row = warp * 8 + r;
        const int i = i0 + row;
        const int ja = j0 + lane, jb = j0 + lane + 32;
        float s0 = Ss[row * SM::SS_LD + lane], s1 = Ss[row * SM::SS_LD + lane + 32];
        if (!in_window(i, ja, W, shape)) s0 += pre0;
        if (!in_window(i, jb, W, shape)) s1 += pre1;
        s0 = (ja <= i && ja < T) ? s0 * scale_log2e : -INFINITY;
        s1 = (jb <= i && jb < T) ? s1 * scale_log2e : -INFINITY;
        float mx = fmaxf(s0, s1);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float m_old = m_s[row];
        const float m_new = fmaxf(m_old, mx);
        const float p0 = exp2f(s0 - m_new), p1 = exp2f(s1 - m_new);
        float sum = p0 + p1;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        Ss[row * SM::SS_LD + lane] = p0;
        Ss[row * SM::SS_LD + lane + 32] = p1;
        __syncwarp();
        if (lane == 0) {
          const float a = exp2f(m_old - m_new);
          alpha_s[row] = a;
          l_s[row] = l_s[row] * a + sum;
          m_s[row] = m_new;
        }
      }
      __syncwarp();
    }

    // ---- O = alpha * O + P V   (rows 4*ty .. 4*ty+3 belong to this thread's own warp)
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const float a = alpha_s[4 * ty + r];
#pragma unroll
      for (int e = 0; e < EV; ++e) O[r][e] *= a;
    }
    const int jmax = min(BN, i1 - j0 + 1);  // keys beyond the last valid row carry P = 0
#pragma unroll 2
    for (int j = 0; j < jmax; ++j) {
      float p[4], vv[EV];
#pragma unroll
      for (int r = 0; r < 4; ++r) p[r] = Ss[(4 * ty + r) * SM::SS_LD + j];
#pragma unroll
      for (int e = 0; e < EV; ++e) vv[e] = Vs[j * D + tx + 16 * e];
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int e = 0; e < EV; ++e) O[r][e] = fmaf(p[r], vv[e], O[r][e]);
    }
  }

  __syncwarp();
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int row = 4 * ty + r;
    if (row < rows_valid) {
      const float inv = 1.0f / l_s[row];
      TIn* op = out + ((size_t)bh * T + i0 + row) * D;
#pragma unroll
      for (int e = 0; e < EV; ++e) op[tx + 16 * e] = from_f32<TIn>(O[r][e] * inv);
    }
  }
}

cudaError_t launch_hybrid_attn_generic(const Shape& s, const Workspace& w, const void* q,
                                       const void* k, const void* v, void* out, int T, int window,
                                       int shape, int dtype, cudaStream_t st) {
  const dim3 grid((T + BM - 1) / BM, s.B * s.H);
  const float scale_log2e = 1.4426950408889634f / sqrtf((float)s.d);
  cudaError_t err = cudaSuccess;
#define LAUNCH(TIN, DD)                                                                         \
  do {                                                                                          \
    auto kern = hybrid_attn_generic_kernel<TIN, DD>;                                            \
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,               \
                               (int)GenSmem<DD>::bytes);                                        \
    if (err != cudaSuccess) return err;                                                         \
    kern<<<grid, NT, GenSmem<DD>::bytes, st>>>((const TIN*)q, (const TIN*)k, (const TIN*)v,     \
                                                (TIN*)out, w.dq, w.row_nnz, w.idx, w.qhat_tile, \
                                                T, s.T_max, s.n_tiles, s.H, s.g(), window,      \
                                                shape, scale_log2e);                            \
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

}  // namespace delta
