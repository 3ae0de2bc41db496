// K2 (tensor-core, telescoped) -- hybrid delta attention for bf16 inputs on sm_100a with every
// score on the tensor cores (Section III-B; Eq. 1, Eq. 4).
//
// Eq. 4's running sum telescopes: R(i)[j] = (sum over rows s <= i of Delta q(s)) . k_j, and by
// Eq. 3 that sum is the reference state q_hat(i), so the out-of-window score of pair (i, j) is
// the dense product q_hat(i).k_j.  For bf16 inputs every element of q_hat is a copy of an input
// element (or 0), hence exactly bf16: the whole out-of-window score matrix is one more
// Q_hat.K^T on the tensor cores, with the rows of Q_hat written by the delta-construction
// kernel.  Nothing is skipped (the zeros of the delta matrix are unstructured, and at the
// sparsity the method reaches a 4-row block of it is nearly dense), but the tensor cores do
// the dense product far faster than the FP32 pipes do the sparse one.
//
// One CTA owns 128 query rows of one head: 16 compute warps and a control warp.  The control
// thread streams K and V tiles with TMA and issues, per 128-key tile, Q_hat.K^T (and Q.K^T if
// the tile touches the window) into a double-buffered tensor-memory score region, one tile
// ahead of the softmax.  Compute threads work row-per-thread straight out of tensor memory:
// thread (row, quarter) reads 32 score columns of its row, selects exact or telescoped per
// element, exchanges the row maximum with the three other quarters through shared memory,
// exponentiates, writes its 32 probabilities as bf16 into the operand layout of the P.V
// product, and rescales/accumulates its 16 output columns from the previous tile's P.V.
//
// Head dimensions 64 and 128 (template parameter).
//
// Every wait on an mbarrier is bounded (see tc_common.cuh); after a time-out the protocol
// still runs to its end, nothing is stored and the status word records DELTA_ERR_TIMEOUT.
#include <cuda.h>

#include "k2_tc.cuh"
#include "tc_common.cuh"

namespace delta {

using namespace tc;

namespace {

constexpr int BM = 128, BN = 128, NCWARP = 16, NCTHR = NCWARP * 32, NTHR = NCTHR + 32;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TMEM_SH = 0;        // telescoped scores, two buffers of 128 columns
constexpr uint32_t TMEM_SX = 256;      // exact scores, 128 columns
constexpr uint32_t TMEM_O = 384;       // P.V tile, d columns (d <= 128)
constexpr uint32_t SZ_BLK = 128 * 64 * 2;             // one [128 rows][64 elements] bf16 block, 16 KiB

// Shared-memory map for head dimension D.  Operand tiles are D/64 blocks of [128][64] bf16 in
// the 128-byte-swizzle layout.  d = 64: keys double buffered; d = 128: one key buffer (the
// next tile's keys are fetched as soon as this tile's score products are done).
template <int D> struct TqSmem {
  static constexpr uint32_t NKB = D / 64;                 // 64-element blocks per row
  static constexpr uint32_t SZ_TILE = NKB * SZ_BLK;       // one [128][D] operand tile
  static constexpr uint32_t NKBUF = (D == 64) ? 2 : 1;
  static constexpr uint32_t OFF_Q = 0;
  static constexpr uint32_t OFF_QH = OFF_Q + SZ_TILE;
  static constexpr uint32_t OFF_K = OFF_QH + SZ_TILE;
  static constexpr uint32_t OFF_V = OFF_K + NKBUF * SZ_TILE;   // two buffers
  static constexpr uint32_t OFF_P = OFF_V + 2 * SZ_TILE;       // bf16 [2][128 rows][64 keys]
  static constexpr uint32_t OFF_PMAX = OFF_P + 2 * SZ_BLK;     // fp32 [2][128 rows][4 quarters]
  static constexpr uint32_t OFF_BAR = OFF_PMAX + 2 * 128 * 4 * 4;
  static constexpr uint32_t OFF_MISC = OFF_BAR + 16 * 8;
  static constexpr uint32_t BYTES = OFF_MISC + 16 + 1024;
  static_assert(BYTES <= 227 * 1024, "shared memory budget");
};

enum Bar {
  BAR_Q = 0, BAR_K0, BAR_K1, BAR_V0, BAR_V1, BAR_S0, BAR_S1, BAR_O, BAR_KX,   // one arrival (+ bytes)
  BAR_SFREE0, BAR_SFREE1,                                             // 16 arrivals: scores read
  BAR_P,                                                              // 16 arrivals: P written
  BAR_QH,                                                             // 16 arrivals: reference-query tile built
  NUM_BARS
};

struct TqParams {
  __nv_bfloat16* out;
  unsigned long long* counters;
  const float* ckpt;           // [B,H,n_ckpt,D] reference in front of every 8-row block (query deltas only)
  int T, T_max, n_ckpt, H, g, W, shape;
  int reverse;       // strategy (2): Eq. 2-3 runs from row T-1 down to row 0
  int basis_row;     // the un-thresholded basis row (0, or T-1 in reverse), -1 if there is none
  float scale_log2e, theta;
};


// Barrier of the four warps that share a tensor-memory lane quadrant (ids 1..4, 128 threads).
// Immediate ids: with a register operand the compiler reserves all sixteen hardware barriers
// for the CTA and no other kernel's CTA can share the SM.
__device__ __forceinline__ void quad_sync(int qd) {
  switch (qd) {
    case 0: asm volatile("bar.sync 1, 128;" ::: "memory"); break;
    case 1: asm volatile("bar.sync 2, 128;" ::: "memory"); break;
    case 2: asm volatile("bar.sync 3, 128;" ::: "memory"); break;
    default: asm volatile("bar.sync 4, 128;" ::: "memory"); break;
  }
}

}  // namespace

// KEY = false: query deltas (strategy 1): telescoped scores Q_hat.K^T.  The 128 reference rows
// of the tile are rebuilt in shared memory from the query tile and the references the chain
// kernel left in front of every 8-row block (Eq. 2-3 re-run over 8 rows, blocks in parallel),
// so the sequential chain kernel does not have to store them and tm_qh is unused.  KEY = true: key deltas (strategy 3): the column recursion telescopes to
// S[i][j] = q_i.k_hat(j), so the telescoped scores are Q.K_hat^T; tm_qh maps the reference key
// rows (per KV head), which take the place of the key tiles in the ring, and the original keys
// are fetched only for tiles that touch the window.
template <int D, bool KEY>
__global__ void __launch_bounds__(NTHR, 1)
hybrid_attn_tcq_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_qh,
                       const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                       const TqParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw);
  using SM = TqSmem<D>;
  constexpr uint32_t NKB = SM::NKB, SZ_TILE = SM::SZ_TILE, NKBUF = SM::NKBUF;
  constexpr uint32_t OFF_Q = SM::OFF_Q, OFF_QH = SM::OFF_QH, OFF_K = SM::OFF_K, OFF_V = SM::OFF_V,
                     OFF_P = SM::OFF_P, OFF_PMAX = SM::OFF_PMAX, OFF_BAR = SM::OFF_BAR, OFF_MISC = SM::OFF_MISC;
  float* sPmax = reinterpret_cast<float*>(sm + OFF_PMAX);
  volatile uint32_t* sMisc = reinterpret_cast<volatile uint32_t*>(sm + OFF_MISC);
  volatile uint32_t* abort_flag = sMisc + 1;
  const uint32_t bar0 = base + OFF_BAR;
#define BAR(i) (bar0 + 8u * (uint32_t)(i))

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qt = (int)gridDim.y - 1 - (int)blockIdx.y;  // heaviest query tiles of every head first
  const int bh = blockIdx.x;
  const int b = bh / p.H, h = bh - b * p.H;
  const int bkv = b * (p.H / p.g) + h / p.g;
  const int i0 = qt * BM;
  const int T = p.T, W = p.W, shape = p.shape;
  const int i1 = min(i0 + BM, T) - 1;

  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     base + OFF_MISC),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    for (int i = 0; i < NUM_BARS; ++i) mbar_init(BAR(i), (i >= BAR_SFREE0) ? (uint32_t)NCWARP : 1u);
    sMisc[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sMisc[0];

  // Keys that some row of this query tile scores exactly: ex_lo <= j <= ex_hi (empty if W = 0).
  // Block window: the window blocks that rows i0..i1 fall into; sliding: i0-W+1 .. i1.
  // Computed once: the per-tile test below must not divide.
  int ex_lo = 1, ex_hi = 0;
  if (W > 0) {
    if (shape == 0) { ex_lo = (i0 / W) * W; ex_hi = (i1 / W) * W + W - 1; }
    else { ex_lo = i0 - W + 1; ex_hi = i1; }
  }
  auto tile_needs_exact = [&](int jt) -> bool {
    const int j0 = jt * BN, j1 = min(j0 + BN, T) - 1;
    return j1 >= ex_lo && j0 <= ex_hi;
  };

  if (warp == NCWARP) {
    // =========================== control warp ===============================================
    if (lane == 0) {
      const uint32_t IDESC_QK = make_idesc(BN, 0);
      const uint32_t IDESC_PV = make_idesc(D, 1);
      // one [128][D] tile = NKB boxes of [128][64]
      auto load_tile = [&](uint32_t dst, const CUtensorMap* tm, uint32_t bar, int row0, int outer) {
#pragma unroll
        for (uint32_t kb = 0; kb < NKB; ++kb) tma_load_3d(dst + kb * SZ_BLK, tm, bar, 64 * kb, row0, outer);
      };
      const CUtensorMap* tm_ring = KEY ? &tm_qh : &tm_k;   // what streams through the key ring
      mbar_expect_tx(BAR(BAR_Q), SZ_TILE);
      load_tile(base + OFF_Q, &tm_q, BAR(BAR_Q), i0, bh);
      // everything up to here is independent of the delta-construction kernel in front of
      // this one (programmatic stream serialisation): wait for its results now
      asm volatile("griddepcontrol.wait;" ::: "memory");
      mbar_expect_tx(BAR(BAR_K0), SZ_TILE);
      load_tile(base + OFF_K, tm_ring, BAR(BAR_K0), 0, bkv);
      mbar_expect_tx(BAR(BAR_V0), SZ_TILE);
      load_tile(base + OFF_V, &tm_v, BAR(BAR_V0), 0, bkv);
      if (NKBUF == 2 && qt >= 1) {
        mbar_expect_tx(BAR(BAR_K1), SZ_TILE);
        load_tile(base + OFF_K + SZ_TILE, tm_ring, BAR(BAR_K1), BN, bkv);
      }
      int n_kx = 0;    // exact key tiles fetched so far (key deltas only)
      // key buffer and barrier parity of tile t
      auto kbuf = [&](int t) { return NKBUF == 2 ? (t & 1) : 0; };
      auto kpar = [&](int t) { return NKBUF == 2 ? ((t >> 1) & 1) : (t & 1); };
      // scores of tile t: Q_hat.K^T into buffer t&1, plus Q.K^T if the tile touches the window
      auto issue_scores = [&](int t) {
        const int bf = t & 1;
        const bool exact = tile_needs_exact(t);
        if (KEY && exact) {
          // original keys of a window tile: into the slot the reference queries use otherwise
          // (its previous reader, the last window tile's product, is done: see the callers)
          mbar_expect_tx(BAR(BAR_KX), SZ_TILE);
          load_tile(base + OFF_QH, &tm_k, BAR(BAR_KX), t * BN, bkv);
        }
        mbar_wait(BAR(BAR_K0 + kbuf(t)), kpar(t), abort_flag);
        tc_fence_after();
        const uint32_t kb = base + OFF_K + kbuf(t) * SZ_TILE;
        const uint32_t a_tele = base + (KEY ? OFF_Q : OFF_QH);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc_mma(tmem + TMEM_SH + bf * 128,
                 make_desc(a_tele + (ks >> 2) * SZ_BLK + (ks & 3) * 32, 16, 1024),
                 make_desc(kb + (ks >> 2) * SZ_BLK + (ks & 3) * 32, 16, 1024), IDESC_QK, ks > 0 ? 1u : 0u);
        if (exact) {
          uint32_t kx = kb;
          if (KEY) {
            mbar_wait(BAR(BAR_KX), n_kx & 1, abort_flag);
            ++n_kx;
            tc_fence_after();
            kx = base + OFF_QH;
          }
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            tc_mma(tmem + TMEM_SX, make_desc(base + OFF_Q + (ks >> 2) * SZ_BLK + (ks & 3) * 32, 16, 1024),
                   make_desc(kx + (ks >> 2) * SZ_BLK + (ks & 3) * 32, 16, 1024), IDESC_QK, ks > 0 ? 1u : 0u);
        }
        tc_commit(BAR(BAR_S0 + bf));
      };
      mbar_wait(BAR(BAR_Q), 0, abort_flag);
      if (!KEY) mbar_wait(BAR(BAR_QH), 0, abort_flag);   // the compute warps have built Q_hat
      issue_scores(0);
      for (int t = 0; t <= qt; ++t) {
        const bool more = t < qt;
        const int nb = (t + 1) & 1;
        const bool next_exact = more && tile_needs_exact(t + 1);
        // the key buffer of tile t is free once its score products are done: refill it
        mbar_wait(BAR(BAR_S0 + (t & 1)), (t >> 1) & 1, abort_flag);
        const int tn = t + (int)NKBUF;         // the tile that takes this buffer next
        if (tn <= qt) {
          mbar_expect_tx(BAR(BAR_K0 + kbuf(tn)), SZ_TILE);
          load_tile(base + OFF_K + kbuf(tn) * SZ_TILE, tm_ring, BAR(BAR_K0 + kbuf(tn)), tn * BN, bkv);
        }
        // next tile's scores one tile ahead, unless it needs the single exact-score buffer
        if (more && !next_exact) {
          if (t >= 1) mbar_wait(BAR(BAR_SFREE0 + nb), ((t - 1) >> 1) & 1, abort_flag);
          issue_scores(t + 1);
        }
        if (t >= 1) mbar_wait(BAR(BAR_O), (t - 1) & 1, abort_flag);   // P.V(t-1) done: its V buffer is free
        if (more) {
          mbar_expect_tx(BAR(BAR_V0 + nb), SZ_TILE);
          load_tile(base + OFF_V + nb * SZ_TILE, &tm_v, BAR(BAR_V0 + nb), (t + 1) * BN, bkv);
        }
        // P.V of this tile
        mbar_wait(BAR(BAR_P), t & 1, abort_flag);
        mbar_wait(BAR(BAR_V0 + (t & 1)), (t >> 1) & 1, abort_flag);
        tc_fence_after();
        const uint32_t vbase = base + OFF_V + (t & 1) * SZ_TILE;
#pragma unroll
        for (int ks = 0; ks < BN / 16; ++ks)
          tc_mma(tmem + TMEM_O, make_desc(base + OFF_P + (ks >> 2) * SZ_BLK + (ks & 3) * 32, 16, 1024),
                 make_desc(vbase + ks * 2048, SZ_BLK, 1024), IDESC_PV, ks > 0 ? 1u : 0u);
        tc_commit(BAR(BAR_O));
        if (next_exact) {
          // every compute warp has read tile t's scores (it wrote P after that)
          mbar_wait(BAR(BAR_SFREE0 + (t & 1)), (t >> 1) & 1, abort_flag);
          if (t >= 1) mbar_wait(BAR(BAR_SFREE0 + nb), ((t - 1) >> 1) & 1, abort_flag);
          issue_scores(t + 1);
        }
      }
    }
    __syncwarp();
  } else {
    // =========================== compute warps: row per thread ==============================
    const int qd = warp & 3, sub = warp >> 2;     // tensor-memory lane quadrant / column quarter
    const int row = 32 * qd + lane;
    const int i = i0 + row;
    const uint32_t lane_sel = (uint32_t)(32 * qd) << 16;
    const float scale = p.scale_log2e;
    constexpr int OC = D / 4;      // output columns per thread (a quarter of the head dimension)
    float O[OC];
#pragma unroll
    for (int c = 0; c < OC; ++c) O[c] = 0.0f;
    float m_run = -INFINITY, l_part = 0.0f, alpha_prev = 1.0f;
    int wlo = 0, whi = 0;       // exact keys of row i: wlo <= j < whi
    if (W > 0) {
      if (shape == 0) { wlo = (i / W) * W; whi = wlo + W; }
      else { wlo = i - W + 1; whi = i + 1; }
    }

    if (!KEY) {
      // ---- reference-query tile.  The chain kernel left the reference in front of every 8-row
      // block; thread (channel c, row segment) re-runs Eq. 2-3 over its blocks from there (the
      // reference after row r is the last fired q[.][c] at or below r) and writes the rows of
      // Q_hat straight into the operand layout.  Blocks are independent of one another.
      constexpr int NSEG = NCTHR / D, SEG = BM / NSEG;   // 8 x 16 rows (d=64), 4 x 32 (d=128)
      const int c = tid % D, seg = tid / D;
      // byte offset of element (r, c) inside a [128][D] operand tile (128-byte swizzle)
      auto elem_off = [&](int r) -> uint32_t {
        return (uint32_t)(c >> 6) * SZ_BLK + (uint32_t)r * 128u + ((((uint32_t)(c & 63) >> 3) ^ ((uint32_t)r & 7u)) << 4) +
               ((uint32_t)c & 7u) * 2u;
      };
      float ref[SEG / DELTA_CKPT_ROWS];
      asm volatile("griddepcontrol.wait;" ::: "memory");    // the chain kernel's checkpoints
#pragma unroll
      for (int bk = 0; bk < SEG / DELTA_CKPT_ROWS; ++bk) {
        const int r0 = i0 + seg * SEG + bk * DELTA_CKPT_ROWS;
        ref[bk] = (r0 < T) ? p.ckpt[((size_t)bh * p.n_ckpt + r0 / DELTA_CKPT_ROWS) * D + c] : 0.0f;
      }
      mbar_wait(BAR(BAR_Q), 0, abort_flag);      // the query tile has landed
#pragma unroll
      for (int bk = 0; bk < SEG / DELTA_CKPT_ROWS; ++bk) {
        float cur = ref[bk];
#pragma unroll
        for (int rr = 0; rr < DELTA_CKPT_ROWS; ++rr) {
          const int r8 = p.reverse ? DELTA_CKPT_ROWS - 1 - rr : rr;   // strategy (2): from the top
          const int r = seg * SEG + bk * DELTA_CKPT_ROWS + r8;
          const uint32_t off = elem_off(r);
          const uint32_t xb = *reinterpret_cast<const uint16_t*>(sm + OFF_Q + off);
          const float x = __uint_as_float(xb << 16);
          // rows past the end of the sequence carry no state (in reverse they come first)
          const bool fire = (i0 + r < T) && ((fabsf(__fsub_rn(x, cur)) > p.theta) || (i0 + r == p.basis_row));
          cur = fire ? x : cur;
          // exact: the reference is a copy of an input element (or the zero it starts from)
          *reinterpret_cast<uint16_t*>(sm + OFF_QH + off) = (uint16_t)(__float_as_uint(cur) >> 16);
        }
      }
      fence_proxy_async();      // the tile was written through the generic proxy, the tensor cores read it
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(BAR_QH));
    }

    for (int jt = 0; jt <= qt; ++jt) {
      const int bf = jt & 1;
      const int jc0 = jt * BN + 32 * sub;      // first key of this thread's 32 columns
      const bool need_exact = tile_needs_exact(jt);
      const bool diag = (jt == qt);

      mbar_wait(BAR(BAR_S0 + bf), (jt >> 1) & 1, abort_flag);
      tc_fence_after();
      float s[32];
      {
        float v[16];
        tc_ld16(tmem + TMEM_SH + bf * 128 + 32 * sub + lane_sel, v);
#pragma unroll
        for (int c = 0; c < 16; ++c) s[c] = v[c];
        tc_ld16(tmem + TMEM_SH + bf * 128 + 32 * sub + 16 + lane_sel, v);
#pragma unroll
        for (int c = 0; c < 16; ++c) s[16 + c] = v[c];
      }
      if (need_exact) {
        // hybrid select (Section III-B): exact score inside the window
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          float v[16];
          tc_ld16(tmem + TMEM_SX + 32 * sub + 16 * hf + lane_sel, v);
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const int j = jc0 + 16 * hf + c;
            if (j >= wlo && j < whi) s[16 * hf + c] = v[c];
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(BAR_SFREE0 + bf));
      if (diag) {
#pragma unroll
        for (int c = 0; c < 32; ++c)
          if (jc0 + c > i) s[c] = -INFINITY;     // causal mask on the diagonal tile
      }
      // row maximum: own 32 columns, then the three other quarters through shared memory
      float mx = fmax3(s[0], s[1], s[2]);
#pragma unroll
      for (int c = 3; c < 31; c += 2) mx = fmax3(mx, s[c], s[c + 1]);
      mx = fmaxf(mx, s[31]);
      sPmax[(bf * BM + row) * 4 + sub] = mx;
      quad_sync(qd);   // the four warps of this quadrant
      const float4 pm = *reinterpret_cast<const float4*>(sPmax + (bf * BM + row) * 4);
      mx = fmaxf(fmaxf(pm.x, pm.y), fmaxf(pm.z, pm.w));
      const float m_new = fmaxf(m_run, mx * scale);
      const float al = ex2(m_run - m_new);
      m_run = m_new;
      float2 sum2 = make_float2(0.0f, 0.0f);
      const float2 sc2 = make_float2(scale, scale), nm2 = make_float2(-m_new, -m_new);
#pragma unroll
      for (int c = 0; c < 32; c += 2) {
        const float2 t = ffma2(make_float2(s[c], s[c + 1]), sc2, nm2);
        s[c] = ex2(t.x);
        s[c + 1] = ex2(t.y);
        sum2 = fadd2(sum2, make_float2(s[c], s[c + 1]));
      }
      l_part = fmaf(l_part, al, sum2.x + sum2.y);

      // the previous tile's P.V is done: the P buffer may be rewritten
      if (jt > 0) mbar_wait(BAR(BAR_O), (jt - 1) & 1, abort_flag);

      // P as bf16 in the operand layout: this thread's 32 keys are 4 chunks of 16 bytes
      {
        unsigned char* prow = sm + OFF_P + (size_t)(sub >> 1) * SZ_BLK + (size_t)row * 128;
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const __nv_bfloat162 t2 = __floats2bfloat162_rn(s[8 * q4 + 2 * e], s[8 * q4 + 2 * e + 1]);
            w[e] = *reinterpret_cast<const uint32_t*>(&t2);
          }
          const int chunk = 4 * (sub & 1) + q4;
          *reinterpret_cast<uint4*>(prow + ((chunk ^ (row & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      // previous tile's P.V: rescale and accumulate (its tensor-memory tile is rewritten by
      // this tile's product, which is issued only after every warp has arrived below)
      if (jt > 0) {
        tc_fence_after();
#pragma unroll
        for (int h16 = 0; h16 < OC / 16; ++h16) {
          float v[16];
          tc_ld16(tmem + TMEM_O + OC * sub + 16 * h16 + lane_sel, v);
          const float2 ap2 = make_float2(alpha_prev, alpha_prev);
#pragma unroll
          for (int c = 0; c < 16; c += 2) {
            const float2 o = ffma2(make_float2(O[16 * h16 + c], O[16 * h16 + c + 1]), ap2, make_float2(v[c], v[c + 1]));
            O[16 * h16 + c] = o.x;
            O[16 * h16 + c + 1] = o.y;
          }
        }
        tc_fence_before();
      }
      alpha_prev = al;
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(BAR_P));
    }

    // ---- last tile's P.V, row sum over the four quarters, normalisation, store
    mbar_wait(BAR(BAR_O), qt & 1, abort_flag);
    tc_fence_after();
    sPmax[(((qt + 1) & 1) * BM + row) * 4 + sub] = l_part;
    quad_sync(qd);
    const float4 lp = *reinterpret_cast<const float4*>(sPmax + (((qt + 1) & 1) * BM + row) * 4);
    const float inv = 1.0f / ((lp.x + lp.y) + (lp.z + lp.w));
    const bool store = (i < T) && !*abort_flag;
#pragma unroll
    for (int h16 = 0; h16 < OC / 16; ++h16) {
      float v[16];
      tc_ld16(tmem + TMEM_O + OC * sub + 16 * h16 + lane_sel, v);
      if (store) {
        uint32_t w[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const __nv_bfloat162 t2 = __floats2bfloat162_rn(
              fmaf(O[16 * h16 + 2 * c], alpha_prev, v[2 * c]) * inv,
              fmaf(O[16 * h16 + 2 * c + 1], alpha_prev, v[2 * c + 1]) * inv);
          w[c] = *reinterpret_cast<const uint32_t*>(&t2);
        }
        uint4* op = reinterpret_cast<uint4*>(p.out + ((size_t)bh * T + i) * D + OC * sub + 16 * h16);
        op[0] = make_uint4(w[0], w[1], w[2], w[3]);
        op[1] = make_uint4(w[4], w[5], w[6], w[7]);
      }
    }
    tc_fence_before();
  }

  __syncthreads();
  if (tid == 0 && sMisc[1]) atomicMax(&p.counters[CNT_STATUS], (unsigned long long)DELTA_ERR_TIMEOUT);
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS)
                 : "memory");
  }
#undef BAR
}

template <int D, bool KEY>
static cudaError_t launch_tcq(const Shape& s, const Workspace& w, const void* q, const void* k, const void* v,
                              void* out, int T, float theta, int init, int window, int shape, bool reverse,
                              cudaStream_t st) {
  const uint64_t BH = (uint64_t)s.B * s.H, BKV = (uint64_t)s.B * s.H_kv;
  const uint64_t ref_heads = KEY ? BKV : BH;   // the reference rows follow the delta stream
  CUtensorMap tq, tqh, tk, tv;
  const bool ok =
      encode3(&tq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, q, D, (uint64_t)T, BH, D * 2, (uint64_t)T * D * 2, 64, 128,
              CU_TENSOR_MAP_SWIZZLE_128B) &&
      encode3(&tqh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, w.qhat_rows, D, (uint64_t)T, ref_heads, D * 2,
              (uint64_t)s.T_max * D * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B) &&
      encode3(&tk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, k, D, (uint64_t)T, BKV, D * 2, (uint64_t)s.T_max * D * 2, 64,
              128, CU_TENSOR_MAP_SWIZZLE_128B) &&
      encode3(&tv, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, v, D, (uint64_t)T, BKV, D * 2, (uint64_t)s.T_max * D * 2, 64,
              128, CU_TENSOR_MAP_SWIZZLE_128B);
  if (!ok) return cudaErrorInvalidValue;
  cudaError_t err = cudaFuncSetAttribute(hybrid_attn_tcq_kernel<D, KEY>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)TqSmem<D>::BYTES);
  if (err != cudaSuccess) return err;
  TqParams p;
  p.out = (__nv_bfloat16*)out;
  p.counters = w.counters;
  p.ckpt = w.ckpt;
  p.T_max = s.T_max; p.n_ckpt = s.n_ckpt();
  p.theta = theta; p.reverse = reverse ? 1 : 0;
  p.basis_row = (init == DELTA_INIT_BASIS_EXACT) ? (reverse ? T - 1 : 0) : -1;
  p.T = T; p.H = s.H; p.g = s.g(); p.W = window; p.shape = shape;
  p.scale_log2e = 1.4426950408889634f / sqrtf((float)s.d);
  // Launched with programmatic stream serialisation: the CTAs become resident and run their
  // prologue (tensor-memory allocation, barrier setup, query-tile load) while the delta chain
  // kernel in front is still running; they wait for its results with griddepcontrol.wait.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)BH, (T + BM - 1) / BM);
  cfg.blockDim = dim3(NTHR);
  cfg.dynamicSmemBytes = TqSmem<D>::BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  err = cudaLaunchKernelEx(&cfg, hybrid_attn_tcq_kernel<D, KEY>, tq, tqh, tk, tv, p);
  count_launch();
  return err != cudaSuccess ? err : cudaGetLastError();
}

bool tcq_kernel_shape(int d) { return d == 64 || d == 128; }

cudaError_t launch_hybrid_attn_tcq(const Shape& s, const Workspace& w, const void* q, const void* k,
                                   const void* v, void* out, int T, float theta, int init, int window,
                                   int shape, bool key_deltas, bool reverse, cudaStream_t st) {
  if (key_deltas && reverse) return cudaErrorNotSupported;
  if (!w.qhat_rows) return cudaErrorNotSupported;
  if (s.d == 64)
    return key_deltas ? launch_tcq<64, true>(s, w, q, k, v, out, T, theta, init, window, shape, reverse, st)
                      : launch_tcq<64, false>(s, w, q, k, v, out, T, theta, init, window, shape, reverse, st);
  if (s.d == 128)
    return key_deltas ? launch_tcq<128, true>(s, w, q, k, v, out, T, theta, init, window, shape, reverse, st)
                      : launch_tcq<128, false>(s, w, q, k, v, out, T, theta, init, window, shape, reverse, st);
  return cudaErrorNotSupported;
}

}  // namespace delta
