// K2 (tensor-core, telescoped) -- hybrid delta attention for bf16 inputs on sm_100a with every
// score on the tensor cores (Section III-B; Eq. 1, Eq. 4).
//
// Eq. 4's running sum telescopes: R(i)[j] = (sum over rows s <= i of Delta q(s)) . k_j, and by
// Eq. 3 that sum is the reference state q_hat(i), so the out-of-window score of pair (i, j) is
// the dense product q_hat(i).k_j.  For bf16 inputs every element of q_hat is a copy of an input
// element (or 0), hence exactly bf16: the whole out-of-window score matrix is one more
// Q_hat.K^T on the tensor cores.  Nothing is skipped (the zeros of the delta matrix are
// unstructured, and at the sparsity the method reaches a 4-row block of it is nearly dense),
// but the tensor cores do the dense product far faster than the FP32 pipes do the sparse one.
//
// Organisation.  One CTA owns TWO 128-row query tiles of one head, a short one (tile p) and a
// long one (tile n-1-p), so that every CTA of a head walks the same number of key tiles in
// total; both read the same key and value tiles out of one shared-memory ring.  Ten warps:
//   warps 0-3  softmax of query tile A, warps 4-7 softmax of query tile B: ONE THREAD PER SCORE
//              ROW.  A thread reads its 128 scores of a key tile out of tensor memory, takes the
//              row maximum and the exponentials without talking to any other thread, and writes
//              the probabilities back into tensor memory as bf16, over the scores it has read;
//   warp 8     one thread issues every tcgen05.mma: scores S = Q_hat.K^T (A and B operands in
//              shared memory) and O += P.V with P read from tensor memory;
//   warp 9     one thread streams key and value tiles by TMA.
// The output tile stays in tensor memory for the whole key loop (the products accumulate);
// a row is rescaled only when its running maximum has grown by more than 2^8 since the scale
// it is stored at, by the softmax thread that owns the row.  While one group of softmax warps
// exponentiates, the tensor cores work on the other group's products.
//
// A key tile that some row of the query tile scores exactly (Section III-B window) takes two
// passes through the same score buffer: the telescoped product first, which the threads read
// into registers, then Q.K^T, from which they take the in-window elements.
//
// Head dimensions 64 and 128 (template parameter).
//
// Every wait on an mbarrier is bounded; after a time-out the protocol still runs to its end,
// nothing is stored and the status word records DELTA_ERR_TIMEOUT.
#include <cuda.h>

#include "k2_tc.cuh"
#include "tc_common.cuh"

namespace delta {

using namespace tc;

namespace {

constexpr int BM = 128, BN = 128;
constexpr int NSW = 8;                     // softmax warps: 4 per query tile
constexpr int WARP_MMA = 8, WARP_TMA = 9;
constexpr int NTHR = 320;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TMEM_S = 0;             // scores of tile A at column 0, of tile B at column 128
constexpr uint32_t TMEM_O = 256;           // output tile of A at 256, of B at 256 + D
constexpr uint32_t SZ_BLK = 128 * 64 * 2;  // one [128 rows][64 elements] bf16 block, 16 KiB
constexpr float RESCALE_LOG2 = 8.0f;       // a row is rescaled when its maximum grew by more than 2^8

// Shared-memory map for head dimension D.  Operand tiles are D/64 blocks of [128][64] bf16 in
// the 128-byte-swizzle layout.  Query deltas: the two query tiles and their reference tiles;
// key deltas: the two query tiles and one tile of original keys for window tiles.
template <int D, bool KEY> struct TqSmem {
  static constexpr uint32_t NKB = D / 64;                 // 64-element blocks per row
  static constexpr uint32_t SZ_TILE = NKB * SZ_BLK;       // one [128][D] operand tile
  static constexpr uint32_t NKS = 2;                      // key ring stages
  static constexpr uint32_t NVS = (D == 64 || KEY) ? 2 : 1;   // value ring stages
  static constexpr uint32_t OFF_Q = 0;                    // query tiles A, B
  static constexpr uint32_t OFF_QH = OFF_Q + 2 * SZ_TILE; // reference tiles A, B (query deltas) / key tile (key deltas)
  static constexpr uint32_t OFF_K = OFF_QH + (KEY ? 1 : 2) * SZ_TILE;
  static constexpr uint32_t OFF_V = OFF_K + NKS * SZ_TILE;
  static constexpr uint32_t OFF_BAR = OFF_V + NVS * SZ_TILE;
  static constexpr uint32_t OFF_MISC = OFF_BAR + 32 * 8;
  static constexpr uint32_t BYTES = OFF_MISC + 16 + 1024;
  static_assert(BYTES <= 227 * 1024, "shared memory budget");
};

enum Bar {
  BAR_Q = 0,                 // both query tiles landed (one arrival + bytes)
  BAR_QH,                    // reference-query tiles built (8 warps)
  BAR_KFULL0, BAR_KFULL1, BAR_KFREE0, BAR_KFREE1,
  BAR_VFULL0, BAR_VFULL1, BAR_VFREE0, BAR_VFREE1,
  BAR_KXFULL, BAR_KXFREE,    // original keys of a window tile (key deltas)
  BAR_SFULL_A, BAR_SFULL_B,  // a score product is complete (tcgen05.commit)
  BAR_PRDY_A, BAR_PRDY_B,    // probabilities written (4 warps)
  BAR_SXREQ_A, BAR_SXREQ_B,  // telescoped scores read, exact pass may overwrite them (4 warps)
  BAR_ODONE_A, BAR_ODONE_B,  // last P.V complete
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

// Keys that some row of the query tile [i0, i1] scores exactly: lo <= j <= hi (empty if W = 0).
// Block window: the window blocks that rows i0..i1 fall into; sliding: i0-W+1 .. i1.
struct ExactRange { int lo, hi; };
__device__ __forceinline__ ExactRange exact_range(int i0, int i1, int W, int shape) {
  ExactRange r{1, 0};
  if (W > 0) {
    if (shape == 0) { r.lo = (i0 / W) * W; r.hi = (i1 / W) * W + W - 1; }
    else { r.lo = i0 - W + 1; r.hi = i1; }
  }
  return r;
}

}  // namespace

// KEY = false: query deltas (strategy 1, or 2 with p.reverse): telescoped scores Q_hat.K^T.  The
// reference rows of both query tiles are rebuilt in shared memory from the query tiles and the
// references the chain kernel left in front of every 8-row block (Eq. 2-3 re-run over 8 rows,
// blocks in parallel); tm_qh is unused.  KEY = true: key deltas (strategy 3): the column
// recursion telescopes to S[i][j] = q_i.k_hat(j), so the telescoped scores are Q.K_hat^T; tm_qh
// maps the reference-key rows (per KV head), which take the place of the key tiles in the ring,
// and the original keys are fetched only for tiles that touch the window.
template <int D, bool KEY>
__global__ void __launch_bounds__(NTHR, 1)
hybrid_attn_tcq_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_qh,
                       const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                       const TqParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw);
  using SM = TqSmem<D, KEY>;
  constexpr uint32_t NKB = SM::NKB, SZ_TILE = SM::SZ_TILE, NKS = SM::NKS, NVS = SM::NVS;
  constexpr uint32_t OFF_Q = SM::OFF_Q, OFF_QH = SM::OFF_QH, OFF_K = SM::OFF_K, OFF_V = SM::OFF_V,
                     OFF_BAR = SM::OFF_BAR, OFF_MISC = SM::OFF_MISC;
  volatile uint32_t* sMisc = reinterpret_cast<volatile uint32_t*>(sm + OFF_MISC);
  volatile uint32_t* abort_flag = sMisc + 1;
  const uint32_t bar0 = base + OFF_BAR;
#define BAR(i) (bar0 + 8u * (uint32_t)(i))

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int bh = blockIdx.x;
  const int b = bh / p.H, h = bh - b * p.H;
  const int bkv = b * (p.H / p.g) + h / p.g;
  const int T = p.T, W = p.W, shape = p.shape;
  const int n_qt = (T + BM - 1) / BM;
  // the CTA's two query tiles: X = 0 (A, the short one) and X = 1 (B, the long one)
  const int qt_of[2] = {(int)blockIdx.y, n_qt - 1 - (int)blockIdx.y};
  const bool has_b = qt_of[1] > qt_of[0];
  const int n_of[2] = {qt_of[0] + 1, has_b ? qt_of[1] + 1 : 0};     // key tiles each one walks
  const int n_max = has_b ? n_of[1] : n_of[0];

  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     base + OFF_MISC),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    for (int i = 0; i < NUM_BARS; ++i) {
      uint32_t cnt = 1;
      if (i == BAR_QH) cnt = NSW;
      if (i == BAR_PRDY_A || i == BAR_PRDY_B || i == BAR_SXREQ_A || i == BAR_SXREQ_B) cnt = 4;
      mbar_init(BAR(i), cnt);
    }
    sMisc[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sMisc[0];

  // does key tile t hold a key that some row of query tile X scores exactly?
  ExactRange ex[2];
#pragma unroll
  for (int X = 0; X < 2; ++X) {
    const int i0 = qt_of[X] * BM;
    ex[X] = exact_range(i0, min(i0 + BM, T) - 1, W, shape);
  }
  auto needs_exact = [&](int X, int t) -> bool {
    const int j0 = t * BN, j1 = min(j0 + BN, T) - 1;
    return j1 >= ex[X].lo && j0 <= ex[X].hi;
  };

  if (warp == WARP_TMA) {
    // =========================== loader ====================================================
    if (lane == 0) {
      auto load_tile = [&](uint32_t dst, const CUtensorMap* tm, uint32_t bar, int row0, int outer) {
#pragma unroll
        for (uint32_t kb = 0; kb < NKB; ++kb) tma_load_3d(dst + kb * SZ_BLK, tm, bar, 64 * kb, row0, outer);
      };
      mbar_expect_tx(BAR(BAR_Q), (has_b ? 2u : 1u) * SZ_TILE);
      load_tile(base + OFF_Q, &tm_q, BAR(BAR_Q), qt_of[0] * BM, bh);
      if (has_b) load_tile(base + OFF_Q + SZ_TILE, &tm_q, BAR(BAR_Q), qt_of[1] * BM, bh);
      // key deltas: the ring streams reference-key rows, which the finish kernel in front of
      // this one writes (programmatic stream serialisation): wait for them.  Keys and values
      // themselves are inputs.
      if (KEY) asm volatile("griddepcontrol.wait;" ::: "memory");
      const CUtensorMap* tm_ring = KEY ? &tm_qh : &tm_k;
      int n_kx = 0;
      for (int t = 0; t < n_max; ++t) {
        const uint32_t ks = (uint32_t)t % NKS, vs = (uint32_t)t % NVS;
        if (t >= (int)NKS) mbar_wait(BAR(BAR_KFREE0 + ks), ((t / NKS) - 1) & 1, abort_flag);
        mbar_expect_tx(BAR(BAR_KFULL0 + ks), SZ_TILE);
        load_tile(base + OFF_K + ks * SZ_TILE, tm_ring, BAR(BAR_KFULL0 + ks), t * BN, bkv);
        if (KEY && ((t < n_of[0] && needs_exact(0, t)) || (t < n_of[1] && needs_exact(1, t)))) {
          if (n_kx > 0) mbar_wait(BAR(BAR_KXFREE), (n_kx - 1) & 1, abort_flag);
          mbar_expect_tx(BAR(BAR_KXFULL), SZ_TILE);
          load_tile(base + OFF_QH, &tm_k, BAR(BAR_KXFULL), t * BN, bkv);
          ++n_kx;
        }
        if (t >= (int)NVS) mbar_wait(BAR(BAR_VFREE0 + vs), ((t / NVS) - 1) & 1, abort_flag);
        mbar_expect_tx(BAR(BAR_VFULL0 + vs), SZ_TILE);
        load_tile(base + OFF_V + vs * SZ_TILE, &tm_v, BAR(BAR_VFULL0 + vs), t * BN, bkv);
      }
    }
    __syncwarp();
  } else if (warp == WARP_MMA) {
    // =========================== tensor-core issue ==========================================
    if (lane == 0) {
      const uint32_t IDESC_QK = make_idesc(BN, 0);
      const uint32_t IDESC_PV = make_idesc(D, 1);
      int k_seen = -1, v_seen = -1;        // highest tile whose keys / values were waited for
      auto wait_k = [&](int t) {
        if (t > k_seen) { mbar_wait(BAR(BAR_KFULL0 + (uint32_t)t % NKS), (t / NKS) & 1, abort_flag); k_seen = t; tc_fence_after(); }
      };
      auto wait_v = [&](int t) {
        if (t > v_seen) { mbar_wait(BAR(BAR_VFULL0 + (uint32_t)t % NVS), (t / NVS) & 1, abort_flag); v_seen = t; tc_fence_after(); }
      };
      // S_X = A . B^T into the score buffer of tile X
      auto scores = [&](int X, uint32_t a, uint32_t bq) {
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc_mma(tmem + TMEM_S + 128u * X, make_desc(a + (ks >> 2) * SZ_BLK + (ks & 3) * 32, 16, 1024),
                 make_desc(bq + (ks >> 2) * SZ_BLK + (ks & 3) * 32, 16, 1024), IDESC_QK, ks > 0 ? 1u : 0u);
        tc_commit(BAR(BAR_SFULL_A + X));
      };
      auto tele = [&](int X, int t) {     // telescoped scores of key tile t
        wait_k(t);
        scores(X, base + (KEY ? OFF_Q : OFF_QH) + (uint32_t)X * SZ_TILE, base + OFF_K + ((uint32_t)t % NKS) * SZ_TILE);
      };
      mbar_wait(BAR(BAR_Q), 0, abort_flag);
      if (!KEY) mbar_wait(BAR(BAR_QH), 0, abort_flag);   // the softmax warps have built Q_hat
      tc_fence_after();
      tele(0, 0);
      if (has_b) tele(1, 0);
      int n_kx = 0, n_sx[2] = {0, 0};
      for (int t = 0; t < n_max; ++t) {
        // ---- exact passes of window tiles (rare: the last tiles of a query tile)
        bool any_x = false;
#pragma unroll
        for (int X = 0; X < 2; ++X) {
          if (t < n_of[X] && needs_exact(X, t)) {
            if (KEY && !any_x) { mbar_wait(BAR(BAR_KXFULL), n_kx & 1, abort_flag); }
            any_x = true;
            mbar_wait(BAR(BAR_SXREQ_A + X), n_sx[X] & 1, abort_flag);     // telescoped scores are in registers
            ++n_sx[X];
            tc_fence_after();
            scores(X, base + OFF_Q + (uint32_t)X * SZ_TILE,
                   KEY ? base + OFF_QH : base + OFF_K + ((uint32_t)t % NKS) * SZ_TILE);
          }
        }
        if (KEY && any_x) { tc_commit(BAR(BAR_KXFREE)); ++n_kx; }
        tc_commit(BAR(BAR_KFREE0 + (uint32_t)t % NKS));   // every product that reads this key stage is issued
        // ---- P.V of this tile, then the next tile's scores of the same query tile at once
#pragma unroll
        for (int X = 0; X < 2; ++X) {
          if (t >= n_of[X]) continue;
          mbar_wait(BAR(BAR_PRDY_A + X), t & 1, abort_flag);
          tc_fence_after();
          wait_v(t);
          const uint32_t vb = base + OFF_V + ((uint32_t)t % NVS) * SZ_TILE;
#pragma unroll
          for (int ks = 0; ks < BN / 16; ++ks)
            tc_mma_ts(tmem + TMEM_O + (uint32_t)(D * X), tmem + TMEM_S + 128u * X + 8u * ks,
                      make_desc(vb + ks * 2048, SZ_BLK, 1024), IDESC_PV, (t > 0 || ks > 0) ? 1u : 0u);
          if (t == n_of[X] - 1) tc_commit(BAR(BAR_ODONE_A + X));
          if (t + 1 < n_of[X]) tele(X, t + 1);
        }
        tc_commit(BAR(BAR_VFREE0 + (uint32_t)t % NVS));
      }
    }
    __syncwarp();
  } else {
    // =========================== softmax warps: one thread per score row ====================
    const int X = warp >> 2;                       // query tile of this warp group
    const int row = 32 * (warp & 3) + lane;        // tensor-memory lane = row of the tile
    const int qt = qt_of[X];
    const int i0 = qt * BM, i = i0 + row;
    const uint32_t lane_sel = (uint32_t)(32 * (warp & 3)) << 16;
    const uint32_t t_s = tmem + TMEM_S + 128u * X + lane_sel;
    const uint32_t t_o = tmem + TMEM_O + (uint32_t)(D * X) + lane_sel;
    const float scale = p.scale_log2e;
    const int n_tiles = n_of[X];

    if (!KEY) {
      // ---- reference-query tiles.  The chain kernel left the reference in front of every 8-row
      // block; thread (channel c, row segment) re-runs Eq. 2-3 over its blocks from there (the
      // reference after row r is the last fired q[.][c] at or below r) and writes the rows of
      // Q_hat straight into the operand layout.  Blocks are independent of one another.
      constexpr int SEG = 2 * BM / ((NSW * 32) / D);     // rows per thread: 64 (d = 64), 128 (d = 128)
      constexpr int NBK = SEG / DELTA_CKPT_ROWS;
      const int c = tid % D, seg = tid / D;
      const int Xs = (seg * SEG) / BM;                   // which query tile the segment lies in
      const int r_seg = (seg * SEG) % BM;                // its first row inside that tile
      const int i0s = qt_of[Xs] * BM;
      const bool live = (Xs == 0) || has_b;
      auto elem_off = [&](int r) -> uint32_t {   // byte offset of (r, c) in a [128][D] tile, 128-byte swizzle
        return (uint32_t)(c >> 6) * SZ_BLK + (uint32_t)r * 128u + ((((uint32_t)(c & 63) >> 3) ^ ((uint32_t)r & 7u)) << 4) +
               ((uint32_t)c & 7u) * 2u;
      };
      float ref[NBK];
      asm volatile("griddepcontrol.wait;" ::: "memory");    // the chain kernel's checkpoints
      if (live) {
#pragma unroll
        for (int bk = 0; bk < NBK; ++bk) {
          const int r0 = i0s + r_seg + bk * DELTA_CKPT_ROWS;
          ref[bk] = (r0 < T) ? p.ckpt[((size_t)bh * p.n_ckpt + r0 / DELTA_CKPT_ROWS) * D + c] : 0.0f;
        }
      }
      mbar_wait(BAR(BAR_Q), 0, abort_flag);      // the query tiles have landed
      if (live) {
        const unsigned char* qs = sm + OFF_Q + (size_t)Xs * SZ_TILE;
        unsigned char* qh = sm + OFF_QH + (size_t)Xs * SZ_TILE;
#pragma unroll
        for (int bk = 0; bk < NBK; ++bk) {
          float cur = ref[bk];
#pragma unroll
          for (int rr = 0; rr < DELTA_CKPT_ROWS; ++rr) {
            const int r8 = p.reverse ? DELTA_CKPT_ROWS - 1 - rr : rr;   // strategy (2): from the top
            const int r = r_seg + bk * DELTA_CKPT_ROWS + r8;
            const uint32_t off = elem_off(r);
            const uint32_t xb = *reinterpret_cast<const uint16_t*>(qs + off);
            const float x = __uint_as_float(xb << 16);
            // rows past the end of the sequence carry no state (in reverse they come first)
            const bool fire = (i0s + r < T) && ((fabsf(__fsub_rn(x, cur)) > p.theta) || (i0s + r == p.basis_row));
            cur = fire ? x : cur;
            // exact: the reference is a copy of an input element (or the zero it starts from)
            *reinterpret_cast<uint16_t*>(qh + off) = (uint16_t)(__float_as_uint(cur) >> 16);
          }
        }
      }
      fence_proxy_async();      // written through the generic proxy, read by the tensor cores
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(BAR_QH));
    }

    if (n_tiles > 0) {
      int wlo = 0, whi = 0;       // exact keys of row i: wlo <= j < whi
      if (W > 0) {
        if (shape == 0) { wlo = (i / W) * W; whi = wlo + W; }
        else { wlo = i - W + 1; whi = i + 1; }
      }
      float m_used = -INFINITY;   // the scale (log2 domain) the row's P and O are stored at
      float l_sum = 0.0f;
      int s_phase = 0;
      for (int t = 0; t < n_tiles; ++t) {
        mbar_wait(BAR(BAR_SFULL_A + X), s_phase & 1, abort_flag);
        ++s_phase;
        tc_fence_after();
        float s[128];
        {
          uint32_t u[128];
          tc_ld128(t_s, u);
#pragma unroll
          for (int c = 0; c < 128; ++c) s[c] = __uint_as_float(u[c]);
        }
        if (needs_exact(X, t)) {
          // hybrid select (Section III-B): hand the buffer back for the exact product, then take
          // the in-window elements from it
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(BAR(BAR_SXREQ_A + X));
          mbar_wait(BAR(BAR_SFULL_A + X), s_phase & 1, abort_flag);
          ++s_phase;
          tc_fence_after();
          const int j0 = t * BN;
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            uint32_t u[32];
            tc_ld32(t_s + 32u * ch, u);
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const int j = j0 + 32 * ch + c;
              if (j >= wlo && j < whi) s[32 * ch + c] = __uint_as_float(u[c]);
            }
          }
        }
        if (t == qt) {
          const int j0 = t * BN;
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (j0 + c > i) s[c] = -INFINITY;     // causal mask on the diagonal tile
        }
        float mx = fmax3(s[0], s[1], s[2]);
#pragma unroll
        for (int c = 3; c < 127; c += 2) mx = fmax3(mx, s[c], s[c + 1]);
        mx = fmaxf(mx, s[127]);
        const float m_new = fmaxf(m_used, mx * scale);
        if (t == 0) {
          m_used = m_new;                          // nothing accumulated yet
        } else {
          // S_full of this tile was committed behind P.V of the previous one, so the output tile
          // holds every product up to tile t-1.  Rescale the rows whose maximum ran away.
          const bool grow = (m_new - m_used) > RESCALE_LOG2;
          if (__any_sync(0xffffffffu, grow)) {
            const float al = grow ? ex2(m_used - m_new) : 1.0f;
            if (grow) { l_sum *= al; m_used = m_new; }
#pragma unroll
            for (int ch = 0; ch < D / 32; ++ch) {
              uint32_t u[32];
              tc_ld32(t_o + 32u * ch, u);
#pragma unroll
              for (int c = 0; c < 32; ++c) u[c] = __float_as_uint(__uint_as_float(u[c]) * al);
              tc_st32(t_o + 32u * ch, u);
            }
            tc_wait_st();
          }
        }
        // probabilities, row sum, bf16 pairs back into tensor memory over the scores
        const float2 sc2 = make_float2(scale, scale), nm2 = make_float2(-m_used, -m_used);
        float2 sum2 = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t w[32];
#pragma unroll
          for (int c = 0; c < 64; c += 2) {
            const float2 e = ffma2(make_float2(s[64 * hf + c], s[64 * hf + c + 1]), sc2, nm2);
            const float p0 = ex2(e.x), p1 = ex2(e.y);
            sum2 = fadd2(sum2, make_float2(p0, p1));
            const __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
            w[c >> 1] = *reinterpret_cast<const uint32_t*>(&pk);
          }
          tc_st32(t_s + 32u * hf, w);
        }
        l_sum += sum2.x + sum2.y;
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(BAR_PRDY_A + X));
      }

      // ---- normalise and store the row
      mbar_wait(BAR(BAR_ODONE_A + X), 0, abort_flag);
      tc_fence_after();
      const float inv = 1.0f / l_sum;
      const bool store = (i < T) && !*abort_flag;
#pragma unroll
      for (int ch = 0; ch < D / 32; ++ch) {
        uint32_t u[32];
        tc_ld32(t_o + 32u * ch, u);
        if (store) {
          uint32_t w[16];
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const __nv_bfloat162 t2 = __floats2bfloat162_rn(__uint_as_float(u[2 * c]) * inv, __uint_as_float(u[2 * c + 1]) * inv);
            w[c] = *reinterpret_cast<const uint32_t*>(&t2);
          }
          uint4* op = reinterpret_cast<uint4*>(p.out + ((size_t)bh * T + i) * D + 32 * ch);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) op[q4] = make_uint4(w[4 * q4], w[4 * q4 + 1], w[4 * q4 + 2], w[4 * q4 + 3]);
        }
      }
      tc_fence_before();
    }
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
                                         (int)TqSmem<D, KEY>::BYTES);
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
  // prologue (tensor-memory allocation, barrier setup, query, key and value loads) while the
  // delta chain kernel in front is still running; they wait for its results with
  // griddepcontrol.wait.
  const int n_qt = (T + BM - 1) / BM;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)BH, (unsigned)((n_qt + 1) / 2));
  cfg.blockDim = dim3(NTHR);
  cfg.dynamicSmemBytes = TqSmem<D, KEY>::BYTES;
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
