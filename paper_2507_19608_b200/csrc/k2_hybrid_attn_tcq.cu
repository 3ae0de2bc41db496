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
// Organisation.  One CTA owns one 128-row query tile of one head and walks its key tiles up to
// the diagonal; the key tiles are dealt alternately to two groups of softmax warps, each with
// its own score buffer, running maximum, row sum and output tile in tensor memory (the two
// partial results are merged once, at the end).  Ten warps:
//   warps 0-3  softmax of the even key tiles, warps 4-7 of the odd ones: ONE THREAD PER SCORE
//              ROW.  A thread reads its 128 scores of a key tile out of tensor memory, takes the
//              row maximum and the exponentials without talking to any other thread, and writes
//              the probabilities back into tensor memory as bf16, over the scores it has read;
//   warp 8     one thread issues the score products S = Q_hat.K^T (A and B operands in shared
//              memory); warp 9: one thread issues O += P.V with P read from tensor memory (for
//              d = 128, where P lies over S, warp 8 issues both in turn);
//   warp 10    one thread streams key and value tiles by TMA through a ring of stages.

// The output tiles stay in tensor memory for the whole key loop (the products accumulate);
// a row is rescaled only when its running maximum has grown by more than 2^8 since the scale
// it is stored at, by the softmax thread that owns the row.  While one group exponentiates,
// the tensor cores work on the other group's products, also for a query tile that is alone
// on its SM.
//
// Key tiles and the window (Section III-B).  A tile none of whose pairs is inside the window is
// scored by the telescoped product alone; a tile all of whose causal pairs are inside it by
// Q.K^T alone; a mixed tile takes the telescoped product first and then, one half of 64 keys
// at a time, hands the half the threads have read into registers back for Q.K^T, from which
// they take the in-window elements.
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
constexpr int NSW = 8;                     // softmax warps: two groups of 4
constexpr int WARP_QK = 8, WARP_PV = 9, WARP_TMA = 10;
constexpr int NTHR = 352;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TMEM_S = 0;             // score buffer of group 0 at column 0, of group 1 at column 128
constexpr uint32_t TMEM_O = 256;           // output tile of group 0 at 256, of group 1 at 256 + D
constexpr uint32_t TMEM_P64 = 384;         // d = 64: probabilities of group 0 at 384, of group 1 at 448
constexpr uint32_t SZ_BLK = 128 * 64 * 2;  // one [128 rows][64 elements] bf16 block, 16 KiB
constexpr float RESCALE_LOG2 = 8.0f;       // a row is rescaled when its maximum grew by more than 2^8
#ifndef DELTA_POLY_EVERY
#define DELTA_POLY_EVERY 4
#endif
constexpr int POLY_EVERY = DELTA_POLY_EVERY; // every n-th pair of exponentials by polynomial (0: none)
static_assert(POLY_EVERY == 0 || POLY_EVERY == 2 || POLY_EVERY == 4 || POLY_EVERY == 8 || POLY_EVERY == 16, "");

// Shared-memory map for head dimension D.  Operand tiles are D/64 blocks of [128][64] bf16 in
// the 128-byte-swizzle layout.  OFF_QH holds the reference-query tile (query deltas) or the
// original keys of a window tile (key deltas).  When the key loop is over, the ring space
// carries the exchange buffer of the final merge.
template <int D, bool PAIR> struct TqSmem {
  static constexpr uint32_t NKB = D / 64;                 // 64-element blocks per row
  static constexpr uint32_t SZ_TILE = NKB * SZ_BLK;       // one [128][D] operand tile
  static constexpr uint32_t NQ = PAIR ? 2 : 1;            // query tiles (heads) per CTA
  static constexpr uint32_t NKS = PAIR ? 3 : (D == 64) ? 4 : 3;      // key ring stages
  static constexpr uint32_t NVS = PAIR ? 3 : (D == 64) ? 4 : 2;      // value ring stages
  static constexpr uint32_t OFF_Q = 0;                    // [NQ] query tiles
  static constexpr uint32_t OFF_QH = OFF_Q + NQ * SZ_TILE;   // [NQ] reference-query tiles
  // d = 64, query deltas: two operand tiles mixed by row halves, [Q rows 0-63; Q_hat rows
  // 64-127] and [Q_hat rows 0-63; Q rows 64-127] (mixed tiles of block windows whose edges
  // fall on multiples of 64)
  static constexpr uint32_t OFF_QM = OFF_QH + NQ * SZ_TILE;  // [NQ][2]
  static constexpr uint32_t OFF_K = OFF_QM + ((D == 64) ? 2 * NQ * SZ_TILE : 0);
  static constexpr uint32_t OFF_V = OFF_K + NKS * SZ_TILE;
  static constexpr uint32_t OFF_BAR = OFF_V + NVS * SZ_TILE;
  static constexpr uint32_t OFF_MISC = OFF_BAR + 40 * 8;
  static constexpr uint32_t BYTES = OFF_MISC + 16 + 1024;
  static constexpr uint32_t XCH_FLOATS = 2 * 128 * (D / 2 + 2);   // merge exchange: [group][column][row]
  static_assert(XCH_FLOATS * 4 <= (NKS + NVS) * SZ_TILE, "the exchange buffer fits the ring space");
  static_assert(!PAIR || D == 64, "head pairs: d = 64 only");
  static_assert(BYTES <= 227 * 1024, "shared memory budget");
};

enum Bar {
  BAR_Q = 0,                 // query tile landed (one arrival + bytes)
  BAR_QH,                    // reference-query tile built (8 warps)
  BAR_KFULL0,                // + stage (up to 4)
  BAR_KFREE0 = BAR_KFULL0 + 4,
  BAR_VFULL0 = BAR_KFREE0 + 4,
  BAR_VFREE0 = BAR_VFULL0 + 4,
  BAR_KXFULL = BAR_VFREE0 + 4, BAR_KXFREE,    // original keys of a window tile (key deltas)
  BAR_SFULL0, BAR_SFULL1,    // a score product of the group is complete (tcgen05.commit)
  BAR_PRDY0, BAR_PRDY1,      // probabilities written (4 warps)
  BAR_SXREQ0, BAR_SXREQ1,    // telescoped scores read, the exact pass may overwrite them (4 warps)
  BAR_ODONE0, BAR_ODONE1,    // the group's last P.V is complete
  BAR_SCONS0, BAR_SCONS1,    // scores read, the next product may overwrite the buffer (4 warps; d = 64)
  BAR_PFREE0, BAR_PFREE1,    // a P.V is complete, the probabilities may be overwritten (d = 64)
  NUM_BARS
};
static_assert(NUM_BARS <= 40, "barrier space");

struct TqParams {
  __nv_bfloat16* out;
  unsigned long long* counters;
  const float* ckpt;           // [B,H,n_ckpt,D] reference in front of every 8-row block (query deltas only)
  int T, T_max, n_ckpt, H, g, W, shape;
  int BH;            // heads in all (batch x query heads)
  int n_one;         // two-head layout: the n_one heaviest query tiles of every head go one head per CTA
  int reverse;       // strategy (2): Eq. 2-3 runs from row T-1 down to row 0
  int basis_row;     // the un-thresholded basis row (0, or T-1 in reverse), -1 if there is none
  float scale_log2e, theta;
};

// Barrier of the eight softmax warps (id 1, 256 threads; immediate id: a register operand would
// make the compiler reserve all sixteen hardware barriers).
__device__ __forceinline__ void softmax_groups_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Maximum of the 32-column chunk Q of a score row; MASKED: only the columns up to `lane`.
template <int Q, bool MASKED>
__device__ __forceinline__ float chunk_max(const uint32_t (&u)[128], int lane) {
  float m0 = __uint_as_float(u[32 * Q]), m1 = -INFINITY;
#pragma unroll
  for (int c = 1; c < 32; c += 2) {
    const float a0 = __uint_as_float(u[32 * Q + c]);
    const float a1 = (c + 1 < 32) ? __uint_as_float(u[32 * Q + c + 1]) : -INFINITY;
    if (!MASKED) {
      m0 = fmax3(m0, a0, a1);
    } else {
      m0 = fmaxf(m0, c <= lane ? a0 : -INFINITY);
      m1 = fmaxf(m1, c + 1 <= lane ? a1 : -INFINITY);
    }
  }
  return fmaxf(m0, m1);
}

// Eq. 2-3 re-run over nbk 8-row blocks of two neighbouring channels of a query tile in shared
// memory (128-byte swizzle, offs[rr] = offset of row rr of a block), from the references in
// front of the blocks (ck[bk * ck_stride], `first` = the first block's, already loaded; the
// next block's is fetched while a block is worked on; the block loop is not unrolled: this code
// runs once per CTA and straight-line code costs more to fetch than it saves); writes the
// reference rows into the operand tile at qh_dst and, with
// `quarters`, the two row-mixed operand tiles at qm_dst ([Q rows 0-63; Q_hat rows 64-127] and
// the reverse).  REV: strategy (2), rows from the top.  CHECK: the tile holds rows past the
// end of the sequence (row0 + r >= T) or the un-thresholded basis row.
template <bool REV, bool CHECK>
__device__ __forceinline__ void build_ref_rows(const unsigned char* q_src, unsigned char* qh_dst, unsigned char* qm_dst,
                                               uint32_t sz_tile, const uint32_t (&offs)[DELTA_CKPT_ROWS],
                                               const float* ck, int ck_stride, float2 first, int nbk, float theta,
                                               bool quarters, int seg_row0, int row0, int T, int basis_row) {
  float2 nxt = first;
#pragma unroll 1
  for (int bk = 0; bk < nbk; ++bk) {
    float cur0 = nxt.x, cur1 = nxt.y;
    // (a block that starts inside the sequence has its reference: T <= T_max bounds the index)
    if (bk + 1 < nbk)
      nxt = (row0 + seg_row0 + (bk + 1) * DELTA_CKPT_ROWS < T)
                ? *reinterpret_cast<const float2*>(ck + (size_t)(bk + 1) * ck_stride) : make_float2(0.0f, 0.0f);
    const bool low = (seg_row0 + bk * DELTA_CKPT_ROWS) < 64;
    unsigned char* const m_q = qm_dst + (low ? 0u : sz_tile);     // takes the query rows of this block
    unsigned char* const m_h = qm_dst + (low ? sz_tile : 0u);     // takes the reference rows
#pragma unroll
    for (int rr = 0; rr < DELTA_CKPT_ROWS; ++rr) {
      const int r8 = REV ? DELTA_CKPT_ROWS - 1 - rr : rr;
      const uint32_t off = (uint32_t)bk * 1024u + offs[r8];
      const uint32_t xw = *reinterpret_cast<const uint32_t*>(q_src + off);
      const float x0 = __uint_as_float(xw << 16), x1 = __uint_as_float(xw & 0xffff0000u);
      bool f0 = fabsf(__fsub_rn(x0, cur0)) > theta, f1 = fabsf(__fsub_rn(x1, cur1)) > theta;
      if (CHECK) {
        // rows past the end of the sequence carry no state (in reverse they come first)
        const int gi = row0 + seg_row0 + bk * DELTA_CKPT_ROWS + r8;
        const bool basis = gi == basis_row, valid = gi < T;
        f0 = (f0 || basis) && valid;
        f1 = (f1 || basis) && valid;
      }
      cur0 = f0 ? x0 : cur0;
      cur1 = f1 ? x1 : cur1;
      // exact: the reference is a copy of an input element (or the zero it starts from)
      const uint32_t hw = __byte_perm(__float_as_uint(cur0), __float_as_uint(cur1), 0x7632);
      *reinterpret_cast<uint32_t*>(qh_dst + off) = hw;
      if (quarters) {
        *reinterpret_cast<uint32_t*>(m_q + off) = xw;
        *reinterpret_cast<uint32_t*>(m_h + off) = hw;
      }
    }
  }
}

}  // namespace

// KEY = false: query deltas (strategy 1, or 2 with p.reverse): telescoped scores Q_hat.K^T.  The
// reference rows of the query tile are rebuilt in shared memory from the query tile and the
// references the chain kernel left in front of every 8-row block (Eq. 2-3 re-run over 8 rows,
// blocks in parallel); tm_qh is unused.  KEY = true: key deltas (strategy 3): the column
// recursion telescopes to S[i][j] = q_i.k_hat(j), so the telescoped scores are Q.K_hat^T; tm_qh
// maps the reference-key rows (per KV head), which take the place of the key tiles in the ring,
// and the original keys are fetched only for tiles that touch the window.
// MIXED = false: no key tile of the launch is mixed (no window; a block window of whole
// 128-key tiles; or, query deltas at d = 64, a block window whose edges fall on multiples of
// 64): the code of the mixed tiles is left out,
// and with it every register spill of the kernel.
// FORM: 0 = every CTA one head; 1 = every CTA two heads; 2 = two-head layout, the form of a CTA
// follows its place in the grid (see below).
template <int D, bool KEY, int FORM, bool MIXED>
__global__ void __launch_bounds__(NTHR, 1)
hybrid_attn_tcq_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_qh,
                       const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                       const TqParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw);
  constexpr bool PAIR = FORM != 0;       // the layout holds two query tiles
  using SM = TqSmem<D, PAIR>;
  constexpr uint32_t NKB = SM::NKB, SZ_TILE = SM::SZ_TILE, NKS = SM::NKS, NVS = SM::NVS;
  constexpr uint32_t OFF_Q = SM::OFF_Q, OFF_QH = SM::OFF_QH, OFF_K = SM::OFF_K, OFF_V = SM::OFF_V,
                     OFF_BAR = SM::OFF_BAR, OFF_MISC = SM::OFF_MISC, OFF_QM = SM::OFF_QM;
  volatile uint32_t* sMisc = reinterpret_cast<volatile uint32_t*>(sm + OFF_MISC);
  volatile uint32_t* abort_flag = sMisc + 1;
  const uint32_t bar0 = base + OFF_BAR;
#define BAR(i) (bar0 + 8u * (uint32_t)(i))

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // Heaviest query tiles of every head first.  PAIR (the layout holds two query tiles): a
  // one-dimensional grid; its first BH * n_one CTAs take the n_one heaviest query tiles of every
  // head in the one-head form (key tiles dealt to the two softmax groups, merge at the end), the
  // others the same query tile of two neighbouring heads of one KV group, bh and bh + 1 (group
  // X of the softmax warps takes head bh + X and every key tile).  pr: this CTA is of the
  // second kind.
  int qt, bh;
  bool pr = false;
  if (PAIR) {
    const int nqt = (p.T + BM - 1) / BM, idx = (int)blockIdx.x, n1 = (FORM == 1) ? 0 : p.BH * p.n_one;
    if (FORM == 2 && idx < n1) {
      qt = nqt - 1 - idx / p.BH;
      bh = idx % p.BH;
    } else {
      const int j = idx - n1, hp = p.BH / 2;
      pr = true;
      qt = nqt - ((FORM == 1) ? 0 : p.n_one) - 1 - j / hp;
      bh = 2 * (j % hp);
    }
  } else {
    qt = (int)gridDim.y - 1 - (int)blockIdx.y;
    bh = (int)blockIdx.x;
  }
  const int b = bh / p.H, h = bh - b * p.H;
  const int bkv = b * (p.H / p.g) + h / p.g;
  const int T = p.T, W = p.W, shape = p.shape;
  const int i0 = qt * BM;
  const int i1 = min(i0 + BM, T) - 1;
  const int n = qt + 1;                                 // key tiles up to the diagonal
  // A unit is one (key tile, group) pair, issued and consumed in the order u = 0, 1, 2, ...;
  // unit u belongs to group u & 1 and is that group's (u >> 1)-th.  Key-split form: unit u is
  // key tile u; head-pair form: units 2t and 2t + 1 are key tile t for the two heads.
  const int U = pr ? 2 * n : n;
  auto tile_of = [&](int u) -> int { return pr ? (u >> 1) : u; };
  // d = 128 fills tensor memory with two score buffers and two output tiles: the probabilities
  // overwrite the scores they come from and a group's next score product has to follow its
  // P.V (one issuing thread does both).  d = 64 leaves room for the probabilities beside the
  // scores: the next score product is issued as soon as the group has read the buffer, by a
  // thread of its own, while another thread issues the P.V products.
  constexpr bool ALIAS = (D == 128);

  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     base + OFF_MISC),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp == WARP_TMA) {
    // the loader warp sets the barriers up (a thread takes barrier `lane` and, for the few past
    // 32, `lane + 32`) and has the query tile on its way before the CTA has even met: the
    // query tile is what the prologue waits for
    static_assert(NUM_BARS <= 64, "two barriers per thread at most");
#pragma unroll
    for (int i = lane; i < NUM_BARS; i += 32) {
      uint32_t cnt = 1;
      if (i == BAR_QH) cnt = NSW;
      if (i == BAR_PRDY0 || i == BAR_PRDY1 || i == BAR_SXREQ0 || i == BAR_SXREQ1 || i == BAR_SCONS0 ||
          i == BAR_SCONS1)
        cnt = 4;
      mbar_init(BAR(i), cnt);
    }
    if (lane == 0) sMisc[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
    __syncwarp();
    if (lane == 0) {
      const uint32_t nq = pr ? 2u : 1u;
      mbar_expect_tx(BAR(BAR_Q), nq * SZ_TILE);
      for (uint32_t x = 0; x < nq; ++x)
#pragma unroll
        for (uint32_t kb = 0; kb < NKB; ++kb)
          tma_load_3d(base + OFF_Q + x * SZ_TILE + kb * SZ_BLK, &tm_q, BAR(BAR_Q), 64 * kb, i0, bh + (int)x);
    }
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
  // Keys j with full_lo <= j <= full_hi are inside the window of EVERY row of the tile (block
  // window: the rows lie in one block; sliding: the keys within W of the first row).
  int full_lo = 1, full_hi = 0;
  if (W > 0) {
    if (shape == 0) { if (i1 < ex_lo + W) { full_lo = ex_lo; full_hi = ex_lo + W - 1; } }
    else { full_lo = i1 - W + 1; full_hi = i1; }
  }
  // A block window whose edges fall on multiples of 64 splits a mixed tile into quarters (row
  // half x key half) that are each wholly inside or outside the window: with the row-mixed
  // operand tiles such a tile needs no second pass (d = 64, query deltas).
  const bool quarters = (D == 64) && !KEY && shape == 0 && W > 0 && (W % 64) == 0;
  // 0: telescoped scores only, 1: mixed, 2: exact scores only, 3: mixed by quarters
  auto tile_class = [&](int t) -> int {
    const int j0 = t * BN, j1 = min(j0 + BN, T) - 1;
    if (!(j1 >= ex_lo && j0 <= ex_hi)) return 0;
    if (j0 >= full_lo && j1 <= full_hi) return 2;
    return quarters ? 3 : 1;
  };

  if (warp == WARP_TMA) {
    // =========================== loader ====================================================
    if (lane == 0) {
      auto load_tile = [&](uint32_t dst, const CUtensorMap* tm, uint32_t bar, int row0, int outer) {
#pragma unroll
        for (uint32_t kb = 0; kb < NKB; ++kb) tma_load_3d(dst + kb * SZ_BLK, tm, bar, 64 * kb, row0, outer);
      };
      // (the query tile is already on its way: see the set-up)
      // key deltas: the ring streams reference-key rows, which the finish kernel in front of
      // this one writes (programmatic stream serialisation): wait for them.  Queries, keys and
      // values themselves are inputs.
      if (KEY) asm volatile("griddepcontrol.wait;" ::: "memory");
      const CUtensorMap* tm_ring = KEY ? &tm_qh : &tm_k;
      int n_kx = 0;
      for (int t = 0; t < n; ++t) {
        const uint32_t ks = (uint32_t)t % NKS, vs = (uint32_t)t % NVS;
        if (t >= (int)NKS) mbar_wait(BAR(BAR_KFREE0 + ks), ((t / NKS) - 1) & 1, abort_flag);
        mbar_expect_tx(BAR(BAR_KFULL0 + ks), SZ_TILE);
        // (key deltas: a tile scored exactly throughout needs the original keys, not the reference keys)
        const int cls = tile_class(t);
        load_tile(base + OFF_K + ks * SZ_TILE, (KEY && cls == 2) ? &tm_k : tm_ring, BAR(BAR_KFULL0 + ks), t * BN, bkv);
        if (MIXED && KEY && cls == 1) {
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
  } else if (warp == WARP_QK) {
    // =========================== tensor-core issue: scores (d = 128: and P.V) ================
    if (lane == 0) {
      const uint32_t IDESC_QK = make_idesc(BN, 0);
      const uint32_t IDESC_PV = make_idesc(D, 1);
      // S = A . B^T into the score buffer of group X
      auto scores = [&](uint32_t X, uint32_t a, uint32_t bq) {
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc_mma(tmem + TMEM_S + 128u * X, make_desc(a + (ks >> 2) * SZ_BLK + (ks & 3) * 32, 16, 1024),
                 make_desc(bq + (ks >> 2) * SZ_BLK + (ks & 3) * 32, 16, 1024), IDESC_QK, ks > 0 ? 1u : 0u);
        tc_commit(BAR(BAR_SFULL0 + X));
      };
      const uint32_t IDESC_QK64 = make_idesc(64, 0);
      int n_kx = 0, n_sx0 = 0, n_sx1 = 0;
      // first scores of unit u, for group u & 1: telescoped, or exact where the whole tile
      // lies inside the window
      auto first_scores = [&](int u) {
        const int t = tile_of(u);
        const uint32_t X = (uint32_t)u & 1u;
        const uint32_t qsel = pr ? X * SZ_TILE : 0u;         // the group's own query tiles
        mbar_poll(BAR(BAR_KFULL0 + (uint32_t)t % NKS), (t / NKS) & 1, abort_flag);
        tc_fence_after();
        // query deltas: Q for an exact tile, Q_hat otherwise, against the keys; key deltas: Q
        // against what the loader put into the stage (original keys for an exact tile)
        const int cls = tile_class(t);
        const uint32_t ring = base + OFF_K + ((uint32_t)t % NKS) * SZ_TILE;
        if (cls == 3) {
          // each half of 64 keys against the operand tile whose row halves are Q where the
          // quarter lies inside the window and Q_hat where it does not
          const int rb0 = i0 / W, rb1 = (i0 + 64) / W;
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            const int jb = (t * BN + 64 * hf) / W;
            const bool in0 = rb0 == jb, in1 = rb1 == jb;
            const uint32_t a = base + (in0 ? (in1 ? OFF_Q + qsel : OFF_QM + 2 * qsel)
                                           : (in1 ? OFF_QM + 2 * qsel + SZ_TILE : OFF_QH + qsel));
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks)
              tc_mma(tmem + TMEM_S + 128u * X + 64u * hf, make_desc(a + (ks >> 2) * SZ_BLK + (ks & 3) * 32, 16, 1024),
                     make_desc(ring + 8192u * hf + (ks >> 2) * SZ_BLK + (ks & 3) * 32, 16, 1024), IDESC_QK64,
                     ks > 0 ? 1u : 0u);
          }
          tc_commit(BAR(BAR_SFULL0 + X));
          return;
        }
        const bool q_exact = KEY || cls == 2;
        scores(X, base + (q_exact ? OFF_Q : OFF_QH) + qsel, ring);
      };
      mbar_poll(BAR(BAR_Q), 0, abort_flag);
      if (!KEY) mbar_poll(BAR(BAR_QH), 0, abort_flag);   // the softmax warps have built Q_hat
      tc_fence_after();
      first_scores(0);
      if (U > 1) first_scores(1);
      for (int u = 0; u < U; ++u) {
        const int t = tile_of(u);
        const uint32_t X = (uint32_t)u & 1u;
        if (MIXED && tile_class(t) == 1) {
          // mixed tile: Q.K^T over each half of 64 keys once the group has that half's
          // telescoped scores in registers
          if (KEY) mbar_poll(BAR(BAR_KXFULL), n_kx & 1, abort_flag);   // (head pairs: the same tile for both heads)
          int& n_sx = X ? n_sx1 : n_sx0;
          const uint32_t kx = KEY ? base + OFF_QH : base + OFF_K + ((uint32_t)t % NKS) * SZ_TILE;
          const uint32_t qx = base + OFF_Q + (pr ? X * SZ_TILE : 0u);
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            mbar_poll(BAR(BAR_SXREQ0 + X), n_sx & 1, abort_flag);
            ++n_sx;
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks)
              tc_mma(tmem + TMEM_S + 128u * X + 64u * hf,
                     make_desc(qx + (ks >> 2) * SZ_BLK + (ks & 3) * 32, 16, 1024),
                     make_desc(kx + 8192u * hf + (ks >> 2) * SZ_BLK + (ks & 3) * 32, 16, 1024), IDESC_QK64,
                     ks > 0 ? 1u : 0u);
            tc_commit(BAR(BAR_SFULL0 + X));
          }
          if (KEY && (!pr || X == 1u)) { tc_commit(BAR(BAR_KXFREE)); ++n_kx; }
        }
        // every product that reads this key stage is issued (head pairs: after the second head's)
        if (!pr || X == 1u) tc_commit(BAR(BAR_KFREE0 + (uint32_t)t % NKS));
        if (ALIAS) {
          // P.V of this tile into the group's output tile, then the group's next scores at once
          mbar_poll(BAR(BAR_VFULL0 + (uint32_t)t % NVS), (t / NVS) & 1, abort_flag);
          mbar_poll(BAR(BAR_PRDY0 + X), (u >> 1) & 1, abort_flag);
          tc_fence_after();
          const uint32_t vb = base + OFF_V + ((uint32_t)t % NVS) * SZ_TILE;
#pragma unroll
          for (int ks = 0; ks < BN / 16; ++ks)
            tc_mma_ts(tmem + TMEM_O + (uint32_t)D * X, tmem + TMEM_S + 128u * X + 8u * ks,
                      make_desc(vb + ks * 2048, SZ_BLK, 1024), IDESC_PV, (u >= 2 || ks > 0) ? 1u : 0u);
          tc_commit(BAR(BAR_VFREE0 + (uint32_t)t % NVS));
          if (u + 2 >= U) tc_commit(BAR(BAR_ODONE0 + X));   // the group's last product
          else first_scores(u + 2);
        } else if (u + 2 < U) {
          // the group's next scores as soon as it has read this unit's
          mbar_poll(BAR(BAR_SCONS0 + X), (u >> 1) & 1, abort_flag);
          first_scores(u + 2);
        }
      }
    }
    __syncwarp();
  } else if (warp == WARP_PV) {
    // =========================== tensor-core issue: P.V (d = 64) ============================
    if (!ALIAS && lane == 0) {
      const uint32_t IDESC_PV = make_idesc(D, 1);
      for (int u = 0; u < U; ++u) {
        const int t = tile_of(u);
        const uint32_t X = (uint32_t)u & 1u;
        mbar_poll(BAR(BAR_VFULL0 + (uint32_t)t % NVS), (t / NVS) & 1, abort_flag);
        mbar_poll(BAR(BAR_PRDY0 + X), (u >> 1) & 1, abort_flag);
        tc_fence_after();
        const uint32_t vb = base + OFF_V + ((uint32_t)t % NVS) * SZ_TILE;
#pragma unroll
        for (int ks = 0; ks < BN / 16; ++ks)
          tc_mma_ts(tmem + TMEM_O + (uint32_t)D * X, tmem + TMEM_P64 + 64u * X + 8u * ks,
                    make_desc(vb + ks * 2048, SZ_BLK, 1024), IDESC_PV, (u >= 2 || ks > 0) ? 1u : 0u);
        if (!pr || X == 1u) tc_commit(BAR(BAR_VFREE0 + (uint32_t)t % NVS));
        if (u + 2 >= U) tc_commit(BAR(BAR_ODONE0 + X));   // the group's last product
        else tc_commit(BAR(BAR_PFREE0 + X));              // the group may write its next probabilities
      }
    }
    __syncwarp();
  } else {
    // =========================== softmax warps: one thread per score row ====================
    const uint32_t X = (uint32_t)warp >> 2;        // group: units u with u & 1 == X
    const int bh_x = bh + (pr ? (int)X : 0);       // the head whose rows this group holds
    const uint32_t qsel = pr ? X * SZ_TILE : 0u;   // its query tiles in shared memory
    const int w4 = warp & 3;
    const int row = 32 * w4 + lane;                // tensor-memory lane = row of the tile
    const int i = i0 + row;
    const uint32_t lane_sel = (uint32_t)(32 * (warp & 3)) << 16;
    const uint32_t t_s = tmem + TMEM_S + 128u * X + lane_sel;
    const uint32_t t_o = tmem + TMEM_O + (uint32_t)D * X + lane_sel;
    const uint32_t t_p = ALIAS ? t_s : tmem + TMEM_P64 + 64u * X + lane_sel;   // bf16 probabilities
    const float scale = p.scale_log2e;

    auto build_tile = [&]() {
      // ---- reference-query tile.  The chain kernel left the reference in front of every 8-row
      // block; thread (channel pair, row segment) re-runs Eq. 2-3 over its blocks from there (the
      // reference after row r is the last fired q[.][c] at or below r) and writes the rows of
      // Q_hat straight into the operand layout, two channels (one 32-bit word) at a time.
      // Blocks are independent of one another.  (head pairs: each group builds its own head's tile)
      const int NBT = pr ? NSW * 16 : NSW * 32;      // threads per tile
      const int SEG = BM / (NBT / (D / 2));          // rows per thread: 16, 32 or 64
      const int nbk = SEG / DELTA_CKPT_ROWS;
      const int tb = pr ? (tid & (NBT - 1)) : tid;
      const int c = 2 * (tb % (D / 2)), seg = tb / (D / 2);   // first channel of the pair, segment
      // byte offset of (row rr of an 8-row block, channel c) in a [128][D] tile with 128-byte
      // swizzle, less the block's own offset (8 rows = 1024 bytes, so r & 7 = rr)
      uint32_t offs[DELTA_CKPT_ROWS];
#pragma unroll
      for (int rr = 0; rr < DELTA_CKPT_ROWS; ++rr)
        offs[rr] = (uint32_t)rr * 128u + ((((uint32_t)(c & 63) >> 3) ^ (uint32_t)rr) << 4) + ((uint32_t)c & 7u) * 2u;
      const uint32_t thr_off = (uint32_t)(c >> 6) * SZ_BLK + (uint32_t)(seg * SEG) * 128u;
      asm volatile("griddepcontrol.wait;" ::: "memory");    // the chain kernel's checkpoints
      // the finish kernel behind needs the chain's results and nothing of this kernel's: once
      // every CTA has come by here (the last wave included) it may run on the SMs left idle
      if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
      const int r00 = i0 + seg * SEG;              // the thread's first row
      const float* const ck = p.ckpt + ((size_t)bh_x * p.n_ckpt + r00 / DELTA_CKPT_ROWS) * D + c;
      const float2 ref0 = (r00 < T && DELTA_IN(min(r00 + SEG - 1, T - 1) / DELTA_CKPT_ROWS, p.n_ckpt, p.counters))
                              ? *reinterpret_cast<const float2*>(ck) : make_float2(0.0f, 0.0f);
      mbar_wait(BAR(BAR_Q), 0, abort_flag);      // the query tile has landed
      const unsigned char* const q_src = sm + OFF_Q + qsel + thr_off;
      unsigned char* const qh_dst = sm + OFF_QH + qsel + thr_off;
      unsigned char* const qm_dst = sm + OFF_QM + 2 * qsel + thr_off;
      const bool check = (i0 + BM > T) || (p.basis_row >= i0 && p.basis_row < i0 + BM);
#define BUILD(REV, CHECK)                                                                              \
  build_ref_rows<REV, CHECK>(q_src, qh_dst, qm_dst, SZ_TILE, offs, ck, D, ref0, nbk, p.theta, quarters, seg * SEG, \
                                  i0, T, p.basis_row)
      if (p.reverse) { if (check) BUILD(true, true); else BUILD(true, false); }
      else { if (check) BUILD(false, true); else BUILD(false, false); }
#undef BUILD
      fence_proxy_async();      // written through the generic proxy, read by the tensor cores
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(BAR_QH));
    };

    int wlo = 0, whi = 0;       // exact keys of row i: wlo <= j < whi
    if (W > 0) {
      if (shape == 0) { wlo = (i / W) * W; whi = wlo + W; }
      else { wlo = i - W + 1; whi = i + 1; }
    }
    float m_used = -INFINITY;   // the scale (log2 domain) the row's P and O are stored at
    float l_sum = 0.0f;
    uint32_t s_phase = 0;
    // d = 64: the score buffer has been read (the next product may overwrite it) / the
    // previous P.V of the group is complete (the probabilities may be overwritten and the
    // output tile holds every earlier product of the group; waited for once per tile, as late
    // as the tile allows)
    auto s_consumed = [&]() {
      if (!ALIAS) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(BAR_SCONS0 + X));
      }
    };
    bool pv_waited = false;
    auto p_free = [&](int u) {
      if (!ALIAS && u >= 2 && !pv_waited) {
        mbar_wait(BAR(BAR_PFREE0 + X), ((u >> 1) - 1) & 1, abort_flag);
        tc_fence_after();
        pv_waited = true;
      }
    };
    // Rescale of the group's output tile.  The group's previous P.V is complete (d = 128: S_full
    // of this tile was committed behind it by the same thread; d = 64: p_free waits for it),
    // so the output tile holds every product so far; the rows whose maximum ran away since the
    // scale they are stored at are brought to the new one (whole warp together: the
    // tensor-memory accesses are warp-wide).
    // has_o: the output tile holds earlier products of the group; has_p0: the first half of this
    // tile's probabilities is already stored (second half of a mixed tile)
    auto settle_scale = [&](int u, float mx, bool has_o, bool has_p0) {
      const float m_new = fmaxf(m_used, mx * scale);
      if (!has_o && !has_p0) { m_used = m_new; return; }     // nothing stored at the old scale yet
      const bool grow = (m_new - m_used) > RESCALE_LOG2;
      if (__any_sync(0xffffffffu, grow)) {
        const float al = grow ? ex2(m_used - m_new) : 1.0f;
        if (grow) { l_sum *= al; m_used = m_new; }
        if (has_o) {
          p_free(u);
#pragma unroll
          for (int ch = 0; ch < D / 32; ++ch) {
            uint32_t u[32];
            tc_ld32(t_o + 32u * ch, u);
#pragma unroll
            for (int c = 0; c < 32; ++c) u[c] = __float_as_uint(__uint_as_float(u[c]) * al);
            tc_st32(t_o + 32u * ch, u);
          }
        }
        if (has_p0) {
          uint32_t u[32];
          tc_ld32(t_p, u);
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            const float lo_ = __uint_as_float(u[c] << 16) * al, hi_ = __uint_as_float(u[c] & 0xffff0000u) * al;
            const __nv_bfloat162 pk = __floats2bfloat162_rn(lo_, hi_);
            u[c] = *reinterpret_cast<const uint32_t*>(&pk);
          }
          tc_st32(t_p, u);
        }
        tc_wait_st();
      }
    };
    // 64 scores -> probabilities at the row's scale, bf16 pairs into tensor-memory columns
    // [32 hf, 32 hf + 32) of the probability buffer, row sum
    // live: how many of the half's two 32-column chunks hold anything but masked scores (the
    // same for every thread of the warp; the others' probabilities are zero without being computed)
    auto exp_store = [&](const float (&v)[64], int hf, int u, int live) {
      const float2 sc2 = make_float2(scale, scale), nm2 = make_float2(-m_used, -m_used);
      float2 sum_a = make_float2(0.0f, 0.0f), sum_b = make_float2(0.0f, 0.0f);
      uint32_t w[32];
#pragma unroll
      for (int qq = 0; qq < 2; ++qq) {
        if (qq < live) {
#pragma unroll
          for (int c = 32 * qq; c < 32 * qq + 32; c += 4) {
            const float2 e0 = ffma2(make_float2(v[c], v[c + 1]), sc2, nm2);
            const float2 e1 = ffma2(make_float2(v[c + 2], v[c + 3]), sc2, nm2);
            // one pair in POLY_EVERY on the FMA pipe instead of the exponential unit
            const bool poly = POLY_EVERY > 0 && (((c >> 1) + 1) % POLY_EVERY) == POLY_EVERY - 1;   // (POLY_EVERY: 2, 4, 8, 16)
            const float p0 = ex2(e0.x), p1 = ex2(e0.y);
            const float2 pp = poly ? ex2_poly2(e1) : make_float2(ex2(e1.x), ex2(e1.y));
            const float p2 = pp.x, p3 = pp.y;
            sum_a = fadd2(sum_a, make_float2(p0, p1));
            sum_b = fadd2(sum_b, make_float2(p2, p3));
            const __nv_bfloat162 pk0 = __floats2bfloat162_rn(p0, p1), pk1 = __floats2bfloat162_rn(p2, p3);
            w[c >> 1] = *reinterpret_cast<const uint32_t*>(&pk0);
            w[(c >> 1) + 1] = *reinterpret_cast<const uint32_t*>(&pk1);
          }
        } else {
#pragma unroll
          for (int c = 16 * qq; c < 16 * qq + 16; ++c) w[c] = 0u;
        }
      }
      p_free(u);      // the group's previous P.V has read the probabilities
      tc_st32(t_p + 32u * hf, w);
      l_sum += (sum_a.x + sum_a.y) + (sum_b.x + sum_b.y);
    };
    auto max64 = [&](const float (&v)[64]) -> float {
      float mx0 = fmax3(v[0], v[1], v[2]), mx1 = fmax3(v[3], v[4], v[5]);
      float mx2 = fmax3(v[6], v[7], v[8]), mx3 = fmax3(v[9], v[10], v[11]);
#pragma unroll
      for (int c = 12; c < 60; c += 8) {
        mx0 = fmax3(mx0, v[c], v[c + 1]); mx1 = fmax3(mx1, v[c + 2], v[c + 3]);
        mx2 = fmax3(mx2, v[c + 4], v[c + 5]); mx3 = fmax3(mx3, v[c + 6], v[c + 7]);
      }
      mx0 = fmax3(mx0, v[60], v[61]); mx1 = fmax3(mx1, v[62], v[63]);
      return fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
    };

    if (!KEY) build_tile();
    for (int u = (int)X; u < U; u += 2) {
      const int t = tile_of(u);
      mbar_wait(BAR(BAR_SFULL0 + X), s_phase & 1u, abort_flag);
      ++s_phase;
      tc_fence_after();
      const int j0 = t * BN;
      const bool diag = (t == qt);
      pv_waited = false;
      if (!MIXED || tile_class(t) != 1) {
        // ---- the common tile: two passes over the score buffer, the row maximum first, then the
        // exponentials in halves of 64 columns
        float mx;
        {
          uint32_t u[128];
          tc_ld128(t_s, u);
          if (!diag) {
            float m0 = fmax3(__uint_as_float(u[0]), __uint_as_float(u[1]), __uint_as_float(u[2]));
            float m1 = fmax3(__uint_as_float(u[3]), __uint_as_float(u[4]), __uint_as_float(u[5]));
            float m2 = fmax3(__uint_as_float(u[6]), __uint_as_float(u[7]), __uint_as_float(u[8]));
            float m3 = fmax3(__uint_as_float(u[9]), __uint_as_float(u[10]), __uint_as_float(u[11]));
#pragma unroll
            for (int c = 12; c < 124; c += 8) {
              m0 = fmax3(m0, __uint_as_float(u[c]), __uint_as_float(u[c + 1]));
              m1 = fmax3(m1, __uint_as_float(u[c + 2]), __uint_as_float(u[c + 3]));
              m2 = fmax3(m2, __uint_as_float(u[c + 4]), __uint_as_float(u[c + 5]));
              m3 = fmax3(m3, __uint_as_float(u[c + 6]), __uint_as_float(u[c + 7]));
            }
            m0 = fmax3(m0, __uint_as_float(u[124]), __uint_as_float(u[125]));
            m1 = fmax3(m1, __uint_as_float(u[126]), __uint_as_float(u[127]));
            mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
          } else {
            // causal mask on the diagonal tile.  The warp's rows are 32 w4 .. 32 w4 + 31 of the
            // tile: the 32-column chunks in front of chunk w4 are unmasked for all of them, chunk
            // w4 is masked behind each thread's own column, the chunks after it entirely
            mx = (w4 == 0) ? chunk_max<0, true>(u, lane) : chunk_max<0, false>(u, lane);
            if (w4 >= 1) mx = fmaxf(mx, (w4 == 1) ? chunk_max<1, true>(u, lane) : chunk_max<1, false>(u, lane));
            if (w4 >= 2) mx = fmaxf(mx, (w4 == 2) ? chunk_max<2, true>(u, lane) : chunk_max<2, false>(u, lane));
            if (w4 >= 3) mx = fmaxf(mx, chunk_max<3, true>(u, lane));
          }
        }
        settle_scale(u, mx, u >= 2, false);
        // the exponentials, one half of 64 columns at a time
        auto exp_half = [&](int hf) {
          float v[64];
          {
            uint32_t u[64];
            tc_ld64(t_s + 64u * hf, u);
#pragma unroll
            for (int c = 0; c < 64; ++c) v[c] = __uint_as_float(u[c]);
          }
          if (hf == 1) s_consumed();
          int live = 2;
          if (diag) {
            live = min(max(w4 + 1 - 2 * hf, 0), 2);
            // chunk w4 of the tile, if it lies in this half: masked behind the thread's own column
            // (selects on every element of the half: no index may depend on w4)
#pragma unroll
            for (int qq = 0; qq < 2; ++qq) {
              const bool part = w4 == 2 * hf + qq;
#pragma unroll
              for (int c = 1; c < 32; ++c) v[32 * qq + c] = (part && c > lane) ? -INFINITY : v[32 * qq + c];
            }
          }
          exp_store(v, hf, u, live);
        };
        if (D == 64) {
          // (two copies of the code: 8 % faster in the steady state than a loop)
          exp_half(0);
          exp_half(1);
        } else {
          // (d = 128: the two-copy form spills)
#pragma unroll 1
          for (int hf = 0; hf < 2; ++hf) exp_half(hf);
        }
      } else {
        // ---- a mixed tile (Section III-B hybrid select), one half of 64 keys at a time: the
        // half's telescoped scores go to registers, its columns go back for the exact product,
        // the in-window elements are taken from that
        auto mixed_half = [&](int hf) {
          float v[64];
          {
            uint32_t u[64];
            tc_ld64(t_s + 64u * hf, u);
#pragma unroll
            for (int c = 0; c < 64; ++c) v[c] = __uint_as_float(u[c]);
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(BAR(BAR_SXREQ0 + X));
          mbar_wait(BAR(BAR_SFULL0 + X), s_phase & 1u, abort_flag);
          ++s_phase;
          tc_fence_after();
#pragma unroll
          for (int ch = 0; ch < 2; ++ch) {
            uint32_t u[32];
            tc_ld32(t_s + 64u * hf + 32u * ch, u);
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const int j = j0 + 64 * hf + 32 * ch + c;
              if (j >= wlo && j < whi) v[32 * ch + c] = __uint_as_float(u[c]);
            }
          }
          if (hf == 1) s_consumed();
          if (diag) {
#pragma unroll
            for (int c = 0; c < 64; ++c)
              if (j0 + 64 * hf + c > i) v[c] = -INFINITY;
          }
          settle_scale(u, max64(v), u >= 2, hf == 1);
          exp_store(v, hf, u, 2);
        };
        if (D == 64) {
          mixed_half(0);
          mixed_half(1);
        } else {
#pragma unroll 1
          for (int hf = 0; hf < 2; ++hf) mixed_half(hf);
        }
      }
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(BAR_PRDY0 + X));
    }

    if (pr) {
      // ---- head pairs: the group's output tile is the whole result of its head's rows
      mbar_wait(BAR(BAR_ODONE0 + X), 0, abort_flag);
      tc_fence_after();
      const float inv = 1.0f / l_sum;
      const bool store = (i < T) && !*abort_flag && DELTA_IN(i, T, p.counters);
#pragma unroll
      for (int ch = 0; ch < D / 32; ++ch) {
        uint32_t u[32];
        tc_ld32(t_o + 32u * ch, u);
        if (store) {
          uint32_t w[16];
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const __nv_bfloat162 t2 = __floats2bfloat162_rn(__uint_as_float(u[c]) * inv, __uint_as_float(u[c + 1]) * inv);
            w[c >> 1] = *reinterpret_cast<const uint32_t*>(&t2);
          }
          uint4* op = reinterpret_cast<uint4*>(p.out + ((size_t)bh_x * T + i) * D + 32 * ch);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) op[q4] = make_uint4(w[4 * q4], w[4 * q4 + 1], w[4 * q4 + 2], w[4 * q4 + 3]);
        }
      }
      tc_fence_before();
    } else {
    // ---- merge the two groups' partial results, normalise, store.  Each group reads its own
    // output row from tensor memory, keeps the half of the columns it will store (group 0 the
    // lower half) and hands the other half, with its maximum and row sum, to the other group
    // through shared memory (the ring space: every product and every load is complete by then).
    const bool have = (int)X < n;                 // group 1 of a one-tile query tile has nothing
    // (both groups' last products: the exchange buffer lies over key stages the other group's
    // products may still be reading)
    mbar_wait(BAR(BAR_ODONE0), 0, abort_flag);
    if (n > 1) mbar_wait(BAR(BAR_ODONE1), 0, abort_flag);
    tc_fence_after();
    constexpr int HC = D / 2;                     // columns per group in the store
    float* xch = reinterpret_cast<float*>(sm + OFF_K);             // [group][HC + 2][128 rows]
    float* mine = xch + (size_t)X * (HC + 2) * 128;                // what this group leaves for the other
    const float* theirs = xch + (size_t)(X ^ 1u) * (HC + 2) * 128;
    const uint32_t t_give = t_o + (X ? 0u : (uint32_t)HC);          // the half the other group stores
    const uint32_t t_keep = t_o + (X ? (uint32_t)HC : 0u);
#pragma unroll
    for (int ch = 0; ch < HC / 32; ++ch) {
      uint32_t u[32];
      if (have) tc_ld32(t_give + 32u * ch, u);
#pragma unroll
      for (int c = 0; c < 32; ++c) mine[(32 * ch + c) * 128 + row] = have ? __uint_as_float(u[c]) : 0.0f;
    }
    mine[HC * 128 + row] = m_used;
    mine[(HC + 1) * 128 + row] = l_sum;
    softmax_groups_sync();
    const float m_o = theirs[HC * 128 + row], l_o = theirs[(HC + 1) * 128 + row];
    const float m_all = fmaxf(m_used, m_o);
    const float a_me = ex2(m_used - m_all), a_o = ex2(m_o - m_all);     // ex2(-inf) = 0 for an empty group
    const float inv = 1.0f / (l_sum * a_me + l_o * a_o);
    const float f_me = a_me * inv, f_o = a_o * inv;
    const bool store = (i < T) && !*abort_flag && DELTA_IN(i, T, p.counters);
#pragma unroll
    for (int ch = 0; ch < HC / 32; ++ch) {
      uint32_t u[32];
      if (have) tc_ld32(t_keep + 32u * ch, u);
      if (store) {
        uint32_t w[16];
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          const float k0 = have ? __uint_as_float(u[c]) : 0.0f, k1 = have ? __uint_as_float(u[c + 1]) : 0.0f;
          const float o0 = k0 * f_me + theirs[(32 * ch + c) * 128 + row] * f_o;
          const float o1 = k1 * f_me + theirs[(32 * ch + c + 1) * 128 + row] * f_o;
          const __nv_bfloat162 t2 = __floats2bfloat162_rn(o0, o1);
          w[c >> 1] = *reinterpret_cast<const uint32_t*>(&t2);
        }
        uint4* op = reinterpret_cast<uint4*>(p.out + ((size_t)bh * T + i) * D + HC * X + 32 * ch);
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

template <int D, bool KEY, int FORM, bool MIXED>
static cudaError_t launch_tcq_m(const Shape& s, const Workspace& w, const void* q, const void* k, const void* v,
                                void* out, int T, float theta, int init, int window, int shape, bool reverse,
                                int n_one, cudaStream_t st) {
  constexpr bool PAIR = FORM != 0;
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
  cudaError_t err = cudaFuncSetAttribute(hybrid_attn_tcq_kernel<D, KEY, FORM, MIXED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)TqSmem<D, PAIR>::BYTES);
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
  cudaLaunchConfig_t cfg = {};
  const int nqt = (T + BM - 1) / BM;
  p.BH = (int)BH;
  p.n_one = (FORM == 2) ? (n_one < nqt ? n_one : nqt) : 0;
  cfg.gridDim = PAIR ? dim3((unsigned)(BH * p.n_one + BH / 2 * (nqt - p.n_one))) : dim3((unsigned)BH, (unsigned)nqt);
  cfg.blockDim = dim3(NTHR);
  cfg.dynamicSmemBytes = TqSmem<D, PAIR>::BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  err = cudaLaunchKernelEx(&cfg, hybrid_attn_tcq_kernel<D, KEY, FORM, MIXED>, tq, tqh, tk, tv, p);
  count_launch();
  return err != cudaSuccess ? err : cudaGetLastError();
}

// Can a key tile be mixed (partly inside the window with no quarter structure)?  Mirrors the
// kernel's tile classes.
template <int D, bool KEY>
static bool mixed_tiles_possible(int window, int shape) {
  if (window <= 0) return false;
  // a block window of whole tiles: every key tile lies inside one block or outside it
  if (shape == 0 && (window % BN) == 0) return false;
  const bool quarters = (D == 64) && !KEY && shape == 0 && (window % 64) == 0;
  return !quarters;
}

template <int D, bool KEY, int FORM>
static cudaError_t launch_tcq(const Shape& s, const Workspace& w, const void* q, const void* k, const void* v,
                              void* out, int T, float theta, int init, int window, int shape, bool reverse,
                              int n_one, cudaStream_t st) {
  return mixed_tiles_possible<D, KEY>(window, shape)
             ? launch_tcq_m<D, KEY, FORM, true>(s, w, q, k, v, out, T, theta, init, window, shape, reverse, n_one, st)
             : launch_tcq_m<D, KEY, FORM, false>(s, w, q, k, v, out, T, theta, init, window, shape, reverse, n_one, st);
}

bool tcq_kernel_shape(int d) { return d == 64 || d == 128; }

cudaError_t launch_hybrid_attn_tcq(const Shape& s, const Workspace& w, const void* q, const void* k,
                                   const void* v, void* out, int T, float theta, int init, int window,
                                   int shape, bool key_deltas, bool reverse, int form, cudaStream_t st) {
  if (key_deltas && reverse) return cudaErrorNotSupported;
  if (!w.qhat_rows) return cudaErrorNotSupported;
  const bool two_heads_ok = s.d == 64 && (s.g() % 2) == 0;
  if ((form == 2 || form == 3) && !two_heads_ok) return cudaErrorNotSupported;
  if (s.d == 64) {
    // Two heads of a KV group per CTA share every key and value tile and need no merge, but a
    // head's key tiles are then walked by one softmax group instead of two.  That pays once
    // there are at least two such CTAs per SM (stack layer: 0.925 of the one-head form's time).
    // On a smaller grid that the one-head form cannot place in one wave, the heaviest query
    // tiles of every head go one head per CTA and the rest two heads per CTA, as many of the
    // former as one wave of SMs allows.
    const long BH = (long)s.B * s.H, nqt = (T + BM - 1) / BM, sms = device_sm_count();
    int n_one = -1;                       // -1: the one-head kernel
    if (form == 2) n_one = 0;
    else if (form == 3) n_one = 1;
    else if (form == 0 && two_heads_ok) {
      if (BH / 2 * nqt >= 2 * sms) n_one = 0;
      else if (BH * nqt > sms && BH / 2 * nqt <= sms) n_one = (int)((sms - BH / 2 * nqt) / (BH / 2));
    }
    if (key_deltas) {
      if (n_one == 0)
        return launch_tcq<64, true, 1>(s, w, q, k, v, out, T, theta, init, window, shape, reverse, 0, st);
      if (n_one > 0)
        return launch_tcq<64, true, 2>(s, w, q, k, v, out, T, theta, init, window, shape, reverse, n_one, st);
      return launch_tcq<64, true, 0>(s, w, q, k, v, out, T, theta, init, window, shape, reverse, 0, st);
    }
    if (n_one == 0)
      return launch_tcq<64, false, 1>(s, w, q, k, v, out, T, theta, init, window, shape, reverse, 0, st);
    if (n_one > 0)
      return launch_tcq<64, false, 2>(s, w, q, k, v, out, T, theta, init, window, shape, reverse, n_one, st);
    return launch_tcq<64, false, 0>(s, w, q, k, v, out, T, theta, init, window, shape, reverse, 0, st);
  }
  if (s.d == 128)
    return key_deltas
               ? launch_tcq<128, true, 0>(s, w, q, k, v, out, T, theta, init, window, shape, reverse, 0, st)
               : launch_tcq<128, false, 0>(s, w, q, k, v, out, T, theta, init, window, shape, reverse, 0, st);
  return cudaErrorNotSupported;
}

}  // namespace delta
