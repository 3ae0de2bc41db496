// K2 (tensor-core) -- fused hybrid delta attention for bf16 inputs on sm_100a
// (Section III-B; Eq. 1, Eq. 4; construction strategy (1) of Section III-A).
//
// One CTA owns 128 query rows of one head and walks the 128-key tiles up to the diagonal.
// 16 compute warps and one control warp; the work is split by what it is:
//   * dense contractions run on the 5th-generation tensor cores (tcgen05.mma issued by the
//     control thread, operands staged in shared memory by TMA, accumulators in tensor memory):
//     the exact Q.K^T of tiles that touch the window, and P.V of every tile;
//   * the out-of-window scores are Eq. 4's running sum of sparse delta products and stay on the
//     FP32 pipes, because the zeros of a thresholded delta matrix are unstructured.  A compute
//     warp owns 8 consecutive rows and all 128 keys of the tile (4 keys per lane).  Rows are
//     taken in blocks of 4: the OR of the 4 rows' mask words says which channels fired anywhere
//     in the block (ballot-style mask words, popc for list positions); channels whose 4x1 delta
//     block is all zero are never touched, every other channel costs one 16-byte key load
//     (channel-major fp32 key tile) and one 16-byte delta load for a 4x4 register tile of
//     multiply-adds.  Prefix sums over the rows turn the per-row products into R(i)[j]; the part
//     of the recursion in front of the warp's rows comes from the other warps' totals and from
//     the seed q_hat(i0-1).k_j (the reference in front of the tile telescopes all earlier rows);
//   * scale, causal mask, hybrid select and the online softmax run in the same key-per-lane
//     layout (row reductions as an 8-row butterfly); exact scores come out of tensor memory
//     row-per-thread and are transposed through shared memory; P goes to shared memory as bf16
//     in the tensor-core operand layout; the P.V tile product is read back from tensor memory
//     row-per-thread and accumulated in registers with the softmax rescale.
// Warps are decoupled: the channel-major key tile is double buffered and every hand-over
// (tile loaded / tile consumed / block totals ready / P ready / P.V done) is an mbarrier, so a
// warp that has finished its delta update moves on to its softmax while others still
// multiply.  Only tiles that touch the window synchronise the compute warps with a barrier.
//
// Every wait on an mbarrier is bounded; a wait that runs out records DELTA_ERR_TIMEOUT in the
// device status word, every later wait returns at once, the protocol still runs to its end (so
// no barrier is left short of arrivals) and the CTA frees its tensor memory and stores nothing.
#include <cuda.h>

#include "k2_tc.cuh"
#include "tc_common.cuh"

namespace delta {

using namespace tc;

namespace {

constexpr int BM = 128, BN = 128, NCWARP = 16, NCTHR = NCWARP * 32, NTHR = NCTHR + 32;
constexpr int TC_D = 64;                 // head dimension served by this kernel
constexpr uint32_t TMEM_COLS = 256;      // S: columns 0..127, O: columns 128..191
constexpr uint32_t TMEM_S = 0, TMEM_O = 128;

// shared-memory map (offsets from a 1024-byte aligned base)
constexpr uint32_t SZ_TILE = 128 * 64 * 2;               // one bf16 operand tile, 16 KiB
constexpr uint32_t ROW_B = 128 * 4;                      // one channel row of the fp32 tiles
constexpr uint32_t PAD_OFF = 64 * ROW_B;                 // row 64 of both fp32 tiles: padding target
constexpr uint32_t SZ_KT = 65 * ROW_B + 512;             // one channel-major key buffer (33792)
constexpr uint32_t OFF_Q = 0;
constexpr uint32_t OFF_K = OFF_Q + SZ_TILE;
constexpr uint32_t OFF_V = OFF_K + SZ_TILE;              // two buffers
constexpr uint32_t OFF_P = OFF_V + 2 * SZ_TILE;          // bf16 [2][128 rows][64 keys]
constexpr uint32_t OFF_KT = OFF_P + 2 * SZ_TILE;         // two buffers fp32 [64 channels + 1][128 keys]
constexpr uint32_t OFF_SX = OFF_KT;                      // fp32 [128][128] exact scores (over both)
constexpr uint32_t OFF_DQT = OFF_KT + 2 * SZ_KT;         // fp32 [64 channels + 1][128 rows]
constexpr uint32_t LIST_LD = 68;                         // list entries per block: 64 + one padding quad
constexpr uint32_t OFF_LIST = OFF_DQT + 65 * ROW_B;      // u32 [32 blocks][LIST_LD]: fired channel * ROW_B
constexpr uint32_t OFF_CNT = OFF_LIST + 32 * LIST_LD * 4;  // u32 [32]: list length / 4
constexpr uint32_t OFF_TOT = OFF_CNT + 32 * 4;           // fp32 [2][16][128]
constexpr uint32_t OFF_SEED = OFF_TOT + 2 * 16 * 128 * 4;  // fp32 [2][128]
constexpr uint32_t OFF_ALPHA = OFF_SEED + 2 * 128 * 4;   // fp32 [2][128]
constexpr uint32_t OFF_M = OFF_ALPHA + 2 * 128 * 4;      // fp32 [128] running max (scaled, log2 domain)
constexpr uint32_t OFF_L = OFF_M + 128 * 4;              // fp32 [128] running sum
constexpr uint32_t OFF_QHAT = OFF_L + 128 * 4;           // fp32 [64]
constexpr uint32_t OFF_BAR = OFF_QHAT + 64 * 4;          // mbarriers
constexpr uint32_t OFF_MISC = OFF_BAR + 16 * 8;          // tmem slot, abort flag
constexpr uint32_t SMEM_USED = OFF_MISC + 16;
constexpr uint32_t SMEM_BYTES = SMEM_USED + 1024;        // slack for the alignment of the base
static_assert(OFF_P % 1024 == 0 && OFF_KT % 1024 == 0 && SZ_KT % 1024 == 0, "1024-byte alignment");
static_assert(2 * SZ_KT >= 128 * 128 * 4, "exact-score buffer must fit in the two key buffers");
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");

enum Bar {
  BAR_Q = 0, BAR_K, BAR_V0, BAR_V1, BAR_S, BAR_O,     // one arrival (+ bytes) per phase
  BAR_KT_FULL0, BAR_KT_FULL1,                         // one arrival + bytes
  BAR_KT_EMPTY0, BAR_KT_EMPTY1,                       // 16 arrivals: every compute warp is done with it
  BAR_DELTA0, BAR_DELTA1,                             // 16 arrivals: block totals and seed written
  BAR_P,                                              // 16 arrivals: P tile written
  BAR_SX,                                             // 16 arrivals: exact scores consumed
  NUM_BARS
};

__device__ __forceinline__ void compute_barrier() {   // the 16 compute warps only
  asm volatile("bar.sync 1, %0;" ::"n"(NCTHR) : "memory");
}

// Reduction of 8 per-lane values (one per row of the warp's row group) over the 32 lanes in
// 9 shuffles: the halves of the value set are exchanged while the lane distance halves.  On
// return every lane holds the warp-wide result of row (lane >> 2) & 7.
template <bool IS_MAX>
__device__ __forceinline__ float reduce8(const float (&v)[8], int lane) {
  auto op = [](float a, float b) { return IS_MAX ? fmaxf(a, b) : a + b; };
  float w[4], u[2];
  const bool h16 = lane & 16, h8 = lane & 8, h4 = lane & 4;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float send = h16 ? v[i] : v[i + 4], keep = h16 ? v[i + 4] : v[i];
    w[i] = op(keep, __shfl_xor_sync(0xffffffffu, send, 16));
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const float send = h8 ? w[i] : w[i + 2], keep = h8 ? w[i + 2] : w[i];
    u[i] = op(keep, __shfl_xor_sync(0xffffffffu, send, 8));
  }
  const float send = h4 ? u[0] : u[1], keep = h4 ? u[1] : u[0];
  float z = op(keep, __shfl_xor_sync(0xffffffffu, send, 4));
  z = op(z, __shfl_xor_sync(0xffffffffu, z, 2));
  z = op(z, __shfl_xor_sync(0xffffffffu, z, 1));
  return z;
}

struct TcParams {
  const float* dq;
  const uint32_t* mask;
  const float* qhat_tile;
  __nv_bfloat16* out;
  unsigned long long* counters;
  int T, T_max, n_tiles64, H, g, W, shape;
  float scale_log2e;
};

}  // namespace

__global__ void __launch_bounds__(NTHR, 1)
hybrid_attn_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                      const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_kt,
                      const TcParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw);

  float* sdQt = reinterpret_cast<float*>(sm + OFF_DQT);
  uint32_t* sList = reinterpret_cast<uint32_t*>(sm + OFF_LIST);
  uint32_t* sCnt = reinterpret_cast<uint32_t*>(sm + OFF_CNT);
  float* sTot = reinterpret_cast<float*>(sm + OFF_TOT);
  float* sSeed = reinterpret_cast<float*>(sm + OFF_SEED);
  float* sAlpha = reinterpret_cast<float*>(sm + OFF_ALPHA);
  float* sM = reinterpret_cast<float*>(sm + OFF_M);
  float* sL = reinterpret_cast<float*>(sm + OFF_L);
  float* sQhat = reinterpret_cast<float*>(sm + OFF_QHAT);
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
  const int i1 = min(i0 + BM, T) - 1;           // last valid row of the tile

  // ---- set-up: tensor memory, barriers ----------------------------------------------------
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     base + OFF_MISC),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    for (int i = 0; i < NUM_BARS; ++i)
      mbar_init(BAR(i), (i >= BAR_KT_EMPTY0) ? (uint32_t)NCWARP : 1u);
    sMisc[1] = 0;  // abort flag
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sMisc[0];

  auto tile_needs_exact = [&](int jt) -> bool {
    if (W <= 0) return false;
    const int j0 = jt * BN, j1 = min(j0 + BN, T) - 1;
    if (shape == 0) return (i0 / W <= j1 / W) && (j0 / W <= i1 / W);
    return max(0, i0 - j1) < W;
  };
  auto tile_all_in = [&](int jt) -> bool {
    if (W <= 0) return false;
    const int j0 = jt * BN, j1 = min(j0 + BN, T) - 1;
    if (shape == 0) return (i0 / W == i1 / W) && (j0 / W == j1 / W) && (i0 / W == j0 / W);
    return (i1 - j0) < W;
  };

  if (warp == NCWARP) {
    // =========================== control warp: TMA and tensor-core issue =====================
    if (lane == 0) {
      const uint32_t IDESC_QK = make_idesc(BN, 0);
      const uint32_t IDESC_PV = make_idesc(TC_D, 1);
      if (W > 0) {
        mbar_expect_tx(BAR(BAR_Q), SZ_TILE);
        tma_load_3d(base + OFF_Q, &tm_q, BAR(BAR_Q), 0, i0, bh);
      }
      mbar_expect_tx(BAR(BAR_KT_FULL0), 64 * ROW_B);
      tma_load_3d(base + OFF_KT, &tm_kt, BAR(BAR_KT_FULL0), 0, 0, bkv);
      mbar_expect_tx(BAR(BAR_V0), SZ_TILE);
      tma_load_3d(base + OFF_V, &tm_v, BAR(BAR_V0), 0, 0, bkv);
      if (tile_needs_exact(0)) {
        mbar_expect_tx(BAR(BAR_K), SZ_TILE);
        tma_load_3d(base + OFF_K, &tm_k, BAR(BAR_K), 0, 0, bkv);
      }
      int nk = 0;   // exact tiles so far: parity of BAR_K, BAR_S, BAR_SX
      for (int t = 0; t <= qt; ++t) {
        const bool exact = tile_needs_exact(t);
        const bool more = t < qt;
        const int nb = (t + 1) & 1;
        auto load_next_keys = [&]() {
          mbar_expect_tx(BAR(BAR_KT_FULL0 + nb), 64 * ROW_B);
          tma_load_3d(base + OFF_KT + nb * SZ_KT, &tm_kt, BAR(BAR_KT_FULL0 + nb), (t + 1) * BN, 0, bkv);
          if (tile_needs_exact(t + 1)) {
            mbar_expect_tx(BAR(BAR_K), SZ_TILE);
            tma_load_3d(base + OFF_K, &tm_k, BAR(BAR_K), 0, (t + 1) * BN, bkv);
          }
        };
        if (exact) {   // exact Q.K^T of a tile that touches the window
          mbar_wait(BAR(BAR_K), nk & 1, abort_flag);
          if (nk == 0) mbar_wait(BAR(BAR_Q), 0, abort_flag);
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < TC_D / 16; ++ks) {
            const uint64_t da = make_desc(base + OFF_Q + ks * 32, 16, 1024);
            const uint64_t db = make_desc(base + OFF_K + ks * 32, 16, 1024);
            tc_mma(tmem + TMEM_S, da, db, IDESC_QK, ks > 0 ? 1u : 0u);
          }
          tc_commit(BAR(BAR_S));
        }
        if (t >= 1) mbar_wait(BAR(BAR_O), (t - 1) & 1, abort_flag);   // P.V(t-1) done: its V buffer is free
        if (more) {
          mbar_expect_tx(BAR(BAR_V0 + nb), SZ_TILE);
          tma_load_3d(base + OFF_V + nb * SZ_TILE, &tm_v, BAR(BAR_V0 + nb), 0, (t + 1) * BN, bkv);
        }
        if (!exact) {
          if (more) {
            if (t >= 1) mbar_wait(BAR(BAR_KT_EMPTY0 + nb), ((t - 1) >> 1) & 1, abort_flag);
            load_next_keys();
          }
        } else {
          // the exact scores of this tile lie over both key buffers: reload only once consumed
          mbar_wait(BAR(BAR_SX), nk & 1, abort_flag);
          if (more) load_next_keys();
          ++nk;
        }
        // P.V on the tensor cores
        mbar_wait(BAR(BAR_P), t & 1, abort_flag);
        mbar_wait(BAR(BAR_V0 + (t & 1)), (t >> 1) & 1, abort_flag);
        tc_fence_after();
        const uint32_t vbase = base + OFF_V + (t & 1) * SZ_TILE;
#pragma unroll
        for (int ks = 0; ks < BN / 16; ++ks) {
          const uint64_t da = make_desc(base + OFF_P + (ks >> 2) * SZ_TILE + (ks & 3) * 32, 16, 1024);
          const uint64_t db = make_desc(vbase + ks * 2048, SZ_TILE, 1024);
          tc_mma(tmem + TMEM_O, da, db, IDESC_PV, ks > 0 ? 1u : 0u);
        }
        tc_commit(BAR(BAR_O));
      }
    }
    __syncwarp();
  } else {
    // =========================== compute warps ===============================================
    const int qd = warp & 3, sub = warp >> 2;     // tensor-memory lane quadrant / slot in it
    const int rg = qd * 4 + sub;                  // row group: rows 8*rg .. 8*rg+7
    const int my_row = 32 * qd + lane;            // row this thread owns in row-per-thread phases
    const int rho = (lane >> 2) & 7;              // row of the group whose reductions this lane ends up with

    // ---- stage the query tile: deltas channel-major, per 4-row block the list of channels that
    // fired anywhere in the block (OR of the mask words, popc for the position), the seed
    // reference, the softmax state
    {
      const float* dqp = p.dq + ((size_t)bh * p.T_max + i0) * TC_D;
      const int r_sub = lane >> 3, c_sub = lane & 7;
      for (int it = warp; it < 32 * 8; it += NCWARP) {
        const int rb = it >> 3, cb = it & 7;
        const int r = rb * 4 + r_sub, c = cb * 8 + c_sub;
        const float x = (i0 + r < T) ? dqp[(size_t)r * TC_D + c] : 0.0f;
        sdQt[c * BM + r] = x;
      }
      if (tid < 128) {               // row 64 of the fp32 tiles: where list padding points
        sdQt[64 * BM + tid] = 0.0f;
        reinterpret_cast<float*>(sm + OFF_KT)[64 * BN + tid] = 0.0f;
        reinterpret_cast<float*>(sm + OFF_KT + SZ_KT)[64 * BN + tid] = 0.0f;
      }
      {
        const int blk = tid >> 4, sl = tid & 15;     // 16 threads per block of 4 rows
        unsigned long long u = 0;
        const uint32_t* mp = p.mask + ((size_t)bh * p.T_max + i0 + blk * 4) * 2;
#pragma unroll
        for (int r = 0; r < 4; ++r)
          if (i0 + blk * 4 + r < T)
            u |= (unsigned long long)mp[r * 2] | ((unsigned long long)mp[r * 2 + 1] << 32);
        const int n = __popcll(u);
        uint32_t* lp = sList + blk * LIST_LD;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int c = sl * 4 + k;
          if ((u >> c) & 1ull) lp[__popcll(u & ((1ull << c) - 1ull))] = (uint32_t)c * ROW_B;
        }
        // pad to a multiple of 4 and add one more quad: the loop reads one quad ahead
        const int n4 = (n + 3) >> 2;
        if (sl < 7 && n + sl < n4 * 4 + 4) lp[n + sl] = PAD_OFF;
        if (sl == 0) sCnt[blk] = (uint32_t)n4;
      }
      if (tid < TC_D) sQhat[tid] = p.qhat_tile[((size_t)bh * p.n_tiles64 + 2 * qt) * TC_D + tid];
      if (tid < BM) { sM[tid] = -INFINITY; sL[tid] = 0.0f; }
    }
    float O[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) O[i] = 0.0f;
    compute_barrier();

    const float scale = p.scale_log2e;
    int n_exact = 0;          // exact tiles seen so far (parity of BAR_S)

    for (int jt = 0; jt <= qt; ++jt) {
      const int j0 = jt * BN;
      const int bf = jt & 1;
      const bool need_exact = tile_needs_exact(jt);
      const bool need_delta = !tile_all_in(jt);
      const bool diag = (jt == qt);

      // ---- Eq. 4 on the FP32 pipes: block-sparse 4x4 register tiles over fired channels
      float Sl[8][4];
#pragma unroll
      for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int k = 0; k < 4; ++k) Sl[r][k] = 0.0f;
      mbar_wait(BAR(BAR_KT_FULL0 + bf), (jt >> 1) & 1, abort_flag);
      if (need_delta) {
        float run[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        const uint32_t ktb = base + OFF_KT + bf * SZ_KT + 16 * lane;
#pragma unroll
        for (int g4 = 0; g4 < 2; ++g4) {
          float a[4][4];
#pragma unroll
          for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int k = 0; k < 4; ++k) a[r][k] = 0.0f;
          const int blk = rg * 2 + g4;
          const uint32_t dqb = base + OFF_DQT + 16 * blk;
          const uint32_t lpa = base + OFF_LIST + blk * (LIST_LD * 4);
          const int n4 = (int)sCnt[blk];
          // software pipeline over single entries: the loads of the next entry are in flight
          // while the current entry's 16 multiply-adds issue
          uint4 e = lds128u(lpa);
          float4 kvA, dvA, kvB, dvB;
          auto mac16 = [&](const float4& kv, const float4& dv) {
            const float kk[4] = {kv.x, kv.y, kv.z, kv.w};
            const float dd[4] = {dv.x, dv.y, dv.z, dv.w};
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
              for (int k = 0; k < 4; ++k) a[r][k] = fmaf(dd[r], kk[k], a[r][k]);
          };
          kvA = lds128(ktb + e.x); dvA = lds128(dqb + e.x);
          for (int q4 = 0; q4 < n4; ++q4) {
            kvB = lds128(ktb + e.y); dvB = lds128(dqb + e.y);
            mac16(kvA, dvA);
            kvA = lds128(ktb + e.z); dvA = lds128(dqb + e.z);
            mac16(kvB, dvB);
            kvB = lds128(ktb + e.w); dvB = lds128(dqb + e.w);
            e = lds128u(lpa + 16 * (q4 + 1));      // next quad (the list carries one padding quad)
            mac16(kvA, dvA);
            kvA = lds128(ktb + e.x); dvA = lds128(dqb + e.x);
            mac16(kvB, dvB);
          }
#pragma unroll
          for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              run[k] += a[r][k];
              Sl[g4 * 4 + r][k] = run[k];
            }
        }
        *reinterpret_cast<float4*>(sTot + (bf * 16 + rg) * BN + 4 * lane) =
            make_float4(run[0], run[1], run[2], run[3]);
        // seed q_hat(i0-1).k_j: this warp serves keys 8*warp .. 8*warp+7, 16 channels per lane
        if (qt > 0) {
          const int kq = lane & 7, cq = lane >> 3;
          const float* kp = reinterpret_cast<const float*>(sm + OFF_KT + bf * SZ_KT) + cq * 16 * BN + 8 * warp + kq;
          float sd = 0.0f;
#pragma unroll
          for (int cc = 0; cc < 16; ++cc) sd = fmaf(sQhat[cq * 16 + cc], kp[cc * BN], sd);
          sd += __shfl_xor_sync(0xffffffffu, sd, 8);
          sd += __shfl_xor_sync(0xffffffffu, sd, 16);
          if (lane < 8) sSeed[bf * BN + 8 * warp + lane] = sd;
        } else if (lane < 8) {
          sSeed[bf * BN + 8 * warp + lane] = 0.0f;
        }
      }
      fence_proxy_async();   // generic reads of the key tile are ordered before its next bulk write
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(BAR(BAR_KT_EMPTY0 + bf));
        mbar_arrive(BAR(BAR_DELTA0 + bf));
      }

      // ---- previous tile's P.V: rescale and accumulate (row-per-thread)
      if (jt > 0) {
        mbar_wait(BAR(BAR_O), (jt - 1) & 1, abort_flag);
        tc_fence_after();
        float v[16];
        tc_ld16(tmem + TMEM_O + 16 * sub + ((uint32_t)(32 * qd) << 16), v);
        const float al = sAlpha[((jt - 1) & 1) * BM + my_row];
#pragma unroll
        for (int i = 0; i < 16; ++i) O[i] = fmaf(O[i], al, v[i]);
        tc_fence_before();
      }

      // ---- every warp's block totals and seed slice are written
      mbar_wait(BAR(BAR_DELTA0 + bf), (jt >> 1) & 1, abort_flag);

      // ---- exact scores: tensor memory (row per thread) -> shared memory, 16-byte XOR swizzle
      if (need_exact) {
        mbar_wait(BAR(BAR_S), n_exact & 1, abort_flag);
        tc_fence_after();
        unsigned char* sx_row = sm + OFF_SX + (size_t)my_row * 512;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          float v[16];
          tc_ld16(tmem + TMEM_S + 32 * sub + 16 * half + ((uint32_t)(32 * qd) << 16), v);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const int chunk = 8 * sub + 4 * half + q4;
            *reinterpret_cast<float4*>(sx_row + ((chunk ^ lane) << 4)) =
                make_float4(v[4 * q4], v[4 * q4 + 1], v[4 * q4 + 2], v[4 * q4 + 3]);
          }
        }
        tc_fence_before();
        compute_barrier();     // exact scores visible to the warps that own the rows
      }

      // ---- pass 1: hybrid select (Section III-B): exact inside the window, running sum outside
      {
        float bs[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        if (need_delta) {
          const float4 s4 = *reinterpret_cast<const float4*>(sSeed + bf * BN + 4 * lane);
          bs[0] = s4.x; bs[1] = s4.y; bs[2] = s4.z; bs[3] = s4.w;
          for (int r2 = 0; r2 < rg; ++r2) {
            const float4 t4 = *reinterpret_cast<const float4*>(sTot + (bf * 16 + r2) * BN + 4 * lane);
            bs[0] += t4.x; bs[1] += t4.y; bs[2] += t4.z; bs[3] += t4.w;
          }
        }
#pragma unroll
        for (int r = 0; r < 8; ++r) {
          const int row = rg * 8 + r;
          const int i = i0 + row;
#pragma unroll
          for (int k = 0; k < 4; ++k) Sl[r][k] += bs[k];
          if (need_exact) {
            int wlo, whi;   // exact keys of row i: wlo <= j < whi
            if (shape == 0) { wlo = (i / W) * W; whi = wlo + W; }
            else { wlo = i - W + 1; whi = i + 1; }
            const float4 e4 = *reinterpret_cast<const float4*>(sm + OFF_SX + (size_t)row * 512 +
                                                               ((lane ^ (row & 31)) << 4));
            const float ex[4] = {e4.x, e4.y, e4.z, e4.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int j = j0 + 4 * lane + k;
              if (j >= wlo && j < whi) Sl[r][k] = ex[k];
            }
          }
          if (diag) {
#pragma unroll
            for (int k = 0; k < 4; ++k)
              if (4 * lane + k > row) Sl[r][k] = -INFINITY;   // causal mask on the diagonal tile
          }
        }
      }
      if (need_exact) {
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(BAR_SX));   // this warp no longer needs the exact-score buffer
        ++n_exact;
      }

      // ---- pass 2: scale, online softmax (Eq. 1); P as bf16 in the operand layout
      {
        float v8[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) v8[r] = fmaxf(fmaxf(Sl[r][0], Sl[r][1]), fmaxf(Sl[r][2], Sl[r][3]));
        const float zmax = reduce8<true>(v8, lane);          // raw maximum of row rho
        const int row_o = rg * 8 + rho;
        const float m_old = sM[row_o];
        const float m_new = fmaxf(m_old, zmax * scale);
        const float al = ex2(m_old - m_new);
        float mn[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) mn[r] = __shfl_sync(0xffffffffu, m_new, 4 * r);
#pragma unroll
        for (int r = 0; r < 8; ++r) {
          const int row = rg * 8 + r;
#pragma unroll
          for (int k = 0; k < 4; ++k) Sl[r][k] = ex2(fmaf(Sl[r][k], scale, -mn[r]));
          v8[r] = (Sl[r][0] + Sl[r][1]) + (Sl[r][2] + Sl[r][3]);
          const __nv_bfloat162 lo = __floats2bfloat162_rn(Sl[r][0], Sl[r][1]);
          const __nv_bfloat162 hi = __floats2bfloat162_rn(Sl[r][2], Sl[r][3]);
          uint2 pk;
          pk.x = *reinterpret_cast<const uint32_t*>(&lo);
          pk.y = *reinterpret_cast<const uint32_t*>(&hi);
          unsigned char* pp = sm + OFF_P + (size_t)(lane >> 4) * SZ_TILE + (size_t)row * 128 +
                              ((((lane & 15) >> 1) ^ (row & 7)) << 4) + ((lane & 1) << 3);
          *reinterpret_cast<uint2*>(pp) = pk;
        }
        const float zsum = reduce8<false>(v8, lane);
        if ((lane & 3) == 0) {
          sAlpha[bf * BM + row_o] = al;
          sL[row_o] = fmaf(sL[row_o], al, zsum);
          sM[row_o] = m_new;
        }
      }
      fence_proxy_async();   // P was written through the generic proxy, the tensor cores read it
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(BAR_P));
    }

    // ---- last tile's P.V, normalisation, store -------------------------------------------
    mbar_wait(BAR(BAR_O), qt & 1, abort_flag);
    tc_fence_after();
    float v[16];
    tc_ld16(tmem + TMEM_O + 16 * sub + ((uint32_t)(32 * qd) << 16), v);
    const float al = sAlpha[(qt & 1) * BM + my_row];
    const float inv = 1.0f / sL[my_row];
    if (i0 + my_row < T && !*abort_flag) {
      uint32_t w[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const __nv_bfloat162 t2 = __floats2bfloat162_rn(fmaf(O[2 * i], al, v[2 * i]) * inv,
                                                        fmaf(O[2 * i + 1], al, v[2 * i + 1]) * inv);
        w[i] = *reinterpret_cast<const uint32_t*>(&t2);
      }
      uint4* op = reinterpret_cast<uint4*>(p.out + ((size_t)bh * T + i0 + my_row) * TC_D + 16 * sub);
      op[0] = make_uint4(w[0], w[1], w[2], w[3]);
      op[1] = make_uint4(w[4], w[5], w[6], w[7]);
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

// ---------------------------------------------------------------------------------------
namespace tc {
EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      f = nullptr;
    return (EncodeTiledFn)f;
  }();
  return fn;
}

bool encode3(CUtensorMap* m, CUtensorMapDataType dt, const void* ptr, uint64_t inner, uint64_t rows,
             uint64_t outer, uint64_t row_stride_b, uint64_t outer_stride_b, uint32_t box_inner,
             uint32_t box_rows, CUtensorMapSwizzle sw) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {inner, rows, outer};
  const cuuint64_t strides[2] = {row_stride_b, outer_stride_b};
  const cuuint32_t box[3] = {box_inner, box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, dt, 3, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
}  // namespace tc

bool tc_kernel_shape(int d) { return d == TC_D; }
bool tc_kernel_available(int d) { return d == TC_D && encode_fn() != nullptr; }

cudaError_t launch_hybrid_attn_tc(const Shape& s, const Workspace& w, const void* q, const void* k,
                                  const void* v, void* out, int T, int window, int shape,
                                  cudaStream_t st) {
  if (s.d != TC_D || !w.kt) return cudaErrorNotSupported;
  const int ld = (s.T_max + 3) / 4 * 4;
  const uint64_t BH = (uint64_t)s.B * s.H, BKV = (uint64_t)s.B * s.H_kv;
  CUtensorMap tq, tk, tv, tkt;
  const bool ok =
      encode3(&tq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, q, TC_D, (uint64_t)T, BH, TC_D * 2,
              (uint64_t)T * TC_D * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B) &&
      encode3(&tk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, k, TC_D, (uint64_t)T, BKV, TC_D * 2,
              (uint64_t)s.T_max * TC_D * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B) &&
      encode3(&tv, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, v, TC_D, (uint64_t)T, BKV, TC_D * 2,
              (uint64_t)s.T_max * TC_D * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B) &&
      encode3(&tkt, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, w.kt, (uint64_t)T, TC_D, BKV, (uint64_t)ld * 4,
              (uint64_t)ld * TC_D * 4, 128, 64, CU_TENSOR_MAP_SWIZZLE_NONE);
  if (!ok) return cudaErrorInvalidValue;

  cudaError_t err;
  err = cudaFuncSetAttribute(hybrid_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)SMEM_BYTES);
  if (err != cudaSuccess) return err;
  TcParams p;
  p.dq = w.dq; p.mask = w.mask; p.qhat_tile = w.qhat_tile; p.out = (__nv_bfloat16*)out;
  p.counters = w.counters;
  p.T = T; p.T_max = s.T_max; p.n_tiles64 = s.n_tiles; p.H = s.H; p.g = s.g(); p.W = window; p.shape = shape;
  p.scale_log2e = 1.4426950408889634f / sqrtf((float)s.d);
  const dim3 grid((unsigned)BH, (T + BM - 1) / BM);
  hybrid_attn_tc_kernel<<<grid, NTHR, SMEM_BYTES, st>>>(tq, tk, tv, tkt, p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace delta
