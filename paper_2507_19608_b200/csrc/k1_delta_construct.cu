// K1 -- delta construction (Section II-C, Eq. 2-3; Section III-A strategies (1), (2), (3)), in
// two kernels.
//
// delta_chain_kernel: the token-sequential part.  Eq. 3 makes every channel a chain along the
// tokens (the reference is the last value that fired), so the only parallelism is across
// channels: one thread per channel, one CTA per (batch, head, 32 channels) of the stream (query
// heads, or KV heads for key deltas).  The chain itself is three dependent FP32 operations per
// token and a lone warp issues slowly, so everything else is kept off it: a producer warp
// streams the rows into a ring of shared-memory stages with TMA (the rows do not depend on the
// carried state), helper warps precompute everything about a four-row sub-block that does not
// involve the carried state (see the kernel), and the chain warp stores nothing but the
// reference in front of every 8-row block (and every 64-row tile, and the final one).  Given
// those checkpoints every 8-row block of Eq. 2-3 is independent of the others: fire bits,
// delta values, mask words and reference rows are recomputed from them by row-parallel code
// (the finish kernel below, the attention kernel for its own query tile).
//
// delta_finish_kernel: everything that is parallel over rows -- Eq. 2-3 over 8-row blocks
// from the checkpoints: delta values, mask words and (key deltas) the reference-key rows;
// per-row and per-tile non-zero counts, the compacted channel indices, the counters behind
// Eq. 6 -- plus, for query deltas, two passes over the keys that prefill needs anyway: the
// hand-off row R(T-1)[j] = q_hat(T-1).k_j for decode and, for the tensor-core attention kernel
// with the FP32 delta path, the channel-major fp32 copy of the keys.
#include "delta_internal.cuh"
#include "tc_common.cuh"

namespace delta {

namespace {

constexpr int RC = 64;       // rows per ring stage (= one 64-row tile)
constexpr int NS = 6;        // stages of staged rows
constexpr int NZ = 2;        // stages of sub-block tables
constexpr int CH = 32;       // channels per CTA: one chain warp, thread = channel
constexpr int SBR = 4;       // rows per sub-block
constexpr int NSB = RC / SBR;
constexpr int NHELP = 3;     // warps that build the sub-block tables
constexpr int Z_STAGE = NSB * 2 * CH;    // float4 per table stage: per (sub-block, channel) x0..x3 and z0..z2
constexpr int CHAIN_THREADS = 32 * (1 + NHELP + 1);

template <typename TIn> __device__ __forceinline__ float lds_elem(const TIn* p);
template <> __device__ __forceinline__ float lds_elem<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float lds_elem<__nv_bfloat16>(const __nv_bfloat16* p) {
  return __uint_as_float((uint32_t)(*reinterpret_cast<const uint16_t*>(p)) << 16);
}

// Does the reference x_ref fire on value x (Eq. 3: one IEEE subtraction, strict compare, NaN false)?
__device__ __forceinline__ bool fires(float x, float x_ref, float theta) {
  return fabsf(__fsub_rn(x, x_ref)) > theta;
}

// Tight bounded poll of an mbarrier phase for the chain warp (a suspended wait wakes up late,
// and the hand-over is on the chain's path); false once the CTA has given up.
__device__ __forceinline__ bool poll_ok(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  if (mbar_test_wait(bar, parity)) return true;
  mbar_poll(bar, parity, abort_flag);
  return *abort_flag == 0;
}
// The helpers' waits: suspended (they run ahead of the chain warp, and where several CTAs share
// an SM a spinning helper would take issue slots from another CTA's chain warp).
__device__ __forceinline__ bool wait_ok(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  if (mbar_test_wait(bar, parity)) return true;
  mbar_wait(bar, parity, abort_flag);
  return *abort_flag == 0;
}

}  // namespace

// The chain of Eq. 3 costs three dependent operations per row (subtract, compare, select), about
// 17 clocks.  Most of that can be taken off the carried state.  Over a sub-block of four rows
// x0..x3 (in processing order) the state r either survives, or the first row i that fires
// against r replaces it -- and from there on the chain no longer depends on r: the state at the
// end of the sub-block is z_i, the end state of the chain that starts with reference x_i at
// row i.  z_3 = x3, z_2 = fires(x3, x2) ? x3 : x2, and in general z_i = z_j for the first j > i
// that fires against x_i (x_i if none does): six pair tests per sub-block, none of which
// involves r.  Helper warps compute the z tables a stage ahead; the chain warp then does, per
// sub-block, four tests against r in parallel and a two-level select: the dependent path is
// subtract, compare, three selects per FOUR rows.  Every test is the same subtraction and
// comparison the sequential chain would make, so the result is bit-identical.
//
// One CTA per (head, 32 channels): warp 0 carries the chain (thread = channel), warps 1-3 build
// the tables, warp 4 streams the rows in with TMA.  Stages that hold the un-thresholded basis
// row or are cut short by the end of the sequence take the sequential form from the staged
// values.
template <typename TIn, int D>
__global__ void __launch_bounds__(CHAIN_THREADS) delta_chain_kernel(
    const __grid_constant__ CUtensorMap tm_x, float* __restrict__ qhat_tile, float* __restrict__ qhat_out,
    float* __restrict__ ckpt, unsigned long long* __restrict__ counters, int T, int n_tiles, int n_ckpt,
    float theta, int basis_exact, int reverse, uint4* zero_ptr, unsigned zero_n16) {
  // tm_x: the stream that becomes the delta matrix as [heads][rows 0..T-1][D]; box = [64 rows][32 channels]
  constexpr int NSL = D / CH;                      // channel slices (CTAs) per head
  constexpr uint32_t RAW_STAGE_BYTES = RC * CH * sizeof(TIn);
  extern __shared__ __align__(128) unsigned char dyn[];
  TIn* raw = reinterpret_cast<TIn*>(dyn);                                   // [NS][RC][CH]
  float4* zb = reinterpret_cast<float4*>(dyn + NS * RAW_STAGE_BYTES);       // [NZ][NSB][x | z][CH]
  __shared__ __align__(8) unsigned long long bars[2 * NS + 2 * NZ];
  __shared__ uint32_t s_abort;

  const int bh = blockIdx.x / NSL, sl = blockIdx.x - bh * NSL;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[NS]);
  const uint32_t zfull0 = smem_u32(&bars[2 * NS]), zfree0 = smem_u32(&bars[2 * NS + NZ]);
  volatile uint32_t* abort_flag = &s_abort;
  const int n_chunks = (T + RC - 1) / RC;
  // the deferred clearing of a state reset (counters, tickets, second reference buffer): nothing
  // of this launch or of the kernels behind it touches that span before this kernel is complete
  if (zero_ptr && blockIdx.x == 0)
    for (unsigned i = tid; i < zero_n16; i += blockDim.x) zero_ptr[i] = make_uint4(0u, 0u, 0u, 0u);

  if (tid < 2 * NS + 2 * NZ) {      // one barrier per thread
    const uint32_t cnt = (tid < NS) ? 1u : (tid < 2 * NS) ? (uint32_t)NHELP : (tid < 2 * NS + NZ) ? (uint32_t)NHELP : 1u;
    tc::mbar_init(full0 + 8 * tid, cnt);
    if (tid == 0) s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    tc::fence_proxy_async();
  }
  if (tid == 32 * (1 + NHELP))
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_x) : "memory");
  __syncthreads();
  // a kernel launched behind this one with programmatic stream serialisation may become
  // resident and run its prologue now; it sees this kernel's results only after its own
  // grid-dependency wait
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // Which of the four compute warps carries the chain rotates with the CTA: where several CTAs
  // share an SM their chain warps, the busiest, then sit on different schedulers.
  const int cw = (int)blockIdx.x & 3;
  if (warp == 1 + NHELP) {
    // ---- producer: keeps up to NS stages of rows in flight
    if (lane == 0) {
      const uint32_t raw0 = smem_u32(raw);
      for (int i = 0; i < n_chunks && !*abort_flag; ++i) {
        const int s = i % NS;
        if (i >= NS) mbar_wait(empty0 + 8 * s, ((i / NS) - 1) & 1, abort_flag);
        const int ci = reverse ? n_chunks - 1 - i : i;      // stage of the head in token order
        tc::mbar_expect_tx(full0 + 8 * s, RAW_STAGE_BYTES); // rows past T arrive as zeros
        tc::tma_load_3d(raw0 + s * RAW_STAGE_BYTES, &tm_x, full0 + 8 * s, sl * CH, ci * RC, bh);
      }
    }
  } else if (warp != cw) {
    // ---- helpers: helper hw takes sub-blocks hw, hw + 3, ... of every stage; rows in processing
    // order (reverse: from the stage's last row down), tables in processing order of the sub-blocks
    const int hw = (warp - cw - 1) & 3;      // 0, 1, 2
    int s = 0, zs = 0;
    uint32_t ph_full = 0, ph_zfree = 0;      // parity of the completion waited for next
    for (int i = 0; i < n_chunks; ++i) {
      if (!wait_ok(full0 + 8 * s, ph_full, abort_flag)) break;
      const TIn* rows = raw + (size_t)s * RC * CH + lane;
      constexpr int NJ = (NSB + NHELP - 1) / NHELP;
      float y[NJ][SBR];        // every load in front of the first store (both are shared memory)
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        const int sb = min(hw + NHELP * j, NSB - 1);
#pragma unroll
        for (int k = 0; k < SBR; ++k) y[j][k] = lds_elem<TIn>(rows + (sb * SBR + (reverse ? SBR - 1 - k : k)) * CH);
      }
      if (i >= NZ && !wait_ok(zfree0 + 8 * zs, ph_zfree, abort_flag)) break;
      float4* zp = zb + (size_t)zs * Z_STAGE + lane;
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        const int sb = hw + NHELP * j;
        if (sb < NSB) {
          const float z2 = fires(y[j][3], y[j][2], theta) ? y[j][3] : y[j][2];
          float z1 = fires(y[j][3], y[j][1], theta) ? y[j][3] : y[j][1];
          z1 = fires(y[j][2], y[j][1], theta) ? z2 : z1;
          float z0 = fires(y[j][3], y[j][0], theta) ? y[j][3] : y[j][0];
          z0 = fires(y[j][2], y[j][0], theta) ? z2 : z0;
          z0 = fires(y[j][1], y[j][0], theta) ? z1 : z0;
          float4* o = zp + (reverse ? NSB - 1 - sb : sb) * (2 * CH);
          o[0] = make_float4(y[j][0], y[j][1], y[j][2], y[j][3]);
          o[CH] = make_float4(z0, z1, z2, 0.0f);
        }
      }
      __syncwarp();
      if (lane == 0) {
        tc::mbar_arrive(zfull0 + 8 * zs);
        tc::mbar_arrive(empty0 + 8 * s);
      }
      if (++s == NS) { s = 0; ph_full ^= 1u; }
      if (++zs == NZ) { zs = 0; if (i >= NZ) ph_zfree ^= 1u; }
    }
  } else {
    // ---- chain warp: thread owns channel c
    const int c = sl * CH + lane;
    float r = 0.0f;           // reference state, starts at zero (Eq. 3)
    int zs = 0;
    uint32_t ph_zfull = 0;
    static_assert(RC == DELTA_TILE_ROWS, "one tile reference per stage");
    float* const ckpt_c = ckpt + (size_t)bh * n_ckpt * D + c;
    float* const qtile = qhat_tile ? qhat_tile + (size_t)bh * n_tiles * D + c : nullptr;
    const ptrdiff_t cstep = reverse ? -(ptrdiff_t)D : (ptrdiff_t)D;
    int t0 = reverse ? (n_chunks - 1) * RC : 0;       // first row of the stage, stepped by dt
    const int dt = reverse ? -RC : RC;
    // checkpoint of the 8-row block the processing order enters next (full stages step it)
    float* cp = ckpt_c + (size_t)((t0 + (reverse ? RC - SBR : 0)) / DELTA_CKPT_ROWS) * D;
    bool ready = false;       // the stage's tables were seen complete during the stage before
    for (int i = 0; i < n_chunks; ++i, t0 += dt) {
      const int nrows = min(RC, T - t0);
      if (qhat_tile && DELTA_IN(t0 / DELTA_TILE_ROWS, n_tiles, counters)) qtile[(size_t)(t0 / DELTA_TILE_ROWS) * D] = r;
      if (!ready && !poll_ok(zfull0 + 8 * zs, ph_zfull, abort_flag)) break;
      const int zs_next = (zs + 1 == NZ) ? 0 : zs + 1;
      const uint32_t ph_next = (zs + 1 == NZ) ? ph_zfull ^ 1u : ph_zfull;
      const float4* zp = zb + (size_t)zs * Z_STAGE + lane;
      const bool has_basis = basis_exact && i == 0;      // row 0, or row T-1 in reverse
      if (nrows == RC) {
        float4 x = zp[0], z = zp[CH];
#pragma unroll
        for (int lsb = 0; lsb < NSB; ++lsb) {
          // the next sub-block's tables while this one is worked on
          const float4 xn = zp[(lsb + 1 < NSB ? lsb + 1 : lsb) * (2 * CH)];
          const float4 zn = zp[(lsb + 1 < NSB ? lsb + 1 : lsb) * (2 * CH) + CH];
          if ((lsb & 1) == 0) {
            // the reference in front of an 8-row block (reverse: in front of its highest row)
            if (DELTA_IN((size_t)(cp - ckpt_c) / D, n_ckpt, counters)) *cp = r;
            cp += cstep;
          }
          // (a look at the next stage's barrier a few sub-blocks before the end: the answer is
          // back by the time it is needed)
          if (lsb == NSB - 4) ready = mbar_test_wait(zfull0 + 8 * zs_next, ph_next);
          const bool p3 = fires(x.w, r, theta), p2 = fires(x.z, r, theta);
          bool p0 = fires(x.x, r, theta);
          if (lsb == 0) p0 = p0 || has_basis;      // the basis row is taken un-thresholded
          const bool p1 = fires(x.y, r, theta);
          float b = p3 ? x.w : r;
          b = p2 ? z.z : b;
          const float a = p0 ? z.x : z.y;          // the first of rows 0, 1 that fired, if one did
          r = (p0 || p1) ? a : b;
          x = xn; z = zn;
        }
      } else {
        // a stage cut short by the end of the sequence: row by row from the staged values
        ready = false;
        for (int lsb = 0; lsb < NSB; ++lsb) {
          const float4 x4 = zp[lsb * (2 * CH)];
          const float xs[SBR] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
          for (int k = 0; k < SBR; ++k) {
            const int l = lsb * SBR + k;
            const int pr = reverse ? RC - 1 - l : l;     // row of the stage
            if (pr < nrows) {
              const int t = t0 + pr;
              const bool at_ckpt = reverse ? ((t % DELTA_CKPT_ROWS) == DELTA_CKPT_ROWS - 1 || pr == nrows - 1)
                                           : (t % DELTA_CKPT_ROWS) == 0;
              if (at_ckpt && DELTA_IN(t / DELTA_CKPT_ROWS, n_ckpt, counters))
                ckpt_c[(size_t)(t / DELTA_CKPT_ROWS) * D] = r;
              const bool basis_here = has_basis && (reverse ? pr == nrows - 1 : pr == 0);
              r = (basis_here || fires(xs[k], r, theta)) ? xs[k] : r;
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(zfree0 + 8 * zs);
      if (nrows != RC) cp = ckpt_c + (size_t)((t0 + dt + (reverse ? RC - SBR : 0)) / DELTA_CKPT_ROWS) * D;
      zs = zs_next; ph_zfull = ph_next;
    }
    if (!*abort_flag && qhat_out) qhat_out[(size_t)bh * D + c] = r;
  }
  __syncthreads();
  if (tid == 0 && s_abort) atomicMax(&counters[CNT_STATUS], (unsigned long long)DELTA_ERR_TIMEOUT);
}


static cudaError_t launch_delta_chain_tables(const Shape& s, const Workspace& w, const void* q, int T, float theta,
                                            int dtype, int init, bool key_stream, bool reverse, void* zero_ptr,
                                            size_t zero_bytes, cudaStream_t st) {
  const int heads = s.B * (key_stream ? s.H_kv : s.H);
  const int src_rows = key_stream ? s.T_max : T;
  const int basis = (init == DELTA_INIT_BASIS_EXACT) ? 1 : 0;
  const bool f32 = dtype == DELTA_F32;
  const size_t esz = f32 ? sizeof(float) : sizeof(__nv_bfloat16);
  CUtensorMap tm;
  if (!tc::encode3(&tm, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, q, (uint64_t)s.d,
                   (uint64_t)T, (uint64_t)heads, (uint64_t)s.d * esz, (uint64_t)src_rows * s.d * esz, CH, RC,
                   CU_TENSOR_MAP_SWIZZLE_NONE))
    return cudaErrorInvalidValue;
  cudaError_t err = cudaSuccess;
#define LAUNCH(TIN, DD)                                                                          \
  do {                                                                                           \
    auto kern = delta_chain_kernel<TIN, DD>;                                                     \
    const size_t smem = (size_t)NS * RC * CH * sizeof(TIN) + (size_t)NZ * Z_STAGE * sizeof(float4); \
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);    \
    if (err != cudaSuccess) return err;                                                          \
    kern<<<heads * (DD / CH), CHAIN_THREADS, smem, st>>>(tm, w.qhat_tile, w.qhat[0], w.ckpt, w.counters, T, \
                                                         s.n_tiles, s.n_ckpt(), theta, basis, reverse ? 1 : 0, \
                                                         (uint4*)zero_ptr, (unsigned)(zero_bytes / 16)); \
  } while (0)
  if (f32) {
    if (s.d == 64) LAUNCH(float, 64); else LAUNCH(float, 128);
  } else {
    if (s.d == 64) LAUNCH(__nv_bfloat16, 64); else LAUNCH(__nv_bfloat16, 128);
  }
#undef LAUNCH
  count_launch();
  return err != cudaSuccess ? err : cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// delta_chain_rows_kernel: the chain row by row, for streams of many heads.  One CTA per (batch,
// head): D/32 chain warps (thread = channel) + one producer warp that streams the head's rows
// into a ring of shared-memory stages with bulk copies.  Per row one shared-memory load, one
// widening, the three dependent operations of Eq. 2-3 and a checkpoint store every 8 rows.  It
// does 3 times fewer instructions and 10 times less shared-memory traffic per row than the
// kernel above, whose tables (32 bytes written and read per element) saturate the shared-memory
// bandwidth of an SM from about two CTAs per SM on: with every head of a large batch resident
// at once this one is faster (stack layer: 59 us against 82), with few heads the other one
// (a single Llama layer: 14.3 us against 18.4).
namespace {

constexpr int RROWS = 64;    // rows per ring stage
constexpr int RSTAGES = 4;   // ring stages

// One element of the staged rows by shared-memory address, widened to fp32.
template <typename TIn> __device__ __forceinline__ float lds_row_elem(uint32_t addr);
template <> __device__ __forceinline__ float lds_row_elem<float>(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}
template <> __device__ __forceinline__ float lds_row_elem<__nv_bfloat16>(uint32_t addr) {
  uint32_t u;
  asm volatile("ld.shared.u16 %0, [%1];" : "=r"(u) : "r"(addr));
  return __uint_as_float(u << 16);
}

// One ring stage of the chain for one thread (= one channel): rows t0 .. t0+nrows-1, the
// thread's values at rows[r * D]; updates the reference qh and leaves it in front of every
// 8-row block (ckptp).  basis_row: the stage's first row is the un-thresholded basis.
template <typename TIn, int D>
__device__ __forceinline__ void chain_stage(const TIn* rows, int t0, int nrows, bool basis_row, float& qh,
                                            float theta, float* ckptp, int n_ckpt, unsigned long long* counters) {
  if (nrows == RROWS && !basis_row) {
    // full stage, no basis row: nothing but loads, the dependent chain and the checkpoints
    float x[RROWS];
    const uint32_t saddr = smem_u32(rows);
#pragma unroll
    for (int r = 0; r < RROWS; ++r) x[r] = lds_row_elem<TIn>(saddr + (uint32_t)(r * D * sizeof(TIn)));
#pragma unroll
    for (int r = 0; r < RROWS; ++r) {
      if ((r % DELTA_CKPT_ROWS) == 0 && DELTA_IN((t0 + r) / DELTA_CKPT_ROWS, n_ckpt, counters))
        ckptp[(size_t)((t0 + r) / DELTA_CKPT_ROWS) * D] = qh;
      const float diff = __fsub_rn(x[r], qh);      // one IEEE subtraction
      const bool fire = fabsf(diff) > theta;       // strict; NaN compares false
      qh = fire ? x[r] : qh;
    }
  } else {
    for (int r = 0; r < nrows; ++r) {
      if (((t0 + r) % DELTA_CKPT_ROWS) == 0 && DELTA_IN((t0 + r) / DELTA_CKPT_ROWS, n_ckpt, counters))
        ckptp[(size_t)((t0 + r) / DELTA_CKPT_ROWS) * D] = qh;
      const float x = to_f32(rows[r * D]);
      const bool fire = (r == 0 && basis_row) || (fabsf(__fsub_rn(x, qh)) > theta);
      qh = fire ? x : qh;
    }
  }
}

// Strategy (2): the same stage of the query stream taken from its last row down to its first.
// The checkpoint of an 8-row block is the reference before the block's highest row.
// basis_last: the stage's last row is row T-1, the un-thresholded basis of this order.
template <typename TIn, int D>
__device__ __forceinline__ void chain_stage_rev(const TIn* rows, int t0, int nrows, bool basis_last, float& qh,
                                                float theta, float* ckptp, int n_ckpt, unsigned long long* counters) {
  if (nrows == RROWS && !basis_last) {
    float x[RROWS];
    const uint32_t saddr = smem_u32(rows);
#pragma unroll
    for (int r = 0; r < RROWS; ++r) x[r] = lds_row_elem<TIn>(saddr + (uint32_t)(r * D * sizeof(TIn)));
#pragma unroll
    for (int r = RROWS - 1; r >= 0; --r) {
      if ((r % DELTA_CKPT_ROWS) == DELTA_CKPT_ROWS - 1 && DELTA_IN((t0 + r) / DELTA_CKPT_ROWS, n_ckpt, counters))
        ckptp[(size_t)((t0 + r) / DELTA_CKPT_ROWS) * D] = qh;
      const float diff = __fsub_rn(x[r], qh);
      const bool fire = fabsf(diff) > theta;
      qh = fire ? x[r] : qh;
    }
  } else {
    for (int r = nrows - 1; r >= 0; --r) {
      if ((((t0 + r) % DELTA_CKPT_ROWS) == DELTA_CKPT_ROWS - 1 || r == nrows - 1) &&
          DELTA_IN((t0 + r) / DELTA_CKPT_ROWS, n_ckpt, counters))
        ckptp[(size_t)((t0 + r) / DELTA_CKPT_ROWS) * D] = qh;
      const float x = to_f32(rows[r * D]);
      const bool fire = (r == nrows - 1 && basis_last) || (fabsf(__fsub_rn(x, qh)) > theta);
      qh = fire ? x : qh;
    }
  }
}

}  // namespace

template <typename TIn, int D>
__global__ void __launch_bounds__(D + 32) delta_chain_rows_kernel(
    const TIn* __restrict__ q, float* __restrict__ qhat_tile, float* __restrict__ qhat_out,
    float* __restrict__ ckpt, unsigned long long* __restrict__ counters, int T, int n_tiles, int n_ckpt,
    float theta, int basis_exact, int src_rows, int reverse, uint4* zero_ptr, unsigned zero_n16) {
  // q: the stream that becomes the delta matrix, [heads][src_rows][D] with rows 0..T-1 read
  // (queries: src_rows = T; keys in the KV-cache layout: src_rows = T_max)
  constexpr int NW = D / 32;                       // chain warps
  constexpr uint32_t ROW_BYTES = D * sizeof(TIn);
  constexpr uint32_t STAGE_BYTES = RROWS * ROW_BYTES;
  extern __shared__ __align__(128) unsigned char ring[];   // [RSTAGES][RROWS][D] of TIn
  __shared__ __align__(8) unsigned long long bars[2 * RSTAGES];   // full[RSTAGES], empty[RSTAGES]
  __shared__ int s_fail;

  const int bh = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[RSTAGES]);
  const int n_chunks = (T + RROWS - 1) / RROWS;
  // the deferred clearing of a state reset (see the table kernel)
  if (zero_ptr && blockIdx.x == 0)
    for (unsigned i = tid; i < zero_n16; i += blockDim.x) zero_ptr[i] = make_uint4(0u, 0u, 0u, 0u);

  if (tid == 0) {
    for (int s = 0; s < RSTAGES; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full0 + 8 * s), "r"(1) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty0 + 8 * s), "r"(NW) : "memory");
    }
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // a kernel launched behind this one with programmatic stream serialisation may become
  // resident and run its prologue now; it sees this kernel's results only after its own
  // grid-dependency wait
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == NW) {
    // ---- producer: keeps up to RSTAGES stages of query rows in flight
    if (lane == 0) {
      const unsigned char* src = reinterpret_cast<const unsigned char*>(q) + (size_t)bh * src_rows * ROW_BYTES;
      const uint32_t ring0 = smem_u32(ring);
      for (int i = 0; i < n_chunks; ++i) {
        const int s = i % RSTAGES;
        if (i >= RSTAGES && !mbar_wait(empty0 + 8 * s, ((i / RSTAGES) - 1) & 1)) { s_fail = 1; break; }
        const int ci = reverse ? n_chunks - 1 - i : i;      // stage of the head in token order
        const int rows = min(RROWS, T - ci * RROWS);
        const uint32_t bytes = (uint32_t)rows * ROW_BYTES;
        // (bounds-checking build: the stage's rows lie inside the head's rows of the stream)
        if (!DELTA_IN((size_t)ci * RROWS + rows - 1, src_rows, counters)) { s_fail = 1; break; }
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full0 + 8 * s),
                     "r"(bytes)
                     : "memory");
        asm volatile(
            "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                ring0 + s * STAGE_BYTES),
            "l"(src + (size_t)ci * STAGE_BYTES), "r"(bytes), "r"(full0 + 8 * s)
            : "memory");
      }
    }
  } else {
    // ---- chain warps: thread c owns channel c
    const int c = tid;
    float* ckptp = ckpt + (size_t)bh * n_ckpt * D + c;
    float qh = 0.0f;          // reference state, starts at zero (Eq. 3)
    bool failed = false;
    for (int i = 0; i < n_chunks; ++i) {
      const int s = i % RSTAGES;
      const int t0 = (reverse ? n_chunks - 1 - i : i) * RROWS;
      if (qhat_tile && (t0 % DELTA_TILE_ROWS) == 0 && DELTA_IN(t0 / DELTA_TILE_ROWS, n_tiles, counters))
        qhat_tile[((size_t)bh * n_tiles + t0 / DELTA_TILE_ROWS) * D + c] = qh;
      if (!mbar_wait(full0 + 8 * s, (i / RSTAGES) & 1)) { failed = true; break; }
      const TIn* rows = reinterpret_cast<const TIn*>(ring + (size_t)s * STAGE_BYTES) + c;
      const int nrows = min(RROWS, T - t0);
      if (reverse)
        chain_stage_rev<TIn, D>(rows, t0, nrows, t0 + nrows == T && basis_exact, qh, theta, ckptp, n_ckpt, counters);
      else
        chain_stage<TIn, D>(rows, t0, nrows, t0 == 0 && basis_exact, qh, theta, ckptp, n_ckpt, counters);
      __syncwarp();
      if (lane == 0)
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty0 + 8 * s) : "memory");
    }
    if (!failed && qhat_out) qhat_out[(size_t)bh * D + c] = qh;
    if (failed) s_fail = 1;
  }
  __syncthreads();
  if (tid == 0 && s_fail) atomicMax(&counters[CNT_STATUS], (unsigned long long)DELTA_ERR_TIMEOUT);
}


static cudaError_t launch_delta_chain_rows(const Shape& s, const Workspace& w, const void* q, int T, float theta,
                                          int dtype, int init, bool key_stream, bool reverse, void* zero_ptr,
                                          size_t zero_bytes, cudaStream_t st) {
  if (key_stream && reverse) return cudaErrorNotSupported;
  const int grid = s.B * (key_stream ? s.H_kv : s.H);
  const int src_rows = key_stream ? s.T_max : T;
  const int basis = (init == DELTA_INIT_BASIS_EXACT) ? 1 : 0;
  cudaError_t err = cudaSuccess;
#define LAUNCH(TIN, DD)                                                                          \
  do {                                                                                           \
    auto kern = delta_chain_rows_kernel<TIN, DD>;                                                     \
    const size_t smem = (size_t)RSTAGES * RROWS * DD * sizeof(TIN);                                      \
    if (smem > 48 * 1024) {                                                                      \
      err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);  \
      if (err != cudaSuccess) return err;                                                        \
    }                                                                                            \
    kern<<<grid, DD + 32, smem, st>>>((const TIN*)q, w.qhat_tile, w.qhat[0], w.ckpt, w.counters, T, s.n_tiles, \
                                      s.n_ckpt(), theta, basis, src_rows, reverse ? 1 : 0,       \
                                      (uint4*)zero_ptr, (unsigned)(zero_bytes / 16));            \
  } while (0)
  if (dtype == DELTA_F32) {
    if (s.d == 64) LAUNCH(float, 64); else LAUNCH(float, 128);
  } else {
    if (s.d == 64) LAUNCH(__nv_bfloat16, 64); else LAUNCH(__nv_bfloat16, 128);
  }
#undef LAUNCH
  count_launch();
  return err != cudaSuccess ? err : cudaGetLastError();
}

// SMs of the current device (queried once per device).
int device_sm_count() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (!cached[dev]) {
    int n = 0;
    cached[dev] = (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) ? n : 148;
  }
  return cached[dev];
}

cudaError_t launch_delta_chain(const Shape& s, const Workspace& w, const void* q, int T, float theta, int dtype,
                               int init, bool key_stream, bool reverse, void* zero_ptr, size_t zero_bytes,
                               cudaStream_t st) {
  if (key_stream && reverse) return cudaErrorNotSupported;
  if (((uintptr_t)zero_ptr | zero_bytes) & 15u) return cudaErrorInvalidValue;
  // the table kernel while every one of its CTAs (head x 32 channels) has an SM of its own
  const long ctas = (long)s.B * (key_stream ? s.H_kv : s.H) * (s.d / CH);
  if (ctas <= device_sm_count())
    return launch_delta_chain_tables(s, w, q, T, theta, dtype, init, key_stream, reverse, zero_ptr, zero_bytes, st);
  return launch_delta_chain_rows(s, w, q, T, theta, dtype, init, key_stream, reverse, zero_ptr, zero_bytes, st);
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
__global__ void __launch_bounds__(256, 5) delta_finish_kernel(
    uint32_t* __restrict__ mask, uint16_t* __restrict__ row_nnz,
    uint32_t* __restrict__ tile_nnz, uint8_t* __restrict__ idx,
    unsigned long long* __restrict__ counters, const TIn* __restrict__ k,
    const float* __restrict__ qhat, float* __restrict__ R, float* __restrict__ kt, int T,
    int T_max, int n_tiles, int BH, int H, int g, int W, int shape, int n_idx_blocks, int kt_ld,
    int key_stream, const TIn* __restrict__ q, int src_rows, float* __restrict__ dq,
    __nv_bfloat16* __restrict__ ref_rows, const float* __restrict__ ckpt, int n_ckpt, float theta,
    int basis_exact, int reverse, int wait_front) {
  // q: the stream the chain kernel ran over, [heads][src_rows][D]; ref_rows (key deltas): the
  // reference after every row, the cache of reference keys
  constexpr int NW = D / 32;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // Launched with programmatic stream serialisation.  wait_front: the results of everything
  // in front are visible from here on (no effect in an ordinary launch).  Without it (query
  // deltas behind the telescoped attention kernel, of which this kernel needs nothing): every
  // CTA of the attention kernel has released this kernel after its own wait for the chain
  // kernel, so the chain's results are complete; they are read past the L1 cache (ld.global.cg),
  // and the blocks run on the SMs the attention kernel's last wave leaves idle.
  if (wait_front) asm volatile("griddepcontrol.wait;" ::: "memory");
  // key deltas: the attention kernel is serialised programmatically behind this one and may set
  // itself up meanwhile (it waits for this kernel's results itself)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if ((int)blockIdx.x < n_idx_blocks) {
    // ---- one block per (batch, head, 64-row tile); warp w serves rows 8w .. 8w+7
    __shared__ unsigned long long s_red[3][8];
    const int tiles_used = (T + DELTA_TILE_ROWS - 1) / DELTA_TILE_ROWS;
    const int bh = blockIdx.x / tiles_used, tile = blockIdx.x - bh * tiles_used;
    const int t0 = tile * DELTA_TILE_ROWS;
    const int rows = min(DELTA_TILE_ROWS, T - t0);
    const int r_mine = warp * 8 + (lane & 7);        // lanes 0..7 hold one row each
    uint32_t mw[NW];
    {
      // The chain kernel left only the reference in front of every 8-row block.  The warp
      // re-runs Eq. 2-3 over its 8 rows (lane = channel of a mask word): delta values, reference
      // rows (key deltas), and one ballot per row for the mask word.
      const int rbase = t0 + warp * 8;
#pragma unroll
      for (int w2 = 0; w2 < NW; ++w2) {
        const int c = w2 * 32 + lane;
        uint32_t word_mine = 0;
        if (rbase < T && DELTA_IN(rbase / DELTA_CKPT_ROWS, n_ckpt, counters) && DELTA_IN(rbase + 7 < T ? rbase + 7 : T - 1, src_rows, counters) &&
            DELTA_IN(T - 1, T_max, counters)) {
          float ref = __ldcg(&ckpt[((size_t)bh * n_ckpt + rbase / DELTA_CKPT_ROWS) * D + c]);
          float x[8];
#pragma unroll
          for (int r = 0; r < 8; ++r)
            x[r] = (rbase + r < T) ? to_f32(q[((size_t)bh * src_rows + rbase + r) * D + c]) : 0.0f;
#pragma unroll
          for (int rr = 0; rr < 8; ++rr) {
            const int r = reverse ? 7 - rr : rr;         // strategy (2) takes the rows from the top
            const bool live = rbase + r < T;
            bool fire;
            float delta;
            if (rbase + r == (reverse ? T - 1 : 0) && basis_exact) {
              fire = true;                               // the basis vector is kept whole
              delta = x[r];
            } else {
              const float diff = __fsub_rn(x[r], ref);
              fire = fabsf(diff) > theta;
              delta = fire ? diff : 0.0f;
            }
            fire = fire && live;
            if (live) {
              dq[((size_t)bh * T_max + rbase + r) * D + c] = delta;
              ref = fire ? x[r] : ref;
              if (ref_rows) ref_rows[((size_t)bh * T_max + rbase + r) * D + c] = __float2bfloat16_rn(ref);
            }
            const uint32_t word = __ballot_sync(0xffffffffu, fire);
            if ((lane & 7) == r) word_mine = word;
          }
        }
        mw[w2] = word_mine;
        if (lane < 8 && r_mine < rows) mask[((size_t)bh * T_max + t0 + r_mine) * NW + w2] = word_mine;
      }
    }
    unsigned long long done = 0, dense = 0, tsum = 0;
    if (lane < 8 && r_mine < rows && DELTA_IN(t0 + r_mine, T_max, counters)) {
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
    __syncthreads();
    if (tid == 0) {
      unsigned long long a = 0, b2 = 0, c2 = 0;
      for (int w2 = 0; w2 < 8; ++w2) { a += s_red[0][w2]; b2 += s_red[1][w2]; c2 += s_red[2][w2]; }
      if (DELTA_IN(tile, n_tiles, counters)) tile_nnz[(size_t)bh * n_tiles + tile] = (uint32_t)a;
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
    qh[hh][c] = __ldcg(&qhat[((size_t)b * H + kvh * g + hh) * D + c]);
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
      if (j0 + j < T && DELTA_IN(j0 + j, T_max, counters)) R[((size_t)b * H + kvh * g + hh) * T_max + j0 + j] = acc;
    }
  }
}

cudaError_t launch_delta_finish(const Shape& s, const Workspace& w, const void* q, const void* k, int T,
                                float theta, int window, int shape, int dtype, int init, bool want_kt,
                                bool key_stream, bool reverse, int programmatic, cudaStream_t st) {
  // programmatic: 0 = ordinary launch, 1 = programmatic serialisation, 2 = the same and the kernel
  // does not wait for the kernel in front (see the kernel)
  // key deltas: the index/counter pass runs over the KV heads and there is no hand-off row
  const int BH = s.B * (key_stream ? s.H_kv : s.H);
  const int tiles_used = (T + DELTA_TILE_ROWS - 1) / DELTA_TILE_ROWS;
  const int n_idx_blocks = BH * tiles_used;
  const int n_key_blocks = key_stream ? 0 : s.B * s.H_kv * ((T + 63) / 64);
  const int kt_ld = (s.T_max + 3) / 4 * 4;
  float* kt = (want_kt && w.kt) ? w.kt : nullptr;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(n_idx_blocks + n_key_blocks));
  cfg.blockDim = dim3(256);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = programmatic ? 1 : 0;
  cudaError_t err = cudaSuccess;
#define LAUNCH(TIN, DD)                                                                          \
  err = cudaLaunchKernelEx(&cfg, delta_finish_kernel<TIN, DD>,                                   \
      w.mask, w.row_nnz, w.tile_nnz, w.idx, w.counters, (const TIN*)k, (const float*)w.qhat[0], w.R, kt, T,    \
      s.T_max, s.n_tiles, BH, s.H, s.g(), window, shape, n_idx_blocks, kt_ld, key_stream ? 1 : 0,   \
      key_stream ? (const TIN*)k : (const TIN*)q, key_stream ? s.T_max : T, w.dq,                 \
      key_stream ? w.qhat_rows : (__nv_bfloat16*)nullptr, (const float*)w.ckpt, s.n_ckpt(), theta, \
      init == DELTA_INIT_BASIS_EXACT ? 1 : 0, reverse ? 1 : 0, programmatic == 2 ? 0 : 1)
  if (dtype == DELTA_F32) {
    if (s.d == 64) LAUNCH(float, 64); else LAUNCH(float, 128);
  } else {
    if (s.d == 64) LAUNCH(__nv_bfloat16, 64); else LAUNCH(__nv_bfloat16, 128);
  }
#undef LAUNCH
  count_launch();
  return err != cudaSuccess ? err : cudaGetLastError();
}

}  // namespace delta
