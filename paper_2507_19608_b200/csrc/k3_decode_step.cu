// K3 -- one decode step of strategy (1) carried past prefill (Section III-A "Decoding Stage
// Considerations", Section III-B "Decoding Stage", Section III-C).  HBM-bound: one streaming
// pass over the K and V cache plus a read-modify-write of the carried score row R.
//
// Grid = (key splits, batch x KV heads).  A CTA serves the G query heads that share one KV
// head, so every cached key and value row is read once for the group.  It
//   0. thresholds q_new against the carried reference (Eq. 2-3) for its G heads,
//   1. streams its slice of the key cache: R[j] += dq . k_j (Eq. 4), exact q_new . k_j for the
//      W_d most recent keys, and for the key that arrives now R[n] = q_hat . k_new; appends
//      k_new / v_new to the cache,
//   2. turns its slice of scores into un-normalised probabilities (slice max, sum),
//   3. accumulates P.V over its slice of the value cache,
//   4. stores (max, sum, partial output); the last CTA of a (batch, KV head) to finish merges
//      the slices and writes the output rows.
#include "delta_internal.cuh"

namespace delta {

namespace {
constexpr int DNT = 256, DNW = DNT / 32;

__device__ __forceinline__ void load8(const float* p, float (&x)[8]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  const float4 b = *reinterpret_cast<const float4*>(p + 4);
  x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&x)[8]) {
  const uint4 u = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    x[2 * i] = __uint_as_float(w[i] << 16);
    x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void copy8(float* dst, const float* src) {
  *reinterpret_cast<float4*>(dst) = *reinterpret_cast<const float4*>(src);
  *reinterpret_cast<float4*>(dst + 4) = *reinterpret_cast<const float4*>(src + 4);
}
__device__ __forceinline__ void copy8(__nv_bfloat16* dst, const __nv_bfloat16* src) {
  *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
}
}  // namespace

template <typename TC, int D, int G>
__global__ void __launch_bounds__(DNT) decode_step_kernel(
    const TC* __restrict__ q_new, const TC* __restrict__ k_new, const TC* __restrict__ v_new,
    TC* __restrict__ k_cache, TC* __restrict__ v_cache, TC* __restrict__ out,
    const float* __restrict__ qhat_in, float* __restrict__ qhat_out, float* __restrict__ R,
    float* __restrict__ partial, uint32_t* __restrict__ ticket,
    unsigned long long* __restrict__ counters, int n, int T_max, int H, int chunk, int nsplit,
    float theta, int W, float scale_log2e) {
  constexpr int LPK = D / 8;     // lanes per key row (8 elements each)
  constexpr int KPW = 32 / LPK;  // key rows per warp iteration
  extern __shared__ __align__(16) float dsm[];
  float* q_s = dsm;              // [G][D]
  float* dq_s = q_s + G * D;     // [G][D]
  float* qh_s = dq_s + G * D;    // [G][D]
  float* red = qh_s + G * D;     // [DNW][G][D]
  float* ml_s = red + DNW * G * D;  // [2][G]: slice max, slice sum
  float* sc = ml_s + 2 * 8;      // [G][chunk]
  __shared__ int s_last;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.x, bkv = blockIdx.y;
  const int H_kv = H / G;
  const int b = bkv / H_kv, kvh = bkv - b * H_kv;
  const int L = n + 1;  // keys after this step
  const int j0 = split * chunk;
  const int len = max(0, min(chunk, L - j0));

  // ---- 0. delta of the new query rows against the carried reference (Eq. 2-3)
  int fired_total = 0;
  for (int e0 = 0; e0 < G * D; e0 += DNT) {
    const int e = e0 + tid;
    bool fire = false;
    if (e < G * D) {
      const int hh = e / D, c = e - hh * D;
      const size_t o = ((size_t)b * H + kvh * G + hh) * D + c;
      const float x = to_f32(q_new[o]);
      const float old = qhat_in[o];
      const float diff = __fsub_rn(x, old);
      fire = fabsf(diff) > theta;
      q_s[e] = x;
      dq_s[e] = fire ? diff : 0.0f;
      const float nq = fire ? x : old;
      qh_s[e] = nq;
      if (split == 0) qhat_out[o] = nq;
    }
    fired_total += __syncthreads_count(fire);
  }
  if (split == 0 && tid == 0) {
    const int n_in = min(L, max(W, 0));
    const int n_out = L - n_in;
    atomicAdd(&counters[CNT_DECODE_NNZ], (unsigned long long)fired_total);
    atomicAdd(&counters[CNT_DECODE_ELEMS], (unsigned long long)G * D);
    atomicAdd(&counters[CNT_DECODE_MACS_DONE],
              (unsigned long long)n_in * D * G + (unsigned long long)n_out * fired_total);
    atomicAdd(&counters[CNT_DECODE_MACS_DENSE], (unsigned long long)L * D * G);
  }

  const int sub = lane / LPK;       // which key row of the warp iteration
  const int c0 = (lane % LPK) * 8;  // first of this lane's 8 channels
  const TC* kc = k_cache + (size_t)bkv * T_max * D;
  const TC* vc = v_cache + (size_t)bkv * T_max * D;

  // ---- 1. scores of this slice
  for (int jb = warp * KPW; jb < len; jb += DNW * KPW) {
    const int jj = jb + sub;
    const int j = j0 + jj;
    const bool valid = jj < len;
    const bool is_new = valid && (j == n);
    const bool warp_has_new = (j0 + jb <= n) && (n < j0 + jb + KPW);
    const bool warp_in_win = (n - (j0 + jb + KPW - 1)) < W;  // some row of this iteration is exact
    float kv[8];
    if (valid) {
      const TC* src = is_new ? (k_new + (size_t)bkv * D + c0) : (kc + (size_t)j * D + c0);
      load8(src, kv);
      if (is_new) copy8(k_cache + ((size_t)bkv * T_max + n) * D + c0, src);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) kv[e] = 0.0f;
    }
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
      float pd = 0.0f, pq = 0.0f, pr = 0.0f;
      const float* dqh = dq_s + hh * D + c0;
#pragma unroll
      for (int e = 0; e < 8; ++e) pd = fmaf(dqh[e], kv[e], pd);
      if (warp_in_win) {
        const float* qh = q_s + hh * D + c0;
#pragma unroll
        for (int e = 0; e < 8; ++e) pq = fmaf(qh[e], kv[e], pq);
      }
      if (warp_has_new) {
        const float* rh = qh_s + hh * D + c0;
#pragma unroll
        for (int e = 0; e < 8; ++e) pr = fmaf(rh[e], kv[e], pr);
      }
#pragma unroll
      for (int o = LPK / 2; o > 0; o >>= 1) {
        pd += __shfl_xor_sync(0xffffffffu, pd, o);
        if (warp_in_win) pq += __shfl_xor_sync(0xffffffffu, pq, o);
        if (warp_has_new) pr += __shfl_xor_sync(0xffffffffu, pr, o);
      }
      if (valid && (lane % LPK) == 0) {
        float* Rp = R + ((size_t)b * H + kvh * G + hh) * T_max + j;
        const float Rn = is_new ? pr : (*Rp + pd);
        *Rp = Rn;
        const float s = (n - j < W) ? pq : Rn;
        sc[hh * chunk + jj] = s * scale_log2e;
      }
    }
  }
  __syncthreads();

  // ---- 2. slice max and un-normalised probabilities (warp hh serves head hh)
  if (warp < G) {
    float* s = sc + warp * chunk;
    float mx = -INFINITY;
    for (int jj = lane; jj < len; jj += 32) mx = fmaxf(mx, s[jj]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = 0.0f;
    for (int jj = lane; jj < len; jj += 32) {
      const float p = exp2f(s[jj] - mx);
      s[jj] = p;
      sum += p;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) { ml_s[warp] = mx; ml_s[8 + warp] = sum; }
  }
  __syncthreads();

  // ---- 3. partial P.V over this slice
  float acc[G][8];
#pragma unroll
  for (int hh = 0; hh < G; ++hh)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[hh][e] = 0.0f;
  for (int jb = warp * KPW; jb < len; jb += DNW * KPW) {
    const int jj = jb + sub;
    const int j = j0 + jj;
    if (jj < len) {
      const bool is_new = (j == n);
      const TC* src = is_new ? (v_new + (size_t)bkv * D + c0) : (vc + (size_t)j * D + c0);
      float vv[8];
      load8(src, vv);
      if (is_new) copy8(v_cache + ((size_t)bkv * T_max + n) * D + c0, src);
#pragma unroll
      for (int hh = 0; hh < G; ++hh) {
        const float p = sc[hh * chunk + jj];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[hh][e] = fmaf(p, vv[e], acc[hh][e]);
      }
    }
  }
#pragma unroll
  for (int hh = 0; hh < G; ++hh)
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      float x = acc[hh][e];
#pragma unroll
      for (int o = LPK; o < 32; o <<= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
      acc[hh][e] = x;
    }
  if (sub == 0) {
#pragma unroll
    for (int hh = 0; hh < G; ++hh)
#pragma unroll
      for (int e = 0; e < 8; ++e) red[(warp * G + hh) * D + c0 + e] = acc[hh][e];
  }
  __syncthreads();

  // ---- 4. store the slice result; the last slice to arrive merges all of them
  float* part = partial + ((size_t)bkv * kMaxDecodeSplits + split) * G * (D + 2);
  for (int e = tid; e < G * D; e += DNT) {
    float x = 0.0f;
#pragma unroll
    for (int w2 = 0; w2 < DNW; ++w2) x += red[w2 * G * D + e];
    const int hh = e / D, c = e - hh * D;
    part[hh * (D + 2) + c] = x;
  }
  if (tid < G) {
    part[tid * (D + 2) + D] = ml_s[tid];
    part[tid * (D + 2) + D + 1] = ml_s[8 + tid];
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const uint32_t t = atomicAdd(&ticket[bkv], 1u);
    s_last = (t == (uint32_t)nsplit - 1u);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const float* pbase = partial + (size_t)bkv * kMaxDecodeSplits * G * (D + 2);
  for (int e = tid; e < G * D; e += DNT) {
    const int hh = e / D, c = e - hh * D;
    float M = -INFINITY;
    for (int s2 = 0; s2 < nsplit; ++s2)
      M = fmaxf(M, __ldcg(pbase + ((size_t)s2 * G + hh) * (D + 2) + D));
    float num = 0.0f, den = 0.0f;
    for (int s2 = 0; s2 < nsplit; ++s2) {
      const float* pp = pbase + ((size_t)s2 * G + hh) * (D + 2);
      const float wgt = exp2f(__ldcg(pp + D) - M);
      num = fmaf(wgt, __ldcg(pp + c), num);
      den = fmaf(wgt, __ldcg(pp + D + 1), den);
    }
    out[((size_t)b * H + kvh * G + hh) * D + c] = from_f32<TC>(num / den);
  }
  if (tid == 0) ticket[bkv] = 0;  // ready for the next step
}

cudaError_t launch_decode_step(const Shape& s, const Workspace& w, const void* q_new,
                               const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                               void* out, int n, float theta, int window, int dtype, int qhat_sel,
                               cudaStream_t st) {
  const int L = n + 1;
  const int bkv = s.B * s.H_kv;
  int nsplit = (296 + bkv - 1) / bkv;
  if (nsplit > kMaxDecodeSplits) nsplit = kMaxDecodeSplits;
  const int max_by_len = (L + 31) / 32;
  if (nsplit > max_by_len) nsplit = max_by_len;
  if (nsplit < 1) nsplit = 1;
  int chunk = (L + nsplit - 1) / nsplit;
  chunk = (chunk + 31) / 32 * 32;
  if (chunk > kDecodeChunkMax) {
    chunk = kDecodeChunkMax;
    nsplit = (L + chunk - 1) / chunk;
    if (nsplit > kMaxDecodeSplits) return cudaErrorInvalidValue;
  }
  nsplit = (L + chunk - 1) / chunk;
  const float scale_log2e = 1.4426950408889634f / sqrtf((float)s.d);
  const int G = s.g();
  const dim3 grid(nsplit, bkv);
  const size_t smem = ((size_t)3 * G * s.d + (size_t)DNW * G * s.d + 16 + (size_t)G * chunk) * 4;
  cudaError_t err = cudaSuccess;
#define LAUNCH(TC, DD, GG)                                                                       \
  do {                                                                                           \
    auto kern = decode_step_kernel<TC, DD, GG>;                                                  \
    if (smem > 48 * 1024) {                                                                      \
      err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);  \
      if (err != cudaSuccess) return err;                                                        \
    }                                                                                            \
    kern<<<grid, DNT, smem, st>>>((const TC*)q_new, (const TC*)k_new, (const TC*)v_new,          \
                                  (TC*)k_cache, (TC*)v_cache, (TC*)out, w.qhat[qhat_sel],        \
                                  w.qhat[qhat_sel ^ 1], w.R, w.dec_partial, w.dec_ticket,        \
                                  w.counters, n, s.T_max, s.H, chunk, nsplit, theta, window,     \
                                  scale_log2e);                                                  \
  } while (0)
#define LAUNCH_G(TC, DD)                                         \
  switch (G) {                                                   \
    case 1: LAUNCH(TC, DD, 1); break;                            \
    case 2: LAUNCH(TC, DD, 2); break;                            \
    case 4: LAUNCH(TC, DD, 4); break;                            \
    case 8: LAUNCH(TC, DD, 8); break;                            \
    default: return cudaErrorInvalidValue;                       \
  }
  if (dtype == DELTA_F32) {
    if (s.d == 64) { LAUNCH_G(float, 64) } else { LAUNCH_G(float, 128) }
  } else {
    if (s.d == 64) { LAUNCH_G(__nv_bfloat16, 64) } else { LAUNCH_G(__nv_bfloat16, 128) }
  }
#undef LAUNCH_G
#undef LAUNCH
  count_launch();
  return cudaGetLastError();
}

}  // namespace delta
