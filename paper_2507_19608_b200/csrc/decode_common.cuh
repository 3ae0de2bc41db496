// Pieces shared by the decode-step kernels: tile geometry, 8-element row loads, bounded mbarrier
// waits and bulk copies.
#pragma once
#include "delta_internal.cuh"
#include "mbar.cuh"

namespace delta {
namespace {
constexpr int DNT = 256, DNW = DNT / 32;
constexpr int TILE_BYTES = 16384;      // bytes of keys (and of values) per tile
// CTAs the key slices aim for: one wave of two CTAs per SM (a CTA's ring holds 64 KiB).
// Measured at batch 16, 2049 keys: 128 CTAs 51.6 us, 256 CTAs 37.2 us, 512 CTAs 40 us, 1024 CTAs 45 us.
constexpr int kDecodeTargetCtas = 296;

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
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}

// Tail of a decode-step kernel: reduce the per-thread partial outputs of the CTA's key slice,
// store (partial output, running max, running sum) of the slice, and let the last CTA of the
// (batch, KV head) to arrive merge all slices into the output rows.
//   acc   per-thread partial outputs (8 channels of each of the G heads)
//   red   shared [DNW][G][D] floats, wgt shared >= G * kMaxDecodeSplits floats,
//   st_s  shared [24]: running max [0..7], running sum [8..15]
template <typename TC, int D, int G>
__device__ __forceinline__ void decode_merge_slices(
    float (&acc)[G][8], float* red, float* wgt_s, float* st_s, int* s_last, int s_fail,
    float* __restrict__ partial, uint32_t* __restrict__ ticket, unsigned long long* __restrict__ counters,
    TC* __restrict__ out, int split, int bkv, int nsplit, int b, int H, int kvh) {
  constexpr int LPK = D / 8;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sub = lane / LPK;
  const int c0 = (lane % LPK) * 8;
  // ---- reduce the partial outputs over key lanes and warps
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

  // ---- store the slice result; the last slice to arrive merges all of them
  float* part = partial + ((size_t)bkv * kMaxDecodeSplits + split) * G * (D + 2);
  for (int e = tid; e < G * D; e += DNT) {
    float x = 0.0f;
#pragma unroll
    for (int w2 = 0; w2 < DNW; ++w2) x += red[w2 * G * D + e];
    const int hh = e / D, c = e - hh * D;
    part[hh * (D + 2) + c] = x;
  }
  if (tid < G) {
    part[tid * (D + 2) + D] = st_s[tid];
    part[tid * (D + 2) + D + 1] = st_s[8 + tid];
  }
  if (tid == 0 && s_fail) atomicMax(&counters[CNT_STATUS], (unsigned long long)DELTA_ERR_TIMEOUT);
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const uint32_t tk = atomicAdd(&ticket[bkv], 1u);
    *s_last = (tk == (uint32_t)nsplit - 1u);
  }
  __syncthreads();
  if (!*s_last) return;
  __threadfence();
  // merge: weights of all (head, slice) pairs first (loads in parallel), then the outputs
  const float* pbase = partial + (size_t)bkv * kMaxDecodeSplits * G * (D + 2);
  float* den_s = st_s;           // [G] (running max / sum are already in the partials)
  for (int e = tid; e < G * kMaxDecodeSplits; e += DNT) {
    const int hh = e / kMaxDecodeSplits, s2 = e - hh * kMaxDecodeSplits;
    wgt_s[e] = (s2 < nsplit) ? __ldcg(pbase + ((size_t)s2 * G + hh) * (D + 2) + D) : -INFINITY;
  }
  __syncthreads();
  if (warp < G) {
    float m0 = wgt_s[warp * kMaxDecodeSplits + lane], m1 = wgt_s[warp * kMaxDecodeSplits + 32 + lane];
    float M = fmaxf(m0, m1);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    const float w0 = exp2f(m0 - M), w1 = exp2f(m1 - M);   // slices that do not exist weigh 0
    float den = 0.0f;
    if (lane < nsplit) den = w0 * __ldcg(pbase + ((size_t)lane * G + warp) * (D + 2) + D + 1);
    if (lane + 32 < nsplit) den = fmaf(w1, __ldcg(pbase + ((size_t)(lane + 32) * G + warp) * (D + 2) + D + 1), den);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
    wgt_s[warp * kMaxDecodeSplits + lane] = w0;
    wgt_s[warp * kMaxDecodeSplits + 32 + lane] = w1;
    if (lane == 0) den_s[warp] = den;
  }
  __syncthreads();
  for (int e = tid; e < G * D; e += DNT) {
    const int hh = e / D, c = e - hh * D;
    float num = 0.0f;
    int s2 = 0;
    for (; s2 + 4 <= nsplit; s2 += 4) {
      float x[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) x[u] = __ldcg(pbase + ((size_t)(s2 + u) * G + hh) * (D + 2) + c);
#pragma unroll
      for (int u = 0; u < 4; ++u) num = fmaf(wgt_s[hh * kMaxDecodeSplits + s2 + u], x[u], num);
    }
    for (; s2 < nsplit; ++s2)
      num = fmaf(wgt_s[hh * kMaxDecodeSplits + s2], __ldcg(pbase + ((size_t)s2 * G + hh) * (D + 2) + c), num);
    out[((size_t)b * H + kvh * G + hh) * D + c] = from_f32<TC>(num / den_s[hh]);
  }
  if (tid == 0) ticket[bkv] = 0;  // ready for the next step
}

}  // namespace
}  // namespace delta
