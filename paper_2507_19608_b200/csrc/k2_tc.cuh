// Tensor-core (tcgen05 / TMEM / TMA) hybrid-attention kernel for bf16 inputs: interface.
#pragma once
#include "delta_internal.cuh"

namespace delta {
// Does this build carry a tensor-core prefill kernel for head dimension d?
bool tc_kernel_available(int d);
// Is head dimension d one the tensor-core kernel is written for (no driver query)?
bool tc_kernel_shape(int d);
cudaError_t launch_hybrid_attn_tc(const Shape& s, const Workspace& w, const void* q, const void* k,
                                  const void* v, void* out, int T, int window, int shape,
                                  cudaStream_t st);
// Head dimensions the telescoped kernel is written for.
bool tcq_kernel_shape(int d);
// Telescoped variant: out-of-window scores as Q_hat.K^T (query deltas) or Q.K_hat^T (key deltas)
// on the tensor cores; w.qhat_rows holds the reference rows of the delta stream.
// form: 1 = a CTA owns one head's query tile and splits its key tiles between two softmax
// groups; 2 = a CTA owns the same query tile of two heads of a KV group (d = 64,
// an even number of query heads per KV head; cudaErrorNotSupported otherwise); 3 = form 2 with
// the heaviest query tile of every head in form 1; 0 = chosen by the size of the grid.
cudaError_t launch_hybrid_attn_tcq(const Shape& s, const Workspace& w, const void* q, const void* k,
                                   const void* v, void* out, int T, float theta, int init, int window,
                                   int shape, bool key_deltas, bool reverse, int form, cudaStream_t st);
}  // namespace delta
