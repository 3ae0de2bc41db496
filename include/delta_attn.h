/*
 * delta_attn.h -- C ABI of the B200 (sm_100a) delta-attention library.
 *
 * The library computes DeltaLLM's hybrid attention (arXiv 2507.19608): the query stream of
 * every head is turned into a thresholded delta matrix against a carried reference state
 * (Section II-C, Eq. 2-3; construction strategy (1) of Section III-A), attention scores for
 * keys outside a context window come from the running sum of sparse delta products (Eq. 4),
 * scores inside the window are the full q.k (Section III-B), then scale, causal softmax and
 * the product with V (Eq. 1).  Prefill and single-token decode share one state object
 * (Section III-C; the decode state of strategy (1) is the reference query and the previous
 * score row, Section III-A "Decoding Stage Considerations").
 *
 * Conventions that hold for every entry point unless its comment says otherwise:
 *   - pointers named q, k, v, out, *_cache, *_new, workspace are DEVICE pointers to memory the
 *     caller owns; the library never allocates or frees device memory;
 *   - `stream` is a cudaStream_t passed as void*; calls only enqueue work on it and return
 *     (delta_sparsity_stats and the *_host entry point synchronise it);
 *   - every function returns a delta_status_t; an argument, capacity or call-order error is
 *     found before anything is launched and leaves the state as it was.  DELTA_ERR_CUDA (a
 *     launch or copy the runtime refused) can come after earlier kernels of the same call were
 *     enqueued: the state's position is left unchanged, but workspace and output buffers may
 *     be partly written, so reset the state before using it again;
 *   - tensors are contiguous, row-major, element type from delta_config_t.dtype
 *     (DELTA_F32: float, DELTA_BF16: bfloat16 bit patterns);
 *   - query head h reads KV head h / (H / H_kv).
 */
#ifndef DELTA_ATTN_H_
#define DELTA_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#if defined(DELTA_BUILDING_LIB) && defined(__GNUC__)
#define DELTA_API __attribute__((visibility("default")))
#else
#define DELTA_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

/* Rows per delta tile: per-tile non-zero counters and per-tile reference snapshots use it. */
#define DELTA_TILE_ROWS 64

typedef enum {
  DELTA_OK = 0,
  DELTA_ERR_INVALID_ARG = 1,  /* null pointer, bad size, theta < 0 or not finite, ...          */
  DELTA_ERR_UNSUPPORTED = 2,  /* a configuration this build has no kernel for                  */
  DELTA_ERR_WORKSPACE = 3,    /* workspace too small or not 256-byte aligned                   */
  DELTA_ERR_CAPACITY = 4,     /* sequence would exceed T_max                                   */
  DELTA_ERR_STATE = 5,        /* call order: prefill on a used state, decode before prefill    */
  DELTA_ERR_CUDA = 6,         /* a CUDA runtime call failed (delta_last_cuda_error has it)     */
  DELTA_ERR_TIMEOUT = 7,      /* a bounded device-side wait ran out (status word on device)    */
  DELTA_ERR_SCRATCH_LIMIT = 8, /* problem larger than the built-in scratch of the no-alloc call */
  DELTA_ERR_BOUNDS = 9        /* bounds-checking build only: a kernel formed an index outside its
                                 array; the access was skipped and the status word records it    */
} delta_status_t;

typedef enum { DELTA_F32 = 0, DELTA_BF16 = 1 } delta_dtype_t;

/* Which operand becomes the delta matrix (Section III-A).
 * QUERY = strategy (1), top-down query deltas: one chain per (query head, channel); the carried
 *   decode state is the reference query and the score row R.
 * KEY = strategy (3), the one the paper adopts: the key stream of every KV head is thresholded
 *   (one chain per (KV head, channel)); the out-of-window score of pair (i, j) is the column
 *   recursion S[i][j] = S[i][j-1] + q_i.Delta k(j) = q_i.k_hat(j); the carried decode state is
 *   the reference key, and the library keeps a cache of reference-key rows in its workspace.
 *   bf16 with d = 64 or 128 only (DELTA_ERR_UNSUPPORTED otherwise).  With KEY the delta arrays
 *   of delta_state_view hold one set per KV head: read them as [B * H_kv, ...] from the start
 *   of the view.
 * QUERY_BOTTOM_UP = strategy (2): query deltas with the rows taken from the last token up to
 *   the first, so the basis is the last row and the reference of row i is the last value that
 *   fired among rows i .. T-1.  Prefill only (the method needs the whole sequence before its
 *   first row): decode on such a state returns DELTA_ERR_UNSUPPORTED.  bf16 with d = 64 or 128
 *   only.  All delta arrays of delta_state_view stay indexed by token row; the per-tile
 *   reference snapshot of tile t is the reference before the tile's highest row is processed
 *   and DELTA_VIEW_QHAT is the reference left after row 0. */
typedef enum { DELTA_SRC_QUERY = 0, DELTA_SRC_KEY = 1, DELTA_SRC_QUERY_BOTTOM_UP = 2 } delta_source_t;

/* Shape of the exact-attention region in prefill (Section III-B).  BLOCK: squares of side
 * `window` along the diagonal, anchored at token 0 (pair (i,j) is exact iff i/W == j/W).
 * SLIDING: the `window` most recent keys of every query (exact iff i - j < W).  window = 0
 * means no exact score at all; window >= T means dense attention.  Decode always uses
 * SLIDING (the W_d most recent tokens, the new one included). */
typedef enum { DELTA_WIN_BLOCK = 0, DELTA_WIN_SLIDING = 1 } delta_window_shape_t;

/* Treatment of row 0 in Eq. 2-3.  BASIS_EXACT: the first vector is the un-thresholded basis
 * (Delta q(0) = q(0), reference = q(0), all mask bits set).  ZERO_STATE: the reference
 * starts at 0 and row 0 is thresholded like every other row. */
typedef enum { DELTA_INIT_BASIS_EXACT = 0, DELTA_INIT_ZERO_STATE = 1 } delta_init_t;

typedef struct {
  int32_t B;      /* batch elements                                     */
  int32_t H;      /* query heads                                        */
  int32_t H_kv;   /* key/value heads, H % H_kv == 0, H / H_kv <= 8      */
  int32_t d;      /* head dimension, 64 or 128                          */
  int32_t T_max;  /* capacity in tokens (prefill length + decode steps) */
  delta_dtype_t dtype;
  delta_source_t source;
  delta_window_shape_t prefill_window;
  delta_init_t init;
} delta_config_t;

/* Opaque host object; owns no device memory (everything lives in the caller's workspace). */
typedef struct delta_state delta_state_t;

/* Bytes of device workspace a state with this configuration needs (multiple of 256). */
DELTA_API delta_status_t delta_state_workspace_bytes(const delta_config_t* cfg, size_t* bytes);

/* delta_state_init -- create a state over a caller-owned device workspace (256-byte aligned,
 * at least delta_state_workspace_bytes large) and enqueue the zeroing of the reference state
 * q_hat and all counters (Eq. 3: the reference starts at 0; one small memset).  The score row R
 * is not cleared: prefill writes its entries 0..T-1 and a decode step reads only entries below
 * its position.  *out is a host object the caller releases with delta_state_destroy; the
 * workspace must outlive it. */
DELTA_API delta_status_t delta_state_init(const delta_config_t* cfg, void* workspace, size_t workspace_bytes,
                                void* stream, delta_state_t** out);

/* Back to the freshly initialised condition (position 0, reference 0, counters 0).  Host-side
 * only: the clearing of the device span is done by the first kernel of the next prefill on this
 * state, on that call's stream (`stream` is unused); delta_sparsity_stats reports zeros in
 * between, delta_state_view still shows the old contents until that prefill. */
DELTA_API delta_status_t delta_state_reset(delta_state_t* st, void* stream);

/* Frees the host object only. */
DELTA_API delta_status_t delta_state_destroy(delta_state_t* st);

/* delta_attn_prefill -- hybrid delta attention over T tokens (Section III, prefilling stage).
 *   q, out : [B, H, T, d]            k, v : [B, H_kv, T_max, d] (KV-cache layout, rows 0..T-1 read)
 *   theta  : delta threshold of Eq. 2 (>= 0, finite); |diff| == theta does not fire
 *   window : W of Section III-B (>= 0), shape from the configuration
 * q, k, v and out must be 16-byte aligned.
 * Steps enqueued: delta construction over Q (Eq. 2-3: values, bit mask, per-row and per-tile
 * non-zero counts, compacted channel indices, per-tile reference snapshots), the fused
 * hybrid-attention kernel (exact q.k inside the window, running delta sums outside (Eq. 4),
 * scale 1/sqrt(d), causal online softmax, P.V (Eq. 1)), the hand-off of q_hat(T-1) and
 * R(T-1)[0..T-1] for decode, and the sparsity counters (Eq. 6).
 * H, H_kv, d must equal the configuration.  Needs a fresh or reset state (else
 * DELTA_ERR_STATE); 1 <= T <= T_max (else DELTA_ERR_CAPACITY). */
DELTA_API delta_status_t delta_attn_prefill(delta_state_t* st, const void* q, const void* k, const void* v,
                                  void* out, int32_t T, int32_t H, int32_t H_kv, int32_t d,
                                  float theta, int32_t window, void* stream);

/* delta_attn_prefill_varlen -- one prefill over a batch of sequences of different lengths, each
 * with its own window (Section III-B, Eq. 5: the prefill window follows the input length,
 * W = min(floor(gamma n), W_max); delta_window_from_gamma gives it).
 *   seq_lens : HOST array [B], tokens of every sequence (1 .. T_max)
 *   windows  : HOST array [B], W of every sequence (>= 0), shape from the configuration
 *   q, out   : packed: sequence b occupies [H, seq_lens[b], d] elements, the sequences one behind
 *              the other in batch order (sequence b starts H * d * (seq_lens[0] + .. + seq_lens[b-1])
 *              elements into the array)
 *   k, v     : [B, H_kv, T_max, d] (KV-cache layout; rows 0 .. seq_lens[b]-1 of element b are read)
 * Every sequence is what delta_attn_prefill computes for a batch of one: its own delta chains,
 * window, counters (Eq. 6 sums over the sequences: S_c_eq6 uses sum min(W_b, n_b) / sum n_b) and
 * decode hand-off.  Afterwards the batch elements stand at different positions:
 * delta_state_sequence_position reports each, delta_state_position the longest, and
 * delta_attn_decode_step advances every sequence by one token from where it stands (one kernel
 * launch per batch element while the positions differ).  Needs a fresh or reset state. */
DELTA_API delta_status_t delta_attn_prefill_varlen(delta_state_t* st, const void* q, const void* k, const void* v,
                                         void* out, const int32_t* seq_lens, const int32_t* windows,
                                         float theta, void* stream);

/* delta_attn_prefill_host -- the same call for HOST buffers (q, k, v, out are host pointers
 * with the shapes above; k and v hold T rows per head, i.e. [B, H_kv, T, d]).  `staging` is
 * a DEVICE buffer of at least delta_prefill_staging_bytes(cfg, T) bytes that receives the
 * copies.  Copies in, runs the prefill, copies `out` back and synchronises the stream. */
DELTA_API delta_status_t delta_prefill_staging_bytes(const delta_config_t* cfg, int32_t T, size_t* bytes);
DELTA_API delta_status_t delta_attn_prefill_host(delta_state_t* st, const void* q_host, const void* k_host,
                                       const void* v_host, void* out_host, void* staging,
                                       size_t staging_bytes, int32_t T, float theta,
                                       int32_t window, void* stream);

/* delta_attn_decode_step -- one decoding step for every (batch, head) (Section III-B/C,
 * decoding stage, carried state of strategy (1)).
 *   q_new, out : [B, H, d]     k_new, v_new : [B, H_kv, d]
 *   k_cache, v_cache : [B, H_kv, T_max, d]; rows 0..n-1 are read, row n is written by the call
 * With n the tokens seen so far: Delta q = threshold(q_new - q_hat) and q_hat update (Eq. 2-3);
 * R[j] += Delta q . k_j for every cached key j < n (Eq. 4); R[n] = q_hat . k_new for the key
 * that arrives now; score j is q_new.k_j if n - j < window else R[j]; softmax over the n + 1
 * keys; out = P.V; position becomes n + 1.  Needs n >= 1 (else DELTA_ERR_STATE) and
 * n < T_max (else DELTA_ERR_CAPACITY).
 * Eq. 4's sum telescopes to R[j] = q_hat . k_j (exactly, up to the order of the fp32
 * additions, for bf16 inputs, whose references are copies of input elements); where
 * delta_state_decode_kernel reports 1 the step computes R[j] in that form on the tensor cores
 * and writes it back without reading it.
 * All six tensor pointers must be 16-byte aligned (the kernels stage cache tiles with bulk
 * copies and read rows as 16-byte vectors): DELTA_ERR_INVALID_ARG otherwise, nothing launched.
 * With DELTA_SRC_KEY the step thresholds k_new against the carried reference key instead
 * (Eq. 2-3), appends the reference-key row k_hat(n), and scores key j with q_new.k_j if
 * n - j < window else q_new.k_hat(j). */
DELTA_API delta_status_t delta_attn_decode_step(delta_state_t* st, const void* q_new, const void* k_new,
                                      const void* v_new, void* k_cache, void* v_cache, void* out,
                                      float theta, int32_t window, void* stream);

/* delta_attn_decode_step_noalloc -- the decode step without any workspace.  (The paper has
 * no counterpart: this exists only for callers that cannot allocate device memory.)
 *
 * Who needs it: code running inside an application whose own memory manager has claimed the
 * whole GPU, so that cudaMalloc fails or is not allowed; latency-critical loops that must stay
 * clear of the device-wide synchronisation cudaMalloc/cudaFree imply; plug-ins that are handed
 * nothing but input and output pointers.  This call allocates and frees nothing, on the host
 * side of the driver or on the device, and calls no library routine that does.
 *
 * It performs exactly the step of delta_attn_decode_step, but stateless: the carried state is
 * passed in and out by the caller instead of living in a delta_state_t.
 *   q_new, out       : [B, H, d]        k_new, v_new : [B, H_kv, d]       (element type `dtype`)
 *   k_cache, v_cache : [B, H_kv, T_max, d]; rows 0..n-1 are read, row n is written
 *   qhat_in          : [B, H, d] float, reference state before the step (read only)
 *   qhat_out         : [B, H, d] float, reference state after the step (must differ from qhat_in)
 *   R                : [B, H, T_max] float, score row; entries 0..n-1 are updated in place,
 *                      entry n is written
 *   n                : tokens already in the cache (>= 1, < T_max)
 * All pointers are DEVICE pointers owned by the caller.  The sparsity counters of the regular
 * call are not kept.
 *
 * Scratch: the split-KV partial results and arrival tickets live in a fixed array of 8 MiB +
 * 8 KiB inside the library image; every GPU that loads the library holds it until the process
 * exits.  Limits that follow from its size: B * H_kv <= 1024 and B * H * (d + 2) <= 32768
 * (for example B = 15 at 32 heads of dimension 64); anything larger returns
 * DELTA_ERR_SCRATCH_LIMIT and launches nothing.
 * The first call on each device looks up the array's device address (with that device
 * current); make that first call outside of any stream capture.  Every call shares the one
 * array and finds in it what the previous call left: the parts that must start at zero are
 * cleared on `stream` at the start of the call.  Calls whose kernels may overlap on one GPU
 * (different streams or threads) race on the array: serialise them.
 * All nine pointers must be 16-byte aligned (DELTA_ERR_INVALID_ARG otherwise).
 * The call itself never returns DELTA_ERR_TIMEOUT: a bounded device-side wait that ran out
 * leaves its mark in a status word inside the scratch array, which stays set across later
 * calls until delta_noalloc_device_status reads it. */
DELTA_API delta_status_t delta_attn_decode_step_noalloc(
    const void* q_new, const void* k_new, const void* v_new, void* k_cache, void* v_cache, void* out,
    const float* qhat_in, float* qhat_out, float* R, int32_t n, int32_t B, int32_t H, int32_t H_kv,
    int32_t d, int32_t T_max, delta_dtype_t dtype, float theta, int32_t window, void* stream);

/* delta_noalloc_device_status -- the device status word of delta_attn_decode_step_noalloc on the
 * current device (the paper has no counterpart): copies it to *host_status (HOST pointer),
 * clears it and synchronises `stream`.  0 means every no-alloc step enqueued on `stream` so far
 * ran to its end; DELTA_ERR_TIMEOUT means one of them gave up a bounded wait and its outputs
 * are not valid.  The return value is DELTA_OK or that status.  Allocates nothing. */
DELTA_API delta_status_t delta_noalloc_device_status(uint32_t* host_status, void* stream);

/* Counters of one stage.  S_m = 1 - nnz/elements (sparsity of the delta matrix, Eq. 6);
 * S_c_eq6 = S_m * (1 - W/n) (Eq. 6); S_c_exact = 1 - macs_done/macs_dense where a causal
 * pair costs d multiply-adds inside the window and nnz(Delta q_i) outside it, against d for
 * every causal pair of dense attention. */
typedef struct {
  uint64_t nnz, elements, macs_done, macs_dense;
  double S_m, S_c_eq6, S_c_exact;
} delta_stage_stats_t;

typedef struct {
  delta_stage_stats_t prefill, decode, combined;
  int32_t n;             /* tokens seen so far */
  uint32_t device_status; /* 0, or the DELTA_ERR_* a kernel recorded in the device status word */
} delta_stats_t;

/* delta_sparsity_stats -- copy the device counters to the host and finish Eq. 6.
 * Synchronises `stream`.  host_out is a HOST pointer. */
DELTA_API delta_status_t delta_sparsity_stats(const delta_state_t* st, delta_stats_t* host_out, void* stream);

/* Eq. 5: W_p,max = min(floor(gamma * n), w_max), the product taken in double precision.
 * gamma is a double so that a decimal scaling factor gives the window the formula gives on
 * paper (floor(0.02 * 100) = 2; the float nearest to 0.02 lies below it and would give 1).
 * Returns 0 for n < 0, gamma < 0 or NaN. */
DELTA_API int32_t delta_window_from_gamma(int32_t n, double gamma, int32_t w_max);

/* Device views into the state's workspace, for parity checks and checkpointing.
 * Shapes (T_max rows allocated, rows 0..T-1 valid after a prefill of T tokens):
 *   DQ        float    [B, H, T_max, d]        Delta q(t), +0.0 where not fired
 *   MASK      uint32   [B, H, T_max, d/32]     bit (c % 32) of word (c / 32)
 *   ROW_NNZ   uint16   [B, H, T_max]
 *   TILE_NNZ  uint32   [B, H, ceil(T_max/64)]
 *   IDX       uint8    [B, H, T_max, d]        fired channel ids ascending, 0xFF padding
 *   QHAT_TILE float    [B, H, ceil(T_max/64), d]  reference state before each tile's first row
 *   QHAT      float    [B, H, d]               current reference state
 *   R         float    [B, H, T_max]           current score row (un-scaled), entries 0..n-1
 *   COUNTERS  uint64   [144]                   raw device counters; word 8 is the device status word
 *                                              (0, or the DELTA_ERR_* a kernel recorded), which
 *                                              delta_sparsity_stats reports and returns
 */
typedef enum {
  DELTA_VIEW_DQ = 0, DELTA_VIEW_MASK = 1, DELTA_VIEW_ROW_NNZ = 2, DELTA_VIEW_TILE_NNZ = 3,
  DELTA_VIEW_IDX = 4, DELTA_VIEW_QHAT_TILE = 5, DELTA_VIEW_QHAT = 6, DELTA_VIEW_R = 7, DELTA_VIEW_COUNTERS = 8
} delta_view_t;
DELTA_API delta_status_t delta_state_view(const delta_state_t* st, int32_t what, const void** dev_ptr,
                                size_t* bytes);

/* Tokens seen so far (0 after init/reset); after delta_attn_prefill_varlen, of the longest sequence. */
DELTA_API int32_t delta_state_position(const delta_state_t* st);
/* Tokens seen so far by batch element b (-1 for a bad argument). */
DELTA_API int32_t delta_state_sequence_position(const delta_state_t* st, int32_t b);

/* Which prefill kernel the next delta_attn_prefill on this state will use:
 *   0 = generic CUDA-core kernel (every configuration);
 *   1 = tcgen05/TMA kernel, out-of-window scores by Eq. 4's running sum of sparse delta
 *       products on the FP32 pipes, skipping all-zero delta blocks (bf16, d = 64);
 *   2 = tcgen05/TMA kernel, out-of-window scores by the telescoped form of Eq. 4,
 *       R(i)[j] = q_hat(i).k_j, as one more tensor-core product (bf16, d = 64 or 128).
 *       A CTA takes one head's query tile and splits its key tiles between two softmax
 *       groups, or (d = 64 with an even number of query heads per KV head)
 *       the same query tile of two heads of a KV group, so that every key and value tile
 *       is fetched once for both; which CTAs take which form follows the size of the grid;
 *   3 = kernel 2 with every CTA in the one-head form, 4 = every CTA in the two-heads form,
 *   5 = the two-heads form with the heaviest query tile of every head in the one-head form
 *       (3 to 5 are never chosen as such; for comparison and tests).
 * All compute the same function.  delta_state_set_prefill_kernel forces one
 * (-1 = automatic); forcing a kernel the configuration has none for returns
 * DELTA_ERR_UNSUPPORTED. */
DELTA_API int32_t delta_state_prefill_kernel(const delta_state_t* st);

/* Which kernel the next delta_attn_decode_step of this state would use: 1 = score products
 * on the tensor cores (bf16, d = 64, top-down query deltas or key deltas, at most 73728 keys:
 * the telescoped form of Eq. 4, see delta_attn_decode_step), 0 = the FP32-pipe kernel,
 * -1 for a null state.  Both compute the same step and keep the same state. */
DELTA_API int32_t delta_state_decode_kernel(const delta_state_t* st);

/* Force the decode kernel of a state: 1 = tensor-core scores whatever the slice length
 * (DELTA_ERR_UNSUPPORTED unless bf16, d = 64, top-down query deltas or key deltas), 0 = FP32 pipes, -1 = chosen per
 * step (the default).  Host-side only. */
DELTA_API delta_status_t delta_state_set_decode_kernel(delta_state_t* st, int32_t which);
DELTA_API delta_status_t delta_state_set_prefill_kernel(delta_state_t* st, int32_t which);

/* Key deltas (DELTA_SRC_KEY, bf16): which form of the thresholded key stream the decode steps
 * read (Section III-A "Decoding Stage Considerations", Section III-C: the cache holds the key
 * deltas instead of the keys, plus the last W_d original keys).
 *   packed = 0 (default): dense rows of reference keys k_hat(j), streamed like a key cache;
 *   packed = 1: the delta stream itself -- per key row a bit mask of the elements that fired and
 *     the fired values packed behind one another, the reference key in front of every 32 rows
 *     and the offsets of those 32-row segments; a decode step rebuilds the reference-key rows of
 *     a tile in shared memory from that.  The keys inside the decode window are read from
 *     k_cache.  Same results bit for bit; the bytes a step reads for the keys shrink with the
 *     delta sparsity (delta_key_cache_bytes), the step itself runs on the FP32 pipes.
 * Set it on a fresh or reset state (DELTA_ERR_STATE otherwise): the prefill builds the encoding.
 * The workspace reserves the packed pool for the worst case (every element fires) beside the
 * dense rows the prefill kernel streams, so the choice changes what decoding reads, not what
 * delta_state_workspace_bytes asks for. */
DELTA_API delta_status_t delta_state_set_key_cache(delta_state_t* st, int32_t packed);
/* Bytes of the packed key-delta encoding in use (values, masks, counts, segment bases and
 * offsets over all batch elements and KV heads) and of the dense reference-key rows of the
 * same tokens.  Synchronises `stream`.  DELTA_ERR_UNSUPPORTED unless the packed cache is on. */
DELTA_API delta_status_t delta_key_cache_bytes(const delta_state_t* st, uint64_t* packed_bytes,
                                     uint64_t* dense_bytes, void* stream);

/* Per-kernel timing of delta_attn_prefill.  With profiling enabled the call records a CUDA
 * event in front of and behind each of its kernels on the caller's stream (host-side event
 * objects; no device memory).  delta_state_prefill_kernel_ms waits for the last event and
 * returns the elapsed milliseconds of the most recent prefill in ms[0..3]:
 * [0] delta chain (Eq. 2-3), [1] counts, compacted indices, Eq. 6 counters, decode hand-off and
 * key re-layout, [2] hybrid attention, [3] reserved (0).
 * DELTA_ERR_STATE if profiling is off or no prefill was recorded. */
DELTA_API delta_status_t delta_state_enable_profiling(delta_state_t* st, int32_t enable);
DELTA_API delta_status_t delta_state_prefill_kernel_ms(delta_state_t* st, float* ms);

/* 1 if this library was built with -DDELTA_DEBUG_BOUNDS: every global index the kernels compute
 * by hand is range-checked against the extent of its array, an index out of range is not
 * accessed and DELTA_ERR_BOUNDS goes to the device status word (delta_sparsity_stats reports it).
 * 0 for the regular build, whose kernels carry no such checks.  (Tile copies by TMA are
 * bounded by their tensor maps in both builds.) */
DELTA_API int32_t delta_debug_bounds_build(void);

/* Kernels launched by this library in the calling process since it was loaded. */
DELTA_API uint64_t delta_launch_count(void);

DELTA_API const char* delta_status_string(delta_status_t s);
/* Text of the last CUDA runtime error seen by this library in the calling thread. */
DELTA_API const char* delta_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* DELTA_ATTN_H_ */
