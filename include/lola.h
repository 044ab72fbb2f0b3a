/*
 * lola.h - C ABI of the B200 (sm_100a) LoLA per-layer attention step.
 *
 * LoLA ("Low-Rank Linear Attention with Sparse Caching", arXiv 2505.23666) keeps every past
 * key-value pair of an attention head in exactly one of three memories (section "Mitigating Memory
 * Collisions with Sparse Caching", Fig. 1): a sliding window of the eta most recent pairs, a sparse
 * global cache G of at most lambda pairs, and the linear-attention state H (D x d_v), s (D) of
 * Eq. 5.  Pairs leaving the window are scored, together with all of G, by their self-recall error
 * (Eq. 10) against the current H, s; the lambda highest stay in G (Eq. 12), the rest are folded
 * into H, s (Eq. 13).  The output (Eq. 14) adds the linear term phi(q)^T H, the sparse-cache term
 * and the window term over ONE shared denominator.
 *
 * Conventions for every entry point
 *   - All tensors are row-major with the head dimension innermost and contiguous.
 *   - "dev" pointers are CUDA device pointers on the current device, "host" pointers are ordinary
 *     host memory.  The library never allocates or frees device memory; the caller owns every
 *     buffer (state, W, q, k, v, out) and must keep W and the state buffer alive for the life of
 *     the handle.  Everything a call enqueues goes to the caller's stream; inside a lola_prefill_chunk call
 *     the scoring of the eligible set runs beside the attention kernel (both only read the memories; the
 *     kernels are chained by programmatic dependent launches on that one stream), and the fold follows both.
 *   - Work is enqueued on the given stream (a cudaStream_t passed as void*; NULL = legacy default
 *     stream) and the call returns without synchronising unless stated otherwise.  All calls on
 *     one state must be issued on one stream, or be ordered by the caller.  The kernels of a call are
 *     launched with programmatic stream serialization and read the call's q before they wait for the
 *     work ahead of them in the stream: what writes q, k, v must be complete in the ordinary way (a
 *     copy, or a kernel that does not signal programmatic launch completion before its end).
 *   - Return value: LOLA_OK (0) or a negative error code.  Argument errors are found on the host
 *     before anything is enqueued and leave the state untouched.  Nothing throws, prints or exits.
 *   - One state serves `batch` sequences that advance in lock-step (equal lengths, no padding).
 *     A "unit" is one (batch row, KV head); the n_q_heads / n_kv_heads query heads of a group share
 *     their KV head's feature-map weights and its three memories.
 *   - Token positions are int32 (at most 2^31 - 1 tokens per sequence).
 */
#ifndef LOLA_H_
#define LOLA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  LOLA_OK = 0,
  LOLA_ERR_ARG = -1,         /* null pointer, bad enum, inconsistent view                      */
  LOLA_ERR_SHAPE = -2,       /* sizes out of range (n_tokens > max_chunk, heads not divisible) */
  LOLA_ERR_ALIGN = -3,       /* a device pointer is not 16-byte aligned (state: 256-byte)      */
  LOLA_ERR_SIZE = -4,        /* caller's buffer smaller than lola_state_bytes / staging bytes  */
  LOLA_ERR_UNSUPPORTED = -5, /* shape outside what the kernels are built for                   */
  LOLA_ERR_CUDA = -6,        /* a CUDA runtime call or launch failed                           */
  LOLA_ERR_DEVICE = -7       /* a kernel recorded an internal error in the state's status word */
};

typedef enum { LOLA_F32 = 0, LOLA_BF16 = 1 } lola_dtype;

/* Feature map phi: R^{d} -> R^{2F}, u = x W.
 *   LOLA_PHI_SOFTMAX: [softmax(u), softmax(-u)], each over its F entries (the benchmark workloads);
 *   LOLA_PHI_EXP:     [exp(u), exp(-u)]                                              (Eq. 6).     */
typedef enum { LOLA_PHI_SOFTMAX = 0, LOLA_PHI_EXP = 1 } lola_phi;

/* config flag: run the shape-generic CUDA-core kernels even where tensor-core kernels exist (bf16,
 * F = 64).  Both compute the same function; the flag exists for cross-checks and timing.        */
#define LOLA_FLAG_GENERIC_KERNELS 1u
/* config flags of the cache ablation (appendix "Sparse Cache & Linear Attention Ablation"): the memories are
 * updated as always, but the queries do not see the linear-attention state (the phi(q)^T H and phi(q)^T s terms
 * of Eq. 14 are left out) and / or the sparse cache (its sum in Eq. 14 is left out).  With both set Eq. 14 is
 * softmax attention over the sliding window (and, in a prefill call, the chunk itself).  A query that then sees
 * nothing at all (window = 0 in a generation step) has no defined output.  Generation steps with either flag run
 * as the kernel chain, not as the fused kernel.                                                          */
#define LOLA_FLAG_QUERY_NO_LINEAR 4u
#define LOLA_FLAG_QUERY_NO_SPARSE 8u
#define LOLA_FLAGS_ALL (LOLA_FLAG_GENERIC_KERNELS | LOLA_FLAG_QUERY_NO_LINEAR | LOLA_FLAG_QUERY_NO_SPARSE)

typedef struct lola_config {
  int32_t batch;         /* B >= 1                                                              */
  int32_t n_q_heads;     /* Hq, multiple of n_kv_heads                                          */
  int32_t n_kv_heads;    /* Hkv                                                                 */
  int32_t head_dim;      /* d = d_k = d_v, 64 or 128                                            */
  int32_t feat_half;     /* F in [1, 128]; the state has D = 2F feature rows                    */
  int32_t window;        /* eta >= 0: pairs resident in the sliding window between calls        */
  int32_t sparse;        /* lambda >= 0: slots of the sparse cache; lambda + max_chunk <= 16384 */
  int32_t max_chunk;     /* C >= 1: largest n_tokens a prefill call may pass                    */
  int32_t dtype;         /* lola_dtype of q, k, v, out, W and of the cached keys/values.
                            H, s, scores and all softmax statistics are always fp32.
                            LOLA_BF16 additionally rounds phi(K) and H to bf16 inside the Eq. 10
                            contraction and folds the rounded phi(K) (Eq. 13).                  */
  int32_t phi_kind;      /* lola_phi                                                            */
  float softmax_scale;   /* 0 => 1/sqrt(head_dim) (Eq. 2)                                       */
  uint32_t flags;        /* 0, or an OR of LOLA_FLAG_*                                          */
} lola_config;

/* Opaque host-side handle.  Owns no device memory. */
typedef struct lola_state lola_state;

/* Host arrays for lola_read_state / lola_write_state.  Every pointer is optional on read (NULL =
 * skip).  U = batch * n_kv_heads units, unit index = b * n_kv_heads + h.  Elements of *_k / *_v
 * have the state's dtype (bf16 as raw 16-bit words).                                            */
typedef struct lola_state_view {
  float* H;               /* [U, D, d]   Eq. 5 state, fp32                                      */
  float* s;               /* [U, D]                                                             */
  int32_t* sparse_count;  /* [U]         occupied slots of G: slots 0 .. count-1                */
  int32_t* sparse_pos;    /* [U, lambda] token position held by each slot, -1 = empty           */
  void* sparse_k;         /* [U, lambda, d]                                                     */
  void* sparse_v;         /* [U, lambda, d]                                                     */
  float* sparse_score;    /* [U, lambda] self-recall error at the last scored update (NaN: the
                                         pair has never been scored)                            */
  float* threshold;       /* [U, 2]      lowest kept / highest folded score of the last scored
                                         update (NaN before the first one)                      */
  int32_t* window_count;  /* [U]                                                                */
  int32_t* window_pos;    /* [U, eta]    position held by ring slot j (= position % eta), -1    */
  void* window_k;         /* [U, eta, d] ring-slot order                                        */
  void* window_v;         /* [U, eta, d]                                                        */
  int64_t* n_seen;        /* [B]         tokens consumed so far                                 */
  int32_t* status;        /* [1]         sticky device status word, 0 = healthy                 */
} lola_state_view;

/* Device bytes the caller must provide for one state (a multiple of 256).  0 if cfg is invalid.
 * Holds H, s, the sparse cache with positions and scores, the window ring, for bf16 layers with
 * feat_half = 64 the tensor-core operand images of W (per KV head) and of H (per unit), and the small per-unit
 * work lists the update kernels pass to each other.                                             */
size_t lola_state_bytes(const lola_config* cfg);

/* Pseudo-code `init`: empty window, empty sparse cache, H = 0, s = 0.
 *   W_dev     [Hkv, d, F] feature-map weights in cfg->dtype, device, 16-byte aligned; shared by
 *             queries and keys of the KV head's group.
 *   state_dev device buffer of at least lola_state_bytes(cfg), 256-byte aligned; zeroed
 *             asynchronously on `stream`.
 *   out       receives the handle (host heap; release with lola_destroy_state).
 * Errors: ARG, SHAPE, ALIGN, SIZE, UNSUPPORTED (device is not compute capability 10.x), CUDA.   */
int lola_init_state(const lola_config* cfg, const void* W_dev, void* state_dev, size_t state_bytes,
                    void* stream, lola_state** out);

/* Back to the state lola_init_state leaves (pseudo-code `init`), asynchronously on `stream`. */
int lola_reset_state(lola_state* st, void* stream);

/* Chunkwise inference (section "Chunkwise Inference", Eq. 15): attend, then evict.
 * Every query of the chunk sees, with softmax weights, the sparse cache, the resident window and
 * the chunk itself causally; with linear weights, the H, s of the start of the call (Eq. 14).
 * Then the chunk joins the window; the pairs that no longer fit (oldest first) are scored together
 * with all of G by Eq. 10 against the H, s before the fold, the lambda highest errors stay in G
 * (ties: the older pair stays), and the rest are folded into H, s (Eq. 13).  While fewer than
 * lambda pairs have ever left the window nothing is scored or folded.
 *   q   [B, n_tokens, Hq, d] dev      k, v [B, n_tokens, Hkv, d] dev      out [B, n_tokens, Hq, d] dev
 *   out may be NULL: only the caches advance (q is then ignored and may be NULL).
 *   1 <= n_tokens <= max_chunk.
 * Errors: ARG, SHAPE, ALIGN, CUDA.                                                              */
int lola_prefill_chunk(lola_state* st, const void* q, const void* k, const void* v, int32_t n_tokens,
                       void* out, void* stream);

/* A run of `n_chunks` consecutive prefill chunks of `n_tokens` tokens each in one call (section "Chunkwise
 * Inference": the chunks of a prompt in order; the chunk recurrence is sequential, so the run is enqueued chunk
 * after chunk on `stream`, the kernels of neighbouring chunks overlapping where their dependencies allow).
 * q, k, v, out hold the chunks one after the other: chunk c is the tensor [B, n_tokens, heads, d] that
 * lola_prefill_chunk takes, at byte offset c * (bytes of that tensor), all in device memory.  out (and then q)
 * may be NULL.  Same results, bit for bit, as n_chunks calls of lola_prefill_chunk.
 * Errors: as lola_prefill_chunk, plus SHAPE for n_chunks < 1; the run stops at the first failing chunk.    */
int lola_prefill_chunks(lola_state* st, const void* q, const void* k, const void* v, int32_t n_chunks, int32_t n_tokens,
                        void* out, void* stream);

/* Generation step (Eq. 11-14): update, then attend.  The new pair enters the window; if the window
 * overflows its oldest pair is evicted, E = G u {evicted} is scored against the current H, s, the
 * lowest-error pair of E is folded and the others form G; then Eq. 14 is evaluated over the updated
 * G, H, s and the window including the new pair.
 *   q [B, Hq, d] dev      k, v [B, Hkv, d] dev      out [B, Hq, d] dev (required)
 * Errors: ARG, ALIGN, CUDA.                                                                     */
int lola_decode_step(lola_state* st, const void* q, const void* k, const void* v, void* out, void* stream);

/* lola_decode_step for callers that cannot provide scratch memory at call time.  The paper has no
 * counterpart: this is a packaging variant of the generation step above, same arguments, same
 * results.
 *
 * Who needs it: code that runs where device allocation is closed - a serving loop whose engine has
 * handed all device memory to its own arena and forbids cudaMalloc after start-up, or a plug-in
 * that only receives the persistent memories (H, s, the caches) from its host application.  The
 * step passes small per-unit work lists from its selection kernel to its update kernel (which pairs
 * to fold, which pair moves to which slot).  lola_decode_step keeps them in the caller's state
 * buffer; this variant keeps them in a device array that is part of the library image, so they
 * exist without anybody allocating them.
 *
 * Limits: batch * n_kv_heads <= LOLA_STATIC_MAX_UNITS and batch * n_kv_heads * max_chunk <=
 * LOLA_STATIC_MAX_LIST_ENTRIES, otherwise LOLA_ERR_SIZE and nothing is enqueued.  The array takes
 * (3 * LOLA_STATIC_MAX_LIST_ENTRIES + 4 * LOLA_STATIC_MAX_UNITS) * 4 bytes = 832 KiB on every GPU
 * that loads the library, until the process exits.
 * Set-up: the first call on each device looks up the array's device address (a host-side query,
 * no allocation, with that device current; the look-up is serialised between host threads); make that
 * first call outside any stream capture.
 * Sharing: all states and all calls on a device use the same array and it keeps the last call's
 * contents.  Nothing in it has to start at zero (each step writes every entry before reading it),
 * but two calls that overlap on the GPU (different streams, or different states on different
 * streams) race on it: serialise them.
 * The call itself allocates nothing: no cudaMalloc, cudaFree, or allocating library routine.
 * Errors: as lola_decode_step, plus SIZE.                                                        */
#define LOLA_STATIC_MAX_UNITS 4096
#define LOLA_STATIC_MAX_LIST_ENTRIES 65536
int lola_decode_step_static(lola_state* st, const void* q, const void* k, const void* v, void* out, void* stream);

/* Same two operations for callers whose tensors live in HOST memory.  `staging_dev` is a device
 * buffer of at least lola_staging_bytes(cfg, n_tokens) bytes (256-byte aligned) that the call uses
 * for the device copies of q, k, v and out; inputs are copied in, the step runs, out is copied back
 * and the stream is synchronised before returning, so out_host is valid on return.  Pinned host
 * memory makes the copies asynchronous with respect to the host but is not required.
 * Errors: as above plus SIZE.                                                                   */
size_t lola_staging_bytes(const lola_config* cfg, int32_t n_tokens);
int lola_prefill_chunk_host(lola_state* st, const void* q_host, const void* k_host, const void* v_host,
                            int32_t n_tokens, void* out_host, void* staging_dev, size_t staging_bytes,
                            void* stream);
int lola_decode_step_host(lola_state* st, const void* q_host, const void* k_host, const void* v_host,
                          void* out_host, void* staging_dev, size_t staging_bytes, void* stream);

/* A run of `n_chunks` consecutive prefill chunks of `n_tokens` tokens each from HOST memory in one call
 * (section "Chunkwise Inference": the chunks of a prompt in order).  q_host, k_host, v_host and out_host
 * hold the chunks one after the other; chunk c is the tensor [B, n_tokens, heads, d] that
 * lola_prefill_chunk takes, at byte offset c * (bytes of that tensor).  out_host (and then q_host) may be
 * NULL: the memories are updated and no output is produced.
 * `staging_dev`: device buffer of at least 2 * lola_staging_bytes(cfg, n_tokens) bytes (256-byte
 * aligned): two sets of device copies, so that the copies in of chunk c + 1 and the copy out of chunk
 * c - 1 run beside the kernels of chunk c.  The copies run on two streams that the handle creates at
 * the first such call (host-side objects only; with them seven events); they start after the work
 * already in `stream` and `stream` waits for them at the end.  The call returns after everything is
 * complete: out_host is valid.  Host arrays should be pinned; pageable memory is correct but the copies
 * then do not overlap.  Errors: ARG, SHAPE (n_tokens outside [1, max_chunk], n_chunks < 1), ALIGN, SIZE,
 * CUDA, and those of lola_prefill_chunk (the run stops at the first failing chunk).                */
int lola_prefill_host(lola_state* st, const void* q_host, const void* k_host, const void* v_host, int32_t n_chunks,
                      int32_t n_tokens, void* out_host, void* staging_dev, size_t staging_bytes, void* stream);

/* Copies the three memories to the host arrays of `view` and synchronises `stream`.  The paper has
 * no counterpart; this is how results are inspected and checkpointed.  Returns LOLA_ERR_DEVICE if
 * the sticky status word is non-zero (the arrays are still filled).                             */
int lola_read_state(const lola_state* st, const lola_state_view* view, void* stream);

/* Replaces the three memories by the host arrays of `view` (all of H, s, sparse_count, sparse_pos,
 * sparse_k, sparse_v, window_count, window_pos, window_k, window_v, n_seen are required;
 * sparse_score and threshold are optional).  Window rows may be given in any order: row j of a unit
 * holds position window_pos[j] and is stored at ring slot position % eta.  The view must describe a
 * reachable state: all n_seen equal, window = the last min(eta, n_seen) positions, sparse_count =
 * min(lambda, n_seen - window_count) for every unit; otherwise LOLA_ERR_ARG.  Synchronises.     */
int lola_write_state(lola_state* st, const lola_state_view* view, void* stream);

/* Per-kernel device timing (no counterpart in the paper; used by the benchmark's roofline figures).
 * While enabled, every kernel launch of this handle is bracketed by a pair of CUDA events on the
 * call's stream.  lola_profile_read synchronises `stream`, writes the accumulated milliseconds and
 * launch counts per kernel kind since the last read (arrays of LOLA_N_KERNEL_KINDS) and clears them. */
enum {
  LOLA_KERNEL_ATTEND = 0,  /* Eq. 14: softmax over sparse cache + window + chunk, linear term         */
  LOLA_KERNEL_SCORE = 1,   /* Eq. 10: self-recall error of the eligible set                         */
  LOLA_KERNEL_SELECT = 2,  /* Eq. 12: top-lambda                                                    */
  LOLA_KERNEL_UPDATE = 3,  /* Eq. 13 fold, moves into the sparse cache, window roll                 */
  LOLA_KERNEL_DECODE = 4,  /* fused generation step                                                 */
  LOLA_N_KERNEL_KINDS = 8
};
int lola_profile_enable(lola_state* st, int enable);
int lola_profile_read(lola_state* st, double* ms_by_kind, int64_t* launches_by_kind, void* stream);

/* What the last lola_prefill_chunk / lola_decode_step call of this handle enqueued (no counterpart in the
 * paper).  Several kernel sets compute the same step: the TMA-fed tensor-core kernels serve bf16 layers with
 * feat_half = 64, prefill chunks of at most 64 tokens and sparse caches filled in whole 64-slot blocks; other
 * shapes run on first-generation tensor-core kernels or on shape-generic CUDA-core kernels, which are
 * several times slower.  A caller that cares reads `paths` after a call (host-side; nothing is synchronised).
 * `ctas[kind]` is the number of thread blocks launched per LOLA_KERNEL_* kind.                            */
enum {
  LOLA_PATH_ATTEND_TMA = 1u << 0,        /* Eq. 14 on the TMA-fed warp-specialised kernel                   */
  LOLA_PATH_ATTEND_MMA = 1u << 1,        /* Eq. 14 on the first-generation tensor-core kernel               */
  LOLA_PATH_ATTEND_GENERIC = 1u << 2,    /* Eq. 14 on CUDA cores                                            */
  LOLA_PATH_SCORE_TMA = 1u << 3,         /* Eq. 10 (+ Eq. 12 in the same launch) on the TMA-fed kernel      */
  LOLA_PATH_SCORE_MMA = 1u << 4,
  LOLA_PATH_SCORE_GENERIC = 1u << 5,
  LOLA_PATH_SELECT_KERNEL = 1u << 6,     /* Eq. 12 as a launch of its own                                   */
  LOLA_PATH_APPLY_TMA = 1u << 7,         /* Eq. 13 fold on tensor cores, moves, window roll                 */
  LOLA_PATH_UPDATE_GENERIC = 1u << 8,
  LOLA_PATH_DECODE_FUSED = 1u << 9,      /* the generation step as one kernel (units of up to 8 row tiles)  */
  LOLA_PATH_DECODE_FUSED_LONG = 1u << 10,/* the same for units of 9 to 16 row tiles                         */
  LOLA_PATH_H_IMAGE_REBUILD = 1u << 11   /* (never reported: every kernel reads H itself)                   */
};
typedef struct lola_call_info {
  uint32_t paths;                        /* OR of LOLA_PATH_*                                               */
  int32_t launches;                      /* kernels enqueued by the call                                    */
  int32_t ctas[LOLA_N_KERNEL_KINDS];
} lola_call_info;
int lola_last_call_info(const lola_state* st, lola_call_info* out);

/* Bits of the sticky status word (lola_state_view.status).  Every wait inside a kernel is bounded; a wait
 * that runs out, or an index outside its array, sets a bit, the kernel cleans up and returns, and every
 * later kernel of the state returns at once, so the memories stay as they were when the failure happened.
 * lola_read_state then returns LOLA_ERR_DEVICE; lola_reset_state or lola_write_state clear the word.     */
enum {
  LOLA_STATUS_LISTS = 1, LOLA_STATUS_SCORE_MMA = 2, LOLA_STATUS_ATTEND_MMA = 4, LOLA_STATUS_DECODE = 8,
  LOLA_STATUS_SCORE = 16, LOLA_STATUS_APPLY = 32, LOLA_STATUS_ATTEND = 64, LOLA_STATUS_SELFTEST = 128,
  LOLA_STATUS_PREFILL_RUN = 256
};

/* Failure-path self-test (no counterpart in the paper): enqueues one warp that waits, with the bounded wait
 * every kernel uses, for a completion that never comes; after `limit_us` microseconds (1 .. 250000) the wait
 * gives up and sets LOLA_STATUS_SELFTEST.  Nothing traps and nothing spins without limit; the context stays
 * usable.  Afterwards the state behaves as after any device-side failure (see above).  Errors: ARG, CUDA. */
int lola_selftest_wait_timeout(lola_state* st, int32_t limit_us, void* stream);

/* Number of kernel launches this handle has enqueued so far. */
int64_t lola_launch_count(const lola_state* st);

/* Tokens consumed so far per sequence. */
int64_t lola_tokens_seen(const lola_state* st);

/* For callers that restore the state buffer themselves (a device-to-device copy of a snapshot taken
 * after n_seen tokens): tells the handle how many tokens that buffer has consumed.  Every count the
 * library uses (window fill, occupied slots) follows from this number.                          */
int lola_set_tokens_seen(lola_state* st, int64_t n_seen);

/* Releases the host handle only; device buffers stay with the caller. */
int lola_destroy_state(lola_state* st);

/* Static description of an error code. */
const char* lola_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* LOLA_H_ */
