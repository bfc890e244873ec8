/*
 * nezha.h -- C ABI of the B200 (sm_100a) speculative semantic-ID decode library.
 *
 * One context serves one (model weights, item catalogue) pair on one GPU.  Call order:
 *
 *     nezha_create -> nezha_build_hashset -> nezha_prefill -> nezha_decode (any number of times)
 *
 * Out-of-order calls return NEZHA_ERR_STATE.  Decoding leaves the prompt KV cache untouched, so the same
 * prefilled batch can be decoded repeatedly (in any mode).
 *
 * Conventions
 *   - "device" pointers are CUDA device memory of the GPU that was current at nezha_create; "host" pointers
 *     are ordinary host memory.  The caller owns every buffer it passes in.  The library allocates NO device
 *     memory: everything it needs lives in the caller-provided arena (nezha_arena_bytes tells its size).
 *     Weights are re-laid-out into the arena during nezha_create; the caller's weight buffers are not read
 *     after nezha_create returns.
 *   - All work is enqueued on the CUDA stream given to nezha_create (a cudaStream_t passed as void*; NULL is
 *     the legacy default stream).  Functions that return data to the host synchronise that stream.
 *   - Matrices are row-major [out_features, in_features].  dtype 0: fp32 storage and arithmetic.  dtype 1:
 *     bf16 storage (weights, activations, KV cache), fp32 accumulation, fp32 residual stream, logits and scores.
 *   - Semantic IDs: L codes, level l (1-based) in [0, T[l-1]).  Token ids of the backbone vocabulary:
 *     code c of level l -> sum_{j<l} T[j] + c; placeholder SP_l -> sum(T) + l - 1; BOS -> sum(T) + L;
 *     vocabulary size sum(T) + L + 1.
 *   - Errors: every function returns a nezha_status and never aborts; nezha_last_error gives a message.
 *     Device-side conditions (hash table full, an out-of-range code) are recorded in a device status word
 *     and reported by the next synchronising call.
 */
#ifndef NEZHA_H_
#define NEZHA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define NEZHA_MAX_LEVELS 8

typedef struct nezha_ctx nezha_ctx;

typedef enum {
  NEZHA_OK = 0,
  NEZHA_ERR_ARG = 1,             /* null pointer, size out of the configured range, unsupported shape      */
  NEZHA_ERR_STATE = 2,           /* call order violated                                                     */
  NEZHA_ERR_ARENA_TOO_SMALL = 3,
  NEZHA_ERR_CUDA = 4,            /* a CUDA runtime call failed; message in nezha_last_error                 */
  NEZHA_ERR_HASH_FULL = 5,       /* an insertion exhausted its probe bound                                  */
  NEZHA_ERR_CATALOG = 6,         /* a catalogue or history code outside [0, T_l)                            */
  NEZHA_ERR_UNSUPPORTED = 7
} nezha_status;

typedef struct {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, d_ffn;
  int32_t L;                     /* codes per semantic ID, 1..NEZHA_MAX_LEVELS                              */
  int32_t T[NEZHA_MAX_LEVELS];   /* codebook size per level; prod(T) must be < 2^64 - 1                     */
  int32_t dtype;                 /* 0 = fp32, 1 = bf16                                                      */
  float rope_theta, rms_eps;
  int32_t max_batch, max_beam, max_hist_items;   /* capacity the arena is sized for                         */
} nezha_config;

/* DEVICE pointers; element type given by nezha_config.dtype.  Per-layer arrays are HOST arrays of n_layers
 * device pointers.  head_dim = d_model / n_q_heads. */
typedef struct {
  const void* embed;             /* [vocab, d]                                                              */
  const void* lm_head;           /* [vocab, d]  (untied)                                                    */
  const void* final_norm;        /* [d]                                                                     */
  const void* const* attn_norm;  /* n_layers x [d]                                                          */
  const void* const* wq;         /* n_layers x [n_q_heads*hd, d]                                            */
  const void* const* wk;         /* n_layers x [n_kv_heads*hd, d]                                           */
  const void* const* wv;         /* n_layers x [n_kv_heads*hd, d]                                           */
  const void* const* wo;         /* n_layers x [d, n_q_heads*hd]                                            */
  const void* const* mlp_norm;   /* n_layers x [d]                                                          */
  const void* const* w_gate;     /* n_layers x [d_ffn, d]                                                   */
  const void* const* w_up;       /* n_layers x [d_ffn, d]                                                   */
  const void* const* w_down;     /* n_layers x [d, d_ffn]                                                   */
  const void* const* draft_logit;/* L x [T_l, d]            logit_head_l of Eq. 2                           */
  const void* draft_ws;          /* [d, d]                  Transition of Eq. 3: tanh(Ws s + We e + b)      */
  const void* draft_we;          /* [d, d]                                                                  */
  const void* draft_b;           /* [d]                                                                     */
} nezha_weights;

/* Host-side summary of one nezha_decode call. */
typedef struct {
  int32_t rounds;                /* draft/verify rounds executed (Algorithm 2's while loop); 0 in mode 0     */
  int64_t primary_tokens;        /* code tokens the primary model processed over all rounds                 */
  int64_t drafted;               /* draft tuples produced in round 1, summed over rows                      */
  int64_t accepted_levels;       /* sum over rows, rounds and draft tuples of newly accepted levels          */
} nezha_decode_stats;

/* Optional per-round device outputs of nezha_decode (any pointer may be NULL).  R = L - 1 round slots;
 * slots of rounds that did not run are filled with -1. */
typedef struct {
  int32_t* drafts;               /* device [R, batch, beam, L]  drafted tuples of the round (the draft tree's  */
                                 /*                             level-L nodes, distinct), -1 padded           */
  int32_t* n_draft;              /* device [R, batch]                                                       */
  int32_t* accepted_len;         /* device [R, batch, beam]     largest i with D[k][1..i] in B_i            */
  int32_t* level_reached;        /* device [R, batch]           level m the row had settled after the round */
  int32_t* beams;                /* device [L, batch, beam, L]  the true beam sets B_1..B_L, -1 padded      */
  float*   beam_scores;          /* device [L, batch, beam]                                                 */
  int32_t* tree_codes;           /* device [R, L, batch, beam, L]  the round's draft tree: nodes of level j  */
                                 /*                             (j codes each) at index j - 1, -1 padded      */
  int32_t* tree_count;           /* device [R, L, batch]        nodes per level (-1: the row took no part)  */
} nezha_trace;

/* Decode modes. */
#define NEZHA_MODE_DRAFT 0       /* Algorithm 3 as printed: draft-head beam search + hash-set filter         */
#define NEZHA_MODE_VERIFIED 1    /* Algorithm 2 with Algorithm 3's drafts: primary pass, accept / roll back  */
#define NEZHA_MODE_AR 2          /* Algorithm 1: plain autoregressive beam search, same validity filter      */

/* Bytes of device arena a context with this configuration and catalogue size needs (0 on a bad argument).
 * load_factor in (0, 1): the hash set gets ceil(n_items / load_factor) slots (rounded up to its bucket size). */
size_t nezha_arena_bytes(const nezha_config* cfg, size_t n_items, double load_factor);

/* Create a context.  Inputs of Algorithm 3 (inference): the model with its draft head, and the set V of valid
 * semantic IDs given as catalogue code tuples.
 *   weights        device pointers as described above; copied/re-laid-out into the arena before returning.
 *   catalog_codes  device int32 [n_items, L]; borrowed until nezha_build_hashset has returned.
 *   arena          device, 256-byte aligned, at least nezha_arena_bytes(cfg, n_items, load_factor) bytes;
 *                  borrowed until nezha_destroy.
 *   cuda_stream    cudaStream_t (as void*), borrowed until nezha_destroy.
 * Synchronises the stream.  Errors: NEZHA_ERR_ARG, NEZHA_ERR_UNSUPPORTED (shape the kernels do not cover),
 * NEZHA_ERR_ARENA_TOO_SMALL, NEZHA_ERR_CUDA. */
nezha_status nezha_create(const nezha_config* cfg, const nezha_weights* weights,
                          const int32_t* catalog_codes, size_t n_items, double load_factor,
                          void* arena, size_t arena_bytes, void* cuda_stream, nezha_ctx** out);

/* Eq. 4 + Eq. 5: pack every catalogue tuple into a 64-bit key (level 1 least significant) and insert it
 * into the open-addressing hash set.  Duplicated tuples are legal and counted once.
 *   n_unique  host out (may be NULL): number of distinct keys inserted.
 * Synchronises.  Errors: NEZHA_ERR_CATALOG (code out of range), NEZHA_ERR_HASH_FULL. */
nezha_status nezha_build_hashset(nezha_ctx* ctx, uint64_t* n_unique);

/* Eq. 4: pack code tuples (device int32 [n, L]) into keys (device uint64 [n]).  Asynchronous. */
nezha_status nezha_pack(nezha_ctx* ctx, const int32_t* codes, size_t n, uint64_t* keys);

/* Eq. 5: membership of packed keys (device uint64 [n]) in V; found[i] = 1 or 0 (device uint8 [n]).
 * Asynchronous. */
nezha_status nezha_probe(nezha_ctx* ctx, const uint64_t* keys, size_t n, uint8_t* found);

/* Prefill step of Algorithm 3 (inference): one pass of the primary model over [BOS, history codes, SP_1..SP_L] of every row.
 * Keeps the context KV cache (placeholders are not retained) and the hidden states h_0..h_L.
 *   hist_codes  device int32 [batch, max_n, L]; row b uses its first n_hist[b] items.
 *   n_hist      device int32 [batch], each in [0, max_n]; max_n <= cfg.max_hist_items.
 * Asynchronous.  A code out of range sets NEZHA_ERR_CATALOG, reported by the next synchronising call. */
nezha_status nezha_prefill(nezha_ctx* ctx, const int32_t* hist_codes, const int32_t* n_hist,
                           int32_t batch, int32_t max_n);

/* Decode the next item of every prefilled row: the top `beam_width` valid semantic IDs and their
 * cumulative log-probabilities (Algorithm 3's inference loop in mode 0; Algorithm 2 in mode 1; Algorithm 1 in mode 2).
 *   out_codes   device int32 [batch, beam_width, L], best first, rows past out_count padded with -1
 *   out_scores  device float [batch, beam_width], padded with -inf
 *   out_count   device int32 [batch]
 *   stats       host out, may be NULL
 *   trace       optional per-round device outputs, may be NULL
 * batch must equal the prefilled batch; 1 <= beam_width <= cfg.max_beam.  Synchronises (modes 1 and 2 read a
 * "rows unfinished" counter once per round). */
nezha_status nezha_decode(nezha_ctx* ctx, int32_t batch, int32_t beam_width, int32_t mode,
                          int32_t* out_codes, float* out_scores, int32_t* out_count,
                          nezha_decode_stats* stats, const nezha_trace* trace);

/* Mode 1 with the first round's drafts supplied by the caller instead of the draft head.
 *   drafts   device int32 [batch, beam_width, L];  n_draft device int32 [batch] (tuples used per row).
 * The draft tree of the round is the prefix tree of the tuples: tuples that share their first j codes share one node of
 * level j (one primary-model token); repeated tuples count once, and accepted_len / drafts of the trace index the distinct
 * tuples in order of first appearance.  A tuple with a code outside [0, T_l) is dropped (NEZHA_ERR_CATALOG). */
nezha_status nezha_decode_with_drafts(nezha_ctx* ctx, int32_t batch, int32_t beam_width,
                                      const int32_t* drafts, const int32_t* n_draft,
                                      int32_t* out_codes, float* out_scores, int32_t* out_count,
                                      nezha_decode_stats* stats, const nezha_trace* trace);

/* Mode 1 with the first round's whole draft tree supplied by the caller (Algorithm 2's drafting step replaced; what the
 * draft head itself proposes is such a tree: the beam sets of every level of Algorithm 3).
 *   tree_codes  device int32 [L, batch, beam_width, L]: at index j - 1 the nodes of level j, j codes each (the rest ignored)
 *   tree_count  device int32 [L, batch]: nodes per level and row, each <= beam_width
 * A node whose first j - 1 codes are no node of level j - 1 is dead (never verified).  The layout is that of
 * nezha_trace.beams, so the true beam sets of an earlier call can be passed back as a perfect draft. */
nezha_status nezha_decode_with_draft_tree(nezha_ctx* ctx, int32_t batch, int32_t beam_width,
                                          const int32_t* tree_codes, const int32_t* tree_count,
                                          int32_t* out_codes, float* out_scores, int32_t* out_count,
                                          nezha_decode_stats* stats, const nezha_trace* trace);

/* Variants of the draft head: the ablations of Section 4.3 ("Ablation Study").  Defaults give Eq. 1-3 and Eq. 5 as
 * printed.  Takes effect from the next nezha_decode / nezha_draft_logits call; never touches the primary model, so
 * modes 1 and 2 still return Algorithm 1's result.
 *   NEZHA_OPT_DRAFT_TRANSITION  0: s_{l+1} = tanh(W_s s_l + W_e e_l + b) (Eq. 3)    1: s_{l+1} = s_l + e_l   (NEZHA-3)
 *   NEZHA_OPT_DRAFT_INPUTS      0: logits from h_l + s_l (Eq. 2)   1: from h_l alone, no context state (NEZHA-1)
 *                               2: from s_l alone (NEZHA-2)
 *   NEZHA_OPT_DRAFT_FILTER      1: hash-set filter at the last level (Eq. 5)        0: no filter              (NEZHA-4)
 *   NEZHA_OPT_FINAL_MASK        how the primary model's beam search (modes 1 and 2) answers the validity mask of the last
 *                               level, where every one of the T_L extensions of every beam is tested (Eq. 5):
 *                               0: one hash-set probe per candidate code
 *                               1 (default): it looks the beam's prefix up in a second table, (first L-1 codes) -> bit
 *                                  set of the valid last codes, built by nezha_build_hashset from the same catalogue: one
 *                                  look-up per beam instead of T_L probes, the same answers bit for bit (the set V of
 *                                  Eq. 5 regrouped by prefix; the paper itself only describes the hash set)
 *                               The draft head's K chosen codes per beam (Algorithm 3) are always probed in the hash set.
 *   NEZHA_OPT_LEVEL_FILTER      0 (default): the validity filter acts at the last level only, as Algorithm 3 prints it
 *                               1: at every level (the per-step variant Section 3.4 mentions): a partial ID survives only
 *                                  if some valid ID begins with it -- in the draft head's search (after its per-beam top-K,
 *                                  unless NEZHA_OPT_DRAFT_FILTER is 0) and in the primary model's beam search of modes 1 and 2
 *                                  (before the top-K).  Answered by the same table as NEZHA_OPT_FINAL_MASK 1, which holds the
 *                                  prefixes of every length.  Modes 1 and 2 still agree item for item.
 *   NEZHA_OPT_ADAPTIVE_DRAFT    0 (default): mode 1 drafts in every round, as Algorithm 2 prints it
 *                               1: a request whose round settled only the one level that the verification pass settles
 *                                  anyway -- its drafts gained nothing -- stops drafting and finishes with plain
 *                                  autoregressive steps (an engine policy; the paper has no counterpart).  The result does
 *                                  not change; rounds, primary_tokens and the trace do.
 * Errors: NEZHA_ERR_ARG (unknown option or value). */
#define NEZHA_OPT_DRAFT_TRANSITION 0
#define NEZHA_OPT_DRAFT_INPUTS 1
#define NEZHA_OPT_DRAFT_FILTER 2
#define NEZHA_OPT_FINAL_MASK 3
#define NEZHA_OPT_LEVEL_FILTER 4
#define NEZHA_OPT_ADAPTIVE_DRAFT 5
nezha_status nezha_set_option(nezha_ctx* ctx, int32_t option, int32_t value);

/* ---- stage-wise entry points (the same kernels as nezha_decode, one step at a time) ------------------- */

/* h_0..h_L of the prefilled rows as fp32: device float [batch, L+1, d].  Asynchronous. */
nezha_status nezha_get_hidden(nezha_ctx* ctx, float* out);

/* Algorithm 1's model call and LM head, teacher-forced: for every (row, beam) the primary model runs on the context plus the
 * beam's `level` codes (0 <= level < L) and the LM head of level+1 gives logits.
 *   prefixes  device int32 [batch, n_beams, level] (ignored when level == 0)
 *   logits    device float [batch, n_beams, T[level]]
 * n_beams <= cfg.max_beam.  Asynchronous. */
nezha_status nezha_primary_logits(nezha_ctx* ctx, int32_t batch, int32_t n_beams, int32_t level,
                                  const int32_t* prefixes, float* logits);

/* Eq. 1-3, teacher-forced: the draft head's logits for level+1 after the given codes.
 * Same argument layout as nezha_primary_logits. */
nezha_status nezha_draft_logits(nezha_ctx* ctx, int32_t batch, int32_t n_beams, int32_t level,
                                const int32_t* prefixes, float* logits);

/* One beam-search level (the top-K, union and pruning steps of Algorithm 1 / Algorithm 3) on caller-supplied logits:
 * log-softmax over the codebook, per-beam top `per_beam` codes, optional validity filter of the resulting tuples (at
 * level + 1 == L: Eq. 5 in the hash set; at an earlier level: "some valid ID begins with it", from the prefix map), top
 * beam_width by cumulative log-probability; ties go to the smaller (parent rank, code).
 *   logits [batch, n_beams, T[level]] float, beam_scores [batch, n_beams] float,
 *   beam_codes [batch, n_beams, level] int32, n_live [batch] int32 (beams in use per row)      -- device
 *   out_parent, out_code [batch, beam_width] int32 (-1 padded), out_score [batch, beam_width] float (-inf
 *   padded), out_count [batch] int32                                                           -- device
 *   per_beam: codes kept per beam before filtering (clamped to T[level]); filter: 0/1.
 * Asynchronous. */
nezha_status nezha_select(nezha_ctx* ctx, int32_t batch, int32_t n_beams, int32_t beam_width, int32_t level,
                          int32_t per_beam, int32_t filter,
                          const float* logits, const float* beam_scores, const int32_t* beam_codes,
                          const int32_t* n_live,
                          int32_t* out_parent, int32_t* out_code, float* out_score, int32_t* out_count);

/* The projection GEMM by itself: C[M,N] (op)= A[M,K] * W[N,K]^T with fp32 accumulation, operands in the context's
 * storage type (device pointers, row-major, leading dimensions = K for A and W, N for C).
 *   epilogue 0: C (storage type) = acc;  1: C (float) = acc;  2: C (float) += acc;  3: C (float) = tanh(acc + bias[n])
 *   path     0: the engine's own choice; 1: CUDA-core kernel; 2: tcgen05 kernel (NEZHA_ERR_UNSUPPORTED if the shape
 *               is not covered: bf16 storage, K % 64 == 0, N % 32 == 0); 3: the tcgen05 kernel as the decode calls use
 *               it: for N <= 1024 the K range is accumulated in two interleaved partial sums (two MMA issuers), which
 *               rounds differently from path 2 in the last bits; 4: the weight-streaming tcgen05 kernel that the
 *               decode calls of an engine with at most 128 rows per pass use (M <= 128; W is the 128-row MMA operand,
 *               the K range is split over CTAs and the parts are added in a fixed order that depends on N, K and
 *               the device only; W must not be written by work still in flight on the stream)
 * Used by every projection of the primary model (Algorithm 1's model call), the LM head and the draft head
 * (Eq. 2-3).  Asynchronous. */
nezha_status nezha_gemm(nezha_ctx* ctx, const void* A, const void* W, void* C, int32_t M, int32_t N, int32_t K,
                        int32_t epilogue, const float* bias, int32_t path);

/* ---- for callers that cannot allocate device memory (the paper has no counterpart) ------------------------ */

/* Largest n nezha_contains_noalloc accepts.  The library image carries a key buffer of this many 8-byte entries
 * (8 MiB), which every GPU that loads the library holds until the process exits. */
#define NEZHA_NOALLOC_MAX_TUPLES (1u << 20)

/* Eq. 4 + Eq. 5 in one call without any allocation: found[i] = 1 if the code tuple codes[i, :] is a valid
 * semantic ID, else 0.  Same result as nezha_pack followed by nezha_probe, but the packed keys in between are kept
 * in a fixed buffer inside the library instead of a buffer somebody has to allocate.
 *
 * It exists for callers that must not, or cannot, call cudaMalloc (directly or through an allocating framework)
 * at the point where they need the answer: a serving loop that handed all device memory to its own pool at
 * start-up, a host thread inside a latency-critical section where cudaMalloc's implicit device synchronisation is
 * not acceptable, a plug-in that was given buffers but no allocator.  The call itself performs no cudaMalloc,
 * cudaFree or other allocating routine; the caller still provides the input and the output.
 *
 *   codes  device int32 [n, L]      found  device uint8 [n]      n <= NEZHA_NOALLOC_MAX_TUPLES
 *
 * Asynchronous on the context's stream.  Errors: NEZHA_ERR_ARG (null pointer; n above the maximum, with a message
 * saying so; another GPU than the context's is the current device), NEZHA_ERR_STATE (before nezha_build_hashset), NEZHA_ERR_CUDA.  A code outside [0, T_l) sets
 * NEZHA_ERR_CATALOG, reported by the next synchronising call; that tuple reads as not found.
 *
 * The first call on a device looks up the device address of the built-in buffer (the GPU of the context must be
 * the current device); make that first call before starting any stream capture.  The buffer is one per device and
 * shared by all contexts and streams: it keeps the previous call's keys (each call overwrites the entries it then
 * reads, nothing has to be cleared), and two calls whose kernels can overlap on the GPU -- different streams,
 * different contexts, different host threads -- race on it.  Serialise them. */
nezha_status nezha_contains_noalloc(nezha_ctx* ctx, const int32_t* codes, size_t n, uint8_t* found);

/* ---- instrumentation (the paper has no counterpart: these only measure the library itself) -------------- */

#define NEZHA_PROFILE_CLASSES 16
/* Kernel classes, in index order: gemm, attention, select, norm, rope_append, embed, swiglu, draft_glue, nodes,
 * accept, hash, misc. */
typedef struct {
  int64_t launches[NEZHA_PROFILE_CLASSES];   /* kernels launched per class since the last read                 */
  double  ms[NEZHA_PROFILE_CLASSES];         /* summed CUDA-event time per class (0 unless timing was enabled) */
} nezha_profile;

/* Total kernels this library has launched in the process (all contexts).  Never fails. */
uint64_t nezha_launch_count(void);

/* Turn per-launch CUDA-event timing on (1) or off (0).  Timing adds two event records per launch, so measure
 * throughput with it off.  Synchronises. */
nezha_status nezha_profile_enable(nezha_ctx* ctx, int32_t on);

/* Synchronise, copy out and reset the per-class launch counts and event times (host struct). */
nezha_status nezha_profile_read(nezha_ctx* ctx, nezha_profile* out);

/* Wait for the context's stream and report any pending device-side error. */
nezha_status nezha_sync(nezha_ctx* ctx);

/* Message of the last error of this context ("" if none).  Valid until the next call on the context. */
const char* nezha_last_error(const nezha_ctx* ctx);

/* Release the context (host memory only; the arena stays the caller's). */
void nezha_destroy(nezha_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* NEZHA_H_ */
