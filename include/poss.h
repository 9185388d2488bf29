/*
 * poss.h -- C ABI of the PosS speculative-round library (CUDA, sm_100a).
 *
 * One speculative round of PosS (position-specialist drafting, paper Sections 2-3):
 *   draft   : at draft position i the specialist ceil((i+1)/n) runs an EAGLE-style layer
 *             (fc on [token embedding ; feature] -> one Llama decoder layer with tree-masked
 *             attention over that specialist's own KV cache -> shared LM head -> top-k ->
 *             tree expansion by cumulative log-prob), Eq. 1, Eq. 2, Eq. 7, Eq. 9, Section 3.3;
 *   verify  : the target evaluates all draft tokens in one tree-masked pass and the greedy
 *             accept walk keeps the longest path that matches its own tokens (Section 2.1,
 *             Section 3.1: acceptance of position i implies acceptance of position i-1).
 *
 * Conventions
 *   - Every function returns a poss_status; nothing throws, aborts or traps.
 *   - Pointers are DEVICE pointers owned by the caller unless the name starts with h_.  Tensors (weights,
 *     caches, q, features, outputs) start on a 16-byte boundary; a misaligned one is POSS_E_INVALID where the
 *     call can see it on the host.
 *   - The library allocates no device memory: all scratch lives in the workspace the caller
 *     hands to poss_init (size from poss_workspace_bytes) and must outlive the context.
 *   - All work is enqueued on the stream argument and is asynchronous; no call synchronises
 *     unless its comment says so.  Calls on one context must not overlap on the GPU.
 *   - Weights are borrowed for the life of the context.
 *   - dtype POSS_BF16: weights, KV caches, features and q/out of poss_tree_attention are bf16;
 *     the activation operand of every matrix product is rounded to bf16, accumulation and the
 *     residual stream are fp32.  dtype POSS_FP32 (check mode): everything is fp32.
 *   - Matrices are row-major [out_features][in_features].
 *   - A device-side problem (a bounded wait that ran out) is reported through poss_last_status.
 */
#ifndef POSS_H
#define POSS_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define POSS_API __attribute__((visibility("default")))
#else
#define POSS_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  POSS_OK = 0,
  POSS_E_INVALID = 1,    /* NULL pointer, negative size, unsupported option            */
  POSS_E_SHAPE = 2,      /* model geometry the kernels do not cover                     */
  POSS_E_CAPACITY = 3,   /* request exceeds a capacity fixed at poss_init               */
  POSS_E_WORKSPACE = 4,  /* workspace too small or misaligned                           */
  POSS_E_CUDA = 5,       /* a CUDA runtime/driver call failed                           */
  POSS_E_TIMEOUT = 6     /* a bounded device-side wait ran out (see poss_last_status)   */
} poss_status;

enum { POSS_FP32 = 0, POSS_BF16 = 1 };

/* Compile-time limits of the kernels. */
enum { POSS_MAX_ROWS = 128,      /* rows of any one matrix product (pending + current, or tree rows) */
       POSS_MAX_TOPK = 16,
       POSS_MAX_DEPTH = 16,
       POSS_MAX_BATCH = 16 };    /* sequences of one batched draft round */

typedef struct poss_ctx poss_ctx;
typedef void* poss_stream;       /* a cudaStream_t */

typedef struct {
  int hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab;   /* head_dim in {32, 64, 128} */
  float rope_theta, rms_eps;
  int dtype;                     /* POSS_FP32 | POSS_BF16 */
  int n_specialists;             /* S */
  int positions_per_specialist;  /* n: draft position i is served by specialist
                                    min(ceil((i+1)/n), S)  (Eq. 7 and the n=2 example below it) */
  int max_depth, max_topk, max_total;  /* capacities for depth L, width K, kept tokens T   */
  int draft_kv_slots;            /* slots per specialist cache; a round needs
                                    prefix_len + n_new + (depth-1)*topk of them             */
  int n_target_layers;           /* 0 = drafter only */
  int target_kv_slots;           /* slots per target layer cache */
  int max_batch;                 /* sequences per poss_draft_round_batched call (0 or 1: single rounds only) */
} poss_config;

/* One decoder layer.  fc_w [H][2H]: columns [0,H) multiply the token embedding, [H,2H) the
 * feature (the paper's pair order [x ; f], Eq. 1).  fc_b, norm_in may be NULL (absent / identity).
 * Target layers leave fc_w and fc_b NULL.  Specialists may alias one another's pointers. */
typedef struct {
  const void *fc_w, *fc_b, *norm_in, *wq, *wk, *wv, *wo, *norm_post, *w_gate, *w_up, *w_down;
} poss_layer_w;

/* h_specialist / h_target are HOST arrays of S / n_target_layers structs whose members are device
 * pointers; they are copied by poss_init. embed, lm_head [V][H]; target_final_norm [H]. */
typedef struct {
  const void *embed, *lm_head, *target_final_norm;
  const poss_layer_w *h_specialist;
  const poss_layer_w *h_target;
} poss_weights;

/* Bytes of scratch the context needs (a multiple of 256); 0 if the configuration is invalid. */
POSS_API size_t poss_workspace_bytes(const poss_config* cfg);

/* Creates a context.  workspace: device memory, 256-byte aligned, at least poss_workspace_bytes.
 * Zeroes its state on `stream` and SYNCHRONISES that stream once.  Errors: INVALID, SHAPE,
 * CAPACITY (limits above), WORKSPACE, CUDA. */
POSS_API int poss_init(poss_ctx** out, const poss_config* cfg, const poss_weights* w,
              void* workspace, size_t workspace_bytes, poss_stream stream);
POSS_API int poss_destroy(poss_ctx* ctx);
/* Zeroes the acceptance counters and the device status word (asynchronous). */
POSS_API int poss_reset(poss_ctx* ctx, poss_stream stream);

/* Fills EVERY specialist's cache with the keys/values of n verified pairs [token ; feature]
 * at slots start .. start+n-1 (each specialist keeps its own cache, Section 3.3).
 * draft_kv: [S][2][n_kv_heads][draft_kv_slots][head_dim].  Any n >= 0 (processed in chunks). */
POSS_API int poss_draft_prefill(poss_ctx* ctx, void* draft_kv, int start,
                       const int32_t* tokens, const void* features /*[n][H]*/, int n, poss_stream stream);

/* One draft phase (Eq. 9 position by position; tree drafting with width/depth/total tokens,
 * Section 4.1).  Slots [0, prefix_len) of every specialist cache are valid.  new_tokens /
 * new_features are the n_new >= 1 verified pairs not yet cached; the LAST one is the root pair
 * [x_t ; f_(t-1)].  They are written to slots prefix_len .. prefix_len+n_new-1 of every
 * specialist's cache; tree nodes use the slots behind them and are garbage afterwards.
 * Outputs (node 0 = root, parent -1, score 0, depth 0; nodes in creation order, parent before
 * child): tokens, parents, depth int32[total+1]; scores float[total+1] (cumulative log-prob);
 * anc_mask uint64[total+1][ceil((total+1)/64)] (bit j of row r: j is r or an ancestor of r);
 * n_nodes int32[1] = 1 + min(total, topk + (depth-1)*topk^2).
 * Top-k and selection ties go to the lower index.  Needs n_new + (depth-1)*topk <= POSS_MAX_ROWS.
 * Errors: INVALID, CAPACITY. */
POSS_API int poss_draft_round(poss_ctx* ctx, void* draft_kv, int prefix_len,
                     const int32_t* new_tokens, const void* new_features, int n_new,
                     int depth, int topk, int total_tokens,
                     int32_t* out_tokens, int32_t* out_parents, float* out_scores,
                     int32_t* out_depth, uint64_t* out_anc_mask, int32_t* out_n_nodes,
                     poss_stream stream);

/* One draft phase for `batch` independent sequences at once (the paper measures decoding speed as throughput
 * against vanilla decoding, Section 4.1 "Metrics"; at one sequence every matrix product of a draft step streams its
 * weights for at most 64 rows, so drafting for B sequences in one pass pays each step's weights once for B trees).
 * Every sequence is drafted exactly as by poss_draft_round -- the result of sequence b equals, bit for bit, that of a
 * single-sequence call on its inputs -- and the sequences share depth, topk and total_tokens.
 * h_draft_kv: HOST array of `batch` device pointers, one cache set [S][2][n_kv_heads][draft_kv_slots][head_dim]
 * per sequence; h_prefix_len, h_n_new: HOST int[batch].  new_tokens int32[sum n_new] and new_features
 * [sum n_new][H]: the sequences' verified pairs one after the other (each sequence's last pair is its root).
 * Outputs as in poss_draft_round with a leading batch dimension: tokens, parents, depth int32[batch][total+1],
 * scores float[batch][total+1], anc_mask uint64[batch][total+1][ceil((total+1)/64)], n_nodes int32[batch].
 * The stacked rows of every step (all sequences' pending and current rows) must fit POSS_MAX_ROWS and batch must
 * not exceed the context's max_batch, else POSS_E_CAPACITY.  Errors: INVALID, CAPACITY. */
POSS_API int poss_draft_round_batched(poss_ctx* ctx, int batch, void* const* h_draft_kv, const int* h_prefix_len,
                             const int32_t* new_tokens, const void* new_features, const int* h_n_new,
                             int depth, int topk, int total_tokens,
                             int32_t* out_tokens, int32_t* out_parents, float* out_scores,
                             int32_t* out_depth, uint64_t* out_anc_mask, int32_t* out_n_nodes,
                             poss_stream stream);

/* Tree-masked attention: every draft token attends to the committed context and to its own path in the draft
 * tree only, which is what lets the target check all draft tokens in one parallel pass (Section 2.1, the
 * verification phase) and lets a draft step extend every frontier node at once (Eq. 2: a prediction conditions
 * on its own previously generated features and tokens).  Used by the target pass and by every draft step.
 * q, out [rows][n_q_heads][head_dim]; kv [2][n_kv_heads][kv_slots][head_dim] with the rows' own
 * keys/values already at slots prefix_len+r.  Row r sees slots [0, prefix_len) and slot
 * prefix_len+j for every bit j set in anc_mask[r] (uint64[rows][ceil(rows/64)]).
 * Query head h reads KV head h / (n_q_heads / n_kv_heads).  rows <= POSS_MAX_ROWS.
 * q, kv and out 16-byte aligned (else POSS_E_INVALID). */
POSS_API int poss_tree_attention(poss_ctx* ctx, const void* q, const void* kv, int kv_slots, int prefix_len,
                        int rows, const uint64_t* anc_mask, float scale, void* out, poss_stream stream);

/* Greedy verification (Section 2.1; A_i subset of A_(i-1), Section 3.1).  Give target_logits
 * ([rows][V], context dtype) or target_argmax (int32[rows]); the other is NULL.  Walks from the
 * root to the child whose token equals the target's greedy token while one exists.
 * out_path int32[POSS_MAX_DEPTH+1] (node indices, root first), out_n_accepted int32[1] = a,
 * out_bonus_token int32[1] = target token after the last accepted node, out_new_tokens
 * int32[a+1] and out_new_features [(a+1)][H] = the verified pairs for the next draft round
 * ([token of path[k+1] ; target feature of path[k]], last = [bonus ; feature of path[a]]).
 * Updates the acceptance counters. */
POSS_API int poss_verify_accept(poss_ctx* ctx, const void* target_logits, const int32_t* target_argmax,
                       const void* target_features /*[rows][H]*/, const int32_t* tokens,
                       const int32_t* parents, int rows,
                       int32_t* out_path, int32_t* out_n_accepted, int32_t* out_bonus_token,
                       int32_t* out_new_tokens, void* out_new_features, poss_stream stream);

/* Verification at a temperature > 0 (the rejection-sampling phase of Section 2.1; the paper's second setting,
 * Section 5, temperature 1).  The tree's candidates are deterministic (top-k), i.e. point masses, so the rule is:
 * at the current node p = softmax(target_logits[node] / temperature); the node's children are tested in node
 * order, child x is accepted iff the next uniform u satisfies u < p(x); on rejection p(x) is removed, p is
 * renormalised and the next child is tested; when no child is left the bonus token is drawn from the current p by
 * inverse CDF in token order (first token whose cumulative probability exceeds u).  The emitted tokens are then
 * distributed exactly as the target's own sampling.  target_logits float[rows][V] (device); uniforms
 * float[n_uniforms] in [0, 1) (device), consumed in order: one per tested child, one for the bonus, at most `rows`
 * in all (n_uniforms < rows -> POSS_E_CAPACITY); out_uniforms_used int32[1].  The other outputs are those of
 * poss_verify_accept, and the acceptance counters are updated in the same way. */
POSS_API int poss_verify_sample(poss_ctx* ctx, const float* target_logits, const void* target_features /*[rows][H]*/,
                       const int32_t* tokens, const int32_t* parents, int rows, float temperature,
                       const float* uniforms, int n_uniforms,
                       int32_t* out_path, int32_t* out_n_accepted, int32_t* out_bonus_token,
                       int32_t* out_new_tokens, void* out_new_features, int32_t* out_uniforms_used,
                       poss_stream stream);

/* The verification phase's forward pass (Section 2.1: the target evaluates all draft tokens in parallel in a
 * single forward pass; Section 3.1 uses its per-position greedy tokens to decide acceptance).
 * Target model over `rows` tree rows: row r holds tokens[r], sits at rotary position
 * prefix_len + depth[r], is written to cache slot prefix_len + r and sees the prefix plus its
 * ancestors and itself (anc_mask as above).  A chain (depth r, lower-triangular mask) is plain
 * causal decoding / prefill.  target_kv [layers][2][n_kv_heads][target_kv_slots][head_dim].
 * out_features [rows][H] (after the final norm), out_argmax int32[rows] (ties -> lowest id);
 * out_logits float[rows][V] optional (NULL = never materialised for the caller). */
POSS_API int poss_target_forward(poss_ctx* ctx, void* target_kv, int prefix_len, const int32_t* tokens,
                        const int32_t* depth, const uint64_t* anc_mask, int rows,
                        void* out_features, int32_t* out_argmax, float* out_logits, poss_stream stream);
/* The same pass under the name of its role in a round: tree verification without the logits
 * (poss_target_forward with out_logits = NULL). */
POSS_API int poss_target_verify(poss_ctx* ctx, void* target_kv, int prefix_len, const int32_t* tokens,
                       const int32_t* depth, const uint64_t* anc_mask, int rows,
                       void* out_features, int32_t* out_argmax, poss_stream stream);

/* The target's pass over the prompt, which leaves the features f_j and the cache the first round starts from
 * (Section 2.1: the draft model conditions on the target's features of the committed tokens, Eq. 1).
 * Causal prefill of n prompt tokens from position `start` (chunks of POSS_MAX_ROWS rows).
 * out_features [n][H], out_argmax int32[n] (may be NULL). */
POSS_API int poss_target_prefill(poss_ctx* ctx, void* target_kv, int start, const int32_t* tokens, int n,
                        void* out_features, int32_t* out_argmax, poss_stream stream);

/* Commit of a round (Section 2.1: accepted tokens join the context of the next round; Section 3.3: the caches
 * hold previously verified tokens): the accepted path's cache entries become contiguous behind the prefix.
 * After acceptance: in every target layer move tree slot prefix_len + path[k] to prefix_len + k
 * for k = 1..*n_accepted (path and n_accepted are the device outputs of poss_verify_accept). */
POSS_API int poss_kv_compact(poss_ctx* ctx, void* target_kv, int prefix_len, const int32_t* path,
                    const int32_t* n_accepted, poss_stream stream);

/* Host copies of the counters: rounds R and N_i = rounds that accepted position i
 * (h_accepted_at[0] unused, [1..max_depth]); pos-acc_i = N_i / N_(i-1) (Eq. 3), N_0 = R.
 * SYNCHRONISES the stream. */
POSS_API int poss_get_counters(poss_ctx* ctx, int64_t* h_rounds, int64_t* h_accepted_at, poss_stream stream);

/* Device status word (POSS_OK or POSS_E_TIMEOUT); SYNCHRONISES the stream. */
POSS_API int poss_last_status(poss_ctx* ctx, poss_stream stream);

/* ---- single stages, exported for kernel-level parity tests and roofline timing ---- */

/* out[M][N] (fp32) = x[M][K] . w[N][K]^T (+ bias[N]) (+ residual[M][N], fp32).  x, w, bias in the
 * context dtype.  M <= POSS_MAX_ROWS, K % 8 == 0.  impl: 0 = default for the dtype, 1 = SIMT kernel,
 * 2 = tcgen05 tensor-core kernel (bf16 only; w 16-byte aligned) followed, as inside a round, by the kernel that
 * adds its split-K partials.  A row's result does not depend on M or on the row's place in the batch. */
POSS_API int poss_linear(poss_ctx* ctx, const void* x, int M, const void* w, int N, int K,
                const void* bias, const float* residual, float* out, int impl, poss_stream stream);

/* Shared LM head + log-softmax + top-k over the vocabulary for `rows` feature rows (context
 * dtype): out_ids int32[rows][topk] best first (ties -> lowest id), out_logp float[rows][topk].
 * out_logits float[rows][V] optional debug output (NULL in production). */
POSS_API int poss_lm_head_topk(poss_ctx* ctx, const void* features, int rows, int topk,
                      int32_t* out_ids, float* out_logp, float* out_logits, poss_stream stream);

/* Tree-masked attention for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a packaging variant of poss_tree_attention).
 * Who needs it: code that is handed device pointers but may not call cudaMalloc -- an engine whose
 * memory pools were sized once at start-up, a latency-critical stream where an allocation would
 * force a device-wide synchronisation, a plugin without access to the host application's allocator.
 * Such callers cannot create the workspace a poss_ctx needs, so this entry takes no context: the
 * geometry comes as arguments and the split-KV partial results go to a fixed 8 MiB array inside the
 * library image (resident on every GPU that loads the library until the process exits).
 * Same semantics and layouts as poss_tree_attention; dtype is POSS_FP32 or POSS_BF16.
 * Limit: rows * n_q_heads * (head_dim + 2) floats must fit the 8 MiB array (2,097,152 floats),
 * otherwise POSS_E_CAPACITY; with less room the key range is split fewer ways (never wrongly).
 * The call allocates nothing and calls no allocating routine.  Its first call on a device looks up
 * the array's device address (once per device, that device current); make that first call outside
 * any stream capture.  All calls share the one array and it keeps the previous call's contents:
 * nothing in it has to start at zero (every value read was written by the same call), but two calls
 * that overlap on the GPU -- different streams, no ordering -- race on it.  Serialise them. */
POSS_API int poss_tree_attention_noalloc(const void* q, const void* kv, int kv_slots, int prefix_len,
                                         int rows, int n_q_heads, int n_kv_heads, int head_dim, int dtype,
                                         const uint64_t* anc_mask, float scale, void* out, poss_stream stream);

/* Host-only query (no device is touched): how poss_tree_attention and the draft / target passes cut `total_keys`
 * visible-or-masked keys for a bf16 model with head dimension 128.  The tcgen05 kernel takes up to 10240 keys:
 * groups of 128 keys at absolute positions (group j always holds keys [128 j, 128 j + 128)), two consecutive groups
 * per unit, one partial result per unit, all units merged in key order in one pass.  *keys_per_unit = 128 (one group,
 * at most 128 keys in all) or 256, *n_units = units that hold keys; the cut depends on total_keys alone, never on the
 * rows, the heads or the number of CTAs that share the units.  Returns POSS_OK, or POSS_E_SHAPE for a key count the
 * kernel does not take (the split-KV kernels then run; outputs untouched), POSS_E_INVALID for NULL outputs or
 * total_keys < 1.  The paper has no counterpart. */
POSS_API int poss_attention_plan(int total_keys, int* keys_per_unit, int* n_units);

#ifdef __cplusplus
}
#endif
#endif /* POSS_H */
