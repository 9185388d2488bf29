/*
 * poss_debug.h -- test, tracing and timing surface of the PosS library.
 *
 * Nothing here is part of a speculative round (the paper has no counterpart for any of it): the calls copy
 * intermediate state out for parity tests, time the stages of a round for roofline reports, make a bounded device
 * wait run out without a fault, and switch between kernels that compute the same stage.  A serving integration needs
 * poss.h only.
 */
#ifndef POSS_DEBUG_H
#define POSS_DEBUG_H

#include "poss.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Copies the last draft round's intermediate state out of the workspace (any pointer may be NULL):
 * cand_* [topk + (depth-1)*topk^2] every candidate in creation order (parent = flat index of the
 * parent candidate, -1 = root); frontier int32[depth-1][topk] flat candidate indices expanded at
 * steps 1..depth-1, best first; step_features float[depth][topk][H] the specialist features of the
 * rows expanded at each step (step 0 uses row 0 only); selected int32[n_nodes-1] flat indices kept
 * by the rerank, ascending. */
POSS_API int poss_draft_trace(poss_ctx* ctx, int32_t* cand_tokens, int32_t* cand_parents, float* cand_scores,
                     int32_t* frontier, float* step_features, int32_t* selected, poss_stream stream);
/* The same for sequence `seq` of the last batched draft round (poss_draft_trace is sequence 0). */
POSS_API int poss_draft_trace_seq(poss_ctx* ctx, int seq, int32_t* cand_tokens, int32_t* cand_parents,
                         float* cand_scores, int32_t* frontier, float* step_features, int32_t* selected,
                         poss_stream stream);

/* Device-time bracketing of the draft steps' stages, for roofline reporting.  mode 0: off (also switches the timeline
 * recording below off); mode 1: the LM-head
 * matrix product (the dominant kernel) of every draft step sits between two CUDA events on the launching stream;
 * mode 2: so does every stage kind below (the launches between the two events are the product's kernel, plus the
 * combine kernel for POSS_PROF_ATTENTION and the in-kernel or consumer-side SwiGLU for POSS_PROF_GATE_UP).  The
 * events cut the overlap between neighbouring launches, so mode 2 times each stage in isolation and lengthens the
 * round; at most 1024 brackets between reads.  poss_profile_read SYNCHRONISES on the last event, returns per kind
 * how many launches were bracketed since the previous read and their summed device time in ms (arrays of
 * POSS_PROF_KINDS entries), and starts over.  The target pass is never bracketed. */
enum { POSS_PROF_FC = 0, POSS_PROF_QKV = 1, POSS_PROF_ATTENTION = 2, POSS_PROF_O = 3, POSS_PROF_GATE_UP = 4,
       POSS_PROF_DOWN = 5, POSS_PROF_LM_HEAD = 6, POSS_PROF_KINDS = 7 };
POSS_API int poss_profile(poss_ctx* ctx, int mode);
POSS_API int poss_profile_read(poss_ctx* ctx, int* h_launches, float* h_total_ms);

/* Timeline of the chain of dependent launches (poss_profile mode 3).  Every launch of the library on the current
 * device -- draft steps and target pass alike -- records which kernel it is and the device time (ns, the GPU's global
 * timer) at which its wait for its predecessor returned, i.e. at which the predecessor grid had completed.  The
 * difference between two consecutive records is the earlier kernel's span INSIDE the chain, overlap with its
 * neighbours included (mode 2 cuts that overlap).  Recording adds one store per launch and leaves the chain as it is.
 * It is a property of the device, not of the context: switch it on for one context at a time; poss_profile(ctx, 0)
 * switches it off.  poss_timeline_read SYNCHRONISES the stream, copies up to `capacity` records in launch order
 * (h_kernel[i] a POSS_K_* value, h_time_ns[i]) to the host, stores their number in *h_count and starts over; at most
 * 8192 records are kept between reads.  A matrix product's id tells which product it is. */
enum { POSS_K_OTHER = 0, POSS_K_GATHER_X = 1, POSS_K_EMBED_ROWS = 2, POSS_K_RMSNORM = 3, POSS_K_REDUCE_NORM = 4,
       POSS_K_ROPE_APPEND = 5, POSS_K_ATTN_TC = 6, POSS_K_ATTN_MMA = 7, POSS_K_ATTN_COMBINE_BF16 = 8,
       POSS_K_ATTN_PARTIAL = 9, POSS_K_ATTN_COMBINE = 10, POSS_K_SPLITK_REDUCE = 11, POSS_K_SPLITK_SWIGLU = 12,
       POSS_K_SILU_MUL = 13, POSS_K_CAST = 14, POSS_K_GEMM_SIMT = 15, POSS_K_TOPK_PARTIAL = 16, POSS_K_TOPK_MERGE =
       17, POSS_K_TOPK_MERGE_EXPAND = 18, POSS_K_ARGMAX_PARTIAL = 19, POSS_K_RERANK = 20, POSS_K_ACCEPT_WALK = 21,
       POSS_K_SAMPLE_WALK = 22, POSS_K_KV_COMPACT = 23, POSS_K_CHAIN_MASK = 24, POSS_K_TILE_CONTRIB = 25,
       POSS_K_GEMM_FC = 32, POSS_K_GEMM_QKV = 33, POSS_K_GEMM_O = 34, POSS_K_GEMM_GATE_UP = 35, POSS_K_GEMM_DOWN =
       36,        POSS_K_GEMM_LM_HEAD = 37, POSS_K_GEMM_OTHER = 38, POSS_K_COUNT = 39 };
POSS_API int poss_timeline_read(poss_ctx* ctx, int capacity, int32_t* h_kernel, int64_t* h_time_ns, int* h_count,
                       poss_stream stream);

/* Failure-detection test hook (the paper has no counterpart).  The next `launches` tensor-core launches of this
 * context (matrix products and tcgen05 tree attention alike) withhold one tile from their own pipeline (a product:
 * one activation tile; attention: the value tiles), so the bounded wait on that tile runs out (after about one
 * second): every CTA stops issuing work, waits (bounded) for its copies in flight, frees its tensor memory and
 * returns; the device status word becomes POSS_E_TIMEOUT (poss_last_status) and the launch's results are undefined.
 * Nothing faults and the context stays usable: poss_reset clears the status. */
POSS_API int poss_debug_lose_load(poss_ctx* ctx, int launches);

/* Kernel choices that do not change what is computed (the paper has no counterpart).  option:
 *   POSS_OPT_ATTENTION_TCGEN05 (default 1): bf16 tree attention at head dimension 128 runs on the tcgen05 kernel;
 *     0 sends every call to the split-KV mma.sync kernels (the two group their sums differently and agree to a
 *     bf16 unit);
 *   POSS_OPT_SWIGLU_IN_KERNEL (default 0): the gate/up product is finished by the matrix product's own SwiGLU
 *     epilogue instead of the consumer kernel over parked partials (equal bit for bit wherever both cut the product
 *     into the same CTA ranges).
 * Takes effect from the next call on this context.  Errors: INVALID. */
enum { POSS_OPT_ATTENTION_TCGEN05 = 0, POSS_OPT_SWIGLU_IN_KERNEL = 1 };
POSS_API int poss_debug_option(poss_ctx* ctx, int option, int value);

/* Number of kernels this context has launched so far (host counter). */
POSS_API int64_t poss_launch_count(const poss_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* POSS_DEBUG_H */
