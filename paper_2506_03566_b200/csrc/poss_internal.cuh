// Internal declarations shared by the kernels and the host orchestration of the PosS library.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/poss.h"

typedef __nv_bfloat16 bf16;

// ------------------------------------------------------------------ scalar conversions
template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<bf16>(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

// ------------------------------------------------------------------ row bookkeeping of one draft step
// Rows of a step's projection batch, in order: n_ver verified pairs, then n_lvl pending rows of the
// earlier tree levels 1.. (width K each), then the current level's K rows (cur_level >= 1).  At
// cur_level == 0 the current row is the last verified pair.
struct StepRows {
  int n_ver, n_lvl, cur_level, K, n_new, prefix_len, M, Mc;
};

struct RowInfo {
  int level;  // 0 = verified pair
  int j;      // index among verified pairs, or node index inside its level
};

__host__ __device__ __forceinline__ RowInfo row_info(const StepRows& s, int m) {
  RowInfo r;
  if (m < s.n_ver) { r.level = 0; r.j = m; return r; }
  int mm = m - s.n_ver;
  if (mm < s.n_lvl) { r.level = 1 + mm / s.K; r.j = mm % s.K; return r; }
  r.level = s.cur_level; r.j = mm - s.n_lvl; return r;
}
// KV slot / rotary position of a row (verified pair j: prefix_len + j; node (level,j): behind them).
__host__ __device__ __forceinline__ int row_slot(const StepRows& s, RowInfo r) {
  return r.level == 0 ? s.prefix_len + r.j : s.prefix_len + s.n_new + (r.level - 1) * s.K + r.j;
}
__host__ __device__ __forceinline__ int row_pos(const StepRows& s, RowInfo r) {
  return r.level == 0 ? s.prefix_len + r.j : s.prefix_len + s.n_new - 1 + r.level;
}

// ------------------------------------------------------------------ GEMM segments (one launch, up to 3 weights)
struct GemmSegs {
  const void* w[3];
  int rows[3];
  int n;  // number of segments
};

// ------------------------------------------------------------------ device tree state (in the workspace)
struct TreeState {
  int32_t* cand_tok;      // [NCmax]
  int32_t* cand_parent;   // [NCmax] flat index of the parent candidate, -1 = root
  float* cand_score;      // [NCmax]
  int32_t* node_tok;      // [Lmax][Kmax]   level l >= 1
  int32_t* node_prow;     // [Lmax][Kmax]   row of the parent inside level l-1
  int32_t* node_cand;     // [Lmax][Kmax]   flat candidate index (level 0: -1)
  float* node_score;      // [Lmax][Kmax]
  uint64_t* node_mask;    // [Lmax][Kmax][2] bits over tree slots (level-1)*K + j
  int32_t* selected;      // [Tmax]
};

// ------------------------------------------------------------------ kernel launchers (defined in the .cu files)
struct Launcher {
  cudaStream_t stream;
  int64_t* launches;
  int err;  // sticky poss_status
};

template <typename T>
void launch_gemm_simt(Launcher& L, const T* X, int ldx, int M, const GemmSegs& segs, int K, const T* bias,
                      const float* residual, int ldr, float* out, int ldo);

template <typename T>
void launch_gather_x(Launcher& L, StepRows s, const int32_t* new_tokens, const T* new_features,
                     const TreeState& ts, int Kmax, const T* fb, const T* embed, int H, T* X);
template <typename T>
void launch_embed_rows(Launcher& L, const int32_t* tokens, int rows, const T* embed, int H, float* out);
template <typename T>
void launch_rmsnorm(Launcher& L, const float* x, int rows, int H, const T* gain, float eps, T* out);
template <typename T>
void launch_cast_rows(Launcher& L, const float* x, size_t n, T* out);
void launch_widen_bf16(Launcher& L, const bf16* x, size_t n, float* out);
template <typename T>
void launch_silu_mul(Launcher& L, const float* gu, int rows, int F, T* out);

struct RopeArgs {
  int mode;        // 0 = draft step rows (StepRows mapping), 1 = target rows (slot = base + r, pos = base + depth[r])
  StepRows s;
  int base;
  const int32_t* depth;
  int rows, q_rows;  // q is produced for the last q_rows rows
  int Hq, Hkv, d, cap;
  float theta;
};
template <typename T>
void launch_rope_append(Launcher& L, const RopeArgs& a, const float* qkv, T* kcache, T* vcache, T* qout);

struct AttnArgs {
  int rows, Hq, Hkv, d, cap;
  int n_all;              // slots [0, n_all) visible to every row
  int n_tree;             // masked slots n_all .. n_all + n_tree - 1
  const uint64_t* mask;   // [rows][mask_words]
  int mask_words;
  float scale;
  int n_splits, keys_per_split;
};
template <typename T>
void launch_tree_attention(Launcher& L, const AttnArgs& a, const T* q, const T* kcache, const T* vcache,
                           float* part, T* out);
size_t attn_partial_floats(int rows, int Hq, int d, int n_splits);
void plan_attention_splits(int rows, int Hkv, int total_keys, int max_splits, int* n_splits, int* keys_per_split);
// Plans the key split (at most max_splits ranges; `part` holds attn_partial_floats(rows, Hq, d, max_splits)
// floats) and runs the attention: the tensor-core kernel for bf16 shapes it covers, else the SIMT kernel.
// a.n_splits / a.keys_per_split are filled in here.
template <typename T>
void run_tree_attention(Launcher& L, AttnArgs a, int max_splits, const T* q, const T* kcache, const T* vcache,
                        float* part, T* out);
bool tree_attention_mma_supported(const AttnArgs& a);
void plan_attention_splits_mma(int rows, int Hq, int Hkv, int total_keys, int max_splits, int* n_splits,
                               int* keys_per_split);
void launch_tree_attention_mma(Launcher& L, const AttnArgs& a, const bf16* q, const bf16* kc, const bf16* vc,
                               float* part, bf16* out);

#define POSS_TOPK_CHUNK 2048
void launch_topk_partial(Launcher& L, const float* logits, int rows, int V, int K, float* pmax, float* psum,
                         float* pval, int32_t* pidx, int n_chunks);
void launch_topk_merge(Launcher& L, int rows, int K, int n_chunks, const float* pmax, const float* psum,
                       const float* pval, const int32_t* pidx, int32_t* out_ids, float* out_logp);

void launch_expand(Launcher& L, const TreeState& ts, int Kmax, int step, int Mc, int K, int cand_base, int last,
                   const int32_t* top_ids, const float* top_logp);
void launch_rerank(Launcher& L, const TreeState& ts, int n_cand, int K, int total, int root_tok_index,
                   const int32_t* new_tokens, int32_t* out_tokens, int32_t* out_parents, float* out_scores,
                   int32_t* out_depth, uint64_t* out_mask, int32_t* out_n_nodes);
template <typename T>
void launch_accept_walk(Launcher& L, const int32_t* g, const T* feats, int H, const int32_t* tokens,
                        const int32_t* parents, int rows, int max_depth, int32_t* out_path, int32_t* out_a,
                        int32_t* out_bonus, int32_t* out_new_tokens, T* out_new_features,
                        unsigned long long* counters);
template <typename T>
void launch_kv_compact(Launcher& L, T* target_kv, int layers, int Hkv, int cap, int d, int prefix_len,
                       const int32_t* path, const int32_t* n_accepted);
void launch_chain_mask(Launcher& L, uint64_t* mask, int32_t* depth, int rows);
