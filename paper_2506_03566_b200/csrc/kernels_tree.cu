// Vocabulary top-k / log-softmax, tree expansion, rerank, accept walk and cache compaction.
// Every ordering rule is (value descending, index ascending), so results are unique.
#include "poss_internal.cuh"
#include <math.h>

#define LAUNCH_CHECK(L)                                         \
  do {                                                          \
    ++*(L).launches;                                            \
    if (cudaGetLastError() != cudaSuccess) (L).err = POSS_E_CUDA; \
  } while (0)

#define NEG_INF (-INFINITY)

__device__ __forceinline__ bool better(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

__device__ __forceinline__ void warp_best(float& v, int& i) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    float ov = __shfl_xor_sync(0xffffffffu, v, off);
    int oi = __shfl_xor_sync(0xffffffffu, i, off);
    if (better(ov, oi, v, i)) { v = ov; i = oi; }
  }
}

// ------------------------------------------------------------------ per-chunk max / sum-exp / top-k of fp32 logits
__global__ void __launch_bounds__(256) k_topk_partial(const float* __restrict__ logits, int V, int K,
                                                      float* __restrict__ pmax, float* __restrict__ psum,
                                                      float* __restrict__ pval, int32_t* __restrict__ pidx,
                                                      int n_chunks) {
  __shared__ float vals[POSS_TOPK_CHUNK];
  __shared__ float wv[8];
  __shared__ int wi[8];
  __shared__ float s_max;
  int chunk = blockIdx.x, row = blockIdx.y;
  int lo = chunk * POSS_TOPK_CHUNK;
  int n = min(POSS_TOPK_CHUNK, V - lo);
  const float* src = logits + (size_t)row * V + lo;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float mx = NEG_INF;
  for (int i = threadIdx.x; i < POSS_TOPK_CHUNK; i += 256) {
    float v = i < n ? src[i] : NEG_INF;
    vals[i] = v;
    mx = fmaxf(mx, v);
  }
  for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  if (lane == 0) wv[warp] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = wv[0];
    for (int w = 1; w < 8; ++w) t = fmaxf(t, wv[w]);
    s_max = t;
  }
  __syncthreads();
  float cmax = s_max;
  float se = 0.f;
  for (int i = threadIdx.x; i < n; i += 256) se += expf(vals[i] - cmax);
  for (int off = 16; off > 0; off >>= 1) se += __shfl_xor_sync(0xffffffffu, se, off);
  __syncthreads();
  if (lane == 0) wv[warp] = se;
  __syncthreads();
  size_t pc = (size_t)row * n_chunks + chunk;
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < 8; ++w) t += wv[w];
    pmax[pc] = cmax;
    psum[pc] = t;
  }
  for (int k = 0; k < K; ++k) {
    __syncthreads();
    float bv = NEG_INF;
    int bi = 0x7fffffff;
    for (int i = threadIdx.x; i < n; i += 256) {
      float v = vals[i];
      if (better(v, i, bv, bi)) { bv = v; bi = i; }
    }
    warp_best(bv, bi);
    if (lane == 0) { wv[warp] = bv; wi[warp] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
      float v = wv[0];
      int i = wi[0];
      for (int w = 1; w < 8; ++w) if (better(wv[w], wi[w], v, i)) { v = wv[w]; i = wi[w]; }
      if (i < n) {
        pval[pc * K + k] = v;
        pidx[pc * K + k] = lo + i;
        vals[i] = NEG_INF;
      } else {                       // fewer than K entries in this chunk
        pval[pc * K + k] = NEG_INF;
        pidx[pc * K + k] = 0x7fffffff;
      }
    }
  }
}

void launch_topk_partial(Launcher& L, const float* logits, int rows, int V, int K, float* pmax, float* psum,
                         float* pval, int32_t* pidx, int n_chunks) {
  if (rows <= 0) return;
  dim3 grid(n_chunks, rows);
  k_topk_partial<<<grid, 256, 0, L.stream>>>(logits, V, K, pmax, psum, pval, pidx, n_chunks);
  LAUNCH_CHECK(L);
}

// ------------------------------------------------------------------ merge chunk partials: one warp per row
// Each chunk's list is already ordered best first, so the merge repeatedly takes the best chunk head.
// -inf entries (a chunk shorter than K) never win against a real value.
__global__ void __launch_bounds__(32) k_topk_merge(int K, int n_chunks, const float* __restrict__ pmax,
                                                   const float* __restrict__ psum, const float* __restrict__ pval,
                                                   const int32_t* __restrict__ pidx, int32_t* __restrict__ out_ids,
                                                   float* __restrict__ out_logp) {
  extern __shared__ int heads[];     // [n_chunks]
  int row = blockIdx.x, lane = threadIdx.x;
  const float* rmax = pmax + (size_t)row * n_chunks;
  const float* rsum = psum + (size_t)row * n_chunks;
  float gm = NEG_INF;
  for (int c = lane; c < n_chunks; c += 32) { gm = fmaxf(gm, rmax[c]); heads[c] = 0; }
  for (int off = 16; off > 0; off >>= 1) gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, off));
  float se = 0.f;
  for (int c = lane; c < n_chunks; c += 32) se += rsum[c] * expf(rmax[c] - gm);
  for (int off = 16; off > 0; off >>= 1) se += __shfl_xor_sync(0xffffffffu, se, off);
  float lse = gm + logf(se);
  __syncwarp();
  for (int k = 0; k < K; ++k) {
    float bv = NEG_INF;
    int bi = 0x7fffffff, bc = -1;
    for (int c = lane; c < n_chunks; c += 32) {
      int h = heads[c];
      if (h < K) {
        size_t p = ((size_t)row * n_chunks + c) * K + h;
        float v = pval[p];
        int i = pidx[p];
        if (better(v, i, bv, bi)) { bv = v; bi = i; bc = c; }
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, bv, off);
      int oi = __shfl_xor_sync(0xffffffffu, bi, off);
      int oc = __shfl_xor_sync(0xffffffffu, bc, off);
      if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; bc = oc; }
    }
    if (lane == 0) {
      out_ids[(size_t)row * K + k] = bi;
      out_logp[(size_t)row * K + k] = bv - lse;
      if (bc >= 0) heads[bc] += 1;
    }
    __syncwarp();
  }
}

void launch_topk_merge(Launcher& L, int rows, int K, int n_chunks, const float* pmax, const float* psum,
                       const float* pval, const int32_t* pidx, int32_t* out_ids, float* out_logp) {
  if (rows <= 0) return;
  k_topk_merge<<<rows, 32, n_chunks * sizeof(int), L.stream>>>(K, n_chunks, pmax, psum, pval, pidx, out_ids,
                                                               out_logp);
  LAUNCH_CHECK(L);
}

// ------------------------------------------------------------------ tree expansion after draft step `step`
// Rows r = 0..Mc-1 are the level-`step` frontier.  Appends Mc*K level-(step+1) candidates in
// (row, rank) order with score = row score + logp, then (unless last) picks the K best of them as the
// next frontier, best first, and records for each its token, parent row, score, flat index and the
// tree-slot mask (parent's mask plus its own slot step*K + rank).
__global__ void __launch_bounds__(256) k_expand(TreeState ts, int Kmax, int step, int Mc, int K, int cand_base,
                                                int last, const int32_t* __restrict__ top_ids,
                                                const float* __restrict__ top_logp) {
  __shared__ float sc[POSS_MAX_TOPK * POSS_MAX_TOPK];
  int n = Mc * K;
  for (int c = threadIdx.x; c < n; c += blockDim.x) {
    int r = c / K;
    float ps = step == 0 ? 0.f : ts.node_score[step * Kmax + r];
    int pc = step == 0 ? -1 : ts.node_cand[step * Kmax + r];
    float s = ps + top_logp[c];
    sc[c] = s;
    ts.cand_tok[cand_base + c] = top_ids[c];
    ts.cand_parent[cand_base + c] = pc;
    ts.cand_score[cand_base + c] = s;
  }
  __syncthreads();
  if (last) return;
  int lvl = step + 1;
  for (int c = threadIdx.x; c < n; c += blockDim.x) {
    float s = sc[c];
    int rank = 0;
    for (int o = 0; o < n; ++o) rank += better(sc[o], o, s, c) ? 1 : 0;
    if (rank < K) {
      int r = c / K;
      int at = lvl * Kmax + rank;
      ts.node_tok[at] = top_ids[c];
      ts.node_prow[at] = r;
      ts.node_cand[at] = cand_base + c;
      ts.node_score[at] = s;
      uint64_t m0 = 0, m1 = 0;
      if (step > 0) { m0 = ts.node_mask[(step * Kmax + r) * 2]; m1 = ts.node_mask[(step * Kmax + r) * 2 + 1]; }
      int bit = step * K + rank;
      if (bit < 64) m0 |= 1ull << bit; else m1 |= 1ull << (bit - 64);
      ts.node_mask[at * 2] = m0;
      ts.node_mask[at * 2 + 1] = m1;
    }
  }
}

void launch_expand(Launcher& L, const TreeState& ts, int Kmax, int step, int Mc, int K, int cand_base, int last,
                   const int32_t* top_ids, const float* top_logp) {
  k_expand<<<1, 256, 0, L.stream>>>(ts, Kmax, step, Mc, K, cand_base, last, top_ids, top_logp);
  LAUNCH_CHECK(L);
}

// ------------------------------------------------------------------ rerank: keep the `total` best candidates
// One block.  rank(c) = number of candidates that order before c; kept iff rank < total.  Kept
// candidates are listed in flat (creation) order behind the root, so a parent always precedes its
// children; level of flat index c is 1 for c < K, else 2 + (c - K) / K^2.
__global__ void __launch_bounds__(1024) k_rerank(TreeState ts, int n_cand, int K, int total,
                                                 const int32_t* __restrict__ root_tok,
                                                 int32_t* __restrict__ out_tokens, int32_t* __restrict__ out_parents,
                                                 float* __restrict__ out_scores, int32_t* __restrict__ out_depth,
                                                 uint64_t* __restrict__ out_mask, int32_t* __restrict__ out_n_nodes) {
  extern __shared__ unsigned char smem_raw[];
  float* sc = reinterpret_cast<float*>(smem_raw);               // [n_cand]
  int* newidx = reinterpret_cast<int*>(sc + n_cand);            // [n_cand] node index or 0 if dropped
  int keep = min(total, n_cand);
  int words = (total + 1 + 63) / 64;
  for (int c = threadIdx.x; c < n_cand; c += blockDim.x) sc[c] = ts.cand_score[c];
  __syncthreads();
  for (int c = threadIdx.x; c < n_cand; c += blockDim.x) {
    float s = sc[c];
    int rank = 0;
    for (int o = 0; o < n_cand; ++o) rank += better(sc[o], o, s, c) ? 1 : 0;
    newidx[c] = rank < keep ? 1 : 0;
  }
  __syncthreads();
  if (threadIdx.x == 0) {               // ordered compaction; n_cand is at most a few thousand
    int nxt = 1;
    for (int c = 0; c < n_cand; ++c) {
      if (newidx[c]) { ts.selected[nxt - 1] = c; newidx[c] = nxt++; }
    }
    out_tokens[0] = root_tok[0];
    out_parents[0] = -1;
    out_scores[0] = 0.f;
    out_depth[0] = 0;
    for (int w = 0; w < words; ++w) out_mask[w] = w == 0 ? 1ull : 0ull;
    out_n_nodes[0] = keep + 1;
  }
  __syncthreads();
  for (int c = threadIdx.x; c < n_cand; c += blockDim.x) {
    int node = newidx[c];
    if (!node) continue;
    int pc = ts.cand_parent[c];
    out_tokens[node] = ts.cand_tok[c];
    out_parents[node] = pc < 0 ? 0 : newidx[pc];
    out_scores[node] = sc[c];
    out_depth[node] = c < K ? 1 : 2 + (c - K) / (K * K);
    uint64_t m[4] = {1ull, 0ull, 0ull, 0ull};     // root bit
    int cur = c;
    while (cur >= 0) {
      int nd = newidx[cur];
      m[nd >> 6] |= 1ull << (nd & 63);
      cur = ts.cand_parent[cur];
    }
    for (int w = 0; w < words; ++w) out_mask[(size_t)node * words + w] = m[w];
  }
  // rows beyond n_nodes are zeroed so that callers may read fixed-size arrays
  for (int node = keep + 1 + threadIdx.x; node <= total; node += blockDim.x) {
    out_tokens[node] = 0; out_parents[node] = -1; out_scores[node] = 0.f; out_depth[node] = 0;
    for (int w = 0; w < words; ++w) out_mask[(size_t)node * words + w] = 0ull;
  }
}

void launch_rerank(Launcher& L, const TreeState& ts, int n_cand, int K, int total, int root_tok_index,
                   const int32_t* new_tokens, int32_t* out_tokens, int32_t* out_parents, float* out_scores,
                   int32_t* out_depth, uint64_t* out_mask, int32_t* out_n_nodes) {
  size_t smem = (size_t)n_cand * 8;
  k_rerank<<<1, 1024, smem, L.stream>>>(ts, n_cand, K, total, new_tokens + root_tok_index, out_tokens, out_parents,
                                        out_scores, out_depth, out_mask, out_n_nodes);
  LAUNCH_CHECK(L);
}

// ------------------------------------------------------------------ greedy accept walk (one warp) + hand-over pairs
template <typename T>
__global__ void __launch_bounds__(32) k_accept_walk(const int32_t* __restrict__ g, const T* __restrict__ feats,
                                                    int H, const int32_t* __restrict__ tokens,
                                                    const int32_t* __restrict__ parents, int rows, int max_depth,
                                                    int32_t* __restrict__ out_path, int32_t* __restrict__ out_a,
                                                    int32_t* __restrict__ out_bonus,
                                                    int32_t* __restrict__ out_new_tokens,
                                                    T* __restrict__ out_new_features,
                                                    unsigned long long* __restrict__ counters) {
  __shared__ int path[POSS_MAX_DEPTH + 1];
  int lane = threadIdx.x;
  int cur = 0, a = 0;
  if (lane == 0) path[0] = 0;
  while (a < max_depth) {
    int want = g[cur];
    int found = 0x7fffffff;
    for (int c = 1 + lane; c < rows; c += 32)
      if (parents[c] == cur && tokens[c] == want) found = min(found, c);
    for (int off = 16; off > 0; off >>= 1) found = min(found, __shfl_xor_sync(0xffffffffu, found, off));
    if (found == 0x7fffffff) break;
    cur = found;
    ++a;
    if (lane == 0) path[a] = cur;
  }
  __syncwarp();
  if (lane == 0) {
    out_a[0] = a;
    out_bonus[0] = g[cur];
    atomicAdd(&counters[0], 1ull);                         // rounds
    for (int i = 1; i <= a; ++i) atomicAdd(&counters[i], 1ull);   // N_i
  }
  for (int i = lane; i <= POSS_MAX_DEPTH; i += 32) out_path[i] = i <= a ? path[i] : -1;
  for (int k = lane; k <= a; k += 32) out_new_tokens[k] = k < a ? tokens[path[k + 1]] : g[cur];
  for (int k = 0; k <= a; ++k) {
    const T* src = feats + (size_t)path[k] * H;
    T* dst = out_new_features + (size_t)k * H;
    for (int i = lane; i < H; i += 32) dst[i] = src[i];
  }
}
template <typename T>
void launch_accept_walk(Launcher& L, const int32_t* g, const T* feats, int H, const int32_t* tokens,
                        const int32_t* parents, int rows, int max_depth, int32_t* out_path, int32_t* out_a,
                        int32_t* out_bonus, int32_t* out_new_tokens, T* out_new_features,
                        unsigned long long* counters) {
  k_accept_walk<T><<<1, 32, 0, L.stream>>>(g, feats, H, tokens, parents, rows, max_depth, out_path, out_a, out_bonus,
                                           out_new_tokens, out_new_features, counters);
  LAUNCH_CHECK(L);
}
template void launch_accept_walk<float>(Launcher&, const int32_t*, const float*, int, const int32_t*, const int32_t*,
                                        int, int, int32_t*, int32_t*, int32_t*, int32_t*, float*,
                                        unsigned long long*);
template void launch_accept_walk<bf16>(Launcher&, const int32_t*, const bf16*, int, const int32_t*, const int32_t*,
                                       int, int, int32_t*, int32_t*, int32_t*, int32_t*, bf16*, unsigned long long*);

// ------------------------------------------------------------------ cache compaction after acceptance
// Block (layer*2 + kv, head): copies slot prefix_len + path[k] to prefix_len + k for k = 1..a in
// ascending k.  path[k] >= k, so a source is never overwritten before it is read.
template <typename T>
__global__ void __launch_bounds__(128) k_kv_compact(T* __restrict__ kv, int Hkv, int cap, int d, int prefix_len,
                                                    const int32_t* __restrict__ path,
                                                    const int32_t* __restrict__ n_accepted) {
  int a = n_accepted[0];
  T* base = kv + ((size_t)blockIdx.x * Hkv + blockIdx.y) * (size_t)cap * d;
  for (int k = 1; k <= a; ++k) {
    int src = path[k];
    if (src == k) continue;
    for (int i = threadIdx.x; i < d; i += blockDim.x)
      base[(size_t)(prefix_len + k) * d + i] = base[(size_t)(prefix_len + src) * d + i];
    __syncthreads();
  }
}
template <typename T>
void launch_kv_compact(Launcher& L, T* target_kv, int layers, int Hkv, int cap, int d, int prefix_len,
                       const int32_t* path, const int32_t* n_accepted) {
  dim3 grid(layers * 2, Hkv);
  k_kv_compact<T><<<grid, 128, 0, L.stream>>>(target_kv, Hkv, cap, d, prefix_len, path, n_accepted);
  LAUNCH_CHECK(L);
}
template void launch_kv_compact<float>(Launcher&, float*, int, int, int, int, int, const int32_t*, const int32_t*);
template void launch_kv_compact<bf16>(Launcher&, bf16*, int, int, int, int, int, const int32_t*, const int32_t*);
