// Vocabulary top-k / log-softmax, tree expansion, rerank, accept walk and cache compaction.
// Every ordering rule is (value descending, index ascending), so results are unique.
#include "poss_internal.cuh"
#include <math.h>
#include <string.h>

POSS_TRACE_REGISTER()

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
__global__ void __launch_bounds__(256) k_topk_partial(const float* logits, int V, int K,
                                                      float* pmax, float* psum,
                                                      float* pval, int32_t* pidx,
                                                      int n_chunks) {
  __shared__ float vals[POSS_TOPK_CHUNK];
  __shared__ float wv[8];
  __shared__ int wi[8];
  __shared__ float s_max;
  pdl_enter(POSS_K_TOPK_PARTIAL);
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
  launch_pdl(L, k_topk_partial, grid, dim3(256), 0, logits, V, K, pmax, psum, pval, pidx, n_chunks);
}

// ------------------------------------------------------------------ row argmax partials straight from the logits
// Block (chunk, row): the best (value, lowest id) of POSS_ARGMAX_CHUNK consecutive logits, written in the
// partial-list format of the merge kernel with K = 1 (max = the value, sum = 1).  bf16 logits are read
// as they are (16-byte loads), never widened to a second buffer.
template <typename T>
__global__ void __launch_bounds__(256) k_argmax_partial(const T* logits, int V, float* pmax, float* psum, float* pval,
                                                        int32_t* pidx, int n_chunks) {
  __shared__ float wv[8];
  __shared__ int wi[8];
  pdl_enter(POSS_K_ARGMAX_PARTIAL);
  const int chunk = blockIdx.x, row = blockIdx.y;
  const int lo = chunk * POSS_ARGMAX_CHUNK;
  const int n = min(POSS_ARGMAX_CHUNK, V - lo);
  const T* src = logits + (size_t)row * V + lo;
  constexpr int PER = 16 / sizeof(T);
  float bv = NEG_INF;
  int bi = 0x7fffffff;
  const bool vec = (reinterpret_cast<uintptr_t>(src) & 15) == 0;
  if (vec) {
    const int n_vec = n / PER;
    const uint4* s4 = reinterpret_cast<const uint4*>(src);
    for (int base = 0; base < n_vec; base += 256 * 4) {
      uint4 raw[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        int i = base + u * 256 + threadIdx.x;
        if (i < n_vec) raw[u] = s4[i];
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        int i = base + u * 256 + threadIdx.x;
        if (i < n_vec) {
          const T* e = reinterpret_cast<const T*>(&raw[u]);
#pragma unroll
          for (int q = 0; q < PER; ++q) {
            float v = to_f(e[q]);
            int id = i * PER + q;
            if (better(v, id, bv, bi)) { bv = v; bi = id; }
          }
        }
      }
    }
    for (int i = n_vec * PER + threadIdx.x; i < n; i += 256) {
      float v = to_f(src[i]);
      if (better(v, i, bv, bi)) { bv = v; bi = i; }
    }
  } else {
    for (int i = threadIdx.x; i < n; i += 256) {
      float v = to_f(src[i]);
      if (better(v, i, bv, bi)) { bv = v; bi = i; }
    }
  }
  warp_best(bv, bi);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) { wv[warp] = bv; wi[warp] = bi; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float v = wv[0];
    int i = wi[0];
    for (int w = 1; w < 8; ++w) if (better(wv[w], wi[w], v, i)) { v = wv[w]; i = wi[w]; }
    size_t pc = (size_t)row * n_chunks + chunk;
    pmax[pc] = v;
    psum[pc] = 1.f;
    pval[pc] = v;
    pidx[pc] = i == 0x7fffffff ? i : lo + i;
  }
}
template <typename T>
int launch_argmax_partial(Launcher& L, const T* logits, int rows, int V, float* pmax, float* psum, float* pval,
                          int32_t* pidx) {
  int n_chunks = (V + POSS_ARGMAX_CHUNK - 1) / POSS_ARGMAX_CHUNK;
  if (rows <= 0) return n_chunks;
  launch_pdl(L, k_argmax_partial<T>, dim3(n_chunks, rows), dim3(256), 0, logits, V, pmax, psum, pval, pidx, n_chunks);
  return n_chunks;
}
template int launch_argmax_partial<float>(Launcher&, const float*, int, int, float*, float*, float*, int32_t*);
template int launch_argmax_partial<bf16>(Launcher&, const bf16*, int, int, float*, float*, float*, int32_t*);

// ------------------------------------------------------------------ tree expansion after draft step `step`
// Rows r = 0..Mc-1 are the level-`step` frontier.  Appends Mc*K level-(step+1) candidates in
// (row, rank) order with score = row score + logp, then (unless last) picks the K best of them as the
// next frontier, best first, and records for each its token, parent row, score, flat index and the
// tree-slot mask (parent's mask plus its own slot step*K + rank).  Runs inside one block.
__device__ void expand_block(const TreeState& ts, const ExpandArgs& x, const int32_t* top_ids, const float* top_logp,
                             float* sc) {
  const int K = x.K, Kmax = x.Kmax, step = x.step;
  int n = x.Mc * K;
  for (int c = threadIdx.x; c < n; c += blockDim.x) {
    int r = c / K;
    float ps = step == 0 ? 0.f : ts.node_score[step * Kmax + r];
    int pc = step == 0 ? -1 : ts.node_cand[step * Kmax + r];
    float s = ps + __ldcg(top_logp + c);
    sc[c] = s;
    ts.cand_tok[x.cand_base + c] = __ldcg(top_ids + c);
    ts.cand_parent[x.cand_base + c] = pc;
    ts.cand_score[x.cand_base + c] = s;
  }
  __syncthreads();
  if (x.last) return;
  int lvl = step + 1;
  for (int c = threadIdx.x; c < n; c += blockDim.x) {
    float s = sc[c];
    int rank = 0;
    for (int o = 0; o < n; ++o) rank += better(sc[o], o, s, c) ? 1 : 0;
    if (rank < K) {
      int r = c / K;
      int at = lvl * Kmax + rank;
      ts.node_tok[at] = __ldcg(top_ids + c);
      ts.node_prow[at] = r;
      ts.node_cand[at] = x.cand_base + c;
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

// ------------------------------------------------------------------ merge the partial lists of a row, finish log-softmax
// One block per activation row.  Every list is ordered best first, so the merge repeatedly takes the
// best list head; -inf entries (a list shorter than K) never win against a real value.  The block that
// finishes last (a counter, nobody waits) also runs the tree expansion when the caller asks for it.
__global__ void __launch_bounds__(128) k_topk_merge(int K, int n_lists, const float* pmax,
                                                    const float* psum, const float* pval,
                                                    const int32_t* pidx, int32_t* out_ids,
                                                    float* out_logp, TreeState ts, ExpandArgs x,
                                                    int* done) {
  extern __shared__ unsigned char merge_smem[];
  float* vals = reinterpret_cast<float*>(merge_smem);                 // [n_lists][K]
  int* idxs = reinterpret_cast<int*>(vals + (size_t)n_lists * K);     // [n_lists][K]
  int* heads = idxs + (size_t)n_lists * K;                            // [n_lists]
  __shared__ float red[4];
  __shared__ float s_gm, s_lse;
  __shared__ int s_is_last;
  pdl_enter(POSS_K_TOPK_MERGE);
  const int row = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float* rmax = pmax + (size_t)row * n_lists;
  const float* rsum = psum + (size_t)row * n_lists;
  {
    const float* pv = pval + (size_t)row * n_lists * K;
    const int32_t* pi = pidx + (size_t)row * n_lists * K;
    const int n = n_lists * K;
    for (int base = 0; base < n; base += 128 * 8) {      // eight loads of each kind in flight per thread
      float v[8];
      int x[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        int i = base + u * 128 + threadIdx.x;
        if (i < n) { v[u] = __ldcg(pv + i); x[u] = __ldcg(pi + i); }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        int i = base + u * 128 + threadIdx.x;
        if (i < n) { vals[i] = v[u]; idxs[i] = x[u]; }
      }
    }
  }
  float gm = NEG_INF;
  for (int c = threadIdx.x; c < n_lists; c += 128) { gm = fmaxf(gm, rmax[c]); heads[c] = 0; }
  for (int off = 16; off > 0; off >>= 1) gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, off));
  if (lane == 0) red[warp] = gm;
  __syncthreads();
  if (threadIdx.x == 0) s_gm = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
  __syncthreads();
  gm = s_gm;
  float se = 0.f;
  for (int c = threadIdx.x; c < n_lists; c += 128) {
    float m = rmax[c];
    if (m > NEG_INF) se += rsum[c] * expf(m - gm);
  }
  for (int off = 16; off > 0; off >>= 1) se += __shfl_xor_sync(0xffffffffu, se, off);
  __syncthreads();
  if (lane == 0) red[warp] = se;
  __syncthreads();
  if (threadIdx.x == 0) s_lse = gm + logf(((red[0] + red[1]) + red[2]) + red[3]);
  __syncthreads();
  if (warp == 0) {
    const float lse = s_lse;
    for (int k = 0; k < K; ++k) {
      float bv = NEG_INF;
      int bi = 0x7fffffff, bc = -1;
      for (int c = lane; c < n_lists; c += 32) {
        int h = heads[c];
        if (h < K) {
          float v = vals[c * K + h];
          int i = idxs[c * K + h];
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
  if (!x.enabled) return;
  // ---- the last block to finish expands the tree
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    int prev = atomicAdd(done, 1);
    s_is_last = prev == (int)gridDim.x - 1;
  }
  __syncthreads();
  if (!s_is_last) return;
  __threadfence();
  for (int b = 0; b < x.batch; ++b) {                // vals is free now: Mc*K <= its size is checked by the host
    expand_block(tree_of(ts, b), x, out_ids + (size_t)b * x.Mc * K, out_logp + (size_t)b * x.Mc * K, vals);
    __syncthreads();
  }
  if (threadIdx.x == 0) *done = 0;
}

// ------------------------------------------------------------------ the same for a draft step, in one block per sequence
// A sequence's draft step has at most POSS_MAX_TOPK rows and is followed by the tree expansion, which needs
// every row's result: one block of 1024 threads stages all partial lists of its sequence's rows in shared memory
// with 16-byte loads (one round trip), warp r merges row r, and after one barrier the block expands the
// sequence's tree.  No second kernel, no counter.  Block b: rows [b * rows, (b + 1) * rows), tree state b.
__global__ void __launch_bounds__(1024) k_topk_merge_expand(int rows, int K, int n_lists, const float* pmax,
                                                            const float* psum, const float* pval,
                                                            const int32_t* pidx, int32_t* out_ids, float* out_logp,
                                                            TreeState ts_all, ExpandArgs x) {
  {
    const size_t row0 = (size_t)blockIdx.x * rows;
    pmax += row0 * n_lists; psum += row0 * n_lists;
    pval += row0 * n_lists * K; pidx += row0 * n_lists * K;
    out_ids += row0 * K; out_logp += row0 * K;
  }
  const TreeState ts = tree_of(ts_all, blockIdx.x);
  extern __shared__ __align__(16) unsigned char me_smem[];
  const int per_row = n_lists * K;
  const int total = rows * per_row;
  const int total4 = (total + 3) & ~3;
  float* vals = reinterpret_cast<float*>(me_smem);               // [rows][n_lists][K]
  int* idxs = reinterpret_cast<int*>(vals + total4);             // [rows][n_lists][K]
  float* smax = reinterpret_cast<float*>(idxs + total4);         // [rows][n_lists]
  float* ssum = smax + rows * n_lists;                           // [rows][n_lists]
  int* heads = reinterpret_cast<int*>(ssum + rows * n_lists);    // [rows][n_lists]
  pdl_enter(POSS_K_TOPK_MERGE_EXPAND);
  {
    // 16-byte loads when this sequence's lists start on a 16-byte boundary, else element by element
    const bool al = ((reinterpret_cast<uintptr_t>(pval) | reinterpret_cast<uintptr_t>(pidx)) & 15) == 0;
    const int n4 = al ? total / 4 : 0;
    const float4* pv4 = reinterpret_cast<const float4*>(pval);
    const int4* pi4 = reinterpret_cast<const int4*>(pidx);
    for (int base = 0; base < n4; base += 1024 * 4) {
      float4 v[4];
      int4 q[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        int i = base + u * 1024 + threadIdx.x;
        if (i < n4) { v[u] = __ldcg(pv4 + i); q[u] = __ldcg(pi4 + i); }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        int i = base + u * 1024 + threadIdx.x;
        if (i < n4) { reinterpret_cast<float4*>(vals)[i] = v[u]; reinterpret_cast<int4*>(idxs)[i] = q[u]; }
      }
    }
    for (int i = n4 * 4 + threadIdx.x; i < total; i += 1024) { vals[i] = __ldcg(pval + i); idxs[i] = __ldcg(pidx + i); }
    for (int i = threadIdx.x; i < rows * n_lists; i += 1024) {
      smax[i] = __ldcg(pmax + i);
      ssum[i] = __ldcg(psum + i);
      heads[i] = 0;
    }
  }
  __syncthreads();
  POSS_TRACE_POINT(1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp < rows) {
    const int row = warp;
    const float* rmax = smax + row * n_lists;
    const float* rsum = ssum + row * n_lists;
    const float* rv = vals + (size_t)row * per_row;
    const int* ri = idxs + (size_t)row * per_row;
    int* rh = heads + row * n_lists;
    float gm = NEG_INF;
    for (int c = lane; c < n_lists; c += 32) gm = fmaxf(gm, rmax[c]);
    for (int off = 16; off > 0; off >>= 1) gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, off));
    float se = 0.f;
    for (int c = lane; c < n_lists; c += 32) {
      float m = rmax[c];
      if (m > NEG_INF) se += rsum[c] * expf(m - gm);
    }
    for (int off = 16; off > 0; off >>= 1) se += __shfl_xor_sync(0xffffffffu, se, off);
    const float lse = gm + logf(se);
    POSS_TRACE_POINT(2);
    if (n_lists <= 32 * 6) {
      // each lane keeps the heads of its (at most six) lists in registers: a round is a register scan,
      // one warp reduction and one shared-memory load by the winning lane
      float hv[6];
      int hi[6], hp[6];
#pragma unroll
      for (int j = 0; j < 6; ++j) {
        int c = lane + 32 * j;
        hp[j] = 0;
        hv[j] = c < n_lists ? rv[c * K] : NEG_INF;
        hi[j] = c < n_lists ? ri[c * K] : 0x7fffffff;
      }
      for (int k = 0; k < K; ++k) {
        float bv = hv[0];
        int bi = hi[0], bj = 0;
#pragma unroll
        for (int j = 1; j < 6; ++j) if (better(hv[j], hi[j], bv, bi)) { bv = hv[j]; bi = hi[j]; bj = j; }
        // the warp's best (largest value, then lowest id) with two integer reductions: the value as an
        // order-preserving unsigned key, then the lowest id among the lanes that hold that value
        const uint32_t bits = bv == 0.f ? 0u : __float_as_uint(bv);      // -0 and +0 are one value
        const uint32_t key = (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
        const uint32_t wkey = __reduce_max_sync(0xffffffffu, key);
        const int wi = (int)__reduce_min_sync(0xffffffffu, key == wkey ? (uint32_t)bi : 0xffffffffu);
        const int wl = __ffs(__ballot_sync(0xffffffffu, key == wkey && bi == wi)) - 1;
        const float wv = __shfl_sync(0xffffffffu, bv, wl);
        if (lane == 0) {
          out_ids[(size_t)row * K + k] = wi;
          out_logp[(size_t)row * K + k] = wv - lse;
        }
        if (lane == wl && wi != 0x7fffffff) {
          // advance the winning list
#pragma unroll
          for (int j = 0; j < 6; ++j) {
            if (j == bj) {
              int c = lane + 32 * j, h = ++hp[j];
              hv[j] = h < K ? rv[c * K + h] : NEG_INF;
              hi[j] = h < K ? ri[c * K + h] : 0x7fffffff;
            }
          }
        }
      }
    } else {
      for (int k = 0; k < K; ++k) {
        float bv = NEG_INF;
        int bi = 0x7fffffff, bc = -1;
        for (int c = lane; c < n_lists; c += 32) {
          int h = rh[c];
          if (h < K) {
            float v = rv[c * K + h];
            int i = ri[c * K + h];
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
          if (bc >= 0) rh[bc] += 1;
        }
        __syncwarp();
      }
    }
  }
  POSS_TRACE_POINT(3);
  __syncthreads();                       // every row's ids / log-probs are written (this block's own stores)
  if (x.enabled) expand_block(ts, x, out_ids, out_logp, vals);
  POSS_TRACE_POINT(4);
}

void launch_topk_merge(Launcher& L, int rows, int K, int n_lists, const float* pmax, const float* psum,
                       const float* pval, const int32_t* pidx, int32_t* out_ids, float* out_logp,
                       const TreeState* ts, const ExpandArgs* x, int* done) {
  if (rows <= 0) return;
  ExpandArgs xa;
  memset(&xa, 0, sizeof(xa));
  TreeState t;
  memset(&t, 0, sizeof(t));
  if (x && ts && x->enabled) { xa = *x; t = *ts; }
  const int batch = xa.enabled && xa.batch > 0 ? xa.batch : 1;
  xa.batch = batch;
  if (xa.enabled && rows == batch * xa.Mc && xa.Mc <= POSS_MAX_TOPK) {
    const int rows_seq = xa.Mc;
    size_t total4 = ((size_t)rows_seq * n_lists * K + 3) & ~(size_t)3;
    size_t smem1 = total4 * 8 + (size_t)rows_seq * n_lists * 12;
    if (smem1 < (size_t)xa.Mc * K * 4) smem1 = (size_t)xa.Mc * K * 4;
    if (smem1 <= 200 * 1024) {
      static PerDeviceFlags attr1_done;
      bool* a1 = attr1_done.current();
      if (!a1 || !*a1) {
        if (cudaFuncSetAttribute(k_topk_merge_expand, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) !=
            cudaSuccess) {
          L.err = POSS_E_CUDA;
          return;
        }
        if (a1) *a1 = true;
      }
      launch_pdl(L, k_topk_merge_expand, dim3(batch), dim3(1024), smem1, rows_seq, K, n_lists, pmax, psum, pval, pidx,
                 out_ids, out_logp, t, xa);
      return;
    }
  }
  size_t elems = (size_t)n_lists * K;
  if (xa.enabled && elems < (size_t)xa.Mc * K) elems = (size_t)xa.Mc * K;      // room for the expansion's scores
  size_t smem = elems * 8 + (size_t)n_lists * 4;
  static PerDeviceFlags attr_done;
  bool* a0 = attr_done.current();
  if (!a0 || !*a0) {
    if (cudaFuncSetAttribute(k_topk_merge, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024) != cudaSuccess) {
      L.err = POSS_E_CUDA;
      return;
    }
    if (a0) *a0 = true;
  }
  if (smem > 100 * 1024) { L.err = POSS_E_CAPACITY; return; }
  launch_pdl(L, k_topk_merge, dim3(rows), dim3(128), smem, K, n_lists, pmax, psum, pval, pidx, out_ids, out_logp, t, xa,
             done);
}

// ------------------------------------------------------------------ rerank: keep the `total` best candidates
// One block.  rank(c) = number of candidates that order before c; kept iff rank < total.  Kept
// candidates are listed in flat (creation) order behind the root, so a parent always precedes its
// children; level of flat index c is 1 for c < K, else 2 + (c - K) / K^2.
__global__ void __launch_bounds__(1024) k_rerank(TreeState ts_all, int n_cand, int K, int total, RerankBatch rb,
                                                 const int32_t* new_tokens,
                                                 int32_t* out_tokens, int32_t* out_parents,
                                                 float* out_scores, int32_t* out_depth,
                                                 uint64_t* out_mask, int32_t* out_n_nodes) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ int wtot[32];
  // block b = sequence b: its tree state, its root token, its slice of the outputs
  const TreeState ts = tree_of(ts_all, blockIdx.x);
  const int32_t* root_tok = new_tokens + rb.root_index[blockIdx.x];
  {
    const size_t o = (size_t)blockIdx.x * (total + 1);
    out_tokens += o; out_parents += o; out_scores += o; out_depth += o;
    out_mask += o * ((total + 1 + 63) / 64);
    out_n_nodes += blockIdx.x;
  }
  pdl_enter(POSS_K_RERANK);
  const int n_pad = (n_cand + 3) & ~3;
  float* sc = reinterpret_cast<float*>(smem_raw);               // [n_pad], -inf behind the candidates
  int* newidx = reinterpret_cast<int*>(sc + n_pad);             // [n_cand] node index or 0 if dropped
  int* par = newidx + n_cand;                                   // [n_cand] parent candidate
  int* same = par + n_cand;                                     // [n_cand] candidates that share a count (see below)
  int keep = min(total, n_cand);
  int words = (total + 1 + 63) / 64;
  for (int c = threadIdx.x; c < n_pad; c += blockDim.x) {
    sc[c] = c < n_cand ? ts.cand_score[c] : NEG_INF;
    if (c < n_cand) { par[c] = ts.cand_parent[c]; same[c] = 0; }
  }
  __syncthreads();
  // rank(c) = candidates with a higher score + candidates with the same score and a lower index; kept iff
  // rank < keep.  Two threads per candidate count the higher scores over half of the list each, four scores per
  // load, no branch (counting one by one with an early exit was a chain of dependent shared-memory loads: 13 us
  // for 510 candidates).  Equal scores are rare: candidates with equal scores have equal counts, so a candidate
  // whose count nobody shares has no equal and its rank is its count; only the others look for equals.
  {
    const float4* sc4 = reinterpret_cast<const float4*>(sc);
    const int n4 = n_pad / 4, half4 = (n4 + 1) / 2;
    for (int c0 = 0; c0 < n_cand; c0 += blockDim.x / 2) {
      const int c = c0 + (threadIdx.x >> 1), side = threadIdx.x & 1;
      const float s = c < n_cand ? sc[c] : INFINITY;
      int gt = 0;
      const int lo = side * half4, hi = side ? n4 : half4;
#pragma unroll 4
      for (int o = lo; o < hi; ++o) {
        const float4 x = sc4[o];
        gt += (x.x > s ? 1 : 0) + (x.y > s ? 1 : 0) + (x.z > s ? 1 : 0) + (x.w > s ? 1 : 0);
      }
      gt += __shfl_xor_sync(0xffffffffu, gt, 1);
      if (c < n_cand && side == 0) {
        newidx[c] = gt;
        atomicAdd(&same[gt], 1);                                 // (gt < n_cand: a candidate is not above itself)
      }
    }
  }
  __syncthreads();
  for (int c = threadIdx.x; c < n_cand; c += blockDim.x) {
    int rank = newidx[c];
    if (same[rank] > 1) {
      const float s = sc[c];
      for (int o = 0; o < c; ++o) rank += sc[o] == s ? 1 : 0;
    }
    newidx[c] = rank < keep ? 1 : 0;                             // (entry c is this thread's alone)
  }
  __syncthreads();
  // ordered compaction: node index = 1 + number of kept candidates with a lower flat index
  {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    int base = 0;
    for (int c0 = 0; c0 < n_cand; c0 += blockDim.x) {
      int c = c0 + threadIdx.x;
      bool kept = c < n_cand && newidx[c] != 0;
      unsigned b = __ballot_sync(0xffffffffu, kept);
      if (lane == 0) wtot[warp] = __popc(b);
      __syncthreads();
      int before = base, all = 0;
      for (int w = 0; w < n_warps; ++w) { int t = wtot[w]; if (w < warp) before += t; all += t; }
      if (kept) {
        int node = 1 + before + __popc(b & ((1u << lane) - 1u));
        newidx[c] = node;
        ts.selected[node - 1] = c;
      }
      base += all;
      __syncthreads();
    }
  }
  if (threadIdx.x == 0) {
    out_tokens[0] = root_tok[0];
    out_parents[0] = -1;
    out_scores[0] = 0.f;
    out_depth[0] = 0;
    for (int w = 0; w < words; ++w) out_mask[w] = w == 0 ? 1ull : 0ull;
    out_n_nodes[0] = keep + 1;
  }
  for (int c = threadIdx.x; c < n_cand; c += blockDim.x) {
    int node = newidx[c];
    if (!node) continue;
    int pc = par[c];
    out_tokens[node] = ts.cand_tok[c];
    out_parents[node] = pc < 0 ? 0 : newidx[pc];
    out_scores[node] = sc[c];
    out_depth[node] = c < K ? 1 : 2 + (c - K) / (K * K);
    uint64_t m[4] = {1ull, 0ull, 0ull, 0ull};     // root bit
    int cur = c;
    while (cur >= 0) {
      int nd = newidx[cur];
      m[nd >> 6] |= 1ull << (nd & 63);
      cur = par[cur];
    }
    for (int w = 0; w < words; ++w) out_mask[(size_t)node * words + w] = m[w];
  }
  // rows beyond n_nodes are zeroed so that callers may read fixed-size arrays
  for (int node = keep + 1 + threadIdx.x; node <= total; node += blockDim.x) {
    out_tokens[node] = 0; out_parents[node] = -1; out_scores[node] = 0.f; out_depth[node] = 0;
    for (int w = 0; w < words; ++w) out_mask[(size_t)node * words + w] = 0ull;
  }
}

void launch_rerank(Launcher& L, const TreeState& ts, int n_cand, int K, int total, const RerankBatch& rb,
                   const int32_t* new_tokens, int32_t* out_tokens, int32_t* out_parents, float* out_scores,
                   int32_t* out_depth, uint64_t* out_mask, int32_t* out_n_nodes) {
  size_t smem = (size_t)(n_cand + 4) * 16;
  // (a round's tree slots fit two mask words, so at most 2064 candidates: 33 KB)
  if (smem > 48 * 1024) { L.err = POSS_E_CAPACITY; return; }
  launch_pdl(L, k_rerank, dim3(rb.batch), dim3(1024), smem, ts, n_cand, K, total, rb, new_tokens, out_tokens,
             out_parents, out_scores, out_depth, out_mask, out_n_nodes);
}

// ------------------------------------------------------------------ greedy accept walk + hand-over pairs
// One block.  The tree (tokens, parents) and the target's greedy tokens are staged in shared memory,
// warp 0 walks (every step scans all nodes for the child that carries the wanted token, lowest node
// index first), then the whole block copies the accepted rows' features with 16-byte accesses.
template <typename T>
__global__ void __launch_bounds__(256) k_accept_walk(const int32_t* g, const T* feats, int H, const int32_t* tokens,
                                                     const int32_t* parents, int rows, int max_depth,
                                                     int32_t* out_path, int32_t* out_a, int32_t* out_bonus,
                                                     int32_t* out_new_tokens, T* out_new_features,
                                                     unsigned long long* counters) {
  __shared__ int s_tok[256], s_par[256], s_g[256];
  __shared__ int path[POSS_MAX_DEPTH + 1];
  __shared__ int s_a;
  pdl_enter(POSS_K_ACCEPT_WALK);
  for (int i = threadIdx.x; i < rows; i += blockDim.x) { s_tok[i] = tokens[i]; s_par[i] = parents[i]; s_g[i] = g[i]; }
  __syncthreads();
  const int lane = threadIdx.x & 31;
  if (threadIdx.x < 32) {
    int cur = 0, a = 0;
    if (lane == 0) path[0] = 0;
    while (a < max_depth) {
      int want = s_g[cur];
      int found = 0x7fffffff;
      for (int c = 1 + lane; c < rows; c += 32)
        if (s_par[c] == cur && s_tok[c] == want) found = min(found, c);
      for (int off = 16; off > 0; off >>= 1) found = min(found, __shfl_xor_sync(0xffffffffu, found, off));
      if (found == 0x7fffffff) break;
      cur = found;
      ++a;
      if (lane == 0) path[a] = cur;
    }
    __syncwarp();
    if (lane == 0) {
      s_a = a;
      out_a[0] = a;
      out_bonus[0] = s_g[cur];
      atomicAdd(&counters[0], 1ull);                         // rounds
      for (int i = 1; i <= a; ++i) atomicAdd(&counters[i], 1ull);   // N_i
    }
    for (int i = lane; i <= POSS_MAX_DEPTH; i += 32) out_path[i] = i <= a ? path[i] : -1;
    for (int k = lane; k <= a; k += 32) out_new_tokens[k] = k < a ? s_tok[path[k + 1]] : s_g[cur];
  }
  __syncthreads();
  const int a = s_a;
  constexpr int PER = 16 / sizeof(T);
  const bool vec = (H % PER) == 0 &&
                   ((reinterpret_cast<uintptr_t>(feats) | reinterpret_cast<uintptr_t>(out_new_features)) & 15) == 0;
  if (vec) {
    const int per_row = H / PER;
    for (int i = threadIdx.x; i < (a + 1) * per_row; i += blockDim.x) {
      int k = i / per_row, e = i % per_row;
      reinterpret_cast<uint4*>(out_new_features + (size_t)k * H)[e] =
          reinterpret_cast<const uint4*>(feats + (size_t)path[k] * H)[e];
    }
  } else {
    for (int i = threadIdx.x; i < (a + 1) * H; i += blockDim.x) {
      int k = i / H, e = i % H;
      out_new_features[(size_t)k * H + e] = feats[(size_t)path[k] * H + e];
    }
  }
}
template <typename T>
void launch_accept_walk(Launcher& L, const int32_t* g, const T* feats, int H, const int32_t* tokens,
                        const int32_t* parents, int rows, int max_depth, int32_t* out_path, int32_t* out_a,
                        int32_t* out_bonus, int32_t* out_new_tokens, T* out_new_features,
                        unsigned long long* counters) {
  launch_pdl(L, k_accept_walk<T>, dim3(1), dim3(256), 0, g, feats, H, tokens, parents, rows, max_depth, out_path, out_a,
             out_bonus, out_new_tokens, out_new_features, counters);
}
template void launch_accept_walk<float>(Launcher&, const int32_t*, const float*, int, const int32_t*, const int32_t*,
                                        int, int, int32_t*, int32_t*, int32_t*, int32_t*, float*,
                                        unsigned long long*);
template void launch_accept_walk<bf16>(Launcher&, const int32_t*, const bf16*, int, const int32_t*, const int32_t*,
                                       int, int, int32_t*, int32_t*, int32_t*, int32_t*, bf16*, unsigned long long*);

// ------------------------------------------------------------------ verification at a temperature > 0
// Rejection sampling over the tree's deterministic candidates (each candidate is a point mass): at the current node
// p = softmax(logits / T); its children are tested in node order, child x is accepted iff the next uniform is
// below p(x) / (mass not yet removed); a rejected child's mass is removed; when no child is left the bonus token is
// drawn from what remains by inverse CDF in token order.  One block walks the tree; a level costs two passes over
// the node's logits (maximum, sum of exponentials), the bonus a third one.  The walk is sequential by nature; the
// passes are spread over the block's 1024 threads.  Sums are formed in a fixed order (per-lane strided partial
// sums, warp tree, warps in order), so a call is reproducible.
#define SW_THREADS 1024
template <typename T>
__global__ void __launch_bounds__(SW_THREADS) k_sample_walk(const float* logits, int V, const T* feats, int H,
                                                            const int32_t* tokens, const int32_t* parents, int rows,
                                                            int max_depth, float inv_t, const float* uniforms,
                                                            int32_t* out_path, int32_t* out_a, int32_t* out_bonus,
                                                            int32_t* out_new_tokens, T* out_new_features,
                                                            int32_t* out_used, unsigned long long* counters) {
  __shared__ int s_tok[256], s_par[256];
  __shared__ int path[POSS_MAX_DEPTH + 1];
  __shared__ float red[SW_THREADS / 32];
  __shared__ float wsum[SW_THREADS / 32];
  __shared__ int removed[256];             // tokens of the current node's rejected children
  __shared__ float s_m, s_z, s_rem, s_thr;
  __shared__ int s_next, s_nrem, s_used, s_a, s_bonus, s_warp;
  __shared__ float s_before;
  pdl_enter(POSS_K_SAMPLE_WALK);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = threadIdx.x; i < rows; i += SW_THREADS) { s_tok[i] = tokens[i]; s_par[i] = parents[i]; }
  if (threadIdx.x == 0) { path[0] = 0; s_used = 0; }
  __syncthreads();
  int cur = 0, a = 0;
  const int seg = ((V + 31) / 32 + 31) / 32 * 32;      // tokens per warp in the bonus pass: contiguous, a multiple of 32
  while (true) {
    const float* row = logits + (size_t)cur * V;
    // ---- maximum and sum of exp((l - max) / T)
    float m = -INFINITY;
    for (int i = threadIdx.x; i < V; i += SW_THREADS) m = fmaxf(m, __ldcg(row + i));
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) red[warp] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
      float t = red[0];
      for (int w = 1; w < SW_THREADS / 32; ++w) t = fmaxf(t, red[w]);
      s_m = t;
    }
    __syncthreads();
    m = s_m;
    float z = 0.f;
    for (int i = threadIdx.x; i < V; i += SW_THREADS) z += expf((__ldcg(row + i) - m) * inv_t);
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    __syncthreads();                                    // red[] was read by thread 0 above
    if (lane == 0) red[warp] = z;
    __syncthreads();
    // ---- the node's children, in node order (one thread: a handful of tests)
    if (threadIdx.x == 0) {
      float zz = 0.f;
      for (int w = 0; w < SW_THREADS / 32; ++w) zz += red[w];
      float rem = 0.f;
      int nrem = 0, nxt = -1, used = s_used;
      if (a < max_depth) {
        for (int c = 1; c < rows; ++c) {
          if (s_par[c] != cur) continue;
          const int x = s_tok[c];
          const float e = expf((__ldcg(row + x) - m) * inv_t);
          const float left = zz - rem;
          const float u = uniforms[used++];
          if (left > 0.f && u * left < e) { nxt = c; break; }
          rem += e;
          removed[nrem++] = x;
        }
      }
      s_z = zz; s_rem = rem; s_nrem = nrem; s_next = nxt; s_used = used;
      if (nxt >= 0) path[a + 1] = nxt;
    }
    __syncthreads();
    if (s_next >= 0) { cur = s_next; ++a; continue; }
    break;
  }
  // ---- bonus token: inverse CDF over what is left of the last node's distribution, in token order
  {
    const float* row = logits + (size_t)cur * V;
    const float m = s_m;
    const int nrem = s_nrem;
    const int lo = warp * seg, hi = min(V, lo + seg);
    float part = 0.f;
    for (int i = lo + lane; i < hi; i += 32) part += expf((__ldcg(row + i) - m) * inv_t);
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if (lane == 0) wsum[warp] = part;
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int k = 0; k < nrem; ++k) wsum[removed[k] / seg] -= expf((__ldcg(row + removed[k]) - m) * inv_t);
      float total = 0.f;
      for (int w = 0; w < SW_THREADS / 32; ++w) { wsum[w] = fmaxf(wsum[w], 0.f); total += wsum[w]; }
      const float thr = uniforms[s_used++] * total;
      // the warp whose segment holds the threshold (the last one with mass if rounding runs past the end)
      float before = 0.f;
      int sel = -1, last = 0;
      for (int w = 0; w < SW_THREADS / 32; ++w) {
        if (wsum[w] > 0.f) last = w;
        if (sel < 0 && before + wsum[w] > thr) sel = w;
        if (sel < 0) before += wsum[w];
      }
      if (sel < 0) { sel = last; before = total - wsum[last]; }
      s_warp = sel; s_before = before; s_thr = thr; s_bonus = -1;
    }
    __syncthreads();
    if (warp == s_warp) {
      float cum = s_before;
      const float thr = s_thr;
      int found = -1, last_pos = -1;
      for (int i0 = lo; i0 < hi && found < 0; i0 += 32) {
        const int i = i0 + lane;
        float e = 0.f;
        if (i < hi) {
          e = expf((__ldcg(row + i) - m) * inv_t);
          for (int k = 0; k < nrem; ++k) if (removed[k] == i) e = 0.f;
        }
        float incl = e;
        for (int o = 1; o < 32; o <<= 1) {
          float v = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += v;
        }
        const unsigned hit = __ballot_sync(0xffffffffu, e > 0.f && cum + incl > thr);
        const unsigned pos = __ballot_sync(0xffffffffu, e > 0.f);
        if (pos) last_pos = i0 + 31 - __clz(pos);
        if (hit) found = i0 + __ffs(hit) - 1;
        cum += __shfl_sync(0xffffffffu, incl, 31);
      }
      if (lane == 0) s_bonus = found >= 0 ? found : last_pos;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    s_a = a;
    out_a[0] = a;
    out_bonus[0] = s_bonus;
    out_used[0] = s_used;
    atomicAdd(&counters[0], 1ull);
    for (int i = 1; i <= a; ++i) atomicAdd(&counters[i], 1ull);
  }
  for (int i = threadIdx.x; i <= POSS_MAX_DEPTH; i += SW_THREADS) out_path[i] = i <= a ? path[i] : -1;
  for (int k = threadIdx.x; k <= a; k += SW_THREADS) out_new_tokens[k] = k < a ? s_tok[path[k + 1]] : s_bonus;
  for (int i = threadIdx.x; i < (a + 1) * H; i += SW_THREADS) {
    int k = i / H, e = i % H;
    out_new_features[(size_t)k * H + e] = feats[(size_t)path[k] * H + e];
  }
}
template <typename T>
void launch_sample_walk(Launcher& L, const float* logits, int V, const T* feats, int H, const int32_t* tokens,
                        const int32_t* parents, int rows, int max_depth, float temperature, const float* uniforms,
                        int32_t* out_path, int32_t* out_a, int32_t* out_bonus, int32_t* out_new_tokens,
                        T* out_new_features, int32_t* out_used, unsigned long long* counters) {
  launch_pdl(L, k_sample_walk<T>, dim3(1), dim3(SW_THREADS), 0, logits, V, feats, H, tokens, parents, rows, max_depth,
             1.0f / temperature, uniforms, out_path, out_a, out_bonus, out_new_tokens, out_new_features, out_used,
             counters);
}
template void launch_sample_walk<float>(Launcher&, const float*, int, const float*, int, const int32_t*, const int32_t*,
                                        int, int, float, const float*, int32_t*, int32_t*, int32_t*, int32_t*, float*,
                                        int32_t*, unsigned long long*);
template void launch_sample_walk<bf16>(Launcher&, const float*, int, const bf16*, int, const int32_t*, const int32_t*,
                                       int, int, float, const float*, int32_t*, int32_t*, int32_t*, int32_t*, bf16*,
                                       int32_t*, unsigned long long*);

// ------------------------------------------------------------------ cache compaction after acceptance
// Block (layer*2 + kv, head): copies slot prefix_len + path[k] to prefix_len + k for k = 1..a in
// ascending k.  path[k] >= k, so a source is never overwritten before it is read.
template <typename T>
__global__ void __launch_bounds__(128) k_kv_compact(T* kv, int Hkv, int cap, int d, int prefix_len,
                                                    const int32_t* path,
                                                    const int32_t* n_accepted) {
  pdl_enter(POSS_K_KV_COMPACT);
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
  launch_pdl(L, k_kv_compact<T>, grid, dim3(128), 0, target_kv, Hkv, cap, d, prefix_len, path, n_accepted);
}
template void launch_kv_compact<float>(Launcher&, float*, int, int, int, int, int, const int32_t*, const int32_t*);
template void launch_kv_compact<bf16>(Launcher&, bf16*, int, int, int, int, int, const int32_t*, const int32_t*);
