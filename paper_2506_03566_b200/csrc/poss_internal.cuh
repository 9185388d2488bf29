// Internal declarations shared by the kernels and the host orchestration of the PosS library.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/poss.h"
#include "../../include/poss_debug.h"

typedef __nv_bfloat16 bf16;

// ------------------------------------------------------------------ scalar conversions
template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<bf16>(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

// ------------------------------------------------------------------ row bookkeeping of one draft step
// A draft step over B sequences stacks the rows of all of them into one batch for the matrix products:
//   [ pending rows of sequence 0 | ... | pending rows of sequence B-1 | current rows of sequence 0 | ... ]
// Pending rows of a sequence (keys/values only): n_ver verified pairs, then n_lvl rows of the earlier tree
// levels 1.. (width K each).  Current rows (the whole layer): Mc per sequence -- the root pair (the sequence's
// last verified pair) at level 0, the level's K frontier nodes afterwards.  Mc = 0: a cache fill without
// current rows.
constexpr int MAXB = POSS_MAX_BATCH;
struct BatchRows {
  int B, K, cur_level, Mc, n_lvl;
  int n_pend;             // pending rows of all sequences
  int M;                  // n_pend + B * Mc
  int prefix_len[MAXB], n_new[MAXB];
  int n_ver[MAXB];        // verified pairs among the sequence's pending rows
  int pend_off[MAXB + 1]; // first pending row of each sequence
  int tok_off[MAXB];      // the sequence's verified pairs start here in new_tokens / new_features
};

struct RowRef {
  int seq;
  int level;  // 0 = verified pair
  int j;      // index among the sequence's verified pairs, or node index inside its level
};

__host__ __device__ __forceinline__ RowRef batch_row(const BatchRows& s, int m) {
  RowRef r;
  if (m >= s.n_pend) {
    const int cm = m - s.n_pend;
    r.seq = cm / s.Mc;
    r.level = s.cur_level;
    r.j = s.cur_level == 0 ? s.n_new[r.seq] - 1 : cm - r.seq * s.Mc;
    return r;
  }
  int b = 0;
  while (b + 1 < s.B && m >= s.pend_off[b + 1]) ++b;
  int mm = m - s.pend_off[b];
  r.seq = b;
  if (mm < s.n_ver[b]) { r.level = 0; r.j = mm; return r; }
  mm -= s.n_ver[b];
  r.level = 1 + mm / s.K;
  r.j = mm % s.K;
  return r;
}
// KV slot / rotary position of a row (verified pair j: prefix_len + j; node (level, j): behind them).
__host__ __device__ __forceinline__ int row_slot(const BatchRows& s, RowRef r) {
  return r.level == 0 ? s.prefix_len[r.seq] + r.j : s.prefix_len[r.seq] + s.n_new[r.seq] + (r.level - 1) * s.K + r.j;
}
__host__ __device__ __forceinline__ int row_pos(const BatchRows& s, RowRef r) {
  return r.level == 0 ? s.prefix_len[r.seq] + r.j : s.prefix_len[r.seq] + s.n_new[r.seq] - 1 + r.level;
}
// per-sequence key / value caches of the specialist (or target layer) a launch writes to
struct CachePtrs {
  void* k[MAXB];
  void* v[MAXB];
};

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
  // every array holds one such block per sequence of a batched round, cand_cap / node_cap / 256 elements apart
  int cand_cap, node_cap;
};
// the tree state of sequence b
__host__ __device__ __forceinline__ TreeState tree_of(const TreeState& t, int b) {
  TreeState r = t;
  r.cand_tok += (size_t)b * t.cand_cap; r.cand_parent += (size_t)b * t.cand_cap; r.cand_score += (size_t)b * t.cand_cap;
  r.node_tok += (size_t)b * t.node_cap; r.node_prow += (size_t)b * t.node_cap; r.node_cand += (size_t)b * t.node_cap;
  r.node_score += (size_t)b * t.node_cap; r.node_mask += (size_t)b * t.node_cap * 2;
  r.selected += (size_t)b * 256;
  return r;
}

// ------------------------------------------------------------------ kernel launchers (defined in the .cu files)
struct Launcher {
  cudaStream_t stream;
  int64_t* launches;
  int err;  // sticky poss_status
};

// Programmatic dependent launch.  Every kernel of the library starts with pdl_enter(): it lets the next
// kernel of the stream be scheduled early (that kernel's own pdl_enter, or the GEMM's weight prefetch,
// then overlaps this kernel's tail) and waits until the previous kernel has completed and its writes are
// visible.  Because every kernel waits before it touches memory, completion is transitive along the
// stream and the usual stream-order guarantees hold.  One consequence for the kernels' signatures: a
// kernel is alive while its predecessor still writes, so nothing a predecessor produces may be read
// through the read-only data path.  Pointers to activations, indices and caches therefore carry no
// `const __restrict__` pair (the compiler would turn their loads into non-coherent ones and could hoist
// them above the wait); only weights, which no kernel writes, may.
//
// Timeline recording (poss_profile mode 3).  While it is switched on, thread 0 of block (0,0,0) of every launch
// appends (kernel id, device time at which its wait for the predecessor returned) to a buffer of the context.
// The predecessor grid has completed at that instant, so the difference between two consecutive records is the
// time the earlier kernel held the chain: its span *inside* the chain of dependent launches, overlap with its
// neighbours included.  The buffer pointer is a per-device global of each translation unit (set on the host by
// trace_set_all); when it is NULL, the cost is one predicated load in one thread per launch.
namespace poss_trace {
constexpr int HEADER_WORDS = 8, ROW_WORDS = 2, MAX_ROWS = 8192;
static __device__ unsigned long long* g_buf = nullptr;
typedef bool (*SetFn)(unsigned long long*);
void register_setter(SetFn fn);                      // poss_api.cu: one entry per translation unit with kernels
bool set_all(unsigned long long* device_buf);        // points every translation unit's g_buf at the buffer (or NULL)
// internal linkage on purpose: every translation unit sets its own copy of g_buf
static bool set_local(unsigned long long* p) {
  return cudaMemcpyToSymbol(g_buf, &p, sizeof(p)) == cudaSuccess;
}
}  // namespace poss_trace
// a translation unit that defines kernels places this once at file scope (the type lives in the unit's own
// anonymous namespace, so that each unit registers its own setter)
#define POSS_TRACE_REGISTER()                                                                  \
  namespace {                                                                                  \
  struct PossTraceRegistrar {                                                                  \
    PossTraceRegistrar() { poss_trace::register_setter(&poss_trace::set_local); }              \
  } g_poss_trace_registrar;                                                                    \
  }

__device__ __forceinline__ void pdl_trace(int kernel_id) {
  if (kernel_id >= 0 && threadIdx.x == 0 && (blockIdx.x | blockIdx.y | blockIdx.z) == 0) {
    unsigned long long* buf = poss_trace::g_buf;
    if (buf) {
      unsigned long long t;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
      const unsigned long long i = atomicAdd(buf, 1ull);
      if (i < (unsigned long long)poss_trace::MAX_ROWS) {
        buf[poss_trace::HEADER_WORDS + poss_trace::ROW_WORDS * i] = (unsigned long long)kernel_id;
        buf[poss_trace::HEADER_WORDS + poss_trace::ROW_WORDS * i + 1] = t;
      }
    }
  }
}
// kernel_id: a POSS_K_* value (poss_debug.h); -1 = a second wait inside a kernel whose first one records
__device__ __forceinline__ void pdl_enter(int kernel_id) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  pdl_trace(kernel_id);
}
// The two halves, for kernels with work that needs nothing from a predecessor (index arithmetic on the
// launch parameters, loads of weights): pdl_begin(), that work, pdl_sync(), then everything else.
__device__ __forceinline__ void pdl_begin() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_sync(int kernel_id) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  pdl_trace(kernel_id);
}

// hook for a timeline-recording build; empty in the library
#ifndef POSS_TRACE_POINT
#define POSS_TRACE_POINT(id)
#endif

template <typename... KArgs, typename... Args>
inline void launch_pdl(Launcher& L, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, Args... args) {
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = L.stream;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  ++*L.launches;
  if (cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...) != cudaSuccess) L.err = POSS_E_CUDA;
}

// Per-device "already done" flags for set-up that CUDA keeps per device (a kernel's shared-memory opt-in, a
// cluster shape the device refused): a process may hold contexts on several devices, so the flag is indexed
// by the current device's ordinal.  Devices past the table share its last entry's fate of "never cached".
struct PerDeviceFlags {
  static constexpr int MAX_DEVICES = 64;
  bool done[MAX_DEVICES] = {};
  // the flag of the current device, or NULL when the ordinal cannot be had or does not fit the table
  bool* current() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return nullptr;
    return &done[dev];
  }
};

// ------------------------------------------------------------------ split-K results left for the consumer
// The tensor-core GEMM cuts the (tile, k-block) sequence of a product into one contiguous range per
// CTA.  For products with few tiles it does not reduce the ranges itself: every CTA parks the fp32
// partial of each tile segment it computed (128 weight rows x Npad activation rows) in scratch, and
// the kernel that consumes the product (norm, rotary embedding, plain reduce) adds a tile's partials
// in range order while it loads.  That reduction is spread over all of the consumer's blocks instead of
// running in the last CTA of each tile.  A view with deferred == 0 is a plain fp32 matrix.
//
// Units are k-blocks in (tile, k-block) order; CTA c owns [range_begin(c), range_begin(c + 1)).  A CTA
// numbers the tile segments of its range 0, 1, 2, ... in order (at most `slots` of them) and parks segment
// s in its slot s.  In a SwiGLU product a tile holds 64 gate rows (rows 0..63) and the 64 up rows of the
// same ffn columns (rows 64..127), so a tile covers 64 output columns.
struct SplitKView {
  const float* scratch;   // partial of (cta, slot): scratch + (cta * slots + slot) * Npad * 128, element [m][row in tile]
  const float* direct;    // deferred == 0: the product itself, [M][ld]
  int ld;
  int deferred, Npad, G, kb_total, n_tiles, slots;
  int swiglu;             // tile layout: 0 = 128 output columns, 1 = 64 gate + 64 up rows
  int seg_tiles[3], seg_rows[3];   // tiles / rows of each weight segment (tiles never straddle segments)
  int n_segs;
};

__host__ __device__ __forceinline__ long long splitk_range_begin(long long c, long long groups, int G, int gran) {
  return (c * groups / G) * gran;
}
// the CTA whose range contains unit u
__host__ __device__ __forceinline__ int splitk_cta_of_unit(long long u, long long groups, int G, int gran) {
  long long g = u / gran;                       // group of the unit
  // largest c with floor(c * groups / G) <= g  <=>  c * groups < (g + 1) * G
  long long c = ((g + 1) * G + groups - 1) / groups - 1;
  if (c > G - 1) c = G - 1;
  return (int)c;
}

// Contributors of one tile: CTAs c_first .. c_first + count - 1; the first one's partial sits in its slot
// slot_first (the tile's ordinal among the tiles its range touches), every later one's in slot 0 (their
// ranges begin inside the tile).
struct TileContrib { int c_first, count, slot_first; };
__device__ __forceinline__ TileContrib splitk_tile_contrib(const SplitKView& v, int tile) {
  long long groups = (long long)v.n_tiles * v.kb_total;
  TileContrib t;
  if (groups * v.G < (1ll << 31)) {
    // same arithmetic in 32 bits (the usual case): far cheaper divisions
    unsigned gr = (unsigned)groups, G = (unsigned)v.G, u0 = (unsigned)tile * (unsigned)v.kb_total;
    unsigned cf = ((u0 + 1u) * G + gr - 1u) / gr - 1u;
    unsigned cl = ((u0 + (unsigned)v.kb_total) * G + gr - 1u) / gr - 1u;
    if (cf > G - 1u) cf = G - 1u;
    if (cl > G - 1u) cl = G - 1u;
    t.c_first = (int)cf;
    t.count = (int)(cl - cf) + 1;
    t.slot_first = tile - (int)((cf * gr / G) / (unsigned)v.kb_total);
    return t;
  }
  long long tile_u0 = (long long)tile * v.kb_total;
  t.c_first = splitk_cta_of_unit(tile_u0, groups, v.G, 1);
  int c_last = splitk_cta_of_unit(tile_u0 + v.kb_total - 1, groups, v.G, 1);
  t.count = c_last - t.c_first + 1;
  t.slot_first = tile - (int)(splitk_range_begin(t.c_first, groups, v.G, 1) / v.kb_total);
  return t;
}
// tile and row-in-tile of output column n (columns of the segments are laid side by side)
__device__ __forceinline__ void splitk_locate(const SplitKView& v, int n, int* tile, int* t) {
  if (v.swiglu) { *tile = n >> 6; *t = n & 63; return; }     // gate row; the up row of the same column is t + 64
  int base_tile = 0, nn = n;              // (at most three segments; constant indices keep the view in registers)
  if (v.n_segs > 1 && nn >= v.seg_rows[0]) {
    nn -= v.seg_rows[0]; base_tile += v.seg_tiles[0];
    if (v.n_segs > 2 && nn >= v.seg_rows[1]) { nn -= v.seg_rows[1]; base_tile += v.seg_tiles[1]; }
  }
  *tile = base_tile + nn / 128;
  *t = nn % 128;
}
// Sum of one tile's partials, in range order, for NV 16-byte values that sit at the float offsets off[]
// inside a partial (offset of element [m][t] = m * 128 + t).  The first contributor's loads and those of
// the next three are in flight together; the adds stay in range order.
template <int NV>
__device__ __forceinline__ void splitk_sum(const SplitKView& v, const TileContrib& tc, const int (&off)[NV],
                                           float4 (&acc)[NV]) {
  const size_t part = (size_t)v.Npad * 128, step = (size_t)v.slots * part;
  const float* p = v.scratch + ((size_t)tc.c_first * v.slots + tc.slot_first) * part;
#pragma unroll
  for (int i = 0; i < NV; ++i) acc[i] = __ldcg(reinterpret_cast<const float4*>(p + off[i]));
  p = v.scratch + (size_t)(tc.c_first + 1) * step;          // every later contributor parks in its slot 0
  for (int k = 1; k < tc.count; k += 3, p += 3 * step) {
    const int nb = tc.count - k;
    float4 x0[NV], x1[NV], x2[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) x0[i] = __ldcg(reinterpret_cast<const float4*>(p + off[i]));
    if (nb > 1) {
#pragma unroll
      for (int i = 0; i < NV; ++i) x1[i] = __ldcg(reinterpret_cast<const float4*>(p + step + off[i]));
    }
    if (nb > 2) {
#pragma unroll
      for (int i = 0; i < NV; ++i) x2[i] = __ldcg(reinterpret_cast<const float4*>(p + 2 * step + off[i]));
    }
#pragma unroll
    for (int i = 0; i < NV; ++i) { acc[i].x += x0[i].x; acc[i].y += x0[i].y; acc[i].z += x0[i].z; acc[i].w += x0[i].w; }
    if (nb > 1) {
#pragma unroll
      for (int i = 0; i < NV; ++i) { acc[i].x += x1[i].x; acc[i].y += x1[i].y; acc[i].z += x1[i].z; acc[i].w += x1[i].w; }
    }
    if (nb > 2) {
#pragma unroll
      for (int i = 0; i < NV; ++i) { acc[i].x += x2[i].x; acc[i].y += x2[i].y; acc[i].z += x2[i].z; acc[i].w += x2[i].w; }
    }
  }
}
// four consecutive columns n .. n+3 of row m (n a multiple of 4, so they share a tile); t = n's row in the tile
__device__ __forceinline__ float4 splitk_load4(const SplitKView& v, int m, int n, const TileContrib& tc, int t) {
  if (!v.deferred) return *reinterpret_cast<const float4*>(v.direct + (size_t)m * v.ld + n);
  const int off[1] = {m * 128 + t};
  float4 acc[1];
  splitk_sum<1>(v, tc, off, acc);
  return acc[0];
}
// SiLU as every kernel of the library forms it (the in-kernel SwiGLU epilogue and the consumer kernels must
// agree to the bit: which of them runs depends on the row count)
__device__ __forceinline__ float silu_f(float g) { return g / (1.f + expf(-g)); }

template <typename T>
void launch_gemm_simt(Launcher& L, const T* X, int ldx, int M, const GemmSegs& segs, int K, const T* bias,
                      const float* residual, int ldr, float* out, int ldo);

// fb: the features of the expanded rows, [level][level_rows][H]; the rows of sequence b at level l start at
// b * (l == 0 ? 1 : K)
template <typename T>
void launch_gather_x(Launcher& L, const BatchRows& s, const int32_t* new_tokens, const T* new_features,
                     const TreeState& ts, int Kmax, const T* fb, int level_rows, const T* embed, int H, T* X);
template <typename T>
void launch_embed_rows(Launcher& L, const int32_t* tokens, int rows, const T* embed, int H, float* out);
template <typename T>
void launch_rmsnorm(Launcher& L, const float* x, int rows, int H, const T* gain, float eps, T* out);
template <typename T>
void launch_cast_rows(Launcher& L, const float* x, size_t n, T* out);
template <typename T>
void launch_silu_mul(Launcher& L, const float* gu, int rows, int F, T* out);

struct RopeArgs {
  const double* inv_freq;  // [d/2] theta^(-2j/d), filled at init
  int mode;        // 0 = draft step rows (BatchRows mapping), 1 = target rows (slot = base + r, pos = base + depth[r])
  BatchRows s;
  int base;
  const int32_t* depth;
  int rows, q_rows;  // q is produced for the last q_rows rows
  int Hq, Hkv, d, cap;
  float theta;
};
// caches: per sequence in mode 0, entry 0 in mode 1
template <typename T>
void launch_rope_append(Launcher& L, const RopeArgs& a, const SplitKView& qkv, const CachePtrs& caches, T* qout);
// h[m][n] (fp32) = product + bias[n] + residual[m][n];  xn[m][n] = T(gain[n] * h / rms(h row))  (gain NULL: xn = T(h))
template <typename T>
void launch_reduce_norm(Launcher& L, const SplitKView& prod, int rows, int H, const T* bias, const float* residual,
                        const T* gain, float eps, float* h, T* xn);
// act[m][f] = T(silu(gate_f . x_m) * (up_f . x_m)) from the partials of a SwiGLU product (prod.swiglu == 1)
template <typename T>
void launch_splitk_swiglu(Launcher& L, const SplitKView& prod, int rows, int F, T* act);
// out[m][n] (fp32, may be NULL) = product + bias[n] + residual[m][n]; out_act (may be NULL) the same in T
template <typename T>
void launch_splitk_reduce(Launcher& L, const SplitKView& prod, int rows, int N, const T* bias, const float* residual,
                          int ldr, float* out, int ldo, T* out_act);

struct AttnArgs {
  int rows, Hq, Hkv, d, cap;
  int n_all;              // slots [0, n_all) visible to every row
  int n_tree;             // masked slots n_all .. n_all + n_tree - 1
  const uint64_t* mask;   // [rows][mask_words]
  int mask_words;
  float scale;
  int n_splits, keys_per_split;
  int splits_per_block;   // tensor-core kernel: consecutive splits one block walks (one partial per split all the same)
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
                               int* keys_per_split, int* splits_per_block);
void launch_tree_attention_mma(Launcher& L, const AttnArgs& a, const bf16* q, const bf16* kc, const bf16* vc,
                               float* part, bf16* out);

#define POSS_TOPK_CHUNK 2048
#define POSS_ARGMAX_CHUNK 8192
// per-chunk argmax of fp32 or bf16 logits in the merge kernel's partial format (K = 1); returns the chunk count
template <typename T>
int launch_argmax_partial(Launcher& L, const T* logits, int rows, int V, float* pmax, float* psum, float* pval,
                          int32_t* pidx);
void launch_topk_partial(Launcher& L, const float* logits, int rows, int V, int K, float* pmax, float* psum,
                         float* pval, int32_t* pidx, int n_chunks);
// Tree expansion run by the merge kernel (enabled = 0: merge only).  batch sequences of Mc rows each: rows
// [b * Mc, (b + 1) * Mc) belong to sequence b and expand its tree.
struct ExpandArgs {
  int enabled, Kmax, step, Mc, K, cand_base, last, batch;
};
void launch_topk_merge(Launcher& L, int rows, int K, int n_lists, const float* pmax, const float* psum,
                       const float* pval, const int32_t* pidx, int32_t* out_ids, float* out_logp,
                       const TreeState* ts = nullptr, const ExpandArgs* x = nullptr, int* done = nullptr);

// one block per sequence; root_index[b]: position of sequence b's root token in new_tokens; outputs [batch][total+1]
struct RerankBatch {
  int batch;
  int root_index[MAXB];
};
void launch_rerank(Launcher& L, const TreeState& ts, int n_cand, int K, int total, const RerankBatch& rb,
                   const int32_t* new_tokens, int32_t* out_tokens, int32_t* out_parents, float* out_scores,
                   int32_t* out_depth, uint64_t* out_mask, int32_t* out_n_nodes);
template <typename T>
void launch_sample_walk(Launcher& L, const float* logits, int V, const T* feats, int H, const int32_t* tokens,
                        const int32_t* parents, int rows, int max_depth, float temperature, const float* uniforms,
                        int32_t* out_path, int32_t* out_a, int32_t* out_bonus, int32_t* out_new_tokens,
                        T* out_new_features, int32_t* out_used, unsigned long long* counters);
template <typename T>
void launch_accept_walk(Launcher& L, const int32_t* g, const T* feats, int H, const int32_t* tokens,
                        const int32_t* parents, int rows, int max_depth, int32_t* out_path, int32_t* out_a,
                        int32_t* out_bonus, int32_t* out_new_tokens, T* out_new_features,
                        unsigned long long* counters);
template <typename T>
void launch_kv_compact(Launcher& L, T* target_kv, int layers, int Hkv, int cap, int d, int prefix_len,
                       const int32_t* path, const int32_t* n_accepted);
void launch_chain_mask(Launcher& L, uint64_t* mask, int32_t* depth, int rows);
