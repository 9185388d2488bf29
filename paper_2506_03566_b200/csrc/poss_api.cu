// Host side of the PosS library: context, workspace layout, argument checks and the launch chains
// of a draft round, the target pass and verification.  No device memory is allocated here; every
// buffer is carved out of the caller's workspace.
#include "poss_internal.cuh"
#include "gemm_tc.cuh"
#include <new>
#include <stdlib.h>
#include <string.h>
#include <math.h>

namespace {

constexpr int R = POSS_MAX_ROWS;
constexpr int KMAX = POSS_MAX_TOPK;
constexpr int ATTN_MAX_SPLITS = 48;     // sizes the attention partials: 47 units of 256 keys on the tcgen05 kernel

struct Bump {
  size_t off = 0;
  char* base = nullptr;
  template <typename P> P* take(size_t count, size_t elem) {
    size_t bytes = (count * elem + 255) / 256 * 256;
    P* p = base ? reinterpret_cast<P*>(base + off) : nullptr;
    off += bytes;
    return p;
  }
};

struct Buffers {
  void* X;            // [R][2H] act
  float* h0;          // [R][H]
  void* xn;           // [R][H] act
  float* qkv;         // [R][(Hq+2Hkv)d]
  float* ptmp;        // [R][max(H, (Hq+2Hkv)d)] product of a GEMM that did not leave split-K partials
  void* q;            // [R][Hq d] act
  float* attn_part;
  size_t attn_part_floats;
  int* attn_arrivals;    // arrival counters of the tcgen05 attention (several clusters per KV head), zero between launches
  void* o;            // [R][Hq d] act
  float* h1;          // [R][H]
  void* u;            // [R][H] act
  float* gu;          // [R][2F]
  void* act;          // [R][F] act
  float* fout;        // [Lmax][KMAX][H] fp32 specialist features per level
  void* fb;           // same, act dtype (layer input of the children, LM-head operand)
  float* hx;          // [R][H] target residual stream
  float* tfeat;       // [R][H] target features fp32
  float* logits;      // [R][V]
  float* pmax; float* psum; float* pval; int32_t* pidx;   // top-k partials
  int32_t* top_ids;   // [R][KMAX]
  float* top_logp;    // [R][KMAX]
  uint64_t* chain_mask;  // [R][2]
  int32_t* chain_depth;  // [R]
  int32_t* argmax_tmp;   // [R]
  unsigned long long* counters;  // [POSS_MAX_DEPTH + 2]
  int32_t* status;       // [1]
  int* merge_done;       // [1] block counter of the top-k merge kernel
  double* rope_inv;      // [head_dim / 2] inverse rotary frequencies
  void* tc_scratch;      // split-K partials + tile counters of the tensor-core GEMM
  unsigned long long* timeline;   // records of the timeline mode: header + (kernel id, time) rows
  TreeState ts;
};

}  // namespace

struct poss_ctx {
  poss_config cfg;
  poss_layer_w* spec;
  poss_layer_w* tgt;
  const void *embed, *lm_head, *final_norm;
  Buffers b;
  size_t esize;          // bytes of the context dtype
  int n_chunks;          // vocabulary chunks of the top-k kernels
  int n_cand_max;
  int max_batch;         // sequences a batched draft round may hold
  int level_rows;        // rows per level of fout / fb: max_batch * POSS_MAX_TOPK
  int64_t launches;
  int last_depth, last_topk, last_nodes, last_batch;
  TcGemmPlanCache* tc;
  bool attn_tc;          // tree attention on the tcgen05 kernel where it covers the call
  bool swiglu_in_kernel; // gate/up product finished by the GEMM's own SwiGLU epilogue instead of the consumer kernel
  int prof_mode;         // 0 off, 1 = LM-head launches of the draft steps, 2 = every stage kind of the draft steps,
                         // 3 = timeline records written by the kernels themselves
  int prof_n;
  int prof_kind[1024];   // kind of each bracketed launch
  cudaEvent_t* prof_ev;   // 2 * PROF_MAX events, created on first enable
};
constexpr int PROF_MAX = 1024;

namespace {

int n_cand_of(int depth, int topk) { return topk + (depth - 1) * topk * topk; }

bool config_ok(const poss_config* c, int* why) {
  *why = POSS_E_INVALID;
  if (!c) return false;
  if (c->hidden <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->ffn <= 0 || c->vocab <= 0) return false;
  if (c->dtype != POSS_FP32 && c->dtype != POSS_BF16) return false;
  if (c->n_specialists < 1 || c->positions_per_specialist < 1) return false;
  if (c->n_target_layers < 0 || c->draft_kv_slots < 1) return false;
  if (c->n_target_layers > 0 && c->target_kv_slots < 1) return false;
  *why = POSS_E_SHAPE;
  if (c->head_dim != 32 && c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->n_q_heads % c->n_kv_heads) return false;
  int g = c->n_q_heads / c->n_kv_heads;
  if (!(g == 1 || g == 2 || g == 3 || g == 4 || g == 8)) return false;
  if (c->hidden % 8 || c->ffn % 8) return false;
  *why = POSS_E_CAPACITY;
  if (c->max_depth < 1 || c->max_depth > POSS_MAX_DEPTH) return false;
  if (c->max_topk < 1 || c->max_topk > POSS_MAX_TOPK) return false;
  if (c->max_total < 1 || c->max_total > 255) return false;
  if ((c->max_depth - 1) * c->max_topk > 128) return false;   // tree-slot mask is two 64-bit words
  if ((c->max_depth - 1) * c->max_topk + 1 > R) return false;
  if (c->vocab < c->max_topk) return false;
  if (c->max_batch < 0 || c->max_batch > POSS_MAX_BATCH) return false;
  *why = POSS_OK;
  return true;
}

void layout(const poss_config& c, Bump& bp, Buffers& b, int* n_chunks, int* n_cand_max) {
  size_t es = c.dtype == POSS_BF16 ? 2 : 4;
  size_t H = c.hidden, F = c.ffn, V = c.vocab;
  size_t qd = (size_t)c.n_q_heads * c.head_dim, kd = (size_t)c.n_kv_heads * c.head_dim;
  int L = c.max_depth;
  const size_t NB = c.max_batch > 1 ? c.max_batch : 1;
  *n_chunks = (int)((V + POSS_TOPK_CHUNK - 1) / POSS_TOPK_CHUNK);
  *n_cand_max = n_cand_of(c.max_depth, c.max_topk);
  b.X = bp.take<void>(R * 2 * H, es);
  b.h0 = bp.take<float>(R * H, 4);
  b.xn = bp.take<void>(R * H, es);
  b.qkv = bp.take<float>(R * (qd + 2 * kd), 4);
  b.ptmp = bp.take<float>(R * (H > qd + 2 * kd ? H : qd + 2 * kd), 4);
  b.q = bp.take<void>(R * qd, es);
  b.attn_part_floats = attn_partial_floats(R, c.n_q_heads, c.head_dim, ATTN_MAX_SPLITS);
  b.attn_part = bp.take<float>(b.attn_part_floats, 4);
  b.attn_arrivals = bp.take<int>(tree_attention_tc_arrival_ints(), 4);
  b.o = bp.take<void>(R * qd, es);
  b.h1 = bp.take<float>(R * H, 4);
  b.u = bp.take<void>(R * H, es);
  b.gu = bp.take<float>(R * 2 * F, 4);
  b.act = bp.take<void>(R * F, es);
  b.fout = bp.take<float>((size_t)L * NB * KMAX * H, 4);
  b.fb = bp.take<void>((size_t)L * NB * KMAX * H, es);
  b.hx = bp.take<float>(R * H, 4);
  b.tfeat = bp.take<float>(R * H, 4);
  b.logits = bp.take<float>(R * V, 4);
  size_t n_lists = *n_chunks > TC_MAX_GRID ? *n_chunks : TC_MAX_GRID;   // chunk lists or one list per GEMM CTA
  b.pmax = bp.take<float>((size_t)R * n_lists, 4);
  b.psum = bp.take<float>((size_t)R * n_lists, 4);
  b.pval = bp.take<float>((size_t)R * n_lists * KMAX, 4);
  b.pidx = bp.take<int32_t>((size_t)R * n_lists * KMAX, 4);
  b.top_ids = bp.take<int32_t>(R * KMAX, 4);
  b.top_logp = bp.take<float>(R * KMAX, 4);
  b.chain_mask = bp.take<uint64_t>(R * 2, 8);
  b.chain_depth = bp.take<int32_t>(R, 4);
  b.argmax_tmp = bp.take<int32_t>(R, 4);
  b.counters = bp.take<unsigned long long>(POSS_MAX_DEPTH + 2, 8);
  b.status = bp.take<int32_t>(64, 4);
  b.merge_done = bp.take<int>(64, 4);
  b.rope_inv = bp.take<double>(64, 8);
  b.tc_scratch = bp.take<void>(tc_gemm_scratch_bytes(), 1);
  b.timeline = bp.take<unsigned long long>(poss_trace::HEADER_WORDS + poss_trace::ROW_WORDS * poss_trace::MAX_ROWS, 8);
  // tree state: one block per sequence of a batched round
  b.ts.cand_cap = (*n_cand_max + 3) / 4 * 4;
  b.ts.node_cap = (L + 1) * KMAX;
  b.ts.cand_tok = bp.take<int32_t>(NB * b.ts.cand_cap, 4);
  b.ts.cand_parent = bp.take<int32_t>(NB * b.ts.cand_cap, 4);
  b.ts.cand_score = bp.take<float>(NB * b.ts.cand_cap, 4);
  b.ts.node_tok = bp.take<int32_t>(NB * b.ts.node_cap, 4);
  b.ts.node_prow = bp.take<int32_t>(NB * b.ts.node_cap, 4);
  b.ts.node_cand = bp.take<int32_t>(NB * b.ts.node_cap, 4);
  b.ts.node_score = bp.take<float>(NB * b.ts.node_cap, 4);
  b.ts.node_mask = bp.take<uint64_t>(NB * b.ts.node_cap * 2, 8);
  b.ts.selected = bp.take<int32_t>(NB * 256, 4);
}

inline cudaStream_t S(poss_stream s) { return reinterpret_cast<cudaStream_t>(s); }

// ------------------------------------------------------------------ typed implementation
template <typename T>
struct Impl {
  poss_ctx* c;
  Launcher L;
  Impl(poss_ctx* ctx, poss_stream s) : c(ctx) { L.stream = S(s); L.launches = &ctx->launches; L.err = POSS_OK; }

  // brackets the launches issued between begin and end with two events (profiling only)
  int prof_begin(int kind) {
    if (!c->prof_mode || c->prof_mode == 3 || !in_draft || c->prof_n >= PROF_MAX) return -1;
    if (c->prof_mode == 1 && kind != POSS_PROF_LM_HEAD) return -1;
    int i = c->prof_n++;
    c->prof_kind[i] = kind;
    cudaEventRecord(c->prof_ev[2 * i], L.stream);
    return i;
  }
  void prof_end(int i) { if (i >= 0) cudaEventRecord(c->prof_ev[2 * i + 1], L.stream); }
  bool in_draft = false;

  const T* W(const void* p) const { return reinterpret_cast<const T*>(p); }
  T* A(void* p) const { return reinterpret_cast<T*>(p); }

  // out[M][N] = x . segs^T (+bias) (+residual); picks the tensor-core kernel when it applies
  // out_act (optional, [M][ldo]) receives the same values in the context dtype
  void gemm(const T* x, int ldx, int M, const GemmSegs& segs, int K, const T* bias, const float* residual, int ldr,
            float* out, int ldo, int impl = 0, T* out_act = nullptr, int tag = POSS_K_GEMM_OTHER);
  // x . segs^T handed to a consumer kernel: split-K partials when the tensor-core kernel can leave them,
  // else the plain product in tmp[M][ldo]
  // tag: which product this is (POSS_K_GEMM_*), for the timeline recording
  SplitKView gemm_view(const T* x, int ldx, int M, const GemmSegs& segs, int K, float* tmp, int ldo,
                       int tag = POSS_K_GEMM_OTHER);
  // act[M][F] = T(silu(x . gate^T) * (x . up^T))
  void gemm_swiglu(const T* x, int M, const void* w_gate, const void* w_up, int F, int K, T* act);
  // tree-masked attention: the tcgen05 kernel where it covers the call (bf16, head dimension 128, at most
  // 10240 keys), else the split-KV kernels with their partial buffer
  void attention(const AttnArgs& aa, const T* q, const T* kc, const T* vc, T* out);
  void attention_batch(const AttnArgs& aa, const AttnBatch& ab, const T* q, T* out);
  // per-row max / sum-exp / top-k partial lists of x . lm_head^T without storing the logits; false = not covered
  // logits_out (argmax only, at most 64 rows): the fp32 logits are stored from the same accumulator read
  bool gemm_topk_partials(const T* x, int M, int K, int topk, int* n_lists, bool argmax_only = false,
                          float* logits_out = nullptr);

  // need_logp = false (with K = 1): the caller wants the argmax only; logp is then meaningless
  void lm_head_topk(const T* feats, int rows, int K, int32_t* ids, float* logp, float* logits_out,
                    const ExpandArgs* expand = nullptr, bool need_logp = true) {
    const poss_config& g = c->cfg;
    GemmSegs sg; sg.n = 1; sg.w[0] = c->lm_head; sg.rows[0] = g.vocab;
    float* lg = logits_out ? logits_out : c->b.logits;
    int pr = expand != nullptr ? prof_begin(POSS_PROF_LM_HEAD) : -1;   // the draft steps' launches only
    int n_lists = 0;
    // wanted logits leave the fused path, except where the argmax epilogue can store them on its way
    const bool argmax_only = !need_logp && K == 1;
    const bool store_too = logits_out && argmax_only && rows <= 64;
    bool fused = (!logits_out || store_too) &&
                 gemm_topk_partials(feats, rows, g.hidden, K, &n_lists, argmax_only, store_too ? logits_out : nullptr);
    if (!fused) gemm(feats, g.hidden, rows, sg, g.hidden, nullptr, nullptr, 0, lg, g.vocab, 0, nullptr, POSS_K_GEMM_LM_HEAD);
    prof_end(pr);
    if (!fused) {
      launch_topk_partial(L, lg, rows, g.vocab, K, c->b.pmax, c->b.psum, c->b.pval, c->b.pidx, c->n_chunks);
      n_lists = c->n_chunks;
    }
    launch_topk_merge(L, rows, K, n_lists, c->b.pmax, c->b.psum, c->b.pval, c->b.pidx, ids, logp, &c->b.ts, expand,
                      c->b.merge_done);
  }

  // fc + norm + K/V(+Q) projection + rotary + cache append for one stacked batch of a specialist
  void project_rows(const poss_layer_w& lw, const BatchRows& s, const int32_t* new_tokens, const T* new_features,
                    const CachePtrs& caches, bool with_q) {
    const poss_config& g = c->cfg;
    Buffers& b = c->b;
    int H = g.hidden, qd = g.n_q_heads * g.head_dim, kd = g.n_kv_heads * g.head_dim;
    launch_gather_x<T>(L, s, new_tokens, new_features, b.ts, KMAX, A(b.fb), c->level_rows, W(c->embed), H, A(b.X));
    GemmSegs fc; fc.n = 1; fc.w[0] = lw.fc_w; fc.rows[0] = H;
    int pr = prof_begin(POSS_PROF_FC);
    SplitKView v_fc = gemm_view(A(b.X), 2 * H, s.M, fc, 2 * H, b.ptmp, H, POSS_K_GEMM_FC);
    prof_end(pr);
    launch_reduce_norm<T>(L, v_fc, s.M, H, W(lw.fc_b), nullptr, W(lw.norm_in), g.rms_eps, b.h0, A(b.xn));
    GemmSegs qkv; qkv.n = 3;
    qkv.w[0] = lw.wq; qkv.rows[0] = qd; qkv.w[1] = lw.wk; qkv.rows[1] = kd; qkv.w[2] = lw.wv; qkv.rows[2] = kd;
    pr = prof_begin(POSS_PROF_QKV);
    SplitKView v_qkv = gemm_view(A(b.xn), H, s.M, qkv, H, b.ptmp, qd + 2 * kd, POSS_K_GEMM_QKV);
    prof_end(pr);
    RopeArgs ra;
    ra.inv_freq = b.rope_inv;
    ra.mode = 0; ra.s = s; ra.base = 0; ra.depth = nullptr; ra.rows = s.M; ra.q_rows = with_q ? s.B * s.Mc : 0;
    ra.Hq = g.n_q_heads; ra.Hkv = g.n_kv_heads; ra.d = g.head_dim; ra.cap = g.draft_kv_slots; ra.theta = g.rope_theta;
    launch_rope_append<T>(L, ra, v_qkv, caches, A(b.q));
  }

  // Rows of a cache fill or of draft step `level` for `batch` sequences (first: the step's specialist has not yet
  // cached this round's verified pairs and earlier levels).  level < 0: verified pairs only, no current rows.
  static BatchRows step_rows(int batch, const int* prefix_len, const int* n_new, int K, int level, bool first) {
    BatchRows s;
    memset(&s, 0, sizeof(s));
    s.B = batch; s.K = K; s.cur_level = level < 0 ? 0 : level;
    s.Mc = level < 0 ? 0 : (level == 0 ? 1 : K);
    s.n_lvl = first && level >= 1 ? (level - 1) * K : 0;
    int off = 0, tok = 0;
    for (int b = 0; b < batch; ++b) {
      s.prefix_len[b] = prefix_len[b]; s.n_new[b] = n_new[b];
      // at level 0 the last verified pair is the current row, not a pending one
      s.n_ver[b] = level < 0 ? n_new[b] : (first ? (level == 0 ? n_new[b] - 1 : n_new[b]) : 0);
      s.pend_off[b] = off;
      s.tok_off[b] = tok;
      off += s.n_ver[b] + s.n_lvl;
      tok += n_new[b];
    }
    for (int b = batch; b <= MAXB; ++b) s.pend_off[b] = off;
    s.n_pend = off;
    s.M = off + batch * s.Mc;
    return s;
  }

  // attention output -> O-proj + residual -> MLP + residual; x0 = layer input rows.  The result
  // out = h1 + down(...) is stored in fp32; next_gain != NULL also writes out_act = T(rmsnorm(out) * gain)
  // (the next layer's input norm or the final norm), next_gain == NULL writes out_act = T(out) if given.
  void layer_tail(const poss_layer_w& lw, const float* x0, int rows, float* out, T* out_act = nullptr,
                  const T* next_gain = nullptr) {
    const poss_config& g = c->cfg;
    Buffers& b = c->b;
    int H = g.hidden, qd = g.n_q_heads * g.head_dim, F = g.ffn;
    GemmSegs so; so.n = 1; so.w[0] = lw.wo; so.rows[0] = H;
    int pr = prof_begin(POSS_PROF_O);
    SplitKView v_o = gemm_view(A(b.o), qd, rows, so, qd, b.ptmp, H, POSS_K_GEMM_O);
    prof_end(pr);
    launch_reduce_norm<T>(L, v_o, rows, H, nullptr, x0, W(lw.norm_post), g.rms_eps, b.h1, A(b.u));
    pr = prof_begin(POSS_PROF_GATE_UP);
    gemm_swiglu(A(b.u), rows, lw.w_gate, lw.w_up, F, H, A(b.act));
    prof_end(pr);
    GemmSegs sd; sd.n = 1; sd.w[0] = lw.w_down; sd.rows[0] = H;
    pr = prof_begin(POSS_PROF_DOWN);
    SplitKView v_d = gemm_view(A(b.act), F, rows, sd, F, b.ptmp, H, POSS_K_GEMM_DOWN);
    prof_end(pr);
    if (next_gain) launch_reduce_norm<T>(L, v_d, rows, H, nullptr, b.h1, next_gain, g.rms_eps, out, out_act);
    else launch_splitk_reduce<T>(L, v_d, rows, H, nullptr, b.h1, H, out, H, out_act);
  }

  CachePtrs caches_of(void* const* kvs, int batch, int spec) const {
    const poss_config& g = c->cfg;
    const size_t per_spec = (size_t)2 * g.n_kv_heads * g.draft_kv_slots * g.head_dim;
    CachePtrs cp;
    memset(&cp, 0, sizeof(cp));
    for (int b = 0; b < batch; ++b) {
      T* kc = A(kvs[b]) + (size_t)spec * per_spec;
      cp.k[b] = kc;
      cp.v[b] = kc + per_spec / 2;
    }
    return cp;
  }

  int draft_prefill(void* draft_kv, int start, const int32_t* tokens, const void* features, int n) {
    const poss_config& g = c->cfg;
    void* kvs[1] = {draft_kv};
    for (int s = 0; s < g.n_specialists; ++s) {
      const CachePtrs cp = caches_of(kvs, 1, s);
      for (int off = 0; off < n; off += R) {
        int m = n - off < R ? n - off : R;
        int pl = start + off;
        BatchRows sr = step_rows(1, &pl, &m, 1, -1, true);
        project_rows(c->spec[s], sr, tokens + off, W(features) + (size_t)off * g.hidden, cp, false);
      }
    }
    return L.err;
  }

  // One draft phase for `batch` sequences (batch = 1: poss_draft_round).  Every matrix product runs once over the
  // stacked rows of all sequences; attention runs per sequence on its own cache; the tree state, the expansion and
  // the rerank are per sequence (one block each).
  int draft_round(int batch, void* const* kvs, const int* prefix_len, const int32_t* new_tokens,
                  const void* new_features, const int* n_new, int depth, int K, int total, int32_t* out_tokens,
                  int32_t* out_parents, float* out_scores, int32_t* out_depth, uint64_t* out_mask,
                  int32_t* out_n_nodes) {
    const poss_config& g = c->cfg;
    Buffers& b = c->b;
    int H = g.hidden, n = g.positions_per_specialist, Sn = g.n_specialists;
    bool used[64] = {false};
    int cand_base = 0;
    in_draft = true;
    for (int i = 0; i < depth; ++i) {
      int s = i / n < Sn - 1 ? i / n : Sn - 1;          // specialist ceil((i+1)/n), clamped, 0-based
      bool first = !used[s < 64 ? s : 63];
      used[s < 64 ? s : 63] = true;
      const BatchRows sr = step_rows(batch, prefix_len, n_new, K, i, first);
      const CachePtrs cp = caches_of(kvs, batch, s);
      const poss_layer_w& lw = c->spec[s];
      project_rows(lw, sr, new_tokens, W(new_features), cp, true);
      int pr = prof_begin(POSS_PROF_ATTENTION);
      {
        AttnArgs aa;
        memset(&aa, 0, sizeof(aa));
        aa.rows = sr.Mc; aa.Hq = g.n_q_heads; aa.Hkv = g.n_kv_heads; aa.d = g.head_dim; aa.cap = g.draft_kv_slots;
        aa.n_tree = i * K; aa.mask_words = 2;
        aa.scale = 1.0f / sqrtf((float)g.head_dim);
        AttnBatch ab;
        memset(&ab, 0, sizeof(ab));
        ab.batch = batch;
        for (int bq = 0; bq < batch; ++bq) {
          ab.kc[bq] = reinterpret_cast<const bf16*>(cp.k[bq]);
          ab.vc[bq] = reinterpret_cast<const bf16*>(cp.v[bq]);
          ab.n_all[bq] = prefix_len[bq] + n_new[bq];
          ab.mask[bq] = tree_of(b.ts, bq).node_mask + (size_t)i * KMAX * 2;
        }
        aa.n_all = ab.n_all[0]; aa.mask = ab.mask[0];
        attention_batch(aa, ab, A(b.q), A(b.o));
      }
      prof_end(pr);
      const int Mc_all = batch * sr.Mc;
      float* fo = b.fout + (size_t)i * c->level_rows * H;
      T* fbi = A(b.fb) + (size_t)i * c->level_rows * H;
      layer_tail(lw, b.h0 + (size_t)sr.n_pend * H, Mc_all, fo, fbi);
      ExpandArgs xa;
      xa.enabled = 1; xa.Kmax = KMAX; xa.step = i; xa.Mc = sr.Mc; xa.K = K; xa.cand_base = cand_base;
      xa.last = i == depth - 1; xa.batch = batch;
      lm_head_topk(fbi, Mc_all, K, b.top_ids, b.top_logp, nullptr, &xa);
      cand_base += sr.Mc * K;
    }
    // specialists the round did not reach still cache the verified pairs
    for (int s = 0; s < Sn && s < 64; ++s) {
      if (used[s]) continue;
      const BatchRows sr = step_rows(batch, prefix_len, n_new, K, -1, true);
      project_rows(c->spec[s], sr, new_tokens, W(new_features), caches_of(kvs, batch, s), false);
    }
    RerankBatch rb;
    memset(&rb, 0, sizeof(rb));
    rb.batch = batch;
    for (int bq = 0, tok = 0; bq < batch; ++bq) { tok += n_new[bq]; rb.root_index[bq] = tok - 1; }
    launch_rerank(L, b.ts, cand_base, K, total, rb, new_tokens, out_tokens, out_parents, out_scores, out_depth,
                  out_mask, out_n_nodes);
    c->last_depth = depth; c->last_topk = K; c->last_batch = batch;
    c->last_nodes = 1 + (total < cand_base ? total : cand_base);
    return L.err;
  }

  int tree_attention(const void* q, const void* kv, int kv_slots, int prefix_len, int rows, const uint64_t* mask,
                     float scale, void* out) {
    const poss_config& g = c->cfg;
    AttnArgs aa;
    aa.rows = rows; aa.Hq = g.n_q_heads; aa.Hkv = g.n_kv_heads; aa.d = g.head_dim; aa.cap = kv_slots;
    aa.n_all = prefix_len; aa.n_tree = rows; aa.mask = mask; aa.mask_words = (rows + 63) / 64; aa.scale = scale;
    const T* kc = W(kv);
    const T* vc = kc + (size_t)g.n_kv_heads * kv_slots * g.head_dim;
    attention(aa, W(q), kc, vc, A(out));
    return L.err;
  }

  int target_forward(void* target_kv, int prefix_len, const int32_t* tokens, const int32_t* depth,
                     const uint64_t* mask, int mask_words, int rows, void* out_features, int32_t* out_argmax,
                     float* out_logits) {
    const poss_config& g = c->cfg;
    Buffers& b = c->b;
    int H = g.hidden, qd = g.n_q_heads * g.head_dim, kd = g.n_kv_heads * g.head_dim;
    size_t per_layer = (size_t)2 * g.n_kv_heads * g.target_kv_slots * g.head_dim;
    launch_embed_rows<T>(L, tokens, rows, W(c->embed), H, b.hx);
    launch_rmsnorm<T>(L, b.hx, rows, H, W(c->tgt[0].norm_in), g.rms_eps, A(b.xn));
    for (int li = 0; li < g.n_target_layers; ++li) {
      const poss_layer_w& lw = c->tgt[li];
      T* kc = A(target_kv) + li * per_layer;
      T* vc = kc + per_layer / 2;
      GemmSegs qkv; qkv.n = 3;
      qkv.w[0] = lw.wq; qkv.rows[0] = qd; qkv.w[1] = lw.wk; qkv.rows[1] = kd; qkv.w[2] = lw.wv; qkv.rows[2] = kd;
      SplitKView v_qkv = gemm_view(A(b.xn), H, rows, qkv, H, b.ptmp, qd + 2 * kd, POSS_K_GEMM_QKV);
      RopeArgs ra;
      ra.inv_freq = b.rope_inv;
      ra.mode = 1; ra.base = prefix_len; ra.depth = depth; ra.rows = rows; ra.q_rows = rows;
      ra.Hq = g.n_q_heads; ra.Hkv = g.n_kv_heads; ra.d = g.head_dim; ra.cap = g.target_kv_slots;
      ra.theta = g.rope_theta; memset(&ra.s, 0, sizeof(ra.s));
      CachePtrs cp;
      memset(&cp, 0, sizeof(cp));
      cp.k[0] = kc; cp.v[0] = vc;
      launch_rope_append<T>(L, ra, v_qkv, cp, A(b.q));
      AttnArgs aa;
      aa.rows = rows; aa.Hq = g.n_q_heads; aa.Hkv = g.n_kv_heads; aa.d = g.head_dim; aa.cap = g.target_kv_slots;
      aa.n_all = prefix_len; aa.n_tree = rows; aa.mask = mask; aa.mask_words = mask_words;
      aa.scale = 1.0f / sqrtf((float)g.head_dim);
      attention(aa, A(b.q), kc, vc, A(b.o));
      // the layer's last reduction also applies the norm that follows it: the next layer's input
      // norm, or the final norm (whose output is the feature)
      const bool last = li == g.n_target_layers - 1;
      const T* next_gain = last ? W(c->final_norm) : W(c->tgt[li + 1].norm_in);
      layer_tail(lw, b.hx, rows, b.hx, last ? A(out_features) : A(b.xn), next_gain);
    }
    if (out_argmax || out_logits)
      lm_head_topk(A(out_features), rows, 1, out_argmax ? out_argmax : b.argmax_tmp, b.top_logp, out_logits, nullptr,
                   false);
    return L.err;
  }
};

template <typename T>
void Impl<T>::gemm(const T* x, int ldx, int M, const GemmSegs& segs, int K, const T* bias, const float* residual,
                   int ldr, float* out, int ldo, int impl, T* out_act, int) {
  launch_gemm_simt<T>(L, x, ldx, M, segs, K, bias, residual, ldr, out, ldo);
  if (out_act) launch_cast_rows<T>(L, out, (size_t)M * ldo, out_act);
}
template <>
void Impl<bf16>::gemm(const bf16* x, int ldx, int M, const GemmSegs& segs, int K, const bf16* bias,
                      const float* residual, int ldr, float* out, int ldo, int impl, bf16* out_act, int tag) {
  bool can_tc = tc_gemm_supported(segs, K, ldx, M);
  if (impl == 2 && !can_tc) { L.err = POSS_E_SHAPE; return; }
  if (impl != 1 && can_tc) {
    TcEpilogue ep;
    ep.mode = TC_EPI_STORE; ep.bias = bias; ep.residual = residual; ep.ldr = ldr; ep.out = out; ep.ldo = ldo;
    ep.out_bf = out_act; ep.ldo_bf = ldo; ep.trace_tag = tag;
    launch_gemm_tc(L, c->tc, x, ldx, M, segs, K, ep, c->b.tc_scratch, c->b.status);
  } else {
    launch_gemm_simt<bf16>(L, x, ldx, M, segs, K, bias, residual, ldr, out, ldo);
    if (out_act) launch_cast_rows<bf16>(L, out, (size_t)M * ldo, out_act);
  }
}

template <typename T>
SplitKView Impl<T>::gemm_view(const T* x, int ldx, int M, const GemmSegs& segs, int K, float* tmp, int ldo, int) {
  launch_gemm_simt<T>(L, x, ldx, M, segs, K, nullptr, nullptr, 0, tmp, ldo);
  SplitKView v;
  memset(&v, 0, sizeof(v));
  v.direct = tmp; v.ld = ldo;
  return v;
}
template <>
SplitKView Impl<bf16>::gemm_view(const bf16* x, int ldx, int M, const GemmSegs& segs, int K, float* tmp, int ldo,
                                 int tag) {
  SplitKView v;
  memset(&v, 0, sizeof(v));
  v.direct = tmp; v.ld = ldo;
  if (tc_gemm_supported(segs, K, ldx, M)) {
    TcEpilogue ep;
    ep.mode = TC_EPI_STORE; ep.out = tmp; ep.ldo = ldo; ep.view = &v; ep.trace_tag = tag;
    launch_gemm_tc(L, c->tc, x, ldx, M, segs, K, ep, c->b.tc_scratch, c->b.status);
  } else {
    launch_gemm_simt<bf16>(L, x, ldx, M, segs, K, nullptr, nullptr, 0, tmp, ldo);
  }
  return v;
}

template <typename T>
void Impl<T>::gemm_swiglu(const T* x, int M, const void* w_gate, const void* w_up, int F, int K, T* act) {
  GemmSegs sg; sg.n = 2; sg.w[0] = w_gate; sg.rows[0] = F; sg.w[1] = w_up; sg.rows[1] = F;
  gemm(x, K, M, sg, K, nullptr, nullptr, 0, c->b.gu, 2 * F);
  launch_silu_mul<T>(L, c->b.gu, M, F, act);
}
template <>
void Impl<bf16>::gemm_swiglu(const bf16* x, int M, const void* w_gate, const void* w_up, int F, int K, bf16* act) {
  GemmSegs sg; sg.n = 2; sg.w[0] = w_gate; sg.rows[0] = F; sg.w[1] = w_up; sg.rows[1] = F;
  if (tc_gemm_supported(sg, K, K, M)) {
    TcEpilogue ep;
    ep.mode = TC_EPI_SWIGLU; ep.out_bf = act; ep.ldo_bf = F; ep.trace_tag = POSS_K_GEMM_GATE_UP;
    // The tile segments are left as partials and a consumer kernel spread over all SMs finishes them: the
    // in-kernel finish by the last CTA of each tile is a tail that grows with the row count and, measured, loses
    // even at 10 rows (48.0 vs 46.1 us for the product, 10 us per draft round).  The kernel's own SwiGLU epilogue
    // remains for products whose partials do not fit the scratch.
    SplitKView v;
    if (F % 4 == 0 && !c->swiglu_in_kernel) ep.view = &v;
    launch_gemm_tc(L, c->tc, x, K, M, sg, K, ep, c->b.tc_scratch, c->b.status);
    if (ep.view && v.deferred) launch_splitk_swiglu<bf16>(L, v, M, F, act);
    return;
  }
  gemm(x, K, M, sg, K, nullptr, nullptr, 0, c->b.gu, 2 * F);
  launch_silu_mul<bf16>(L, c->b.gu, M, F, act);
}

template <typename T>
void Impl<T>::attention(const AttnArgs& aa, const T* q, const T* kc, const T* vc, T* out) {
  run_tree_attention<T>(L, aa, ATTN_MAX_SPLITS, q, kc, vc, c->b.attn_part, out);
}
template <>
void Impl<bf16>::attention(const AttnArgs& aa, const bf16* q, const bf16* kc, const bf16* vc, bf16* out) {
  AttnBatch ab;
  memset(&ab, 0, sizeof(ab));
  ab.batch = 1; ab.kc[0] = kc; ab.vc[0] = vc; ab.n_all[0] = aa.n_all; ab.mask[0] = aa.mask;
  if (c->attn_tc && launch_tree_attention_tc(L, c->tc, aa, ab, q, c->b.attn_part, c->b.attn_part_floats,
                                             c->b.attn_arrivals, out, c->b.status))
    return;
  run_tree_attention<bf16>(L, aa, ATTN_MAX_SPLITS, q, kc, vc, c->b.attn_part, out);
}

// the attention of a batched draft step: one launch where the tcgen05 kernel takes it, else sequence by sequence
template <typename T>
void Impl<T>::attention_batch(const AttnArgs& aa, const AttnBatch& ab, const T* q, T* out) {
  const size_t per_seq = (size_t)aa.rows * aa.Hq * aa.d;
  for (int b = 0; b < ab.batch; ++b) {
    AttnArgs ai = aa;
    ai.n_all = ab.n_all[b]; ai.mask = ab.mask[b];
    attention(ai, q + b * per_seq, reinterpret_cast<const T*>(ab.kc[b]), reinterpret_cast<const T*>(ab.vc[b]),
              out + b * per_seq);
  }
}
template <>
void Impl<bf16>::attention_batch(const AttnArgs& aa, const AttnBatch& ab, const bf16* q, bf16* out) {
  if (c->attn_tc && launch_tree_attention_tc(L, c->tc, aa, ab, q, c->b.attn_part, c->b.attn_part_floats,
                                             c->b.attn_arrivals, out, c->b.status))
    return;
  const size_t per_seq = (size_t)aa.rows * aa.Hq * aa.d;
  for (int b = 0; b < ab.batch; ++b) {
    AttnArgs ai = aa;
    ai.n_all = ab.n_all[b]; ai.mask = ab.mask[b];
    run_tree_attention<bf16>(L, ai, ATTN_MAX_SPLITS, q + b * per_seq, ab.kc[b], ab.vc[b], c->b.attn_part, out + b * per_seq);
  }
}

template <typename T>
bool Impl<T>::gemm_topk_partials(const T*, int, int, int, int*, bool, float*) { return false; }
template <>
bool Impl<bf16>::gemm_topk_partials(const bf16* x, int M, int K, int topk, int* n_lists, bool argmax_only,
                                    float* logits_out) {
  GemmSegs sg; sg.n = 1; sg.w[0] = c->lm_head; sg.rows[0] = c->cfg.vocab;
  if (!tc_gemm_supported(sg, K, K, M)) return false;
  TcEpilogue ep;
  ep.mode = TC_EPI_TOPK; ep.topk = topk; ep.argmax_only = argmax_only; ep.trace_tag = POSS_K_GEMM_LM_HEAD;
  ep.out = logits_out; ep.ldo = c->cfg.vocab;
  ep.pmax = c->b.pmax; ep.psum = c->b.psum; ep.pval = c->b.pval; ep.pidx = c->b.pidx; ep.n_lists = n_lists;
  launch_gemm_tc(L, c->tc, x, K, M, sg, K, ep, c->b.tc_scratch, c->b.status);
  return true;
}

}  // namespace

// ------------------------------------------------------------------ timeline recording: per-translation-unit setters
namespace poss_trace {
namespace {
constexpr int MAX_UNITS = 16;
SetFn& setter(int i) { static SetFn fns[MAX_UNITS] = {}; return fns[i]; }
int& n_setters() { static int n = 0; return n; }
}  // namespace
void register_setter(SetFn fn) { if (n_setters() < MAX_UNITS) setter(n_setters()++) = fn; }
bool set_all(unsigned long long* device_buf) {
  bool ok = true;
  for (int i = 0; i < n_setters(); ++i) ok = setter(i)(device_buf) && ok;
  return ok;
}
}  // namespace poss_trace

namespace {

#define DISPATCH(ctx, stream, call)                         \
  ((ctx)->cfg.dtype == POSS_BF16 ? Impl<bf16>(ctx, stream).call : Impl<float>(ctx, stream).call)

}  // namespace

// ====================================================================== C ABI
extern "C" {

size_t poss_workspace_bytes(const poss_config* cfg) {
  int why;
  if (!config_ok(cfg, &why)) return 0;
  Bump bp;
  Buffers b;
  int nc, ncand;
  layout(*cfg, bp, b, &nc, &ncand);
  return bp.off;
}

int poss_init(poss_ctx** out, const poss_config* cfg, const poss_weights* w, void* workspace, size_t workspace_bytes,
              poss_stream stream) {
  if (!out) return POSS_E_INVALID;
  *out = nullptr;
  int why;
  if (!config_ok(cfg, &why)) return why;
  if (!w || !w->embed || !w->lm_head || !w->h_specialist) return POSS_E_INVALID;
  if (cfg->n_target_layers > 0 && (!w->h_target || !w->target_final_norm)) return POSS_E_INVALID;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255)) return POSS_E_WORKSPACE;
  if (workspace_bytes < poss_workspace_bytes(cfg)) return POSS_E_WORKSPACE;
  for (int s = 0; s < cfg->n_specialists; ++s) {
    const poss_layer_w& l = w->h_specialist[s];
    if (!l.fc_w || !l.wq || !l.wk || !l.wv || !l.wo || !l.norm_post || !l.w_gate || !l.w_up || !l.w_down)
      return POSS_E_INVALID;
  }
  for (int s = 0; s < cfg->n_target_layers; ++s) {
    const poss_layer_w& l = w->h_target[s];
    if (!l.wq || !l.wk || !l.wv || !l.wo || !l.norm_post || !l.w_gate || !l.w_up || !l.w_down) return POSS_E_INVALID;
  }
  poss_ctx* c = new (std::nothrow) poss_ctx();
  if (!c) return POSS_E_INVALID;
  c->cfg = *cfg;
  c->spec = (poss_layer_w*)malloc(sizeof(poss_layer_w) * cfg->n_specialists);
  c->tgt = cfg->n_target_layers ? (poss_layer_w*)malloc(sizeof(poss_layer_w) * cfg->n_target_layers) : nullptr;
  memcpy(c->spec, w->h_specialist, sizeof(poss_layer_w) * cfg->n_specialists);
  if (c->tgt) memcpy(c->tgt, w->h_target, sizeof(poss_layer_w) * cfg->n_target_layers);
  c->embed = w->embed; c->lm_head = w->lm_head; c->final_norm = w->target_final_norm;
  c->esize = cfg->dtype == POSS_BF16 ? 2 : 4;
  c->prof_mode = 0; c->prof_n = 0; c->prof_ev = nullptr;
  c->launches = 0; c->last_depth = 0; c->last_topk = 0; c->last_nodes = 0; c->last_batch = 0;
  c->max_batch = cfg->max_batch > 1 ? cfg->max_batch : 1;
  c->level_rows = c->max_batch * KMAX;
  Bump bp;
  bp.base = reinterpret_cast<char*>(workspace);
  layout(*cfg, bp, c->b, &c->n_chunks, &c->n_cand_max);
  c->tc = tc_plan_cache_create();
  c->attn_tc = true;
  c->swiglu_in_kernel = false;
  cudaStream_t st = S(stream);
  bool ok = cudaMemsetAsync(workspace, 0, bp.off, st) == cudaSuccess;
  double inv[64];
  for (int j = 0; j < 64; ++j) inv[j] = pow((double)cfg->rope_theta, -2.0 * j / (double)cfg->head_dim);
  ok = ok && cudaMemcpyAsync(c->b.rope_inv, inv, sizeof(inv), cudaMemcpyHostToDevice, st) == cudaSuccess;
  Launcher L; L.stream = st; L.launches = &c->launches; L.err = POSS_OK;
  launch_chain_mask(L, c->b.chain_mask, c->b.chain_depth, R);
  ok = ok && L.err == POSS_OK && cudaStreamSynchronize(st) == cudaSuccess;
  if (!ok) { poss_destroy(c); return POSS_E_CUDA; }
  *out = c;
  return POSS_OK;
}

int poss_destroy(poss_ctx* c) {
  if (!c) return POSS_E_INVALID;
  if (c->prof_mode == 3) poss_trace::set_all(nullptr);
  tc_plan_cache_destroy(c->tc);
  if (c->prof_ev) {
    for (int i = 0; i < 2 * PROF_MAX; ++i) cudaEventDestroy(c->prof_ev[i]);
    free(c->prof_ev);
  }
  free(c->spec);
  free(c->tgt);
  delete c;
  return POSS_OK;
}

int poss_reset(poss_ctx* c, poss_stream stream) {
  if (!c) return POSS_E_INVALID;
  if (cudaMemsetAsync(c->b.counters, 0, sizeof(unsigned long long) * (POSS_MAX_DEPTH + 2), S(stream)) != cudaSuccess)
    return POSS_E_CUDA;
  if (cudaMemsetAsync(c->b.status, 0, sizeof(int32_t) * 64, S(stream)) != cudaSuccess) return POSS_E_CUDA;
  // what a launch that gave up on a wait may have left behind: arrival counters of the matrix product's tiles
  // and of the top-k merge's blocks (both return to zero by themselves after a launch that ran to its end)
  if (!tc_gemm_clear_counters(c->b.tc_scratch, S(stream))) return POSS_E_CUDA;
  if (cudaMemsetAsync(c->b.merge_done, 0, sizeof(int) * 64, S(stream)) != cudaSuccess) return POSS_E_CUDA;
  if (cudaMemsetAsync(c->b.attn_arrivals, 0, sizeof(int) * tree_attention_tc_arrival_ints(), S(stream)) != cudaSuccess)
    return POSS_E_CUDA;
  return POSS_OK;
}

int poss_draft_prefill(poss_ctx* c, void* draft_kv, int start, const int32_t* tokens, const void* features, int n,
                       poss_stream stream) {
  if (!c || !draft_kv || n < 0 || start < 0) return POSS_E_INVALID;
  if (n == 0) return POSS_OK;
  if (!tokens || !features) return POSS_E_INVALID;
  if (start + n > c->cfg.draft_kv_slots) return POSS_E_CAPACITY;
  return DISPATCH(c, stream, draft_prefill(draft_kv, start, tokens, features, n));
}

namespace {
// host-side checks shared by the single and the batched entry; POSS_OK when the round fits
int check_round(const poss_ctx* c, int batch, const int* prefix_len, const int* n_new, int depth, int topk, int total) {
  const poss_config& g = c->cfg;
  if (batch < 1 || depth < 1 || topk < 1 || total < 1) return POSS_E_INVALID;
  if (batch > c->max_batch || batch > POSS_MAX_BATCH) return POSS_E_CAPACITY;
  if (depth > g.max_depth || topk > g.max_topk || total > g.max_total) return POSS_E_CAPACITY;
  int sum_new = 0;
  for (int b = 0; b < batch; ++b) {
    if (prefix_len[b] < 0 || n_new[b] < 1) return POSS_E_INVALID;
    if (prefix_len[b] + n_new[b] + (depth - 1) * topk > g.draft_kv_slots) return POSS_E_CAPACITY;
    sum_new += n_new[b];
  }
  // the stacked rows of every step must fit one matrix product: at a specialist's first step of the round the
  // verified pairs and all earlier levels ride along as pending rows
  bool used[64] = {false};
  const int n = g.positions_per_specialist, Sn = g.n_specialists;
  for (int i = 0; i < depth; ++i) {
    const int s = i / n < Sn - 1 ? i / n : Sn - 1;
    const bool first = !used[s < 64 ? s : 63];
    used[s < 64 ? s : 63] = true;
    const int cur = batch * (i == 0 ? 1 : topk);
    const int pend = first ? (i == 0 ? sum_new - batch : sum_new + batch * (i - 1) * topk) : 0;
    if (pend + cur > R) return POSS_E_CAPACITY;
  }
  if (sum_new > R) return POSS_E_CAPACITY;       // specialists the round does not reach cache the verified pairs
  return POSS_OK;
}
}  // namespace

int poss_draft_round(poss_ctx* c, void* draft_kv, int prefix_len, const int32_t* new_tokens, const void* new_features,
                     int n_new, int depth, int topk, int total, int32_t* out_tokens, int32_t* out_parents,
                     float* out_scores, int32_t* out_depth, uint64_t* out_mask, int32_t* out_n_nodes,
                     poss_stream stream) {
  if (!c || !draft_kv || !new_tokens || !new_features || !out_tokens || !out_parents || !out_scores || !out_depth ||
      !out_mask || !out_n_nodes)
    return POSS_E_INVALID;
  int rc = check_round(c, 1, &prefix_len, &n_new, depth, topk, total);
  if (rc != POSS_OK) return rc;
  void* kvs[1] = {draft_kv};
  return DISPATCH(c, stream, draft_round(1, kvs, &prefix_len, new_tokens, new_features, &n_new, depth, topk, total,
                                         out_tokens, out_parents, out_scores, out_depth, out_mask, out_n_nodes));
}

int poss_draft_round_batched(poss_ctx* c, int batch, void* const* h_draft_kv, const int* h_prefix_len,
                             const int32_t* new_tokens, const void* new_features, const int* h_n_new, int depth,
                             int topk, int total, int32_t* out_tokens, int32_t* out_parents, float* out_scores,
                             int32_t* out_depth, uint64_t* out_mask, int32_t* out_n_nodes, poss_stream stream) {
  if (!c || !h_draft_kv || !h_prefix_len || !h_n_new || !new_tokens || !new_features || !out_tokens || !out_parents ||
      !out_scores || !out_depth || !out_mask || !out_n_nodes)
    return POSS_E_INVALID;
  if (batch < 1) return POSS_E_INVALID;
  if (batch > POSS_MAX_BATCH) return POSS_E_CAPACITY;
  for (int b = 0; b < batch; ++b)
    if (!h_draft_kv[b]) return POSS_E_INVALID;
  int rc = check_round(c, batch, h_prefix_len, h_n_new, depth, topk, total);
  if (rc != POSS_OK) return rc;
  return DISPATCH(c, stream, draft_round(batch, h_draft_kv, h_prefix_len, new_tokens, new_features, h_n_new, depth, topk,
                                         total, out_tokens, out_parents, out_scores, out_depth, out_mask, out_n_nodes));
}

int poss_draft_trace_seq(poss_ctx* c, int seq, int32_t* cand_tokens, int32_t* cand_parents, float* cand_scores,
                         int32_t* frontier, float* step_features, int32_t* selected, poss_stream stream) {
  if (!c || c->last_depth < 1 || seq < 0 || seq >= c->last_batch) return POSS_E_INVALID;
  cudaStream_t st = S(stream);
  int K = c->last_topk, Ld = c->last_depth, H = c->cfg.hidden;
  size_t nc = n_cand_of(Ld, K);
  const TreeState ts = tree_of(c->b.ts, seq);
  bool ok = true;
  auto cp = [&](void* dst, const void* src, size_t bytes) {
    if (dst && bytes) ok = ok && cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  };
  cp(cand_tokens, ts.cand_tok, nc * 4);
  cp(cand_parents, ts.cand_parent, nc * 4);
  cp(cand_scores, ts.cand_score, nc * 4);
  cp(selected, ts.selected, (size_t)(c->last_nodes - 1) * 4);
  for (int l = 1; l < Ld; ++l) {
    if (frontier) cp(frontier + (size_t)(l - 1) * K, ts.node_cand + (size_t)l * KMAX, (size_t)K * 4);
  }
  for (int l = 0; l < Ld; ++l) {
    // level l holds (l == 0 ? 1 : K) expanded rows per sequence, sequence after sequence
    const size_t mc = l == 0 ? 1 : K;
    if (step_features)
      cp(step_features + (size_t)l * K * H, c->b.fout + ((size_t)l * c->level_rows + (size_t)seq * mc) * H, mc * H * 4);
  }
  return ok ? POSS_OK : POSS_E_CUDA;
}

int poss_draft_trace(poss_ctx* c, int32_t* cand_tokens, int32_t* cand_parents, float* cand_scores, int32_t* frontier,
                     float* step_features, int32_t* selected, poss_stream stream) {
  return poss_draft_trace_seq(c, 0, cand_tokens, cand_parents, cand_scores, frontier, step_features, selected, stream);
}

int poss_tree_attention(poss_ctx* c, const void* q, const void* kv, int kv_slots, int prefix_len, int rows,
                        const uint64_t* anc_mask, float scale, void* out, poss_stream stream) {
  if (!c || !q || !kv || !anc_mask || !out || prefix_len < 0 || rows < 0 || kv_slots < 1) return POSS_E_INVALID;
  // the kernels move keys, values and outputs in 16-byte pieces
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(kv) | reinterpret_cast<uintptr_t>(out)) & 15)
    return POSS_E_INVALID;
  if (((size_t)kv_slots * c->cfg.head_dim * c->esize) & 15) return POSS_E_INVALID;
  if (rows == 0) return POSS_OK;
  if (rows > R) return POSS_E_CAPACITY;
  if (prefix_len + rows > kv_slots) return POSS_E_CAPACITY;
  return DISPATCH(c, stream, tree_attention(q, kv, kv_slots, prefix_len, rows, anc_mask, scale, out));
}

int poss_verify_accept(poss_ctx* c, const void* target_logits, const int32_t* target_argmax,
                       const void* target_features, const int32_t* tokens, const int32_t* parents, int rows,
                       int32_t* out_path, int32_t* out_n_accepted, int32_t* out_bonus, int32_t* out_new_tokens,
                       void* out_new_features, poss_stream stream) {
  if (!c || !target_features || !tokens || !parents || !out_path || !out_n_accepted || !out_bonus ||
      !out_new_tokens || !out_new_features)
    return POSS_E_INVALID;
  if ((target_logits == nullptr) == (target_argmax == nullptr)) return POSS_E_INVALID;
  if (rows < 1) return POSS_E_INVALID;
  if (rows > 256) return POSS_E_CAPACITY;
  Launcher L; L.stream = S(stream); L.launches = &c->launches; L.err = POSS_OK;
  const int32_t* g = target_argmax;
  const poss_config& cf = c->cfg;
  if (target_logits) {
    if (rows > R) return POSS_E_CAPACITY;
    // row argmax over the vocabulary: per-chunk best (ties -> lowest id) read straight from the logits,
    // then the list merge
    int n_lists;
    if (cf.dtype == POSS_BF16)
      n_lists = launch_argmax_partial<bf16>(L, reinterpret_cast<const bf16*>(target_logits), rows, cf.vocab, c->b.pmax,
                                            c->b.psum, c->b.pval, c->b.pidx);
    else
      n_lists = launch_argmax_partial<float>(L, reinterpret_cast<const float*>(target_logits), rows, cf.vocab,
                                             c->b.pmax, c->b.psum, c->b.pval, c->b.pidx);
    launch_topk_merge(L, rows, 1, n_lists, c->b.pmax, c->b.psum, c->b.pval, c->b.pidx, c->b.argmax_tmp, c->b.top_logp);
    g = c->b.argmax_tmp;
  }
  if (cf.dtype == POSS_BF16)
    launch_accept_walk<bf16>(L, g, reinterpret_cast<const bf16*>(target_features), cf.hidden, tokens, parents, rows,
                             POSS_MAX_DEPTH, out_path, out_n_accepted, out_bonus, out_new_tokens,
                             reinterpret_cast<bf16*>(out_new_features), c->b.counters);
  else
    launch_accept_walk<float>(L, g, reinterpret_cast<const float*>(target_features), cf.hidden, tokens, parents, rows,
                              POSS_MAX_DEPTH, out_path, out_n_accepted, out_bonus, out_new_tokens,
                              reinterpret_cast<float*>(out_new_features), c->b.counters);
  return L.err;
}

int poss_verify_sample(poss_ctx* c, const float* target_logits, const void* target_features, const int32_t* tokens,
                       const int32_t* parents, int rows, float temperature, const float* uniforms, int n_uniforms,
                       int32_t* out_path, int32_t* out_n_accepted, int32_t* out_bonus, int32_t* out_new_tokens,
                       void* out_new_features, int32_t* out_uniforms_used, poss_stream stream) {
  if (!c || !target_logits || !target_features || !tokens || !parents || !uniforms || !out_path || !out_n_accepted ||
      !out_bonus || !out_new_tokens || !out_new_features || !out_uniforms_used)
    return POSS_E_INVALID;
  if (rows < 1 || !(temperature > 0.f)) return POSS_E_INVALID;
  if (rows > 256 || n_uniforms < rows) return POSS_E_CAPACITY;
  Launcher L; L.stream = S(stream); L.launches = &c->launches; L.err = POSS_OK;
  const poss_config& cf = c->cfg;
  if (cf.dtype == POSS_BF16)
    launch_sample_walk<bf16>(L, target_logits, cf.vocab, reinterpret_cast<const bf16*>(target_features), cf.hidden,
                             tokens, parents, rows, POSS_MAX_DEPTH, temperature, uniforms, out_path, out_n_accepted,
                             out_bonus, out_new_tokens, reinterpret_cast<bf16*>(out_new_features), out_uniforms_used,
                             c->b.counters);
  else
    launch_sample_walk<float>(L, target_logits, cf.vocab, reinterpret_cast<const float*>(target_features), cf.hidden,
                              tokens, parents, rows, POSS_MAX_DEPTH, temperature, uniforms, out_path, out_n_accepted,
                              out_bonus, out_new_tokens, reinterpret_cast<float*>(out_new_features), out_uniforms_used,
                              c->b.counters);
  return L.err;
}

int poss_target_forward(poss_ctx* c, void* target_kv, int prefix_len, const int32_t* tokens, const int32_t* depth,
                        const uint64_t* anc_mask, int rows, void* out_features, int32_t* out_argmax,
                        float* out_logits, poss_stream stream) {
  if (!c || !target_kv || !tokens || !depth || !anc_mask || !out_features || prefix_len < 0 || rows < 1)
    return POSS_E_INVALID;
  if (c->cfg.n_target_layers < 1) return POSS_E_INVALID;
  if (rows > R) return POSS_E_CAPACITY;
  if (prefix_len + rows > c->cfg.target_kv_slots) return POSS_E_CAPACITY;
  return DISPATCH(c, stream, target_forward(target_kv, prefix_len, tokens, depth, anc_mask, (rows + 63) / 64, rows,
                                            out_features, out_argmax, out_logits));
}

int poss_target_verify(poss_ctx* c, void* target_kv, int prefix_len, const int32_t* tokens, const int32_t* depth,
                       const uint64_t* anc_mask, int rows, void* out_features, int32_t* out_argmax,
                       poss_stream stream) {
  return poss_target_forward(c, target_kv, prefix_len, tokens, depth, anc_mask, rows, out_features, out_argmax,
                             nullptr, stream);
}

int poss_target_prefill(poss_ctx* c, void* target_kv, int start, const int32_t* tokens, int n, void* out_features,
                        int32_t* out_argmax, poss_stream stream) {
  if (!c || !target_kv || !tokens || !out_features || start < 0 || n < 0) return POSS_E_INVALID;
  if (c->cfg.n_target_layers < 1) return POSS_E_INVALID;
  if (start + n > c->cfg.target_kv_slots) return POSS_E_CAPACITY;
  int rc = POSS_OK;
  for (int off = 0; off < n && rc == POSS_OK; off += R) {
    int m = n - off < R ? n - off : R;
    char* of = reinterpret_cast<char*>(out_features) + (size_t)off * c->cfg.hidden * c->esize;
    rc = DISPATCH(c, stream, target_forward(target_kv, start + off, tokens + off, c->b.chain_depth, c->b.chain_mask, 2,
                                            m, of, out_argmax ? out_argmax + off : nullptr, nullptr));
  }
  return rc;
}

int poss_kv_compact(poss_ctx* c, void* target_kv, int prefix_len, const int32_t* path, const int32_t* n_accepted,
                    poss_stream stream) {
  if (!c || !target_kv || !path || !n_accepted || prefix_len < 0) return POSS_E_INVALID;
  if (c->cfg.n_target_layers < 1) return POSS_E_INVALID;
  Launcher L; L.stream = S(stream); L.launches = &c->launches; L.err = POSS_OK;
  const poss_config& g = c->cfg;
  if (g.dtype == POSS_BF16)
    launch_kv_compact<bf16>(L, reinterpret_cast<bf16*>(target_kv), g.n_target_layers, g.n_kv_heads, g.target_kv_slots,
                            g.head_dim, prefix_len, path, n_accepted);
  else
    launch_kv_compact<float>(L, reinterpret_cast<float*>(target_kv), g.n_target_layers, g.n_kv_heads,
                             g.target_kv_slots, g.head_dim, prefix_len, path, n_accepted);
  return L.err;
}

int poss_get_counters(poss_ctx* c, int64_t* h_rounds, int64_t* h_accepted_at, poss_stream stream) {
  if (!c || !h_rounds || !h_accepted_at) return POSS_E_INVALID;
  unsigned long long tmp[POSS_MAX_DEPTH + 2];
  if (cudaMemcpyAsync(tmp, c->b.counters, sizeof(tmp), cudaMemcpyDeviceToHost, S(stream)) != cudaSuccess)
    return POSS_E_CUDA;
  if (cudaStreamSynchronize(S(stream)) != cudaSuccess) return POSS_E_CUDA;
  *h_rounds = (int64_t)tmp[0];
  h_accepted_at[0] = 0;
  for (int i = 1; i <= c->cfg.max_depth; ++i) h_accepted_at[i] = (int64_t)tmp[i];
  return POSS_OK;
}

int poss_last_status(poss_ctx* c, poss_stream stream) {
  if (!c) return POSS_E_INVALID;
  int32_t v = 0;
  if (cudaMemcpyAsync(&v, c->b.status, 4, cudaMemcpyDeviceToHost, S(stream)) != cudaSuccess) return POSS_E_CUDA;
  if (cudaStreamSynchronize(S(stream)) != cudaSuccess) return POSS_E_CUDA;
  return v;
}

int poss_linear(poss_ctx* c, const void* x, int M, const void* w, int N, int K, const void* bias,
                const float* residual, float* out, int impl, poss_stream stream) {
  if (!c || !x || !w || !out || M < 0 || N < 1 || K < 1 || impl < 0 || impl > 2) return POSS_E_INVALID;
  if (M == 0) return POSS_OK;
  if (M > R) return POSS_E_CAPACITY;
  if (K % 8) return POSS_E_SHAPE;
  GemmSegs sg; sg.n = 1; sg.w[0] = w; sg.rows[0] = N;
  if (c->cfg.dtype == POSS_BF16) {
    Impl<bf16> im(c, stream);
    const bf16* xb = reinterpret_cast<const bf16*>(x);
    bool can_tc = tc_gemm_supported(sg, K, K, M);
    if (impl == 2 && !can_tc) return POSS_E_SHAPE;
    if (impl != 1 && can_tc) {
      // the product as the round uses it: split-K partials (or the plain product in `out`) + a reducing consumer
      SplitKView v = im.gemm_view(xb, K, M, sg, K, out, N);
      launch_splitk_reduce<bf16>(im.L, v, M, N, reinterpret_cast<const bf16*>(bias), residual, N, out, N, nullptr);
    } else {
      im.gemm(xb, K, M, sg, K, reinterpret_cast<const bf16*>(bias), residual, N, out, N, 1);
    }
    return im.L.err;
  }
  if (impl == 2) return POSS_E_SHAPE;
  Impl<float> im(c, stream);
  im.gemm(reinterpret_cast<const float*>(x), K, M, sg, K, reinterpret_cast<const float*>(bias), residual, N, out, N,
          impl);
  return im.L.err;
}

int poss_lm_head_topk(poss_ctx* c, const void* features, int rows, int topk, int32_t* out_ids, float* out_logp,
                      float* out_logits, poss_stream stream) {
  if (!c || !features || !out_ids || !out_logp || rows < 0 || topk < 1) return POSS_E_INVALID;
  if (rows == 0) return POSS_OK;
  if (rows > R || topk > POSS_MAX_TOPK || topk > c->cfg.vocab) return POSS_E_CAPACITY;
  if (c->cfg.dtype == POSS_BF16) {
    Impl<bf16> im(c, stream);
    im.lm_head_topk(reinterpret_cast<const bf16*>(features), rows, topk, out_ids, out_logp, out_logits);
    return im.L.err;
  }
  Impl<float> im(c, stream);
  im.lm_head_topk(reinterpret_cast<const float*>(features), rows, topk, out_ids, out_logp, out_logits);
  return im.L.err;
}

int poss_profile(poss_ctx* c, int mode) {
  if (!c || mode < 0 || mode > 3) return POSS_E_INVALID;
  // the kernels' record pointer: the context's buffer in mode 3, nothing otherwise (synchronous host calls)
  if (mode == 3) {
    if (cudaMemset(c->b.timeline, 0, sizeof(unsigned long long) * poss_trace::HEADER_WORDS) != cudaSuccess)
      return POSS_E_CUDA;
    if (!poss_trace::set_all(c->b.timeline)) return POSS_E_CUDA;
  } else if (c->prof_mode == 3) {
    if (!poss_trace::set_all(nullptr)) return POSS_E_CUDA;
  }
  if (mode && mode != 3 && !c->prof_ev) {
    c->prof_ev = (cudaEvent_t*)malloc(sizeof(cudaEvent_t) * 2 * PROF_MAX);
    if (!c->prof_ev) return POSS_E_INVALID;
    for (int i = 0; i < 2 * PROF_MAX; ++i)
      if (cudaEventCreate(&c->prof_ev[i]) != cudaSuccess) return POSS_E_CUDA;
  }
  c->prof_mode = mode;
  c->prof_n = 0;
  return POSS_OK;
}

int poss_profile_read(poss_ctx* c, int* h_launches, float* h_total_ms) {
  if (!c || !h_launches || !h_total_ms) return POSS_E_INVALID;
  for (int k = 0; k < POSS_PROF_KINDS; ++k) { h_launches[k] = 0; h_total_ms[k] = 0.f; }
  if (!c->prof_ev || c->prof_n == 0) return POSS_OK;
  if (cudaEventSynchronize(c->prof_ev[2 * c->prof_n - 1]) != cudaSuccess) return POSS_E_CUDA;
  for (int i = 0; i < c->prof_n; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]) != cudaSuccess) return POSS_E_CUDA;
    h_launches[c->prof_kind[i]] += 1;
    h_total_ms[c->prof_kind[i]] += ms;
  }
  c->prof_n = 0;
  return POSS_OK;
}

int poss_timeline_read(poss_ctx* c, int capacity, int32_t* h_kernel, int64_t* h_time_ns, int* h_count,
                       poss_stream stream) {
  if (!c || !h_kernel || !h_time_ns || !h_count || capacity < 0) return POSS_E_INVALID;
  *h_count = 0;
  cudaStream_t st = S(stream);
  unsigned long long n = 0;
  if (cudaMemcpyAsync(&n, c->b.timeline, sizeof(n), cudaMemcpyDeviceToHost, st) != cudaSuccess) return POSS_E_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return POSS_E_CUDA;
  if (n > (unsigned long long)poss_trace::MAX_ROWS) n = poss_trace::MAX_ROWS;
  if (n > (unsigned long long)capacity) n = capacity;
  if (n) {
    unsigned long long* rows = (unsigned long long*)malloc(sizeof(unsigned long long) * poss_trace::ROW_WORDS * n);
    if (!rows) return POSS_E_INVALID;
    bool ok = cudaMemcpyAsync(rows, c->b.timeline + poss_trace::HEADER_WORDS,
                              sizeof(unsigned long long) * poss_trace::ROW_WORDS * n, cudaMemcpyDeviceToHost,
                              st) == cudaSuccess && cudaStreamSynchronize(st) == cudaSuccess;
    // launches overlap (programmatic dependent launch), so the appends are not strictly in time order
    for (unsigned long long i = 0; ok && i < n; ++i) {
      h_kernel[i] = (int32_t)rows[poss_trace::ROW_WORDS * i];
      h_time_ns[i] = (int64_t)rows[poss_trace::ROW_WORDS * i + 1];
    }
    free(rows);
    if (!ok) return POSS_E_CUDA;
  }
  if (cudaMemsetAsync(c->b.timeline, 0, sizeof(unsigned long long) * poss_trace::HEADER_WORDS, st) != cudaSuccess)
    return POSS_E_CUDA;
  *h_count = (int)n;
  return POSS_OK;
}

int poss_debug_lose_load(poss_ctx* c, int launches) {
  if (!c || launches < 0) return POSS_E_INVALID;
  tc_inject_lost_load(c->tc, launches);
  return POSS_OK;
}

int poss_debug_option(poss_ctx* c, int option, int value) {
  if (!c || (value != 0 && value != 1)) return POSS_E_INVALID;
  if (option == POSS_OPT_ATTENTION_TCGEN05) c->attn_tc = value != 0;
  else if (option == POSS_OPT_SWIGLU_IN_KERNEL) c->swiglu_in_kernel = value != 0;
  else return POSS_E_INVALID;
  return POSS_OK;
}

int poss_attention_plan(int total_keys, int* keys_per_unit, int* n_units) {
  if (!keys_per_unit || !n_units || total_keys < 1) return POSS_E_INVALID;
  int k = 0, n = 0;
  if (!tree_attention_tc_plan(total_keys, &k, &n)) return POSS_E_SHAPE;
  *keys_per_unit = k;
  *n_units = n;
  return POSS_OK;
}

int64_t poss_launch_count(const poss_ctx* c) { return c ? c->launches : 0; }

}  // extern "C"
