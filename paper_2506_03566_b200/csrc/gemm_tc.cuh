// Tensor-core (tcgen05 / TMEM / TMA) skinny GEMM: interface used by the host orchestration.
#pragma once
#include "poss_internal.cuh"

struct TcGemmPlanCache;
TcGemmPlanCache* tc_plan_cache_create();
void tc_plan_cache_destroy(TcGemmPlanCache*);
// test hook: the next `launches` tensor-core launches (products or attention) withhold one tile of their own
// pipeline, so one of their bounded waits runs out
void tc_inject_lost_load(TcGemmPlanCache*, int launches);
// consumes one pending injection (true when this launch has to withhold its tile)
bool tc_take_injection(TcGemmPlanCache*);
size_t tc_gemm_scratch_bytes();
// zeroes the per-tile arrival counters inside the scratch (after a launch that gave up on a wait)
bool tc_gemm_clear_counters(void* scratch, cudaStream_t stream);
// the driver's tensor-map encoder (cuTensorMapEncodeTiled), resolved once; NULL when it cannot be had
void* tc_encode_fn(TcGemmPlanCache*);

// number of SMs of the device the cache was created on (= the persistent grid of the matrix products)
int tc_sm_count(const TcGemmPlanCache*);

// Tree attention on tcgen05 (bf16, head dimension 128, at most 10240 keys).  `part` (part_floats floats) holds one
// partial of 132 floats per (row, head, 256-key unit); `arrivals` (tree_attention_tc_arrival_ints() ints, zero
// between launches, may be NULL) lets more than eight CTAs share one (KV head, query tile).
// Returns false, having launched nothing, when the call is not covered; errors of a launch go to *status.
bool tree_attention_tc_plan(int total_keys, int* keys_per_unit, int* n_units);
size_t tree_attention_tc_arrival_ints();
bool tree_attention_tc_supported(const AttnArgs& a, const void* q, const void* kc, const void* vc, const void* out);
// One launch for `batch` sequences: q / out hold the sequences' rows one after the other (a.rows each), every
// sequence has its own cache, key count a.n_tree + n_all[b] and masks; a.n_all and a.mask are not read.
struct AttnBatch {
  int batch;
  const bf16* kc[MAXB];
  const bf16* vc[MAXB];
  int n_all[MAXB];
  const uint64_t* mask[MAXB];
};
bool launch_tree_attention_tc(Launcher& L, TcGemmPlanCache* cache, const AttnArgs& a, const AttnBatch& ab, const bf16* q,
                              float* part, size_t part_floats, int* arrivals, bf16* out, int32_t* status);

// true when the tensor-core kernel covers this product (bf16, K and leading dimension multiples of 8, ...)
bool tc_gemm_supported(const GemmSegs& segs, int K, int ldx, int M);

constexpr int TC_MAX_GRID = 512;     // upper bound of the persistent grid = of the LM-head partial lists per row

enum { TC_EPI_STORE = 0, TC_EPI_SWIGLU = 1, TC_EPI_TOPK = 2, TC_EPI_PARTIAL = 3 };

// What happens to the accumulators.
//   TC_EPI_STORE : out[m][n] (fp32, may be NULL) = acc + bias[n] + residual[m][n]; out_bf (may be NULL) gets the
//                  same value rounded to bf16.
//   TC_EPI_SWIGLU: segs = {gate, up} with equal row counts F; out_bf[m][f] = bf16(silu(gate_f . x_m) * (up_f . x_m)).
//   TC_EPI_TOPK  : segs = {lm_head}; every CTA leaves, per activation row, the max, the sum of exp(logit - max) and
//                  the topk best (logit, id) pairs of its vocabulary tiles, best first:
//                  pmax/psum [M][n_lists], pval/pidx [M][n_lists][topk]; *n_lists receives the list count.
//   TC_EPI_PARTIAL: nothing is reduced or stored: *view describes the parked partials for the consumer kernel
//                  (see SplitKView).  Only chosen by the launcher when `view` is given and the shape allows it;
//                  otherwise the launcher falls back to TC_EPI_STORE into `out` and *view describes that matrix.
struct TcEpilogue {
  int mode = TC_EPI_STORE;
  const bf16* bias = nullptr;
  const float* residual = nullptr;
  int ldr = 0;
  float* out = nullptr;
  int ldo = 0;
  bf16* out_bf = nullptr;
  int ldo_bf = 0;
  int topk = 0;
  bool argmax_only = false;   // TC_EPI_TOPK with topk == 1 and no use for max / sum-exp: cheaper epilogue, psum = 1
  float* pmax = nullptr;
  float* psum = nullptr;
  float* pval = nullptr;
  int32_t* pidx = nullptr;
  int* n_lists = nullptr;
  SplitKView* view = nullptr;
  int trace_tag = POSS_K_GEMM_OTHER;   // which product this is, for the timeline recording
};

void launch_gemm_tc(Launcher& L, TcGemmPlanCache* cache, const bf16* X, int ldx, int M, const GemmSegs& segs, int K,
                    const TcEpilogue& ep, void* scratch, int32_t* status);
