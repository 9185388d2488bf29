// Skinny bf16 GEMM on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM, operands
// staged by TMA): a persistent, warp-specialised, stream-K kernel with fused epilogues.
//
// out[m][n] = sum_k X[m][k] * W[n][k]  with M <= 128 activation rows and N large.  The product is
// evaluated "swapped": a tile of 128 weight rows is the MMA's M dimension (TMEM lane = weight row n),
// the activation rows are the MMA's N dimension (TMEM column = row m, padded to a multiple of 16).
// The weights, which are all of the traffic, stream through shared memory exactly once in 16 KB TMA
// boxes [128 rows x 64 k] (128-byte swizzle); the small activation tile rides along from L2.
//
// Work split.  The (tile, k-block) pairs of a product form one linear sequence; a fixed grid of CTAs
// cuts it into equal contiguous ranges ("stream-K"), so every SM streams the same number of bytes
// whatever the shape.  A range may start or end inside a tile.  A CTA that holds only part of a tile's
// K range writes its fp32 partial to scratch and bumps the tile's counter; the CTA that arrives last
// adds the partials in range order (never in arrival order) and runs the epilogue.  No CTA waits for
// another one, the result is deterministic, and a row's value depends on the weight shape and the
// grid only, never on M or on the row's place in the batch.
//
// Roles inside a CTA of 192 threads: warp 0 lane 0 issues TMA into a ring of stages; warp 1 lane 0
// issues the MMAs into one of two TMEM accumulators and releases stages with tcgen05.commit; warps
// 2..5 drain the other accumulator (tcgen05.ld, 32 TMEM lanes per warp) and run the epilogue, so the
// epilogue of one tile overlaps the weight stream of the next.
//
// Epilogues: (0) fp32 store with bias / residual and an optional bf16 copy; (1) SwiGLU: the tile holds
// 64 gate rows and 64 up rows of the same ffn columns and the epilogue writes bf16(silu(g) * u);
// (2) LM head: running max / sum-exp / top-k per activation row over the CTA's vocabulary tiles, one
// partial list per CTA, the logits never reach memory (template variant: argmax only, every lane keeps
// its rows' best in registers; with more than 16 activation rows -- batched rounds -- the LM-head product runs
// un-swapped, activation row = TMEM lane, so that one thread owns one row and keeps its running maximum,
// sum and top-k list without any warp-wide exchange); (3) nothing: every tile segment is parked as an fp32 partial and the
// kernel that consumes the product adds a tile's segments in range order while it loads (no counter, no
// last-arriver tail: that reduction is spread over all of the consumer's blocks).
//
// Programmatic dependent launch: the kernel lets its successor start early and itself prefetches
// weight tiles (which no kernel writes) before it waits for its predecessor's results.
//
// Every wait on an mbarrier is bounded; on expiry the CTA raises POSS_E_TIMEOUT in the status word,
// stops issuing work, drains its own copies (bounded), frees its TMEM and returns.
#include "gemm_tc.cuh"
#include "tc_ptx.cuh"
#include <cuda.h>
#include <unordered_map>
#include <string>
#include <string.h>
#include <stdlib.h>
#include <math.h>

POSS_TRACE_REGISTER()

#define LAUNCH_CHECK(L)                                         \
  do {                                                          \
    ++*(L).launches;                                            \
    if (cudaGetLastError() != cudaSuccess) (L).err = POSS_E_CUDA; \
  } while (0)

namespace {

using namespace tcptx;

constexpr int TILE_N = 128;          // weight rows per tile (UMMA M)
constexpr int TILE_K = 64;           // bf16 elements per k-block = one 128-byte swizzle row
constexpr int W_TILE_BYTES = TILE_N * TILE_K * 2;
constexpr int MAX_STAGES = 12;
constexpr int N_THREADS = 192;
constexpr size_t SCRATCH_PARTIAL_BYTES = 96ull << 20;
constexpr int N_COUNTERS = 8192;
constexpr int XCH_STRIDE = 17;

struct TcArgs {
  int M, Npad, n_stages, mode;
  int n_segs, seg_tiles[3], seg_rows[3], seg_col[3];
  int n_tiles, kb_total, gran, slots, pair_tiles;
  int rows_on_lanes;      // LM-head mode with many rows: activation rows are the MMA's M dimension (TMEM lane = row)
  int inject_lost_load;   // test hook: the producer leaves out the activation tile of its first stage
  int trace_tag;          // kernel id for the timeline recording (POSS_K_GEMM_*)
  const bf16* bias;
  const float* residual;
  int ldr;
  float* out;
  int ldo;
  bf16* out_bf;
  int ldo_bf;
  float* scratch;
  int* counters;
  int32_t* status;
  // LM-head mode
  int topk, V;
  float* pmax; float* psum; float* pval; int32_t* pidx;
};

// barrier among the four epilogue warps only
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// e^x for the running sums of the LM-head lists (x <= 0): one multiply and the hardware's 2^x, whose relative error of
// about 2^-22 is far below what the log-sum-exp of a vocabulary row needs; the library's expf costs several times the
// instructions, and the scan of a CTA's last tile is not hidden behind any copy.
__device__ __forceinline__ float exp_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x * 1.4426950408889634f));
  return y;
}

__device__ __forceinline__ bool better(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

struct Segment {
  int tile, kb_begin, kb_end;
};

// ------------------------------------------------------------------ the kernel
// VARIANT 0: every epilogue but those below; 1: LM-head argmax only (lane-local state in registers); 2: LM-head
// lists with the activation rows on the TMEM lanes (more than 16 rows), one thread per row; 3: LM-head lists for up
// to 16 rows, product swapped like everywhere else, the accumulator tile turned through shared memory and eight
// threads per row.  2 and 3 compute a row's maximum and sum with the same operations in the same order, and the K
// best by (value down, id up) do not depend on how they are found, so a row's lists do not depend on how many rows
// share the launch.  Separate instantiations, so that the registers of one epilogue never cost another.
template <int VARIANT>
__global__ void __launch_bounds__(N_THREADS) k_gemm_tc(const __grid_constant__ CUtensorMap map_x,
                                                       const __grid_constant__ CUtensorMap map_w0,
                                                       const __grid_constant__ CUtensorMap map_w1,
                                                       const __grid_constant__ CUtensorMap map_w2, const TcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * MAX_STAGES + 4];
  __shared__ uint32_t tmem_slot;
  __shared__ int s_abort, s_last, s_epi_ok;

  pdl_begin();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* tiles_ptr = smem_raw + (tiles_base - smem_u32(smem_raw));
  constexpr bool ARGMAX = VARIANT == 1;
  constexpr bool rows_on_lanes = VARIANT == 2;
  constexpr bool row_lists = VARIANT == 2 || VARIANT == 3;       // one thread per activation row keeps its lists
  constexpr int XT_LD = TILE_N + 4;                              // row length of the turned tile (variant 3)
  const uint32_t x_tile_bytes = (uint32_t)a.Npad * 128u;
  const int acc_cols = rows_on_lanes ? TILE_N : a.Npad;     // TMEM columns of one accumulator
  const uint32_t stage_bytes = W_TILE_BYTES + x_tile_bytes;
  const int S = a.n_stages;
  auto w_tile = [&](int s) { return tiles_base + (uint32_t)s * stage_bytes; };
  auto x_tile = [&](int s) { return tiles_base + (uint32_t)s * stage_bytes + W_TILE_BYTES; };
  auto full_bar = [&](int s) { return smem_u32(&bars[s]); };
  auto empty_bar = [&](int s) { return smem_u32(&bars[MAX_STAGES + s]); };
  auto acc_full = [&](int b) { return smem_u32(&bars[2 * MAX_STAGES + b]); };
  auto acc_empty = [&](int b) { return smem_u32(&bars[2 * MAX_STAGES + 2 + b]); };
  // mode-specific scratch (behind the ring and, rows on lanes, the 16 KB the last stage's operand read runs into)
  float* extra = reinterpret_cast<float*>(tiles_ptr + (size_t)S * stage_bytes + (VARIANT == 2 ? W_TILE_BYTES : 0));

  const int G = gridDim.x;
  const long long groups = (long long)a.n_tiles * a.kb_total / a.gran;
  const long long u0 = splitk_range_begin(blockIdx.x, groups, G, a.gran);
  const long long u1 = splitk_range_begin(blockIdx.x + 1, groups, G, a.gran);
  const int n_kb = (int)(u1 - u0);
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < 2 * acc_cols) tmem_cols <<= 1;

  if (threadIdx.x == 0) {
    s_abort = 0;
    s_last = 0;
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    prefetch_tensormap(&map_x);
    prefetch_tensormap(&map_w0);
    if (a.n_segs > 1) prefetch_tensormap(&map_w1);
    if (a.n_segs > 2) prefetch_tensormap(&map_w2);
  }
  if (warp == 1) tmem_alloc(smem_u32(&tmem_slot), tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  volatile int* abort_flag = &s_abort;

  // which weight map / first row a tile starts at
  auto tile_seg = [&](int tile, int* ltile) {
    int seg = 0, lt = tile;
    while (seg < a.n_segs - 1 && lt >= a.seg_tiles[seg]) { lt -= a.seg_tiles[seg]; ++seg; }
    *ltile = lt;
    return seg;
  };

  if (warp == 0) {
    if (lane == 0 && n_kb > 0) {
      // ---------------- TMA producer
      const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();   // weights pass through L2 once
      // position of the next k-block to load, advanced without divisions
      struct Cursor { int tile, kb, seg, lt; };
      auto cursor_at = [&](long long u) {
        Cursor c;
        c.tile = (int)(u / a.kb_total);
        c.kb = (int)(u - (long long)c.tile * a.kb_total);
        c.seg = tile_seg(c.tile, &c.lt);
        return c;
      };
      auto advance = [&](Cursor& c) {
        if (++c.kb == a.kb_total) {
          c.kb = 0;
          ++c.tile;
          if (++c.lt == a.seg_tiles[c.seg] && c.seg < a.n_segs - 1) { c.lt = 0; ++c.seg; }
        }
      };
      auto load_w = [&](const Cursor& c, int s) {
        int kcoord = c.kb * TILE_K;
        if (a.pair_tiles) {          // 64 gate rows + 64 up rows of the same ffn columns
          tma_load_2d(w_tile(s), &map_w0, full_bar(s), kcoord, c.tile * 64, pol_w);
          tma_load_2d(w_tile(s) + W_TILE_BYTES / 2, &map_w1, full_bar(s), kcoord, c.tile * 64, pol_w);
        } else {
          const CUtensorMap* mw = c.seg == 0 ? &map_w0 : (c.seg == 1 ? &map_w1 : &map_w2);
          tma_load_2d(w_tile(s), mw, full_bar(s), kcoord, c.lt * TILE_N, pol_w);
        }
      };
      auto load_x = [&](const Cursor& c, int s) {
        tma_load_2d(x_tile(s), &map_x, full_bar(s), c.kb * TILE_K, 0, pol_x);
      };
      // Weights are never written by a kernel: fill the ring with them before waiting for the
      // predecessor, whose results are the activations.  (Asking L2 for further k-blocks at this point
      // was measured and lost: the extra requests delay the latency-bound kernels in between.)
      const int pre = n_kb < S ? n_kb : S;
      Cursor cw = cursor_at(u0), cx = cw;
      for (int it = 0; it < pre; ++it) {
        mbar_expect_tx(full_bar(it), stage_bytes);
        load_w(cw, it);
        advance(cw);
      }
      pdl_sync(a.trace_tag);
      for (int it = 0; it < pre; ++it) { if (!(a.inject_lost_load && it == 0)) load_x(cx, it); advance(cx); }
      int issued = pre, s = 0;
      uint32_t phase = 0;                     // parity of the "empty" completion that frees stage s next
      for (int it = pre; it < n_kb; ++it) {
        if (!mbar_wait(empty_bar(s), phase, abort_flag)) break;
        mbar_expect_tx(full_bar(s), stage_bytes);
        load_w(cw, s);
        load_x(cw, s);
        advance(cw);
        issued = it + 1;
        if (++s == S) { s = 0; phase ^= 1u; }
      }
      if (*abort_flag) {
        // drain: every copy this thread started must land before the CTA's shared memory goes away
        for (int it = max(0, issued - S); it < issued; ++it) {
          uint32_t bar = full_bar(it % S), par = (uint32_t)((it / S) & 1);
          uint64_t t0 = global_ns();
          while (!mbar_try_wait(bar, par) && global_ns() - t0 < WAIT_LIMIT_NS / 4) __nanosleep(64);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && n_kb > 0) {
      // ---------------- MMA issuer
      const uint32_t idesc = rows_on_lanes ? instr_desc_bf16(128, TILE_N) : instr_desc_bf16(TILE_N, a.Npad);
      bool ok = true;
      int it = 0, seg_i = 0, s = 0;
      uint32_t phase = 0;
      int kb_begin = (int)(u0 % a.kb_total);
      while (it < n_kb && ok) {
        int len = min(a.kb_total - kb_begin, n_kb - it);
        kb_begin = 0;                          // every later segment starts a tile
        int buf = seg_i & 1, use = seg_i >> 1;
        if (use > 0) ok = mbar_wait(acc_empty(buf), (uint32_t)((use - 1) & 1), abort_flag);
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(buf * acc_cols);
        for (int i = 0; i < len && ok; ++i, ++it) {
          ok = mbar_wait(full_bar(s), phase, abort_flag);
          if (!ok) break;
          tc_fence_after();
          // swapped: the weight tile is the M operand.  Rows on lanes: the activation tile is, read as 128 rows:
          // the rows past its Npad loaded ones are whatever shared memory follows (the next stage, or the slack
          // behind the ring) and fill accumulator lanes that no thread reads.
          uint64_t ad = smem_desc_sw128(rows_on_lanes ? x_tile(s) : w_tile(s)),
                   bd = smem_desc_sw128(rows_on_lanes ? w_tile(s) : x_tile(s));
#pragma unroll
          for (int kk = 0; kk < TILE_K / 16; ++kk)      // 16 bf16 = 32 bytes = 2 descriptor address units
            umma_bf16(tmem_d, ad + (uint64_t)(2 * kk), bd + (uint64_t)(2 * kk), idesc, (i > 0 || kk > 0) ? 1u : 0u);
          umma_commit(empty_bar(s));
          if (++s == S) { s = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(acc_full(buf));     // arrives once every MMA of this segment has finished
        ++seg_i;
      }
    }
  } else {
    // ---------------- epilogue warps: TMEM lane = weight row
    pdl_sync(-1);
    const int q = warp & 3;                       // TMEM lane quarter this warp may read
    const int t = q * 32 + lane;                  // row inside the tile
    const int K = a.topk;
    // LM-head lists, rows on lanes (variant 2): this thread owns activation row t; running maximum and sum in
    // registers, an unordered list of the K best (value, id) in shared memory, and in registers the list's worst
    // entry: a candidate enters only if it beats that one (a later equal value carries a higher id and loses)
    float* xt = extra;                                           // variant 3: the turned tile [16][XT_LD]
    float* lists = extra;                                        // variant 2: one list per thread
    float* my_val = lists + (size_t)t * K;
    int* my_idx = reinterpret_cast<int*>(lists + (size_t)TILE_N * K) + (size_t)t * K;
    float r_max = -INFINITY, r_sum = 0.f, worst_v = -INFINITY;
    int worst_pos = 0, worst_i = 0x7fffffff;
    if (VARIANT == 2) {
      for (int i = 0; i < K; ++i) { my_val[i] = -INFINITY; my_idx[i] = 0x7fffffff; }
    }
    // sixteen consecutive logits of this thread's row (the first nv of them exist), vocabulary ids from id0 on
    auto scan16 = [&](float* v, int nv, int id0) {
      float cm = -INFINITY;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        if (j >= nv) v[j] = -INFINITY;
        cm = fmaxf(cm, v[j]);
      }
      if (cm > r_max) {                                          // (never -inf here: a real logit is finite)
        r_sum *= exp_fast(r_max - cm);                               // exp(-inf) = 0 at the first chunk
        r_max = cm;
      }
      float add = 0.f;
#pragma unroll
      for (int j = 0; j < 16; ++j) add += exp_fast(v[j] - r_max);   // exp(-inf) = 0 for the columns past the end
      r_sum += add;
      if (cm > worst_v) {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          if (v[j] > worst_v) {                                  // (columns past the end are -inf and never enter)
            my_val[worst_pos] = v[j];
            my_idx[worst_pos] = id0 + j;
            // the list's new worst entry: lowest value, among equals the highest id
            worst_v = my_val[0]; worst_i = my_idx[0]; worst_pos = 0;
            for (int i = 1; i < K; ++i) {
              const float lv = my_val[i];
              const int li = my_idx[i];
              if (lv < worst_v || (lv == worst_v && li > worst_i)) { worst_v = lv; worst_i = li; worst_pos = i; }
            }
          }
        }
      }
    };
    // Variant 3 has 128 threads for at most 16 rows, and the one-thread scan above is a long chain of dependent
    // instructions: the first tile of a CTA, whose list is still empty, took it 28 us (device timestamps, ten rows),
    // later tiles 7 .. 3 us.  Here eight threads share a row: thread (row, s) holds chunk s (16 logits) of the tile
    // and two entries of the row's list (entry k, best first, sits in thread k & 7, slot k >> 3).  Maximum and sum
    // stay the one-thread recurrence bit for bit: chunk s needs the maximum after chunks 0..s (a prefix maximum over
    // the eight threads), its sum of exponentials is then the same expression, and the eight steps of the recurrence
    // are replayed in order by every thread of the row from the shuffled (maximum, sum) pairs.  The list is kept in
    // order and takes a tile's entrants one per round (at most K rounds, a fraction of a microsecond each, none for
    // a tile without entrants).  The K best by (value down, id up) are a set that does not depend on how it is
    // found, so the lists equal the one-thread scan's.
    const int row3 = t >> 3, sub3 = t & 7;
    float ov[2] = {-INFINITY, -INFINITY};
    int oi[2] = {0x7fffffff, 0x7fffffff};
    auto scan_tile3 = [&](int n0, int n_cols) {
      float c_v[16];
      int c_i[16];
#pragma unroll
      for (int j = 0; j < 16; j += 4) {
        const float4 x4 = *reinterpret_cast<const float4*>(xt + row3 * XT_LD + sub3 * 16 + j);
        c_v[j] = x4.x; c_v[j + 1] = x4.y; c_v[j + 2] = x4.z; c_v[j + 3] = x4.w;
      }
      const int nv = n_cols - sub3 * 16, id0 = n0 + sub3 * 16;
      float cm = -INFINITY;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        if (j >= nv) c_v[j] = -INFINITY;
        c_i[j] = j < nv ? id0 + j : 0x7fffffff;
        cm = fmaxf(cm, c_v[j]);
      }
      float pm = cm;                                             // the row's maximum after this chunk
#pragma unroll
      for (int o = 1; o < 8; o <<= 1) {
        const float y = __shfl_up_sync(0xffffffffu, pm, o, 8);
        if (sub3 >= o) pm = fmaxf(pm, y);
      }
      pm = fmaxf(pm, r_max);
      float add = 0.f;
      if (nv > 0) {
#pragma unroll
        for (int j = 0; j < 16; ++j) add += exp_fast(c_v[j] - pm);
      }
#pragma unroll
      for (int s8 = 0; s8 < 8; ++s8) {
        const float cs = __shfl_sync(0xffffffffu, cm, s8, 8), as = __shfl_sync(0xffffffffu, add, s8, 8);
        if (n_cols > 16 * s8) {
          if (cs > r_max) {
            r_sum *= exp_fast(r_max - cs);
            r_max = cs;
          }
          r_sum += as;
        }
      }
      // The row's K-th entry so far: a logit enters only if it beats it (an equal one carries a higher id and
      // loses).  Entrants are taken best first; entrant number r lands at position (old entries better than it) + r,
      // and a row is done once a position reaches K or nothing is left.  Then every thread rebuilds its two entries:
      // an entrant that landed there, or the old entry that moved up by the entrants before it.
      const float kth = __shfl_sync(0xffffffffu, ((K - 1) >> 3) ? ov[1] : ov[0], (K - 1) & 7, 8);
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if (!(c_v[j] > kth) || row3 >= a.M) { c_v[j] = -INFINITY; c_i[j] = 0x7fffffff; }
      if (!__any_sync(0xffffffffu, cm > kth && row3 < a.M)) return;
      const unsigned row_lanes = 0xffu << (lane & 24);
      unsigned taken = 0;                                        // positions entrants took (the same in a row's threads)
      int placed = 0;
      float ev[2] = {0.f, 0.f};
      int ei[2] = {0, 0};
      bool mine0 = false, mine1 = false;
#pragma unroll 1
      for (int r = 0; r < K; ++r) {
        float wv = c_v[0];
        int wi = c_i[0];
#pragma unroll
        for (int i = 1; i < 16; ++i)
          if (better(c_v[i], c_i[i], wv, wi)) { wv = c_v[i]; wi = c_i[i]; }
#pragma unroll
        for (int x = 4; x > 0; x >>= 1) {
          const float yv = __shfl_xor_sync(0xffffffffu, wv, x, 8);
          const int yi = __shfl_xor_sync(0xffffffffu, wi, x, 8);
          if (better(yv, yi, wv, wi)) { wv = yv; wi = yi; }
        }
        const bool real = wi != 0x7fffffff;
        if (!__any_sync(0xffffffffu, real)) break;
        const unsigned b0 = __ballot_sync(0xffffffffu, better(ov[0], oi[0], wv, wi));
        const unsigned b1 = __ballot_sync(0xffffffffu, better(ov[1], oi[1], wv, wi));
        const int pos = __popc(b0 & row_lanes) + __popc(b1 & row_lanes) + placed;
        if (real && pos < K) {
          taken |= 1u << pos;
          ++placed;
          if (sub3 == (pos & 7)) {
            if (pos >> 3) { ev[1] = wv; ei[1] = wi; mine1 = true; }
            else { ev[0] = wv; ei[0] = wi; mine0 = true; }
          }
#pragma unroll
          for (int i = 0; i < 16; ++i)
            if (c_i[i] == wi) { c_v[i] = -INFINITY; c_i[i] = 0x7fffffff; }   // (ids are distinct)
        } else {
          // nothing further of this row enters
#pragma unroll
          for (int i = 0; i < 16; ++i) { c_v[i] = -INFINITY; c_i[i] = 0x7fffffff; }
        }
      }
#pragma unroll
      for (int sl = 0; sl < 2; ++sl) {
        const int k = sub3 + 8 * sl;
        const int src = k - __popc(taken & ((1u << k) - 1u));    // the old entry that ends at k if no entrant did
        const float f0 = __shfl_sync(0xffffffffu, ov[0], src & 7, 8), f1 = __shfl_sync(0xffffffffu, ov[1], src & 7, 8);
        const int g0 = __shfl_sync(0xffffffffu, oi[0], src & 7, 8), g1 = __shfl_sync(0xffffffffu, oi[1], src & 7, 8);
        const bool mine = sl ? mine1 : mine0;
        if (!mine) {
          ev[sl] = (src >> 3) ? f1 : f0;
          ei[sl] = (src >> 3) ? g1 : g0;
        }
        if (k >= K) { ev[sl] = -INFINITY; ei[sl] = 0x7fffffff; }   // entries past K stay fillers
      }
      ov[0] = ev[0]; ov[1] = ev[1];
      oi[0] = ei[0]; oi[1] = ei[1];
    };
    // argmax mode: every lane keeps, in registers, the best (value, id) of its own rows for each of up to
    // 64 activation rows; the lanes are merged once, after the CTA's last tile
    float abv[ARGMAX ? 4 : 1][16];
    int abi[ARGMAX ? 4 : 1][16];
    if (ARGMAX) {
#pragma unroll
      for (int cc = 0; cc < (ARGMAX ? 4 : 1); ++cc)
#pragma unroll
        for (int j = 0; j < 16; ++j) { abv[cc][j] = -INFINITY; abi[cc][j] = 0x7fffffff; }
    }
    bool ok = true;
    int it = 0, seg_i = 0;
    while (it < n_kb && ok) {
      long long u = u0 + it;
      const int tile = (int)(u / a.kb_total);
      const int kb_begin = (int)(u % a.kb_total);
      const int len = min(a.kb_total - kb_begin, n_kb - it);
      const bool whole = len == a.kb_total;
      const int buf = seg_i & 1, use = seg_i >> 1;
      mbar_wait(acc_full(buf), (uint32_t)(use & 1), abort_flag);
      // one verdict for all four warps (their barriers below must stay matched)
      epi_sync();
      if (threadIdx.x == 64) s_epi_ok = *abort_flag == 0;
      epi_sync();
      ok = s_epi_ok != 0;
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * acc_cols);

      // where this thread's row lands
      int lt, seg = 0, col, n_local;
      bool n_ok;
      if (a.mode == 1) {
        n_local = tile * 64 + (t & 63);
        n_ok = n_local < a.seg_rows[0];
        col = n_local;
        lt = tile;
      } else {
        seg = tile_seg(tile, &lt);
        n_local = lt * TILE_N + t;
        n_ok = n_local < a.seg_rows[seg];
        col = a.seg_col[seg] + n_local;
      }

      // ---- epilogue of one 16-column chunk held in v[]
      auto epilogue_chunk = [&](int c0, float* v) {
        if (a.mode == 0) {
          float bv = (a.bias && n_ok) ? __bfloat162float(a.bias[col]) : 0.f;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            int m = c0 + j;
            if (m < a.M && n_ok) {
              float r = v[j] + bv;
              if (a.residual) r += a.residual[(size_t)m * a.ldr + col];
              if (a.out) a.out[(size_t)m * a.ldo + col] = r;
              if (a.out_bf) a.out_bf[(size_t)m * a.ldo_bf + col] = __float2bfloat16_rn(r);
            }
          }
        } else if (a.mode == 1) {
          float* xch = extra;                     // [64][XCH_STRIDE]
          if (t >= 64) {
#pragma unroll
            for (int j = 0; j < 16; ++j) xch[(t - 64) * XCH_STRIDE + j] = v[j];
          }
          epi_sync();
          if (t < 64) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              int m = c0 + j;
              if (m < a.M && n_ok) {
                float g = v[j], up = xch[t * XCH_STRIDE + j];
                a.out_bf[(size_t)m * a.ldo_bf + col] = __float2bfloat16_rn(silu_f(g) * up);
              }
            }
          }
          epi_sync();
        }
      };

      if (ARGMAX) {
        // (argmax launches always hand out whole tiles)
#pragma unroll
        for (int cc = 0; cc < (ARGMAX ? 4 : 1); ++cc) {
          const int c0 = cc * 16;
          if (c0 < a.Npad && c0 < a.M) {
            float v[16];
            tmem_ld16(taddr + (uint32_t)c0, v);
            if (c0 + 16 >= a.Npad || c0 + 16 >= a.M) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(acc_empty(buf));
            }
            if (n_ok) {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if (v[j] > abv[cc][j]) { abv[cc][j] = v[j]; abi[cc][j] = n_local; }   // rows only grow: ties keep the lower id
              if (a.out) {                                       // the caller also wants the logits: same read
#pragma unroll
                for (int j = 0; j < 16; ++j)
                  if (c0 + j < a.M) a.out[(size_t)(c0 + j) * a.ldo + col] = v[j];
              }
            }
          }
        }
      } else if (rows_on_lanes) {
        // (LM-head launches always hand out whole tiles)  Columns = the tile's vocabulary rows.
        const int n0 = lt * TILE_N;
        const int n_cols = min(TILE_N, a.seg_rows[0] - n0);
        for (int c0 = 0; c0 < TILE_N; c0 += 16) {
          float v[16];
          tmem_ld16(taddr + (uint32_t)c0, v);
          if (c0 + 16 >= TILE_N) {                              // last read of this accumulator: hand it back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(buf));
          }
          if (t < a.M && c0 < n_cols) scan16(v, min(16, n_cols - c0), n0 + c0);
        }
      } else if (VARIANT == 3) {
        // (whole tiles; at most 16 activation rows = one chunk of accumulator columns)  The warps turn the tile
        // through shared memory -- lane = vocabulary row in, thread = activation row out -- and the row's thread
        // scans its 128 logits exactly as above.
        const int n0 = lt * TILE_N;
        const int n_cols = min(TILE_N, a.seg_rows[0] - n0);
        {
          float v[16];
          tmem_ld16(taddr, v);
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(acc_empty(buf));
#pragma unroll
          for (int j = 0; j < 16; ++j) xt[j * XT_LD + t] = v[j];
        }
        epi_sync();
        scan_tile3(n0, n_cols);
        epi_sync();                                              // the next tile overwrites the turned tile
      } else if (whole && a.mode != 3) {
        for (int c0 = 0; c0 < a.Npad && c0 < a.M; c0 += 16) {
          float v[16];
          tmem_ld16(taddr + (uint32_t)c0, v);
          if (c0 + 16 >= a.Npad || c0 + 16 >= a.M) {    // last read of this accumulator: hand it back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(buf));
          }
          epilogue_chunk(c0, v);
        }
      } else {
        // partial K range (or a product whose reduction is left to the consumer): park the fp32 partial;
        // unless deferred, the last arriver of the tile finishes it
        // deferred: segment s of the range goes to slot s; else a range's first segment (0) or its trailing one (1)
        const int slot = a.mode == 3 ? seg_i : ((u == u0) ? 0 : 1);
        const size_t part_elems = (size_t)a.Npad * TILE_N;
        float* part = a.scratch + ((size_t)blockIdx.x * a.slots + slot) * part_elems;
        for (int c0 = 0; c0 < a.Npad && c0 < a.M; c0 += 16) {
          float v[16];
          tmem_ld16(taddr + (uint32_t)c0, v);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            int m = c0 + j;
            if (m < a.M) part[(size_t)m * TILE_N + t] = v[j];
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty(buf));
        if (a.mode == 3) { it += len; ++seg_i; continue; }   // the consumer kernel adds the partials
        const long long tile_u0 = (long long)tile * a.kb_total;
        const int c_first = splitk_cta_of_unit(tile_u0, groups, G, a.gran);
        const int c_last = splitk_cta_of_unit(tile_u0 + a.kb_total - 1, groups, G, a.gran);
        epi_sync();
        if (threadIdx.x == 64) {
          // release: the four warps' partial stores (ordered before this by the barrier) become visible
          // before the count; acquire: the last arriver sees every earlier contributor's partial
          int prev;
          asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(prev) : "l"(&a.counters[tile]) : "memory");
          s_last = prev == (c_last - c_first);
        }
        epi_sync();
        const bool last = s_last != 0;
        epi_sync();                                // s_last is rewritten by the next partial segment
        if (last) {
          for (int c0 = 0; c0 < a.Npad && c0 < a.M; c0 += 16) {
            float v[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = 0.f;
            for (int c = c_first; c <= c_last; c += 2) {
              // contributor c: its range begins inside this tile (slot 0) unless it is the first
              // contributor and began earlier (then this tile is its trailing segment, slot 1)
              const bool two = c + 1 <= c_last;
              long long b0 = splitk_range_begin(c, groups, G, a.gran);
              int s0 = (b0 >= tile_u0) ? 0 : 1;
              const float* p0 = a.scratch + ((size_t)c * 2 + s0) * part_elems + t;
              const float* p1 = a.scratch + ((size_t)(c + 1) * 2) * part_elems + t;   // a later contributor: slot 0
              float x0[16], x1[16];
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                int m = c0 + j;
                x0[j] = m < a.M ? __ldcg(p0 + (size_t)m * TILE_N) : 0.f;
                x1[j] = (two && m < a.M) ? __ldcg(p1 + (size_t)m * TILE_N) : 0.f;
              }
#pragma unroll
              for (int j = 0; j < 16; ++j) { v[j] += x0[j]; if (two) v[j] += x1[j]; }
            }
            epilogue_chunk(c0, v);
          }
          if (threadIdx.x == 64) a.counters[tile] = 0;     // ready for the next launch on this stream
        }
      }
      it += len;
      ++seg_i;
    }

    if (ARGMAX) {
      // ---- merge the 128 lanes' bests per activation row.  The ring is idle now (every stage was consumed
      // before the last accumulator was handed to the epilogue), so it serves as the exchange buffer.
      float* xv = reinterpret_cast<float*>(tiles_ptr);                  // [128][65]
      int* xi = reinterpret_cast<int*>(tiles_ptr) + 128 * 65;           // [128][65]
      epi_sync();
#pragma unroll
      for (int cc = 0; cc < (ARGMAX ? 4 : 1); ++cc)
#pragma unroll
        for (int j = 0; j < 16; ++j) { xv[t * 65 + cc * 16 + j] = abv[cc][j]; xi[t * 65 + cc * 16 + j] = abi[cc][j]; }
      epi_sync();
      // two threads per row, each scans 64 lanes' entries, then the pair is merged with a shuffle
      const int m = t >> 1, half_sel = t & 1;
      float bv = -INFINITY;
      int bi = 0x7fffffff;
      if (m < a.M) {
        for (int l = half_sel * 64; l < half_sel * 64 + 64; ++l) {
          float v = xv[l * 65 + m];
          int i = xi[l * 65 + m];
          if (better(v, i, bv, bi)) { bv = v; bi = i; }
        }
      }
      float ov = __shfl_xor_sync(0xffffffffu, bv, 1);
      int oi = __shfl_xor_sync(0xffffffffu, bi, 1);
      if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
      if (m < a.M && half_sel == 0) {
        size_t o = (size_t)m * gridDim.x + blockIdx.x;
        a.pmax[o] = bv; a.psum[o] = 1.f; a.pval[o] = bv; a.pidx[o] = bi;
      }
    }
    if (VARIANT == 3) {
      // ---- the row's list is already in order: entry k sits in thread k & 7, slot k >> 3
      if (row3 < a.M) {
        const size_t o = (size_t)row3 * gridDim.x + blockIdx.x;
#pragma unroll
        for (int k = 0; k < POSS_MAX_TOPK; ++k) {
          if (k < K && sub3 == (k & 7)) {
            a.pval[o * K + k] = ov[k >> 3];
            a.pidx[o * K + k] = oi[k >> 3];
          }
        }
        if (sub3 == 0) {
          a.pmax[o] = r_max;
          a.psum[o] = r_sum;
        }
      }
    } else if (row_lists) {
      // ---- this thread's list, best first (value down, id up), is the CTA's list of its row
      if (t < a.M) {
        const size_t o = (size_t)t * gridDim.x + blockIdx.x;
        for (int k = 0; k < K; ++k) {
          int best = 0;
          float bv = my_val[0];
          int bi = my_idx[0];
          for (int i = 1; i < K; ++i)
            if (better(my_val[i], my_idx[i], bv, bi)) { bv = my_val[i]; bi = my_idx[i]; best = i; }
          a.pval[o * K + k] = bv;
          a.pidx[o * K + k] = bi;
          my_val[best] = -INFINITY;                              // taken: orders behind every remaining entry
          my_idx[best] = 0x7fffffff;
        }
        a.pmax[o] = r_max;
        a.psum[o] = r_sum;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);
  if (threadIdx.x == 0 && *abort_flag) atomicExch(a.status, (int)POSS_E_TIMEOUT);
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct MapKey {
  const void* p; int rows, cols, ld, box_rows;
  bool operator==(const MapKey& o) const {
    return p == o.p && rows == o.rows && cols == o.cols && ld == o.ld && box_rows == o.box_rows;
  }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    size_t h = reinterpret_cast<size_t>(k.p);
    h = h * 1000003u ^ (size_t)k.rows; h = h * 1000003u ^ (size_t)k.cols;
    h = h * 1000003u ^ (size_t)k.ld; h = h * 1000003u ^ (size_t)k.box_rows;
    return h;
  }
};

}  // namespace

struct TcGemmPlanCache {
  EncodeTiledFn encode = nullptr;
  bool tried = false, attr_set = false;
  int inject = 0;          // launches left whose first activation tile is withheld (wait-expiry test hook)
  int grid = 0, sms = 0;
  std::unordered_map<MapKey, CUtensorMap, MapKeyHash> maps;
};

TcGemmPlanCache* tc_plan_cache_create() {
  TcGemmPlanCache* c = new TcGemmPlanCache();
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (sms < 1) sms = 148;
  // The grid is a property of the device, not of a call: the work split (and with it the order in
  // which a tile's partial sums are added) must not change from call to call.
  c->sms = sms;
  c->grid = sms;                       // one persistent CTA per SM
  if (c->grid > TC_MAX_GRID) c->grid = TC_MAX_GRID;
  return c;
}
void tc_plan_cache_destroy(TcGemmPlanCache* p) { delete p; }
int tc_sm_count(const TcGemmPlanCache* c) { return c->sms; }
void tc_inject_lost_load(TcGemmPlanCache* c, int launches) { c->inject = launches < 0 ? 0 : launches; }
bool tc_take_injection(TcGemmPlanCache* c) {
  if (c->inject <= 0) return false;
  --c->inject;
  return true;
}
size_t tc_gemm_scratch_bytes() { return SCRATCH_PARTIAL_BYTES + N_COUNTERS * sizeof(int); }
// The per-tile arrival counters return to zero by themselves after every launch that ran to its end; a launch
// whose bounded wait ran out may leave some behind.
bool tc_gemm_clear_counters(void* scratch, cudaStream_t stream) {
  return cudaMemsetAsync(reinterpret_cast<char*>(scratch) + SCRATCH_PARTIAL_BYTES, 0, N_COUNTERS * sizeof(int),
                         stream) == cudaSuccess;
}

void* tc_encode_fn(TcGemmPlanCache* c) {
  if (!c->tried) {
    c->tried = true;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      c->encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  return reinterpret_cast<void*>(c->encode);
}

bool tc_gemm_supported(const GemmSegs& segs, int K, int ldx, int M) {
  if (M < 1 || M > 128 || K < 8 || (K % 8) || (ldx % 8)) return false;
  for (int i = 0; i < segs.n; ++i)
    if (reinterpret_cast<uintptr_t>(segs.w[i]) & 15) return false;
  return true;
}

namespace {

bool get_map(TcGemmPlanCache* c, const void* p, int rows, int cols, int ld, int box_rows, bool weights,
             CUtensorMap* out) {
  MapKey key{p, rows, cols, ld, box_rows};
  auto it = c->maps.find(key);
  if (it != c->maps.end()) { *out = it->second; return true; }
  if (!tc_encode_fn(c)) return false;
  cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t gstride[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)TILE_K, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMap m;
  CUresult r = c->encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(p), gdim, gstride, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         weights ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (c->maps.size() > 4096) c->maps.clear();
  c->maps.emplace(key, m);
  *out = m;
  return true;
}

}  // namespace

void launch_gemm_tc(Launcher& L, TcGemmPlanCache* cache, const bf16* X, int ldx, int M, const GemmSegs& segs, int K,
                    const TcEpilogue& ep, void* scratch, int32_t* status) {
  TcArgs a;
  memset(&a, 0, sizeof(a));
  a.M = M;
  a.Npad = (M + 15) / 16 * 16;
  a.mode = ep.mode;
  a.pair_tiles = ep.mode == TC_EPI_SWIGLU ? 1 : 0;
  a.n_segs = segs.n;
  const int tile_rows = ep.mode == TC_EPI_SWIGLU ? 64 : TILE_N;
  int n_tiles = 0, col = 0;
  for (int i = 0; i < segs.n; ++i) {
    a.seg_tiles[i] = (segs.rows[i] + tile_rows - 1) / tile_rows;
    a.seg_rows[i] = segs.rows[i];
    a.seg_col[i] = col;
    col += segs.rows[i];
    n_tiles += a.seg_tiles[i];
  }
  if (ep.mode == TC_EPI_SWIGLU) n_tiles = a.seg_tiles[0];   // one tile = 64 gate + 64 up rows
  a.n_tiles = n_tiles;
  a.kb_total = (K + TILE_K - 1) / TILE_K;
  // Leave the reduction to the consumer when the caller can take a view, groups of four columns never
  // straddle a tile and the parked segments fit the scratch (a CTA parks one segment per tile its range
  // touches).
  a.slots = 2;
  if (ep.view) {
    bool ok4 = true;
    for (int i = 0; i < segs.n; ++i) ok4 = ok4 && (segs.rows[i] % 4 == 0);
    long long units = (long long)n_tiles * a.kb_total;
    int g_eff = (long long)cache->grid < units ? cache->grid : (int)units;
    long long range_max = (units + g_eff - 1) / g_eff;
    int slots = (int)((range_max + a.kb_total - 1) / a.kb_total) + 1;
    size_t need = (size_t)cache->grid * slots * a.Npad * TILE_N * sizeof(float);
    bool defer = (ep.mode == TC_EPI_STORE || ep.mode == TC_EPI_SWIGLU) && ok4 && need <= SCRATCH_PARTIAL_BYTES;
    memset(ep.view, 0, sizeof(*ep.view));
    if (defer) {
      a.mode = TC_EPI_PARTIAL;
      a.slots = slots;
    } else {
      ep.view->deferred = 0;
      ep.view->direct = ep.out;
      ep.view->ld = ep.ldo;
    }
  }
  // whole tiles per CTA for the LM-head epilogues (the argmax state lives in registers and only the whole-tile
  // path feeds it; the top-k lists measured slower with split tiles), and whenever the partial buffers or the
  // tile counters could not hold the split.
  const bool argmax = ep.mode == TC_EPI_TOPK && ep.argmax_only && ep.topk == 1 && a.Npad <= 64;
  size_t part_bytes = (size_t)cache->grid * 2 * a.Npad * TILE_N * sizeof(float);
  bool no_split = argmax || a.mode == TC_EPI_TOPK || part_bytes > SCRATCH_PARTIAL_BYTES ||
                  n_tiles > N_COUNTERS;
  a.gran = no_split ? a.kb_total : 1;
  // never more CTAs than ranges to hand out: every CTA of the grid owns at least one k-block
  long long groups = (long long)n_tiles * a.kb_total / a.gran;
  int G = (long long)cache->grid < groups ? cache->grid : (int)groups;
  // Partials left to the consumer: a grid that is a whole multiple of the tile count gives every tile the
  // same number of equal ranges, none straddling two tiles, so each CTA parks one segment and the
  // consumer adds grid/tiles partials instead of one or two more.
  if (a.mode == TC_EPI_PARTIAL && n_tiles * 2 <= G) {
    int per_tile = G / n_tiles;
    if (per_tile > a.kb_total) per_tile = a.kb_total;
    G = per_tile * n_tiles;
  }
  if (ep.n_lists) *ep.n_lists = G;
  if (a.mode == TC_EPI_PARTIAL) {
    SplitKView* v = ep.view;
    v->deferred = 1;
    v->scratch = reinterpret_cast<const float*>(scratch);
    v->Npad = a.Npad; v->G = G; v->kb_total = a.kb_total; v->n_tiles = n_tiles; v->n_segs = segs.n;
    v->slots = a.slots; v->swiglu = ep.mode == TC_EPI_SWIGLU ? 1 : 0;
    for (int i = 0; i < segs.n; ++i) { v->seg_tiles[i] = a.seg_tiles[i]; v->seg_rows[i] = a.seg_rows[i]; }
  }
  // LM head with lists: one thread per activation row.  More than 16 rows: the rows sit on the TMEM lanes; up to
  // 16: the product stays swapped (an eighth of the tensor work) and the tile is turned through shared memory.
  // Both scan a row's logits in the same order with the same operations.
  const bool lists = ep.mode == TC_EPI_TOPK && !argmax;
  a.rows_on_lanes = lists && a.Npad > 16 ? 1 : 0;
  uint32_t stage_bytes = W_TILE_BYTES + (uint32_t)a.Npad * 128u;
  size_t extra = 0;
  if (ep.mode == TC_EPI_SWIGLU) extra = 64 * XCH_STRIDE * sizeof(float);
  // argmax only (no log-probabilities wanted, at most 64 rows): the lane-local epilogue, no running lists
  if (ep.mode == TC_EPI_TOPK && !argmax)
    extra = a.rows_on_lanes ? (size_t)TILE_N * ep.topk * 8                    // one list per thread
                            : (size_t)16 * (TILE_N + 4) * sizeof(float);       // the turned tile
  // rows on lanes: the activation operand is read as 128 rows from a tile that holds Npad of them; the last
  // stage's read runs up to 16 KB past the ring, into this slack (never written, never used)
  const size_t slack = a.rows_on_lanes ? (size_t)W_TILE_BYTES : 0;
  // Ring size (measured on the c2 round): 170 KB = nine 18 KB stages for up to 16 rows (150 KB: +12 us per draft
  // round, 190: +2, 210: +24), 200 KB = eight 24 KB stages at 64 rows (the target pass; 176 and 220 KB: +18 us
  // per pass)
  const int smem_kb = a.Npad <= 16 ? 170 : 200;
  // (the slack and the lists or the turned tile of the LM-head epilogue come on top: the ring keeps its stages)
  const size_t on_top = lists ? slack + extra : 0;
  int stages = (int)(((size_t)smem_kb * 1024u + on_top - extra - slack - 1024u) / stage_bytes);
  while (stages > 2 && (size_t)stages * stage_bytes + slack + extra + 1024 > 225u * 1024u) --stages;
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  if (stages < 2) stages = 2;
  a.n_stages = stages;
  a.inject_lost_load = tc_take_injection(cache) ? 1 : 0;
  a.trace_tag = ep.trace_tag;
  a.bias = ep.bias; a.residual = ep.residual; a.ldr = ep.ldr; a.out = ep.out; a.ldo = ep.ldo;
  a.out_bf = ep.out_bf; a.ldo_bf = ep.ldo_bf;
  a.scratch = reinterpret_cast<float*>(scratch);
  a.counters = reinterpret_cast<int*>(reinterpret_cast<char*>(scratch) + SCRATCH_PARTIAL_BYTES);
  a.status = status;
  a.topk = ep.topk; a.V = segs.rows[0];
  a.pmax = ep.pmax; a.psum = ep.psum; a.pval = ep.pval; a.pidx = ep.pidx;

  CUtensorMap mx, mw[3];
  if (!get_map(cache, X, M, K, ldx, a.Npad, false, &mx)) { L.err = POSS_E_CUDA; return; }
  for (int i = 0; i < 3; ++i) {
    int j = i < segs.n ? i : 0;
    if (!get_map(cache, segs.w[j], segs.rows[j], K, K, tile_rows, true, &mw[i])) { L.err = POSS_E_CUDA; return; }
  }
  size_t smem = (size_t)stages * stage_bytes + slack + extra + 1024;
  if (!cache->attr_set) {
    if (cudaFuncSetAttribute(k_gemm_tc<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(k_gemm_tc<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(k_gemm_tc<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(k_gemm_tc<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024) != cudaSuccess) {
      L.err = POSS_E_CUDA;
      return;
    }
    cache->attr_set = true;
  }
  if (argmax && (size_t)stages * stage_bytes < (size_t)128 * 65 * 8) { L.err = POSS_E_SHAPE; return; }   // exchange buffer
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(G);
  cfg.blockDim = dim3(N_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = L.stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  cudaError_t le = argmax ? cudaLaunchKernelEx(&cfg, k_gemm_tc<1>, mx, mw[0], mw[1], mw[2], a)
                   : a.rows_on_lanes ? cudaLaunchKernelEx(&cfg, k_gemm_tc<2>, mx, mw[0], mw[1], mw[2], a)
                   : lists ? cudaLaunchKernelEx(&cfg, k_gemm_tc<3>, mx, mw[0], mw[1], mw[2], a)
                                     : cudaLaunchKernelEx(&cfg, k_gemm_tc<0>, mx, mw[0], mw[1], mw[2], a);
  if (le != cudaSuccess) L.err = POSS_E_CUDA;
  LAUNCH_CHECK(L);
}
