// Skinny bf16 GEMM on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM, operands
// staged by TMA).
//
// out[m][n] = sum_k X[m][k] * W[n][k]  with M <= 128 activation rows and N large.  The product is
// evaluated "swapped": a tile of 128 weight rows is the MMA's M dimension (TMEM lane = weight row n),
// the activation rows are the MMA's N dimension (TMEM column = row m, padded to a multiple of 16).
// So the weights, which are all of the traffic, stream through shared memory exactly once in 16 KB
// TMA boxes [128 rows x 64 k] (128-byte swizzle), and the small activation tile rides along.
//
// Grid = (weight-row tiles, K splits).  Roles inside a CTA of 128 threads: warp 0 lane 0 issues TMA
// into a ring of stages; warp 1 lane 0 issues the MMAs and releases stages with tcgen05.commit; all
// four warps run the epilogue (tcgen05.ld, 32 TMEM lanes per warp).  With K splits every CTA writes
// its fp32 partial tile to scratch, and the CTA that arrives last at the tile's counter adds the
// partials in split order (never in arrival order) and applies bias / residual: the result is
// deterministic and a row's value does not depend on M.  No CTA ever waits for another CTA.
//
// Every wait on an mbarrier is bounded; on expiry the CTA raises POSS_E_TIMEOUT in the status word,
// stops issuing work, drains its own copies (bounded), frees its TMEM and returns.
#include "gemm_tc.cuh"
#include <cuda.h>
#include <unordered_map>
#include <string>
#include <string.h>

#define LAUNCH_CHECK(L)                                         \
  do {                                                          \
    ++*(L).launches;                                            \
    if (cudaGetLastError() != cudaSuccess) (L).err = POSS_E_CUDA; \
  } while (0)

namespace {

constexpr int TILE_N = 128;          // weight rows per tile (UMMA M)
constexpr int TILE_K = 64;           // bf16 elements per k-block = one 128-byte swizzle row
constexpr int W_TILE_BYTES = TILE_N * TILE_K * 2;
constexpr int MAX_STAGES = 8;
constexpr uint32_t WAIT_LIMIT = 1u << 22;
constexpr size_t SCRATCH_PARTIAL_BYTES = 96ull << 20;
constexpr int N_COUNTERS = 8192;

struct TcArgs {
  int M, Npad, n_stages;
  int n_segs, seg_tiles[3], seg_rows[3], seg_col[3];
  int kb_total, kb_per_split, n_splits;
  const bf16* bias;
  const float* residual;
  int ldr;
  float* out;
  int ldo;
  float* scratch;
  int* counters;
  int32_t* status;
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// bounded wait; returns false when it gave up or when another role already raised the abort flag
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      if (it > 4096u) __nanosleep(64);
    }
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, "
      "[%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory operand descriptor: K-major tile whose rows are 128 bytes (64 bf16), 128-byte swizzle,
// 8-row groups 1024 bytes apart; descriptor version 1 (Blackwell), swizzle code 2 in bits 61..63.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);       // start address, 16-byte units
  d |= (uint64_t)(1024u >> 4) << 32;             // stride between 8-row groups
  d |= 1ull << 46;                               // descriptor version
  d |= 2ull << 61;                               // 128-byte swizzle
  return d;
}
// Instruction descriptor of kind::f16: fp32 accumulate, bf16 x bf16, both operands K-major.
__device__ __forceinline__ uint32_t instr_desc_bf16(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ------------------------------------------------------------------ the kernel
__global__ void __launch_bounds__(128) k_gemm_tc(const __grid_constant__ CUtensorMap map_x,
                                                 const __grid_constant__ CUtensorMap map_w0,
                                                 const __grid_constant__ CUtensorMap map_w1,
                                                 const __grid_constant__ CUtensorMap map_w2, const TcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * MAX_STAGES + 1];
  __shared__ uint32_t tmem_slot;
  __shared__ int s_abort, s_last;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t x_tile_bytes = (uint32_t)a.Npad * 128u;
  const uint32_t stage_bytes = W_TILE_BYTES + x_tile_bytes;
  const int S = a.n_stages;
  auto w_tile = [&](int s) { return tiles_base + (uint32_t)s * stage_bytes; };
  auto x_tile = [&](int s) { return tiles_base + (uint32_t)s * stage_bytes + W_TILE_BYTES; };
  auto full_bar = [&](int s) { return smem_u32(&bars[s]); };
  auto empty_bar = [&](int s) { return smem_u32(&bars[MAX_STAGES + s]); };
  const uint32_t accum_bar = smem_u32(&bars[2 * MAX_STAGES]);

  // which weight tile
  int tile = blockIdx.x, seg = 0, ltile = tile;
  while (seg < a.n_segs - 1 && ltile >= a.seg_tiles[seg]) { ltile -= a.seg_tiles[seg]; ++seg; }
  const CUtensorMap* map_w = seg == 0 ? &map_w0 : (seg == 1 ? &map_w1 : &map_w2);
  const int n0 = ltile * TILE_N;
  const int split = blockIdx.y;
  const int kb0 = split * a.kb_per_split;
  const int nkb = min(a.kb_total, kb0 + a.kb_per_split) - kb0;
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < a.Npad) tmem_cols <<= 1;

  if (threadIdx.x == 0) {
    s_abort = 0;
    s_last = 0;
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(accum_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&tmem_slot), tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  volatile int* abort_flag = &s_abort;

  if (warp == 0 && lane == 0) {
    // ---------------- TMA producer
    int issued = 0;
    for (int i = 0; i < nkb; ++i) {
      int s = i % S;
      if (i >= S && !mbar_wait(empty_bar(s), (uint32_t)((i / S - 1) & 1), abort_flag)) break;
      mbar_expect_tx(full_bar(s), stage_bytes);
      int kcoord = (kb0 + i) * TILE_K;
      tma_load_2d(w_tile(s), map_w, full_bar(s), kcoord, n0);
      tma_load_2d(x_tile(s), &map_x, full_bar(s), kcoord, 0);
      issued = i + 1;
    }
    if (*abort_flag) {
      // drain: every copy this thread started must land before the CTA's shared memory goes away
      for (int i = max(0, issued - S); i < issued; ++i) {
        uint32_t bar = full_bar(i % S), par = (uint32_t)((i / S) & 1);
        for (uint32_t it = 0; it < WAIT_LIMIT && !mbar_try_wait(bar, par); ++it) __nanosleep(64);
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer
    const uint32_t idesc = instr_desc_bf16(TILE_N, a.Npad);
    bool ok = true;
    for (int i = 0; i < nkb && ok; ++i) {
      int s = i % S;
      ok = mbar_wait(full_bar(s), (uint32_t)((i / S) & 1), abort_flag);
      if (!ok) break;
      tc_fence_after();
      uint64_t ad = smem_desc_sw128(w_tile(s)), bd = smem_desc_sw128(x_tile(s));
#pragma unroll
      for (int kk = 0; kk < TILE_K / 16; ++kk)      // 16 bf16 = 32 bytes = 2 descriptor address units
        umma_bf16(tmem_base, ad + (uint64_t)(2 * kk), bd + (uint64_t)(2 * kk), idesc, (i > 0 || kk > 0) ? 1u : 0u);
      umma_commit(empty_bar(s));
    }
    umma_commit(accum_bar);        // arrives once every MMA issued above has finished
  }
  __syncwarp();

  // ---------------- epilogue: all four warps, TMEM lane = weight row
  bool have = mbar_wait(accum_bar, 0u, abort_flag);
  have = have && !*abort_flag;
  tc_fence_after();
  const int t = threadIdx.x;
  const int n_local = n0 + t;
  const bool n_ok = n_local < a.seg_rows[seg];
  const int col = a.seg_col[seg] + n_local;
  const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16);
  if (have) {
    if (a.n_splits == 1) {
      float bv = (a.bias && n_ok) ? __bfloat162float(a.bias[col]) : 0.f;
      for (int c0 = 0; c0 < a.Npad && c0 < a.M; c0 += 16) {
        float v[16];
        tmem_ld16(taddr + (uint32_t)c0, v);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          int m = c0 + j;
          if (m < a.M && n_ok) {
            float r = v[j] + bv;
            if (a.residual) r += a.residual[(size_t)m * a.ldr + col];
            a.out[(size_t)m * a.ldo + col] = r;
          }
        }
      }
    } else {
      float* part = a.scratch + ((size_t)tile * a.n_splits + split) * (size_t)a.Npad * TILE_N;
      for (int c0 = 0; c0 < a.Npad && c0 < a.M; c0 += 16) {
        float v[16];
        tmem_ld16(taddr + (uint32_t)c0, v);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          int m = c0 + j;
          if (m < a.M) part[(size_t)m * TILE_N + t] = v[j];
        }
      }
      __threadfence();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);
  if (threadIdx.x == 0 && *abort_flag) atomicExch(a.status, (int)POSS_E_TIMEOUT);

  if (a.n_splits > 1 && !*abort_flag) {
    if (threadIdx.x == 0) {
      int prev = atomicAdd(&a.counters[tile], 1);
      s_last = prev == a.n_splits - 1;
    }
    __syncthreads();
    if (s_last) {
      __threadfence();
      const float* p0 = a.scratch + (size_t)tile * a.n_splits * (size_t)a.Npad * TILE_N;
      float bv = (a.bias && n_ok) ? __bfloat162float(a.bias[col]) : 0.f;
      for (int m = 0; m < a.M; ++m) {
        float acc = 0.f;
        for (int sp = 0; sp < a.n_splits; ++sp)
          acc += __ldcg(p0 + ((size_t)sp * a.Npad + m) * TILE_N + t);
        if (n_ok) {
          float r = acc + bv;
          if (a.residual) r += a.residual[(size_t)m * a.ldr + col];
          a.out[(size_t)m * a.ldo + col] = r;
        }
      }
      if (threadIdx.x == 0) a.counters[tile] = 0;     // ready for the next launch on this stream
    }
  }
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
  std::unordered_map<MapKey, CUtensorMap, MapKeyHash> maps;
};

TcGemmPlanCache* tc_plan_cache_create() { return new TcGemmPlanCache(); }
void tc_plan_cache_destroy(TcGemmPlanCache* p) { delete p; }
size_t tc_gemm_scratch_bytes() { return SCRATCH_PARTIAL_BYTES + N_COUNTERS * sizeof(int); }

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
  if (!c->tried) {
    c->tried = true;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      c->encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  if (!c->encode) return false;
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

// Split factor and stage count depend on the weight shape only, never on M.
void tc_plan_splits(int n_tiles, int kb_total, int* n_splits, int* kb_per_split) {
  int target = 2 * 148;
  int want = (target + n_tiles - 1) / n_tiles;
  int max_by_k = kb_total / 4;
  if (max_by_k < 1) max_by_k = 1;
  if (want > max_by_k) want = max_by_k;
  if (want < 1) want = 1;
  int per = (kb_total + want - 1) / want;
  *kb_per_split = per;
  *n_splits = (kb_total + per - 1) / per;
}

void launch_gemm_tc(Launcher& L, TcGemmPlanCache* cache, const bf16* X, int ldx, int M, const GemmSegs& segs, int K,
                    const bf16* bias, const float* residual, int ldr, float* out, int ldo, void* scratch,
                    int32_t* status) {
  TcArgs a;
  memset(&a, 0, sizeof(a));
  a.M = M;
  a.Npad = (M + 15) / 16 * 16;
  a.n_segs = segs.n;
  int n_tiles = 0, col = 0;
  for (int i = 0; i < segs.n; ++i) {
    a.seg_tiles[i] = (segs.rows[i] + TILE_N - 1) / TILE_N;
    a.seg_rows[i] = segs.rows[i];
    a.seg_col[i] = col;
    col += segs.rows[i];
    n_tiles += a.seg_tiles[i];
  }
  a.kb_total = (K + TILE_K - 1) / TILE_K;
  tc_plan_splits(n_tiles, a.kb_total, &a.n_splits, &a.kb_per_split);
  size_t part_bytes = (size_t)n_tiles * a.n_splits * a.Npad * TILE_N * sizeof(float);
  if (a.n_splits > 1 && (part_bytes > SCRATCH_PARTIAL_BYTES || n_tiles > N_COUNTERS)) {
    a.n_splits = 1;
    a.kb_per_split = a.kb_total;
  }
  uint32_t stage_bytes = W_TILE_BYTES + (uint32_t)a.Npad * 128u;
  int stages = (int)((100u * 1024u) / stage_bytes);
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  if (stages > a.kb_per_split) stages = a.kb_per_split;
  if (stages < 2) stages = a.kb_per_split < 2 ? 1 : 2;
  a.n_stages = stages;
  a.bias = bias; a.residual = residual; a.ldr = ldr; a.out = out; a.ldo = ldo;
  a.scratch = reinterpret_cast<float*>(scratch);
  a.counters = reinterpret_cast<int*>(reinterpret_cast<char*>(scratch) + SCRATCH_PARTIAL_BYTES);
  a.status = status;

  CUtensorMap mx, mw[3];
  if (!get_map(cache, X, M, K, ldx, a.Npad, false, &mx)) { L.err = POSS_E_CUDA; return; }
  for (int i = 0; i < 3; ++i) {
    int j = i < segs.n ? i : 0;
    if (!get_map(cache, segs.w[j], segs.rows[j], K, K, TILE_N, true, &mw[i])) { L.err = POSS_E_CUDA; return; }
  }
  size_t smem = (size_t)stages * stage_bytes + 1024;
  if (!cache->attr_set) {
    if (cudaFuncSetAttribute(k_gemm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) {
      L.err = POSS_E_CUDA;
      return;
    }
    cache->attr_set = true;
  }
  dim3 grid(n_tiles, a.n_splits);
  k_gemm_tc<<<grid, 128, smem, L.stream>>>(mx, mw[0], mw[1], mw[2], a);
  LAUNCH_CHECK(L);
}
