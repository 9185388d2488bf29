// Tree-masked attention on the 5th-generation tensor cores (bf16, head dimension 128): the kernel of every
// draft step and target layer, from one key up to 10240 keys (prefix 8192 + tree and beyond).
//
// Geometry.  For one KV head the G = Hq/Hkv query heads of all tree rows form one matrix Q' of rows*G
// query rows (query row qi = r*G + g).  The keys are cut into groups of 128 at absolute positions
// (group j = keys [128 j, 128 j + 128)) and two consecutive groups form a unit of 256 keys.  The units of one
// (KV head, 128 query rows) are dealt round-robin to the CTAs that walk them (unit u goes to walker
// u mod n_walk); a walker pipelines its groups:
//   * one thread (warp 16) issues every copy and every product.  TMA brings the query tile once and, per group,
//     128 keys and 128 values (two stages each, loaded two to three groups ahead), 128-byte swizzle, rows past the last key or the last tree row arriving as zeros.  S_g = Q' K_g^T
//     (tcgen05.mma, M = 128 query rows, N = 128 keys, fp32 in TMEM) runs two groups ahead into one of two score
//     buffers; O_g = P_g V_g (two MMAs per 16 keys: hi and lo; V is the MN-major B operand, read as it sits in
//     the cache: [key][d]) goes into one of two output accumulators, one per group of the unit;
//   * sixteen warps do the softmax of one group at a time, one thread per (query row, quarter of the group's
//     keys): scores out of TMEM once (32 registers), ancestor mask, row maximum (the quarters meet through shared
//     memory), p = 2^(s - m), the quarter's share of the row sum; p is written to shared memory as a two-term bf16 split (p = hi + lo), laid
//     out as the A operand of the second product;
//   * when a unit's groups are done the same warps merge the two accumulators and park the 128 x 128 fp32 O of the
//     unit, its maximum and the four quarters' row sums in global memory (short-lived, read back out of L2).
// The walkers of one (KV head, query tile) form one or more thread-block clusters of up to 8 CTAs.  After a
// cluster barrier the CTA of cluster rank j merges its share of the query rows over ALL units in key order and
// writes the bf16 result.  With several clusters, the rank-j CTAs count their arrivals per (KV head, query tile,
// rank) after their own cluster's barrier, and the one that arrives last does rank j's merge: nobody waits for
// another cluster.
//
// The groups and units sit at absolute key positions, every unit is parked on its own and the final merge is
// one flat pass over the units in key order, so a query row's arithmetic depends neither on how many walkers
// there are, nor on where in the tile the row sits, nor on keys it does not see (a masked key enters every sum
// as an exact zero): a token whose visible keys are the prefix and itself gets the same bit pattern whether it
// is verified as the root of a 61-row tree or decoded alone.
//
// Visibility.  Keys [0, n_all) are seen by every row; key n_all + t is seen by row r iff bit t of the
// row's packed ancestor mask is set.
//
// Every wait on an mbarrier is bounded (wall time); on expiry the CTA raises POSS_E_TIMEOUT; every later wait
// then returns at once, the CTA runs through the rest of its (bounded) walk without meaning, still meets its
// cluster at the barrier, keeps the arrival counters consistent, frees its TMEM and returns.
#include "gemm_tc.cuh"
#include "tc_ptx.cuh"
#include <string.h>

POSS_TRACE_REGISTER()

namespace {

using namespace tcptx;

constexpr int D = 128;
constexpr int QT = 128;               // query rows per CTA (UMMA M)
constexpr int KG = 128;               // keys per group: the unit of the softmax, at absolute positions
constexpr int UNIT_KEYS = 2 * KG;     // keys per parked partial
constexpr int N_SOFTMAX = 512;        // sixteen softmax warps: TMEM lane quarter x quarter of the group's keys
constexpr int N_THREADS = N_SOFTMAX + 32;   // + the warp whose first lane issues copies and products
constexpr int MAX_CLUSTER = 8;        // portable cluster size
constexpr int MAX_UNITS = 40;         // 10240 keys (the merge's first pass covers up to 48 units)
constexpr int MAX_ARRIVAL_SETS = 512; // (KV head, query tile) pairs that can run with several clusters
constexpr int O_LD = D + 8;           // floats per parked partial: 128 outputs, four quarter row sums, m, padding
constexpr int TILE = 128 * 128;       // bytes of a [128 rows][64 bf16] tile
constexpr float NEG_BIG = -1.0e30f;
// shared memory: query tile (two 64-column halves), two key stages, two value stages, P as hi and lo (two 64-key
// blocks each)
constexpr uint32_t Q_OFF = 0, K_OFF = 2 * TILE, V_OFF = 6 * TILE, P_HI = 10 * TILE, P_LO = 12 * TILE;
constexpr uint32_t SMEM_TILES = 14 * TILE;                // 224 KB
constexpr uint32_t SMEM_LIMIT = 227 * 1024;               // static + dynamic shared memory a CTA may hold
constexpr uint32_t TMEM_COLS = 512;                       // S0 | S1 | O0 | O1, 128 columns each

// One launch serves `batch` sequences (a batched draft step; 1 otherwise): the same rows per sequence, each
// sequence with its own cache, key count and masks.  blockIdx.z = sequence * q_tiles + query tile.
struct AttnTcArgs {
  int rows, Hq, G, n_q;               // per sequence; n_q = rows * G query rows per KV head
  int batch, q_tiles;
  int n_walk;                         // CTAs that share the units of one (sequence, KV head, query tile)
  int cluster, n_clusters;            // n_walk = cluster * n_clusters
  int mask_words;
  float scale_log2;                   // softmax scale times log2(e)
  int inject_lost_load;               // test hook: the value tiles are never requested
  int n_all[MAXB], total[MAXB];       // keys every row sees / all keys, per sequence
  int n_units[MAXB];                  // 256-key units, per sequence
  const uint64_t* mask[MAXB];
  unsigned long long part_off[MAXB];  // the sequence's partials start here in `part` (floats)
  float* part;                        // per sequence [rows][Hq][n_units][O_LD]: 128 outputs, 4 row-sum shares, m
  uint32_t smem_bytes;                // dynamic shared memory of the launch (the tiles must fit behind the alignment)
  int* arrivals;                      // [batch * query tiles * Hkv][MAX_CLUSTER], zero between launches
  bf16* out;                          // [batch * rows][Hq][D]
  int32_t* status;
};
struct AttnMaps {
  CUtensorMap q;                      // the stacked queries of all sequences
  CUtensorMap k[MAXB], v[MAXB];       // each sequence's keys / values
};

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
// MN-major operand, 128-byte swizzle: 64 elements along N are one 128-byte line, consecutive K (keys) are
// consecutive lines, 8-line groups 1024 bytes apart, the next 64 elements along N `lbo_bytes` further.
__device__ __forceinline__ uint64_t smem_desc_sw128_mn(uint32_t addr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)(1024u >> 4) << 32;
  d |= 1ull << 46;
  d |= 2ull << 61;
  return d;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// barrier among the sixteen softmax warps only
__device__ __forceinline__ void softmax_sync(int id) { asm volatile("bar.sync %0, 512;" ::"r"(id) : "memory"); }
// 16 TMEM columns of this thread's lane into registers, without waiting; tmem_wait16 is the matching wait (it
// names the registers, so nothing that reads them can be scheduled ahead of it)
__device__ __forceinline__ void tmem_ld16_async(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, "
      "[%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_wait16(uint32_t* r) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                 "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :
               : "memory");
}
// Two-term bf16 split of two positive floats, packed low-first: hi = the upper 16 bits, lo = the upper 16 bits
// of the exact remainder x - hi.  hi + lo carries 16 significant bits of x (plain bit operations: conversion
// instructions share the transcendental unit with the exponentials).
__device__ __forceinline__ void split_pack(float x, float y, uint32_t& hi, uint32_t& lo) {
  const uint32_t xb = __float_as_uint(x), yb = __float_as_uint(y);
  hi = __byte_perm(xb, yb, 0x7632);
  const float xr = x - __uint_as_float(xb & 0xffff0000u), yr = y - __uint_as_float(yb & 0xffff0000u);
  lo = __byte_perm(__float_as_uint(xr), __float_as_uint(yr), 0x7632);
}

// ------------------------------------------------------------------ merge of a row's parked units
// One group of LANES threads (half a warp or a warp) per query row, 128 / LANES consecutive output columns per
// thread.  Lane j of the group loads the maxima and row-sum shares of units j, j + LANES, ... (together with the
// first batch of outputs: one round trip for everything when the units fit one batch); the row maximum is a
// shuffle reduction, each unit's weight c_u = 2^(m_u - max) reaches the other lanes by shuffle, and row sum and
// outputs are added in unit order.
// A load past L1 that stays where it is written: the merge wants every load of a batch in flight before the first
// use, and a plain load under a condition is free to sink to its use (one L2 round trip per unit instead of one per
// batch).  The callers clamp the address instead of skipping the load.
__device__ __forceinline__ float4 ld_cg_f4(const float* p) {
  float4 v;
  asm volatile("ld.global.cg.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ float ld_cg_f1(const float* p) {
  float v;
  asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p));
  return v;
}
struct MergeJob {
  int nu, row_lo, row_hi, q0, n_q, G, Hq, head0;
  const float* part;
  bf16* out;
};
template <int LANES>
__device__ __forceinline__ void merge_rows(const MergeJob& job) {
  constexpr int COLS = D / LANES;                  // 8 or 4 output columns per thread
  constexpr int NV = COLS / 4;                     // 16-byte loads per unit
  constexpr int BATCH = LANES == 16 ? 6 : 12;      // units in flight per thread
  constexpr int PER_LANE = LANES == 16 ? 3 : 2;    // units whose (m, l) one lane holds: 48 or 64 >= MAX_UNITS
  const int lane_g = threadIdx.x & (LANES - 1);
  const unsigned mask = LANES == 32 ? 0xffffffffu : ((threadIdx.x & 16) ? 0xffff0000u : 0x0000ffffu);
  const int groups = N_THREADS / LANES;
  const int nu = job.nu;
#pragma unroll 1
  for (int rr = job.row_lo + (int)threadIdx.x / LANES; rr < job.row_hi; rr += groups) {
    const int qj = job.q0 + rr;
    if (qj >= job.n_q) break;                      // rows only grow: the group is done
    const int rj = qj / job.G, gj = qj - rj * job.G;
    const float* src = job.part + (((size_t)rj * job.Hq + job.head0 + gj) * nu) * O_LD;
    const int cg = lane_g * COLS;
    // every load of the first batch before the first use
    float m_l[PER_LANE], l_l[PER_LANE];
    float4 lp[PER_LANE];
#pragma unroll
    for (int j = 0; j < PER_LANE; ++j) {
      const int u = lane_g + LANES * j;
      const float* pu = src + (size_t)(u < nu ? u : nu - 1) * O_LD + D;
      m_l[j] = ld_cg_f1(pu + 4);
      lp[j] = ld_cg_f4(pu);
    }
    float4 x[BATCH][NV];
#pragma unroll
    for (int j = 0; j < BATCH; ++j) {
      const float* pj = src + (size_t)(j < nu ? j : nu - 1) * O_LD + cg;
#pragma unroll
      for (int v = 0; v < NV; ++v) x[j][v] = ld_cg_f4(pj + 4 * v);
    }
    float mm = NEG_BIG;
#pragma unroll
    for (int j = 0; j < PER_LANE; ++j) {
      const bool have = lane_g + LANES * j < nu;
      if (!have) m_l[j] = NEG_BIG;
      mm = fmaxf(mm, m_l[j]);
      l_l[j] = have ? (lp[j].x + lp[j].y) + (lp[j].z + lp[j].w) : 0.f;
    }
#pragma unroll
    for (int o = LANES / 2; o > 0; o >>= 1) mm = fmaxf(mm, __shfl_xor_sync(mask, mm, o));
    float c_l[PER_LANE];
#pragma unroll
    for (int j = 0; j < PER_LANE; ++j) {
      c_l[j] = ex2(m_l[j] - mm);
      l_l[j] *= c_l[j];
    }
    float ll = 0.f, acc[COLS];
#pragma unroll
    for (int j = 0; j < COLS; ++j) acc[j] = 0.f;
    // unit u's weight and weighted row sum sit in lane u % LANES, slot u / LANES
    auto unit_c = [&](int u, float& c, float& l) {
      float cs = c_l[0], ls = l_l[0];
#pragma unroll
      for (int j = 1; j < PER_LANE; ++j)
        if (u >= LANES * j) { cs = c_l[j]; ls = l_l[j]; }
      c = __shfl_sync(mask, cs, u & (LANES - 1), LANES);
      l = __shfl_sync(mask, ls, u & (LANES - 1), LANES);
    };
#pragma unroll 1
    for (int u0 = 0; u0 < nu; u0 += BATCH) {
      if (u0 > 0) {
#pragma unroll
        for (int j = 0; j < BATCH; ++j) {
          const float* pj = src + (size_t)(u0 + j < nu ? u0 + j : nu - 1) * O_LD + cg;
#pragma unroll
          for (int v = 0; v < NV; ++v) x[j][v] = ld_cg_f4(pj + 4 * v);
        }
      }
#pragma unroll
      for (int j = 0; j < BATCH; ++j) {
        if (u0 + j < nu) {
          float c, l;
          unit_c(u0 + j, c, l);
          ll += l;
#pragma unroll
          for (int v = 0; v < NV; ++v) {
            acc[4 * v + 0] = fmaf(x[j][v].x, c, acc[4 * v + 0]);
            acc[4 * v + 1] = fmaf(x[j][v].y, c, acc[4 * v + 1]);
            acc[4 * v + 2] = fmaf(x[j][v].z, c, acc[4 * v + 2]);
            acc[4 * v + 3] = fmaf(x[j][v].w, c, acc[4 * v + 3]);
          }
        }
      }
    }
    const float inv = 1.f / ll;
    uint32_t w[COLS / 2];
#pragma unroll
    for (int j = 0; j < COLS / 2; ++j) {
      __nv_bfloat162 b = __floats2bfloat162_rn(acc[2 * j] * inv, acc[2 * j + 1] * inv);
      w[j] = *reinterpret_cast<uint32_t*>(&b);
    }
    bf16* dst = job.out + ((size_t)rj * job.Hq + job.head0 + gj) * D + cg;
    if (COLS == 8) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[COLS / 2 - 2], w[COLS / 2 - 1]);
    else *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
  }
}

// ------------------------------------------------------------------ the kernel
// 544 threads.  Softmax warp w (0..15) owns TMEM lane quarter q = w & 3 (32 query rows) and quarter cq = w >> 2 of
// a group's eight 16-key chunks; when a unit is parked the same thread owns output columns [32 cq, 32 cq + 32).
// Lane 0 of warp 16 issues the copies and both products.
__global__ void __launch_bounds__(N_THREADS, 1) k_attn_tc(const __grid_constant__ AttnMaps maps, const AttnTcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[10];
  __shared__ uint32_t tmem_slot;
  __shared__ int s_abort, s_last;
  __shared__ float x_max[4][QT];                               // [key quarter][query row]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int walker = blockIdx.x, kvh = blockIdx.y;
  const int seq = blockIdx.z / a.q_tiles, qtile = blockIdx.z - seq * a.q_tiles;
  const int n_all = a.n_all[seq], total = a.total[seq], n_units = a.n_units[seq];
  const CUtensorMap* const map_q = &maps.q;
  const CUtensorMap* const map_k = &maps.k[seq];
  const CUtensorMap* const map_v = &maps.v[seq];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar_q = smem_u32(&bars[0]), bar_p = smem_u32(&bars[7]), bar_pv = smem_u32(&bars[8]),
                 bar_of = smem_u32(&bars[9]);
  auto bar_k = [&](int st) { return smem_u32(&bars[1 + st]); };
  auto bar_v = [&](int st) { return smem_u32(&bars[3 + st]); };
  auto bar_s = [&](int b) { return smem_u32(&bars[5 + b]); };

  // this walker's groups, in the order it meets them: its units walker, walker + n_walk, ...; a unit's second
  // group exists when it holds at least one key
  const int n_my_units = walker < n_units ? (n_units - 1 - walker) / a.n_walk + 1 : 0;
  auto group_of = [&](int gi) { return 2 * (walker + (gi >> 1) * a.n_walk) + (gi & 1); };
  auto keys_of = [&](int grp) {
    int n = total - grp * KG;
    return n < 0 ? 0 : (n > KG ? KG : n);
  };
  int n_g = 2 * n_my_units;
  if (n_g > 0 && keys_of(group_of(n_g - 1)) == 0) --n_g;

  if (warp == 0) {
    if (lane == 0) {
      // (the tiles need SMEM_TILES bytes behind the 1024-byte alignment: checked on the host, and here)
      s_abort = base + SMEM_TILES > smem_u32(smem_raw) + a.smem_bytes ? 1 : 0;
      s_last = 0;
      mbar_init(bar_q, 1);
      mbar_init(bar_k(0), 1);
      mbar_init(bar_k(1), 1);
      mbar_init(bar_v(0), 1);
      mbar_init(bar_v(1), 1);
      mbar_init(bar_s(0), 1);
      mbar_init(bar_s(1), 1);
      mbar_init(bar_p, N_SOFTMAX);
      mbar_init(bar_pv, 1);
      mbar_init(bar_of, N_SOFTMAX);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      prefetch_tensormap(map_q);
      prefetch_tensormap(map_k);
      prefetch_tensormap(map_v);
    }
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_slot), TMEM_COLS);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  volatile int* abort_flag = &s_abort;

  // The successor may start only now that this CTA holds its TMEM columns: a successor's CTA that took
  // columns on this SM first would keep them until this grid has finished, which then could not happen.
  pdl_begin();
  pdl_sync(POSS_K_ATTN_TC);

  if (warp == 16) {
    if (lane == 0 && n_g > 0) {
      // ---------------- copies and products
      int k_loads0 = 0, k_loads1 = 0, v_loads0 = 0, v_loads1 = 0;
      auto load_k = [&](int gi) {
        const int key0 = group_of(gi) * KG, st = gi & 1;
        mbar_expect_tx(bar_k(st), 2u * TILE);
        tma_load_3d(base + K_OFF + st * 2u * TILE, map_k, bar_k(st), 0, key0, kvh);
        tma_load_3d(base + K_OFF + st * 2u * TILE + TILE, map_k, bar_k(st), 64, key0, kvh);
        if (st) ++k_loads1; else ++k_loads0;
      };
      auto load_v = [&](int gi) {
        const int key0 = group_of(gi) * KG, st = gi & 1;
        mbar_expect_tx(bar_v(st), 2u * TILE);
        if (!a.inject_lost_load) {
          tma_load_3d(base + V_OFF + st * 2u * TILE, map_v, bar_v(st), 0, key0, kvh);
          tma_load_3d(base + V_OFF + st * 2u * TILE + TILE, map_v, bar_v(st), 64, key0, kvh);
        }
        if (st) ++v_loads1; else ++v_loads0;
      };
      const uint32_t idesc_s = instr_desc_bf16(QT, KG);
      const uint32_t idesc_o = instr_desc_bf16(QT, D) | (1u << 16);     // B (the values) is MN-major
      auto issue_s = [&](int gi) {
        const uint32_t t_s = tmem_base + (uint32_t)((gi & 1) * KG);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const uint64_t ad = smem_desc_sw128(base + Q_OFF + h * TILE),
                         bd = smem_desc_sw128(base + K_OFF + (uint32_t)(gi & 1) * 2u * TILE + h * TILE);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)          // 16 bf16 = 32 bytes = 2 descriptor address units
            umma_bf16(t_s, ad + (uint64_t)(2 * kk), bd + (uint64_t)(2 * kk), idesc_s, (h | kk) ? 1u : 0u);
        }
        umma_commit(bar_s(gi & 1));
      };
      auto issue_pv = [&](int gi) {
        const int steps = (keys_of(group_of(gi)) + 15) / 16;
        const uint32_t t_o = tmem_base + 2u * KG + (uint32_t)((gi & 1) * D);
        const uint32_t v_base = base + V_OFF + (uint32_t)(gi & 1) * 2u * TILE;
        for (int ks = 0; ks < steps; ++ks) {
          const uint32_t pa = (uint32_t)(ks >> 2) * TILE;
          const uint64_t step = (uint64_t)(2 * (ks & 3));
          const uint64_t ah = smem_desc_sw128(base + P_HI + pa) + step, al = smem_desc_sw128(base + P_LO + pa) + step;
          const uint64_t bd = smem_desc_sw128_mn(v_base + (uint32_t)ks * 2048u, TILE);
          umma_bf16(t_o, ah, bd, idesc_o, ks > 0 ? 1u : 0u);
          umma_bf16(t_o, al, bd, idesc_o, 1u);
        }
        umma_commit(bar_pv);
      };

      mbar_expect_tx(bar_q, 2u * TILE);
      // (query rows past this sequence's last row are the next sequence's or zeros: they are computed and dropped)
      tma_load_4d(base + Q_OFF, map_q, bar_q, 0, 0, kvh, seq * a.rows + qtile * (QT / a.G));
      tma_load_4d(base + Q_OFF + TILE, map_q, bar_q, 64, 0, kvh, seq * a.rows + qtile * (QT / a.G));
      load_k(0);
      load_v(0);
      if (n_g > 1) { load_k(1); load_v(1); }
      bool ok = *abort_flag == 0 && mbar_wait(bar_q, 0, abort_flag) && mbar_wait(bar_k(0), 0, abort_flag);
      if (ok) {
        tc_fence_after();
        issue_s(0);
      }
      if (ok && n_g > 1) {
        ok = mbar_wait(bar_k(1), 0, abort_flag);
        if (ok) {
          tc_fence_after();
          issue_s(1);
        }
        if (ok && n_g > 2) {
          ok = mbar_wait(bar_s(0), 0, abort_flag);            // the first group's scores exist: its keys may go
          if (ok) load_k(2);
        }
      }
      // Group gi: its second product as soon as its P is written; then the scores two groups ahead (into the
      // buffer this group's softmax has just left), the keys three groups ahead (into the stage the scores of
      // group gi + 1 have long left) and the values two groups ahead (into this group's stage).
      for (int gi = 0; gi < n_g && ok; ++gi) {
        ok = mbar_wait(bar_p, (uint32_t)(gi & 1), abort_flag) &&                      // P of this group is written
             mbar_wait(bar_v(gi & 1), (uint32_t)((gi >> 1) & 1), abort_flag);         // its values have landed
        // a unit's accumulators are free again once the previous unit has been read out of them
        if (ok && (gi & 1) == 0 && gi >= 2) ok = mbar_wait(bar_of, (uint32_t)(((gi >> 1) - 1) & 1), abort_flag);
        if (!ok) break;
        tc_fence_after();
        issue_pv(gi);
        if (gi + 2 < n_g) {
          ok = mbar_wait(bar_k(gi & 1), (uint32_t)(((gi + 2) >> 1) & 1), abort_flag);
          if (!ok) break;
          tc_fence_after();
          issue_s(gi + 2);
        }
        if (gi + 3 < n_g) {
          ok = mbar_wait(bar_s((gi + 1) & 1), (uint32_t)(((gi + 1) >> 1) & 1), abort_flag);
          if (!ok) break;
          load_k(gi + 3);
        }
        if (gi + 2 < n_g) {
          ok = mbar_wait(bar_pv, (uint32_t)(gi & 1), abort_flag);                     // this group's values may go
          if (!ok) break;
          load_v(gi + 2);
        }
      }
      if (*abort_flag) {
        // drain: the copies this thread started must land before the CTA's shared memory goes away
        const uint64_t t0 = global_ns();
        auto drain = [&](uint32_t bar, int loads) {
          if (loads <= 0) return;
          const uint32_t par = (uint32_t)((loads - 1) & 1);
          while (!mbar_try_wait(bar, par) && global_ns() - t0 < WAIT_LIMIT_NS / 2) __nanosleep(64);
        };
        drain(bar_q, 1);
        drain(bar_k(0), k_loads0);
        drain(bar_k(1), k_loads1);
        drain(bar_v(0), v_loads0);
        drain(bar_v(1), v_loads1);
      }
    }
  } else {
    // ---------------- softmax and parking: TMEM lane = query row
    const int q = warp & 3, cq = warp >> 2;
    const int row = q * 32 + lane;
    const int qi = qtile * QT + row;
    const bool valid = qi < a.n_q;
    const int r = valid ? qi / a.G : 0;
    uint64_t mk0 = 0, mk1 = 0;
    if (valid) {
      const uint64_t* mask = a.mask[seq];
      mk0 = mask[(size_t)r * a.mask_words];
      if (a.mask_words > 1) mk1 = mask[(size_t)r * a.mask_words + 1];
    }
    float* const part = a.part + a.part_off[seq];
    const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
    float m_g0 = NEG_BIG, m_g1 = NEG_BIG;   // scaled row maximum of the unit's two groups
    float l_g0 = 0.f, l_g1 = 0.f;           // this thread's share (its quarter of the keys) of their row sums

    for (int gi = 0; gi < n_g; ++gi) {
      const int grp = group_of(gi);
      const int key_g = grp * KG;
      const int n_ch = (keys_of(grp) + 15) / 16;               // 16-key chunks of the group that hold keys
      mbar_wait(bar_s(gi & 1), (uint32_t)((gi >> 1) & 1), abort_flag);
      tc_fence_after();
      POSS_TRACE_POINT(1);
      // this thread's two chunks of scores; invisible keys become -inf: they lose every maximum and their 2^x is
      // an exact zero
      uint32_t sr[2][16];
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int c = 2 * cq + j;
        if (c < n_ch) {
          tmem_ld16_async(t_lane + (uint32_t)((gi & 1) * KG + c * 16), sr[j]);
          tmem_wait16(sr[j]);
          const int key0 = key_g + c * 16;
          if (key0 + 16 > n_all) {                             // the chunk reaches the tree slots or the end
            // bit i = key0 + i is visible: 16 bits cut out of (all ones below n_all | the row's ancestor mask)
            const int t0 = key0 - n_all;                       // tree slot of the chunk's first key; > -16
            uint32_t vis;
            if (t0 >= 64) vis = t0 >= 128 ? 0u : (uint32_t)(mk1 >> (t0 - 64));
            else if (t0 > 48) vis = (uint32_t)(mk0 >> t0) | (uint32_t)(mk1 << (64 - t0));
            else if (t0 >= 0) vis = (uint32_t)(mk0 >> t0);
            else vis = ((uint32_t)mk0 << (-t0)) | ((1u << (-t0)) - 1u);
            const int n_valid = total - key0;                  // keys of the chunk that exist
            if (n_valid < 16) vis &= (1u << (n_valid < 0 ? 0 : n_valid)) - 1u;
#pragma unroll
            for (int i = 0; i < 16; ++i)
              if (!((vis >> i) & 1u)) sr[j][i] = 0xff800000u;
          }
          float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int i = 0; i < 16; ++i) m4[i & 3] = fmaxf(m4[i & 3], __uint_as_float(sr[j][i]));
          mx = fmaxf(mx, fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])));
        }
      }
      x_max[cq][row] = mx;
      softmax_sync(1);
      const float mraw = fmaxf(fmaxf(x_max[0][row], x_max[1][row]), fmaxf(x_max[2][row], x_max[3][row]));
      // the scale is positive: the maximum of the scaled scores is the scaled maximum
      const float ms = mraw == -INFINITY ? 0.f : mraw * a.scale_log2;
      // P is one buffer: the previous group's second product must have read it
      if (gi > 0) mbar_wait(bar_pv, (uint32_t)((gi - 1) & 1), abort_flag);
      float ls = 0.f;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int c = 2 * cq + j;
        if (c < n_ch) {
          uint32_t hi[8], lo[8];
          float l4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int i = 0; i < 16; i += 2) {
            const float p0 = ex2(fmaf(__uint_as_float(sr[j][i]), a.scale_log2, -ms));
            const float p1 = ex2(fmaf(__uint_as_float(sr[j][i + 1]), a.scale_log2, -ms));
            l4[i & 3] += p0;
            l4[(i & 3) + 1] += p1;
            split_pack(p0, p1, hi[i >> 1], lo[i >> 1]);
          }
          ls += (l4[0] + l4[1]) + (l4[2] + l4[3]);
          // A operand of P V: k-block of 64 keys, row = query row (128 bytes), 16-byte pieces swizzled by row
          const uint32_t line = (uint32_t)(c >> 2) * TILE + (uint32_t)row * 128u;
          const uint32_t pc = (uint32_t)(c & 3) * 2u, sw = (uint32_t)(row & 7);
          *reinterpret_cast<uint4*>(base_ptr + P_HI + line + ((pc ^ sw) << 4)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          *reinterpret_cast<uint4*>(base_ptr + P_HI + line + (((pc + 1) ^ sw) << 4)) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
          *reinterpret_cast<uint4*>(base_ptr + P_LO + line + ((pc ^ sw) << 4)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
          *reinterpret_cast<uint4*>(base_ptr + P_LO + line + (((pc + 1) ^ sw) << 4)) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // P becomes visible to the tensor core
      tc_fence_before();
      mbar_arrive(bar_p);
      softmax_sync(2);                                         // every quarter has read this group's maxima
      POSS_TRACE_POINT(2);
      {
        const float mg = mraw == -INFINITY ? NEG_BIG : ms;
        if (gi & 1) { m_g1 = mg; l_g1 = ls; } else { m_g0 = mg; l_g0 = ls; }
      }

      if ((gi & 1) == 1 || gi == n_g - 1) {
        // ---- the unit is complete: merge its groups in key order and park (m, l, O) in global memory (it stays in
        // L2).  This thread: its query row, output columns [32 cq, 32 cq + 32).  (A unit whose second group holds
        // no key accumulated nothing there: that accumulator is not read.)
        const bool two = (gi & 1) == 1;
        mbar_wait(bar_pv, (uint32_t)(gi & 1), abort_flag);
        tc_fence_after();
        POSS_TRACE_POINT(3);
        const float m0 = m_g0, m1 = two ? m_g1 : NEG_BIG;
        const float l0 = l_g0, l1 = two ? l_g1 : 0.f;
        const float mu = fmaxf(m0, m1);
        const float c0 = ex2(m0 - mu), c1 = two ? ex2(m1 - mu) : 0.f;
        const int unit = walker + (gi >> 1) * a.n_walk;
        const uint32_t t_o = t_lane + 2u * KG + (uint32_t)(cq * 32);
        float* dst = part + (((size_t)r * a.Hq + kvh * a.G + (qi - r * a.G)) * n_units + unit) * O_LD;
        if (valid) {
          dst[D + cq] = l0 * c0 + l1 * c1;                     // this quarter's share of the unit's row sum
          if (cq == 0) dst[D + 4] = mu;
        }
#pragma unroll 1
        for (int cc = 0; cc < 2; ++cc) {
          uint32_t v0[16], v1[16];
          tmem_ld16_async(t_o + (uint32_t)(cc * 16), v0);
          if (two) tmem_ld16_async(t_o + (uint32_t)(D + cc * 16), v1);
          tmem_wait16(v0);
          if (two) tmem_wait16(v1);
          float v[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            v[j] = __uint_as_float(v0[j]) * c0;
            if (two) v[j] += __uint_as_float(v1[j]) * c1;
          }
          if (valid) {
#pragma unroll
            for (int j = 0; j < 16; j += 4)
              __stcg(reinterpret_cast<float4*>(dst + cq * 32 + cc * 16 + j), make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]));
          }
        }
        tc_fence_before();
        mbar_arrive(bar_of);                                   // the accumulators may take the next unit
        m_g0 = m_g1 = NEG_BIG;
        l_g0 = l_g1 = 0.f;
      }
    }
    if (a.n_clusters > 1) __threadfence();                     // this thread's parked values, before the arrival count
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  POSS_TRACE_POINT(4);

  // ---------------- merge over ALL units, in key order: this cluster rank's share of the query rows.  Within a
  // cluster the partials were written before the cluster barrier (release / acquire at cluster scope); with several
  // clusters the rank's last arriver merges (fence + counter), and nobody waits.  Partials are read past L1.
  const int rank = (int)cluster_rank();
  bool do_merge = true;
  if (a.n_clusters > 1) {
    if (threadIdx.x == 0) {
      int* cnt = a.arrivals + ((size_t)(blockIdx.z * gridDim.y + kvh) * MAX_CLUSTER + rank);
      __threadfence();
      const int prev = atomicAdd(cnt, 1);
      const int last = prev == a.n_clusters - 1;
      if (last) *cnt = 0;                                      // every other arrival is in: ready for the next launch
      __threadfence();
      s_last = last;
    }
    __syncthreads();
    do_merge = s_last != 0;
  }
  if (do_merge) {
    MergeJob job;
    job.nu = n_units;
    job.part = a.part + a.part_off[seq];
    job.out = a.out + (size_t)seq * a.rows * a.Hq * D;
    // the tile's rows that exist, in equal shares
    const int n_here = a.n_q - qtile * QT < QT ? a.n_q - qtile * QT : QT;
    job.row_lo = rank * n_here / a.cluster;
    job.row_hi = (rank + 1) * n_here / a.cluster;
    job.q0 = qtile * QT; job.n_q = a.n_q; job.G = a.G; job.Hq = a.Hq; job.head0 = kvh * a.G;
    // few units: half a warp per row, eight columns per thread, every load of the row in one round trip;
    // many units: a warp per row, four columns per thread, twelve units in flight per thread.  Both add a
    // column's terms in unit order with the same operations, so the result does not depend on the choice.
    if (job.nu <= 6) merge_rows<16>(job);
    else merge_rows<32>(job);
  }

  POSS_TRACE_POINT(5);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, TMEM_COLS);
  if (threadIdx.x == 0 && *abort_flag) atomicExch(a.status, (int)POSS_E_TIMEOUT);
}

}  // namespace

// ------------------------------------------------------------------ host side
// The cut of the keys: a function of the key count alone.  Groups of 128 keys from key 0 on, two per unit; one
// partial per unit.
bool tree_attention_tc_plan(int total, int* unit_keys, int* n_units) {
  if (total < 1 || total > MAX_UNITS * UNIT_KEYS) return false;
  *unit_keys = total <= KG ? KG : UNIT_KEYS;
  *n_units = (total + UNIT_KEYS - 1) / UNIT_KEYS;
  return true;
}

size_t tree_attention_tc_arrival_ints() { return (size_t)MAX_ARRIVAL_SETS * MAX_CLUSTER; }

bool tree_attention_tc_supported(const AttnArgs& a, const void* q, const void* kc, const void* vc, const void* out) {
  if (a.d != D || a.Hkv < 1 || a.Hq % a.Hkv) return false;
  const int G = a.Hq / a.Hkv;
  if (G > QT || QT % G) return false;
  const int total = a.n_all + a.n_tree;
  if (a.rows < 1 || total < 1 || total > MAX_UNITS * UNIT_KEYS) return false;
  if (a.mask_words > 2 || a.n_tree > 128) return false;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(kc) | reinterpret_cast<uintptr_t>(vc) |
       reinterpret_cast<uintptr_t>(out)) & 15)
    return false;
  return true;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// How many clusters of `size` CTAs of the kernel the current device holds at once (0: cannot be had).  Asked once
// per device and size.
static int resident_clusters(int size, size_t smem) {
  constexpr int MAX_DEVICES = 64;
  static int known[MAX_DEVICES][MAX_CLUSTER + 1];              // 0 = not asked yet, -1 = the query failed
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return 0;
  int& slot = known[dev][size];
  if (slot == 0) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(size, 1, 1);
    cfg.blockDim = dim3(N_THREADS);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = size;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, k_attn_tc, &cfg) != cudaSuccess || n < 1) {
      cudaGetLastError();
      n = -1;
    }
    slot = n;
  }
  return slot > 0 ? slot : 0;
}

bool launch_tree_attention_tc(Launcher& L, TcGemmPlanCache* cache, const AttnArgs& a, const AttnBatch& ab, const bf16* q,
                              float* part, size_t part_floats, int* arrivals, bf16* out, int32_t* status) {
  if (ab.batch < 1 || ab.batch > MAXB || !status || !part || (reinterpret_cast<uintptr_t>(part) & 15)) return false;
  EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(tc_encode_fn(cache));
  if (!encode) return false;
  const int G = a.Hkv > 0 ? a.Hq / a.Hkv : 1;
  AttnMaps maps;                       // the launch's tensor maps (copied into the kernel's parameters)
  AttnTcArgs k;
  memset(&k, 0, sizeof(k));
  k.rows = a.rows; k.Hq = a.Hq; k.G = G; k.n_q = a.rows * G;
  k.batch = ab.batch;
  int max_units = 0;
  size_t part_need = 0;
  for (int b = 0; b < ab.batch; ++b) {
    AttnArgs ai = a;
    ai.n_all = ab.n_all[b];
    if (!tree_attention_tc_supported(ai, q, ab.kc[b], ab.vc[b], out) || !ab.mask[b]) return false;
    k.n_all[b] = ab.n_all[b];
    k.total[b] = ab.n_all[b] + a.n_tree;
    int unit_keys = 0;
    if (!tree_attention_tc_plan(k.total[b], &unit_keys, &k.n_units[b])) return false;
    if (k.n_units[b] > max_units) max_units = k.n_units[b];
    k.mask[b] = ab.mask[b];
    k.part_off[b] = part_need;
    part_need += (size_t)a.rows * a.Hq * k.n_units[b] * O_LD;
  }
  if (part_need > part_floats) return false;
  // Shared memory: the tiles behind a 1024-byte alignment of the dynamic part, which starts behind the kernel's
  // static part; together they must fit what a CTA may hold.  (More than half an SM's shared memory, so that two of
  // these CTAs never share an SM: each holds all of the SM's TMEM until its whole cluster has merged.)
  static size_t static_smem = 0;       // a property of the compiled kernel: asked for once
  if (!static_smem) {
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, k_attn_tc) != cudaSuccess) return false;
    static_smem = fa.sharedSizeBytes ? fa.sharedSizeBytes : 1;
  }
  const size_t static_bytes = (static_smem + 15) / 16 * 16;
  const size_t pad = (1024 - static_bytes % 1024) % 1024;
  if (static_bytes + pad + SMEM_TILES > SMEM_LIMIT) return false;
  const size_t smem = SMEM_LIMIT - static_bytes;
  k.smem_bytes = (uint32_t)smem;
  // the shared-memory opt-in is a per-device property of the kernel
  static PerDeviceFlags attr_done;
  bool* attr = attr_done.current();
  if (!attr || !*attr) {
    if (cudaFuncSetAttribute(k_attn_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return false;
    if (attr) *attr = true;
  }
  // Walkers per (sequence, KV head, query tile), as c clusters of s CTAs: the shape with the lowest estimated time.
  // A cluster needs its s SMs inside one GPC, so fewer large clusters are resident at once than the SM count
  // suggests (15 of eight on a 148-SM device), and a shape that needs a second wave takes twice as long; the merge
  // is done by the s CTAs of the cluster that arrives last, so small clusters leave it to few SMs.  Estimates in
  // tenths of a microsecond, from device timestamps: 6.2 us per unit walked, 4 us to start a wave, 1 us + 0.9 us
  // per batch of units for every pass of the merge over a CTA's rows, its reads at 100 GB/s per SM.
  // (Scheduling only: the result does not depend on it.)
  k.q_tiles = (k.n_q + QT - 1) / QT;
  const int sets = a.Hkv * k.q_tiles * ab.batch;
  const bool several = arrivals && sets <= MAX_ARRIVAL_SETS;
  const int tile_rows = k.n_q < QT ? k.n_q : QT;
  long best_cost = -1;
  k.cluster = 1;
  k.n_clusters = 1;
  for (int s = MAX_CLUSTER; s >= 1; --s) {
    if (s > max_units) continue;
    const int fit = resident_clusters(s, smem);
    if (fit < 1) continue;
    int c = fit / sets;
    if (c < 1) c = 1;
    if (c > max_units / s) c = max_units / s;
    if (c > 1 && !several) c = 1;
    const long waves = (sets * c + fit - 1) / fit;
    const long walked = (max_units + s * c - 1) / (s * c);
    const long rows_rank = (tile_rows + s - 1) / s;
    const long passes = (rows_rank + (max_units <= 6 ? 33 : 16)) / (max_units <= 6 ? 34 : 17);
    const long batches = max_units <= 6 ? 1 : (max_units + 11) / 12;
    const long cost = waves * (40 + 62 * walked) + passes * (10 + 9 * batches) +
                      rows_rank * max_units * (O_LD * 4) / 10000 + (c > 1 ? 10 : 0);
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      k.cluster = s;
      k.n_clusters = c;
    }
  }
  k.n_walk = k.cluster * k.n_clusters;
  k.mask_words = a.mask_words;
  k.scale_log2 = a.scale * 1.4426950408889634f;
  k.part = part; k.arrivals = arrivals; k.out = out; k.status = status;
  k.inject_lost_load = tc_take_injection(cache) ? 1 : 0;
  // The maps carry the call's extents (rows, key count): rows past them are filled with zeros by the copy.
  {
    cuuint64_t gdim[4] = {(cuuint64_t)D, (cuuint64_t)G, (cuuint64_t)a.Hkv, (cuuint64_t)(a.rows * ab.batch)};
    cuuint64_t gstr[3] = {(cuuint64_t)D * 2, (cuuint64_t)G * D * 2, (cuuint64_t)a.Hq * D * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)G, 1, (cuuint32_t)(QT / G)};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    if (encode(&maps.q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<bf16*>(q), gdim, gstr, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  for (int b = 0; b < ab.batch; ++b) {
    for (int i = 0; i < 2; ++i) {
      cuuint64_t gdim[3] = {(cuuint64_t)D, (cuuint64_t)k.total[b], (cuuint64_t)a.Hkv};
      cuuint64_t gstr[2] = {(cuuint64_t)D * 2, (cuuint64_t)a.cap * D * 2};
      cuuint32_t box[3] = {64, (cuuint32_t)KG, 1};
      cuuint32_t estr[3] = {1, 1, 1};
      if (encode(i ? &maps.v[b] : &maps.k[b], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
                 const_cast<bf16*>(i ? ab.vc[b] : ab.kc[b]), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                 CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    }
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(k.n_walk, a.Hkv, k.q_tiles * ab.batch);
  cfg.blockDim = dim3(N_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = L.stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  at[1].id = cudaLaunchAttributeClusterDimension;
  at[1].val.clusterDim.x = k.cluster;
  at[1].val.clusterDim.y = 1;
  at[1].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 2;
  // A cluster shape the device does not take is reported at launch, before anything runs: remember it and
  // leave the call to the split-KV kernels.
  static PerDeviceFlags refused[MAX_CLUSTER + 1];
  bool* ref = refused[k.cluster].current();
  if (ref && *ref) return false;
  if (cudaLaunchKernelEx(&cfg, k_attn_tc, maps, k) != cudaSuccess) {
    cudaGetLastError();
    if (ref) *ref = true;
    return false;
  }
  ++*L.launches;
  return true;
}
