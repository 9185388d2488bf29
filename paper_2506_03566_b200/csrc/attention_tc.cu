// Tree-masked attention on the 5th-generation tensor cores (bf16, head dimension 128): the kernel of every
// draft step and target layer whenever the key count fits one pass (at most 2048 keys).
//
// Geometry.  For one KV head the G = Hq/Hkv query heads of all tree rows form one matrix Q' of rows*G
// query rows (query row qi = r*G + g).  The keys are cut into groups of 128 at absolute positions
// (group j = keys [128 j, 128 j + 128)); a CTA owns two consecutive groups, one KV head and 128 query
// rows.  The CTAs of one (KV head, query tile) form one thread-block cluster (1 to 8 of them):
//   1. TMA brings the 128 x 128 query tile and the CTA's 256 keys and values into shared memory
//      (128-byte swizzle; rows past the last key or the last tree row arrive as zeros);
//   2. one thread issues S = Q' K^T (tcgen05.mma, M = 128 query rows, N = 256 keys, fp32 in TMEM);
//   3. sixteen warps take S out of TMEM, one thread per (query row, group, half of the group's keys): scale,
//      ancestor mask, row maximum (the halves meet through shared memory), p = 2^(s - m), row sum; p is written
//      back to shared memory as a two-term bf16 split (p = hi + lo), laid out as the A operand of the next product;
//   4. one thread issues O_g = P_g V_g for both groups (two MMAs per 16 keys: hi and lo; V is the MN-major
//      B operand, read as it sits in the cache: [key][d]), each group into its own TMEM accumulator;
//   5. every CTA merges its two groups and parks (m, l) and the 128 x 128 fp32 O in global memory (one
//      short-lived partial per CTA, read back out of L2); after a cluster barrier CTA j merges its share of
//      the query rows over the cluster's CTAs, in key order, and writes the bf16 result.  (Reading the
//      peers' shared memory instead was measured: the SM-to-SM path moved these rows at a quarter of L2's
//      rate.)
//
// The groups sit at absolute key positions and a query row's arithmetic does not depend on where in the
// tile it sits, nor on keys it does not see (a masked key enters every sum as an exact zero): a token whose
// visible keys are the prefix and itself gets the same bit pattern whether it is verified as the root of a
// 61-row tree or decoded alone.
//
// Visibility.  Keys [0, n_all) are seen by every row; key n_all + t is seen by row r iff bit t of the
// row's packed ancestor mask is set.
//
// Every wait on an mbarrier is bounded (wall time); on expiry the CTA raises POSS_E_TIMEOUT, skips its
// remaining work, still meets its cluster at the barrier, frees its TMEM and returns.
#include "gemm_tc.cuh"
#include "tc_ptx.cuh"
#include <string.h>

POSS_TRACE_REGISTER()

namespace {

using namespace tcptx;

constexpr int D = 128;
constexpr int QT = 128;               // query rows per CTA (UMMA M)
constexpr int N_THREADS = 512;        // sixteen warps: TMEM lane quarter x key group x half of the group
constexpr int KG = 128;               // keys per group: the unit of the softmax partials, at absolute positions
constexpr int MAX_CTA_KEYS = 2 * KG;  // keys per CTA (UMMA N of the first product)
constexpr int MAX_SPLITS = 8;         // portable cluster size
constexpr int O_LD = D + 4;           // floats per parked partial: 128 outputs, m, l, padding to 16 bytes
constexpr int HALF_TILE = QT * 128;   // bytes of a [128 rows][64 bf16] tile
constexpr float NEG_BIG = -1.0e30f;

struct AttnTcArgs {
  int rows, Hq, G, n_q;               // n_q = rows * G query rows per KV head
  int n_all, n_tree, total;
  int cta_keys, n_splits;             // keys per CTA (128 or 256); CTAs per cluster
  uint32_t region_a_bytes;            // Q + K, later P (hi, lo); V sits behind it
  const uint64_t* mask;
  int mask_words;
  float scale_log2;                   // softmax scale times log2(e)
  int inject_lost_load;               // test hook: the value tiles are never requested
  float* part;                        // [rows][Hq][n_splits][O_LD]: a CTA's merged partial, 128 outputs then (m, l)
  bf16* out;
  int32_t* status;
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

// ------------------------------------------------------------------ the kernel
// 512 threads: warp w owns TMEM lane quarter q = w & 3 (32 query rows), key group g = (w >> 2) & 1 and half
// hf = w >> 3 of the group's eight 16-key chunks in the softmax; column quarter cq = w >> 2 (32 output columns) when
// the outputs are parked.  Thread 0 also issues the copies and both products.
__global__ void __launch_bounds__(N_THREADS, 1) k_attn_tc(const __grid_constant__ CUtensorMap map_q,
                                                          const __grid_constant__ CUtensorMap map_k,
                                                          const __grid_constant__ CUtensorMap map_v, const AttnTcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[5];
  __shared__ uint32_t tmem_slot;
  __shared__ int s_abort;
  __shared__ float half_max[2][2][QT], half_sum[2][2][QT];     // [half][group][query row]
  __shared__ float grp_m[2][QT];                               // scaled maximum per group and query row

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, kvh = blockIdx.y, qtile = blockIdx.z;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const int cta_keys = a.cta_keys, ng = cta_keys / KG;
  const uint32_t k_half = (uint32_t)cta_keys * 128u;            // bytes of [cta_keys][64 bf16]
  const uint32_t q_off = 0, k_off = 2 * HALF_TILE;              // region A, first life
  const uint32_t p_hi = 0, p_lo = (uint32_t)(cta_keys / 64) * HALF_TILE;   // region A, second life
  const uint32_t v_off = a.region_a_bytes;
  const uint32_t bar_qk = smem_u32(&bars[0]), bar_v = smem_u32(&bars[1]), bar_s = smem_u32(&bars[2]),
                 bar_p = smem_u32(&bars[3]), bar_o = smem_u32(&bars[4]);
  const uint32_t o_col = (uint32_t)cta_keys;                    // S at column 0, O of group g at o_col + 128 g
  const uint32_t tmem_cols = 2u * (uint32_t)cta_keys;
  const int k_begin = split * cta_keys;
  // keys of group g that exist at all (the rest of the group, if any, is zero fill)
  auto group_keys = [&](int g) {
    int n = a.total - (k_begin + g * KG);
    return n < 0 ? 0 : (n > KG ? KG : n);
  };

  if (warp == 0) {
    if (lane == 0) {
      s_abort = 0;
      mbar_init(bar_qk, 1);
      mbar_init(bar_v, 1);
      mbar_init(bar_s, 1);
      mbar_init(bar_p, N_THREADS);
      mbar_init(bar_o, 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      prefetch_tensormap(&map_v);
    }
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_slot), tmem_cols);
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

  if (threadIdx.x == 0) {
    // ---------------- the copies and the first product
    mbar_expect_tx(bar_qk, 2u * HALF_TILE + 2u * k_half);
    tma_load_4d(base + q_off, &map_q, bar_qk, 0, 0, kvh, qtile * (QT / a.G));
    tma_load_4d(base + q_off + HALF_TILE, &map_q, bar_qk, 64, 0, kvh, qtile * (QT / a.G));
    tma_load_3d(base + k_off, &map_k, bar_qk, 0, k_begin, kvh);
    tma_load_3d(base + k_off + k_half, &map_k, bar_qk, 64, k_begin, kvh);
    mbar_expect_tx(bar_v, 2u * k_half);
    if (!a.inject_lost_load) {
      tma_load_3d(base + v_off, &map_v, bar_v, 0, k_begin, kvh);
      tma_load_3d(base + v_off + k_half, &map_v, bar_v, 64, k_begin, kvh);
    }
    if (mbar_wait(bar_qk, 0, abort_flag)) {
      tc_fence_after();
      const uint32_t idesc = instr_desc_bf16(QT, cta_keys);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint64_t ad = smem_desc_sw128(base + q_off + h * HALF_TILE), bd = smem_desc_sw128(base + k_off + h * k_half);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)          // 16 bf16 = 32 bytes = 2 descriptor address units
          umma_bf16(tmem_base, ad + (uint64_t)(2 * kk), bd + (uint64_t)(2 * kk), idesc, (h | kk) ? 1u : 0u);
      }
      umma_commit(bar_s);
    }
  }
  __syncwarp();

  // ---------------- softmax: TMEM lane = query row
  const int q = warp & 3, g = (warp >> 2) & 1, hf = warp >> 3;
  const int row = q * 32 + lane;
  const int qi = qtile * QT + row;
  const bool valid = qi < a.n_q;
  const int r = valid ? qi / a.G : 0;
  uint64_t mk0 = 0, mk1 = 0;
  if (valid) {
    mk0 = a.mask[(size_t)r * a.mask_words];
    if (a.mask_words > 1) mk1 = a.mask[(size_t)r * a.mask_words + 1];
  }
  const int n_grp = g < ng ? (group_keys(g) + 15) / 16 : 0;          // 16-key chunks of this warp's group
  const int c_lo = hf * 4 < n_grp ? hf * 4 : n_grp, c_hi = hf * 4 + 4 < n_grp ? hf * 4 + 4 : n_grp;
  const int key_g = k_begin + g * KG;
  const uint32_t t_s = tmem_base + ((uint32_t)(q * 32) << 16);
  bool ok = mbar_wait(bar_s, 0, abort_flag);
  tc_fence_after();
  POSS_TRACE_POINT(1);
  // Two passes over this thread's scores, 16 keys per TMEM load, as compact loops: a CTA runs this code once, so
  // every instruction is fetched cold and short bodies that iterate beat straight-line code.  Invisible keys become
  // -inf: they lose every maximum and their 2^x is an exact zero.
  auto chunk = [&](int c, uint32_t* sr) {
    tmem_ld16_async(t_s + (uint32_t)(g * KG + c * 16), sr);
    tmem_wait16(sr);
    const int key0 = key_g + c * 16;
    if (key0 + 16 > a.n_all) {                         // the chunk reaches the tree slots or the end
      // bit j = key0 + j is visible: 16 bits cut out of (all ones below n_all | the row's ancestor mask)
      const int t0 = key0 - a.n_all;                   // tree slot of the chunk's first key; > -16
      uint32_t vis;
      if (t0 >= 64) vis = t0 >= 128 ? 0u : (uint32_t)(mk1 >> (t0 - 64));
      else if (t0 > 48) vis = (uint32_t)(mk0 >> t0) | (uint32_t)(mk1 << (64 - t0));
      else if (t0 >= 0) vis = (uint32_t)(mk0 >> t0);
      else vis = ((uint32_t)mk0 << (-t0)) | ((1u << (-t0)) - 1u);
      const int n_valid = a.total - key0;              // keys of the chunk that exist
      if (n_valid < 16) vis &= (1u << (n_valid < 0 ? 0 : n_valid)) - 1u;
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if (!((vis >> j) & 1u)) sr[j] = 0xff800000u;
    }
  };
  {
    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
    if (ok) {
#pragma unroll 1
      for (int c = c_lo; c < c_hi; ++c) {
        uint32_t sr[16];
        chunk(c, sr);
#pragma unroll
        for (int j = 0; j < 16; ++j) mx[j & 3] = fmaxf(mx[j & 3], __uint_as_float(sr[j]));
      }
    }
    half_max[hf][g][row] = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
  }
  __syncthreads();
  {
    const float mraw = fmaxf(half_max[0][g][row], half_max[1][g][row]);
    // the scale is positive: the maximum of the scaled scores is the scaled maximum
    const float ms = mraw == -INFINITY ? 0.f : mraw * a.scale_log2;
    if (hf == 0) grp_m[g][row] = mraw == -INFINITY ? NEG_BIG : ms;
    float ls[4] = {0.f, 0.f, 0.f, 0.f};
    if (ok) {
#pragma unroll 1
      for (int c = c_lo; c < c_hi; ++c) {
        uint32_t sr[16];
        chunk(c, sr);
        uint32_t hi[8], lo[8];
#pragma unroll
        for (int j = 0; j < 16; j += 2) {
          const float p0 = ex2(fmaf(__uint_as_float(sr[j]), a.scale_log2, -ms));
          const float p1 = ex2(fmaf(__uint_as_float(sr[j + 1]), a.scale_log2, -ms));
          ls[j & 3] += p0;
          ls[(j & 3) + 1] += p1;
          split_pack(p0, p1, hi[j >> 1], lo[j >> 1]);
        }
        // A operand of P V: k-block of 64 keys, row = query row (128 bytes), 16-byte pieces swizzled by row
        const int kc = g * (KG / 16) + c;
        const uint32_t line = (uint32_t)(kc >> 2) * HALF_TILE + (uint32_t)row * 128u;
        const uint32_t pc = (uint32_t)(kc & 3) * 2u, sw = (uint32_t)(row & 7);
        *reinterpret_cast<uint4*>(base_ptr + p_hi + line + ((pc ^ sw) << 4)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4*>(base_ptr + p_hi + line + (((pc + 1) ^ sw) << 4)) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
        *reinterpret_cast<uint4*>(base_ptr + p_lo + line + ((pc ^ sw) << 4)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        *reinterpret_cast<uint4*>(base_ptr + p_lo + line + (((pc + 1) ^ sw) << 4)) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
      }
    }
    half_sum[hf][g][row] = (ls[0] + ls[1]) + (ls[2] + ls[3]);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // P becomes visible to the tensor core
  mbar_arrive(bar_p);
  POSS_TRACE_POINT(2);

  if (threadIdx.x == 0) {
    // ---------------- the second product, once the values and all of P are in shared memory
    const bool v_ok = mbar_wait(bar_v, 0, abort_flag);
    if (v_ok && mbar_wait(bar_p, 0, abort_flag) && *abort_flag == 0) {
      tc_fence_after();
      const uint32_t idesc = instr_desc_bf16(QT, D) | (1u << 16);     // B (the values) is MN-major
      for (int gg = 0; gg < ng; ++gg) {
        const int steps = (group_keys(gg) + 15) / 16;
        for (int ks = 0; ks < steps; ++ks) {
          const int kc = gg * (KG / 16) + ks;                         // 16-key step inside the CTA's keys
          const uint32_t pa = (uint32_t)(kc >> 2) * HALF_TILE;
          const uint64_t step = (uint64_t)(2 * (kc & 3));
          const uint64_t ah = smem_desc_sw128(base + p_hi + pa) + step, al = smem_desc_sw128(base + p_lo + pa) + step;
          const uint64_t bd = smem_desc_sw128_mn(base + v_off + (uint32_t)kc * 2048u, k_half);
          const uint32_t t_o = tmem_base + o_col + (uint32_t)(gg * D);
          umma_bf16(t_o, ah, bd, idesc, ks > 0 ? 1u : 0u);
          umma_bf16(t_o, al, bd, idesc, 1u);
        }
      }
      umma_commit(bar_o);
    }
    if (*abort_flag) {
      // drain: the copies this thread started must land before the CTA's shared memory goes away
      uint64_t t0 = global_ns();
      while (!mbar_try_wait(bar_qk, 0) && global_ns() - t0 < WAIT_LIMIT_NS / 4) __nanosleep(64);
      while (!mbar_try_wait(bar_v, 0) && global_ns() - t0 < WAIT_LIMIT_NS / 2) __nanosleep(64);
    }
  }
  __syncwarp();
  ok = mbar_wait(bar_o, 0, abort_flag);
  tc_fence_after();
  POSS_TRACE_POINT(3);
  __syncthreads();                  // every half's sum and every group's maximum are in place
  if (ok) {
    // park O in global memory (it stays in L2): this warp's 32 query rows, output columns [32 cq, 32 cq + 32), the
    // CTA's groups merged in key order (a group without keys accumulated nothing: it is left out, its TMEM columns
    // are not read)
    const int cq = warp >> 2;
    const bool two = ng == 2 && group_keys(1) > 0;
    const float m0 = grp_m[0][row], m1 = two ? grp_m[1][row] : NEG_BIG;
    const float l0 = half_sum[0][0][row] + half_sum[1][0][row];
    const float l1 = two ? half_sum[0][1][row] + half_sum[1][1][row] : 0.f;
    const float ms = fmaxf(m0, m1);
    const float c0 = ex2(m0 - ms), c1 = two ? ex2(m1 - ms) : 0.f;
    const uint32_t t_o = t_s + o_col + (uint32_t)(cq * 32);
    float* dst = a.part + (((size_t)r * a.Hq + kvh * a.G + (qi - r * a.G)) * a.n_splits + split) * O_LD;
    if (valid && cq == 0) *reinterpret_cast<float2*>(dst + D) = make_float2(ms, l0 * c0 + l1 * c1);
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
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  POSS_TRACE_POINT(4);

  // ---------------- merge over the cluster's CTAs, in key order: this CTA's share of the query rows.  The
  // partials were written before the cluster barrier (release / acquire at cluster scope) and are read past L1.
  {
    const int ns = a.n_splits;
    const int rank = (int)cluster_rank();
    const int row_lo = rank * QT / ns, row_hi = (rank + 1) * QT / ns;
#pragma unroll 1
    for (int item = threadIdx.x; item < (row_hi - row_lo) * 16; item += N_THREADS) {
      const int rr = row_lo + (item >> 4), cg = (item & 15) * 8;
      const int qj = qtile * QT + rr;
      if (qj >= a.n_q) continue;
      const int rj = qj / a.G, gj = qj - rj * a.G;
      const float* src = a.part + (((size_t)rj * a.Hq + kvh * a.G + gj) * ns) * O_LD;
      // every load is in flight before the first use
      float2 ml[MAX_SPLITS];
      float4 x0[MAX_SPLITS], x1[MAX_SPLITS];
#pragma unroll
      for (int j = 0; j < MAX_SPLITS; ++j) {
        if (j < ns) {
          ml[j] = __ldcg(reinterpret_cast<const float2*>(src + (size_t)j * O_LD + D));
          x0[j] = __ldcg(reinterpret_cast<const float4*>(src + (size_t)j * O_LD + cg));
          x1[j] = __ldcg(reinterpret_cast<const float4*>(src + (size_t)j * O_LD + cg + 4));
        }
      }
      float mm = NEG_BIG;
#pragma unroll
      for (int j = 0; j < MAX_SPLITS; ++j)
        if (j < ns) mm = fmaxf(mm, ml[j].x);
      float ll = 0.f, acc[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] = 0.f;
#pragma unroll
      for (int j = 0; j < MAX_SPLITS; ++j) {
        if (j < ns) {
          const float c = ex2(ml[j].x - mm);
          ll += ml[j].y * c;
          acc[0] += x0[j].x * c; acc[1] += x0[j].y * c; acc[2] += x0[j].z * c; acc[3] += x0[j].w * c;
          acc[4] += x1[j].x * c; acc[5] += x1[j].y * c; acc[6] += x1[j].z * c; acc[7] += x1[j].w * c;
        }
      }
      const float inv = 1.f / ll;
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        __nv_bfloat162 b = __floats2bfloat162_rn(acc[2 * j] * inv, acc[2 * j + 1] * inv);
        w[j] = *reinterpret_cast<uint32_t*>(&b);
      }
      *reinterpret_cast<uint4*>(a.out + ((size_t)rj * a.Hq + kvh * a.G + gj) * D + cg) = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }

  POSS_TRACE_POINT(5);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, tmem_cols);
  if (threadIdx.x == 0 && *abort_flag) atomicExch(a.status, (int)POSS_E_TIMEOUT);
}

}  // namespace

// ------------------------------------------------------------------ host side
// The cut of the keys: a function of the key count alone.  Two 128-key groups per CTA (one when there are no more
// than 128 keys), as many CTAs as the keys need.
bool tree_attention_tc_plan(int total, int* cta_keys, int* n_ctas) {
  if (total < 1 || total > MAX_SPLITS * MAX_CTA_KEYS) return false;
  *cta_keys = total <= KG ? KG : MAX_CTA_KEYS;
  *n_ctas = (total + *cta_keys - 1) / *cta_keys;
  return true;
}

bool tree_attention_tc_supported(const AttnArgs& a, const void* q, const void* kc, const void* vc, const void* out) {
  if (a.d != D || a.Hkv < 1 || a.Hq % a.Hkv) return false;
  const int G = a.Hq / a.Hkv;
  if (G > QT || QT % G) return false;
  const int total = a.n_all + a.n_tree;
  if (a.rows < 1 || total < 1 || total > MAX_SPLITS * MAX_CTA_KEYS) return false;
  if (a.mask_words > 2 || a.n_tree > 128) return false;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(kc) | reinterpret_cast<uintptr_t>(vc) |
       reinterpret_cast<uintptr_t>(out)) & 15)
    return false;
  return true;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool launch_tree_attention_tc(Launcher& L, TcGemmPlanCache* cache, const AttnArgs& a, const bf16* q, const bf16* kc,
                              const bf16* vc, float* part, bf16* out, int32_t* status) {
  if (!tree_attention_tc_supported(a, q, kc, vc, out) || !status || !part || (reinterpret_cast<uintptr_t>(part) & 15))
    return false;
  EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(tc_encode_fn(cache));
  if (!encode) return false;
  const int G = a.Hq / a.Hkv, total = a.n_all + a.n_tree;
  AttnTcArgs k;
  memset(&k, 0, sizeof(k));
  k.rows = a.rows; k.Hq = a.Hq; k.G = G; k.n_q = a.rows * G;
  k.n_all = a.n_all; k.n_tree = a.n_tree; k.total = total;
  if (!tree_attention_tc_plan(total, &k.cta_keys, &k.n_splits)) return false;
  k.mask = a.mask; k.mask_words = a.mask_words;
  k.scale_log2 = a.scale * 1.4426950408889634f;
  k.part = part; k.out = out; k.status = status;
  k.inject_lost_load = tc_take_injection(cache) ? 1 : 0;
  const uint32_t k_half = (uint32_t)k.cta_keys * 128u, p_bytes = 2u * (uint32_t)(k.cta_keys / 64) * HALF_TILE;
  uint32_t region_a = 2u * HALF_TILE + 2u * k_half;
  if (region_a < p_bytes) region_a = p_bytes;
  k.region_a_bytes = region_a;                       // a multiple of 1024 either way
  size_t smem = (size_t)region_a + 2u * k_half + 1024u;
  // At least half an SM's shared memory, so that two of these CTAs never share an SM: each holds up to all
  // of the SM's TMEM until its whole cluster has merged, and CTAs of two clusters queued behind each other's
  // TMEM on two SMs would wait forever.
  if (smem < 116u * 1024u) smem = 116u * 1024u;

  // The maps carry the call's extents (rows, key count): rows past them are filled with zeros by the copy.
  CUtensorMap mq, mk, mv;
  {
    cuuint64_t gdim[4] = {(cuuint64_t)D, (cuuint64_t)G, (cuuint64_t)a.Hkv, (cuuint64_t)a.rows};
    cuuint64_t gstr[3] = {(cuuint64_t)D * 2, (cuuint64_t)G * D * 2, (cuuint64_t)a.Hq * D * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)G, 1, (cuuint32_t)(QT / G)};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    if (encode(&mq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<bf16*>(q), gdim, gstr, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  for (int i = 0; i < 2; ++i) {
    cuuint64_t gdim[3] = {(cuuint64_t)D, (cuuint64_t)total, (cuuint64_t)a.Hkv};
    cuuint64_t gstr[2] = {(cuuint64_t)D * 2, (cuuint64_t)a.cap * D * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)k.cta_keys, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    if (encode(i ? &mv : &mk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<bf16*>(i ? vc : kc), gdim, gstr, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  // the shared-memory opt-in is a per-device property of the kernel
  static PerDeviceFlags attr_done;
  bool* attr = attr_done.current();
  if (!attr || !*attr) {
    if (cudaFuncSetAttribute(k_attn_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) return false;
    if (attr) *attr = true;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(k.n_splits, a.Hkv, (k.n_q + QT - 1) / QT);
  cfg.blockDim = dim3(N_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = L.stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  at[1].id = cudaLaunchAttributeClusterDimension;
  at[1].val.clusterDim.x = k.n_splits;
  at[1].val.clusterDim.y = 1;
  at[1].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 2;
  // A cluster shape the device does not take is reported at launch, before anything runs: remember it and
  // leave the call to the split-KV kernels.
  static PerDeviceFlags refused[MAX_SPLITS + 1];
  bool* ref = refused[k.n_splits].current();
  if (ref && *ref) return false;
  if (cudaLaunchKernelEx(&cfg, k_attn_tc, mq, mk, mv, k) != cudaSuccess) {
    cudaGetLastError();
    if (ref) *ref = true;
    return false;
  }
  ++*L.launches;
  return true;
}
