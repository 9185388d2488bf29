// Split-KV tree attention on mma.sync tensor cores (bf16): the kernel for what the tcgen05 kernel does not take
// (head dimension 64, more than 10240 keys, callers without a context workspace) and the comparison partner of
// the tcgen05 kernel in the tests.
//
// Geometry.  For one KV head the G = Hq/Hkv query heads of all tree rows form one matrix Q' of
// rows*G query rows (query row qi = r*G + g).  A block owns (key split, KV head, 64 query rows); each of
// its four warps owns 16 query rows.  The block walks its key range 64 keys at a time: K and V chunks
// are staged in shared memory with 16-byte cp.async copies (double buffered, padded rows so that
// ldmatrix is conflict free), S = Q'K^T and O += P V run on mma.sync m16n8k16 with fp32 accumulators,
// the online softmax lives in registers (row max / row sum reduced with warp shuffles inside a quad).
//
// Precision.  Scores, softmax and the weighted sum are fp32 as in the SIMT kernel: the probabilities
// enter the P V product as an exact two-term bf16 split (p = hi + lo, two MMAs), so nothing is rounded
// to bf16 beyond q, k and v themselves.
//
// Visibility.  Keys [0, n_all) are seen by every row; key n_all + t is seen by row r iff bit t of the
// row's packed ancestor mask is set.  Each block writes an online-softmax partial (m, l, o[d]) per query
// row; k_attn_combine merges the partials in split order.  With one split the block writes the result.
#include "poss_internal.cuh"
#include <string.h>

POSS_TRACE_REGISTER()

namespace {

constexpr float NEG_BIG = -1.0e30f;
constexpr int CHUNK = 64;           // keys per shared-memory stage
constexpr int QROWS = 64;           // query rows per block (16 per warp)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  int sz = valid ? 16 : 0;          // size 0: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                                  uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// p = hi + lo with hi = bf16(p), lo = bf16(p - hi); packs two values (low half = first)
__device__ __forceinline__ void split_pack(float x, float y, uint32_t& hi, uint32_t& lo) {
  __nv_bfloat16 xh = __float2bfloat16_rn(x), yh = __float2bfloat16_rn(y);
  __nv_bfloat16 xl = __float2bfloat16_rn(x - __bfloat162float(xh)), yl = __float2bfloat16_rn(y - __bfloat162float(yh));
  hi = (uint32_t)__bfloat16_as_ushort(xh) | ((uint32_t)__bfloat16_as_ushort(yh) << 16);
  lo = (uint32_t)__bfloat16_as_ushort(xl) | ((uint32_t)__bfloat16_as_ushort(yl) << 16);
}

// NW = warps per block: 4 (64 query rows) or, when one KV head has at most 16 query rows, 1
template <int D, int NW>
__global__ void __launch_bounds__(32 * NW) k_attn_mma(AttnArgs a, const bf16* q,
                                                  const bf16* kcache, const bf16* vcache,
                                                  float* part, bf16* out) {
  constexpr int LD = D + 8;                       // padded shared-memory row, elements
  constexpr int KSTEPS = D / 16;                  // k-steps of Q K^T
  constexpr int NT_D = D / 8;                     // n-tiles of the output
  extern __shared__ __align__(16) unsigned char smem_attn[];
  bf16* Ks = reinterpret_cast<bf16*>(smem_attn);  // [2][CHUNK][LD]
  bf16* Vs = Ks + 2 * CHUNK * LD;                 // [2][CHUNK][LD]

  pdl_enter(POSS_K_ATTN_MMA);

  const int split = blockIdx.x, kvh = blockIdx.y, qtile = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = a.Hq / a.Hkv;
  const int n_q = a.rows * G;                     // query rows of this KV head
  const int quad = lane >> 2, tq = lane & 3;
  const int qi0 = qtile * (16 * NW) + warp * 16 + quad, qi1 = qi0 + 8;
  const bool v0 = qi0 < n_q, v1 = qi1 < n_q;
  const int r0 = v0 ? qi0 / G : 0, r1 = v1 ? qi1 / G : 0;
  const bool warp_active = qtile * (16 * NW) + warp * 16 < n_q;

  // the block walks splits_per_block consecutive splits as one chunk sequence and emits one partial per
  // split: how many splits a block takes is a scheduling choice, the grouping of the sums is not
  const int total = a.n_all + a.n_tree;
  const int split0 = split * a.splits_per_block;
  const int k_begin = split0 * a.keys_per_split;
  const int k_end = min(total, k_begin + a.splits_per_block * a.keys_per_split);
  const int n_chunks = (k_end - k_begin + CHUNK - 1) / CHUNK;
  const int chunks_per_split = a.keys_per_split / CHUNK;
  const bf16* kb = kcache + (size_t)kvh * a.cap * D;
  const bf16* vb = vcache + (size_t)kvh * a.cap * D;

  auto load_chunk = [&](int c, int stage) {
    const int key0 = k_begin + c * CHUNK;
    bf16* kd = Ks + (size_t)stage * CHUNK * LD;
    bf16* vd = Vs + (size_t)stage * CHUNK * LD;
    constexpr int PER_ROW = D / 8;                // 16-byte pieces per key
    for (int i = threadIdx.x; i < CHUNK * PER_ROW; i += 32 * NW) {
      int kr = i / PER_ROW, piece = i % PER_ROW;
      int key = key0 + kr;
      bool ok = key < k_end;
      size_t off = (size_t)(ok ? key : k_begin) * D + piece * 8;
      cp_async16(smem_u32(kd + kr * LD + piece * 8), kb + off, ok);
      cp_async16(smem_u32(vd + kr * LD + piece * 8), vb + off, ok);
    }
    cp_async_commit();
  };

  if (n_chunks > 0) load_chunk(0, 0);

  // query fragments (A operand), straight from global memory
  uint32_t qf[KSTEPS][4];
  {
    const bf16* q0 = q + ((size_t)r0 * a.Hq + kvh * G + (v0 ? qi0 % G : 0)) * D;
    const bf16* q1 = q + ((size_t)r1 * a.Hq + kvh * G + (v1 ? qi1 % G : 0)) * D;
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
      int c = kk * 16 + tq * 2;
      qf[kk][0] = v0 ? *reinterpret_cast<const uint32_t*>(q0 + c) : 0u;
      qf[kk][1] = v1 ? *reinterpret_cast<const uint32_t*>(q1 + c) : 0u;
      qf[kk][2] = v0 ? *reinterpret_cast<const uint32_t*>(q0 + c + 8) : 0u;
      qf[kk][3] = v1 ? *reinterpret_cast<const uint32_t*>(q1 + c + 8) : 0u;
    }
  }
  // ancestor masks of this thread's two rows (at most two 64-bit words: 128 tree slots)
  uint64_t mk0a = 0, mk0b = 0, mk1a = 0, mk1b = 0;
  if (v0) { mk0a = a.mask[(size_t)r0 * a.mask_words]; if (a.mask_words > 1) mk0b = a.mask[(size_t)r0 * a.mask_words + 1]; }
  if (v1) { mk1a = a.mask[(size_t)r1 * a.mask_words]; if (a.mask_words > 1) mk1b = a.mask[(size_t)r1 * a.mask_words + 1]; }

  POSS_TRACE_POINT(1);
  float m0 = NEG_BIG, m1 = NEG_BIG, l0 = 0.f, l1 = 0.f;
  float o[NT_D][4];
#pragma unroll
  for (int j = 0; j < NT_D; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }

  // online-softmax partial (m, l, o[d]) of one split for this thread's two query rows
  auto write_partial = [&](int sp) {
    if (v0) {
      float* pp = part + (((size_t)r0 * a.Hq + kvh * G + qi0 % G) * a.n_splits + sp) * (D + 2);
      if (tq == 0) { pp[0] = m0; pp[1] = l0; }
#pragma unroll
      for (int j = 0; j < NT_D; ++j) *reinterpret_cast<float2*>(pp + 2 + j * 8 + tq * 2) = make_float2(o[j][0], o[j][1]);
    }
    if (v1) {
      float* pp = part + (((size_t)r1 * a.Hq + kvh * G + qi1 % G) * a.n_splits + sp) * (D + 2);
      if (tq == 0) { pp[0] = m1; pp[1] = l1; }
#pragma unroll
      for (int j = 0; j < NT_D; ++j) *reinterpret_cast<float2*>(pp + 2 + j * 8 + tq * 2) = make_float2(o[j][2], o[j][3]);
    }
  };

  for (int c = 0; c < n_chunks; ++c) {
    const int stage = c & 1;
    if (c + 1 < n_chunks) { load_chunk(c + 1, stage ^ 1); cp_async_wait<1>(); }
    else cp_async_wait<0>();
    __syncthreads();
    if (warp_active) {
      const bf16* kd = Ks + (size_t)stage * CHUNK * LD;
      const bf16* vd = Vs + (size_t)stage * CHUNK * LD;
      const int key0 = k_begin + c * CHUNK;
      // ---- S = Q K^T for 16 query rows x 64 keys
      float s[CHUNK / 8][4];
#pragma unroll
      for (int j = 0; j < CHUNK / 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
      // k-steps outside, key tiles inside: consecutive MMAs write different accumulators and pipeline
      // (each accumulator still receives its k-steps in order 0, 1, 2, ...)
#pragma unroll
      for (int kk = 0; kk < KSTEPS; kk += 2) {
#pragma unroll
        for (int j = 0; j < CHUNK / 8; ++j) {
          uint32_t b0, b1, b2, b3;
          uint32_t addr = smem_u32(kd + (j * 8 + (lane & 7)) * LD + kk * 16 + (lane >> 3) * 8);
          ldmatrix_x4(addr, b0, b1, b2, b3);
          mma_bf16(s[j], qf[kk], b0, b1);
          mma_bf16(s[j], qf[kk + 1], b2, b3);
        }
      }
      // ---- scale, visibility, online softmax
      const bool need_mask = key0 + CHUNK > a.n_all;     // the chunk reaches into the tree slots or past the end
      float cmax0 = NEG_BIG, cmax1 = NEG_BIG;
#pragma unroll
      for (int j = 0; j < CHUNK / 8; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float sv = s[j][e] * a.scale;
          if (need_mask) {
            int key = key0 + j * 8 + tq * 2 + (e & 1);
            bool vis = key < k_end;
            if (vis && key >= a.n_all) {
              int t = key - a.n_all;
              uint64_t wsel = (e < 2) ? (t < 64 ? mk0a : mk0b) : (t < 64 ? mk1a : mk1b);
              vis = t < 128 && ((wsel >> (t & 63)) & 1ull);
            }
            if (!vis) sv = NEG_BIG;
          }
          s[j][e] = sv;
          if (e < 2) cmax0 = fmaxf(cmax0, sv); else cmax1 = fmaxf(cmax1, sv);
        }
      }
      cmax0 = fmaxf(cmax0, __shfl_xor_sync(0xffffffffu, cmax0, 1));
      cmax0 = fmaxf(cmax0, __shfl_xor_sync(0xffffffffu, cmax0, 2));
      cmax1 = fmaxf(cmax1, __shfl_xor_sync(0xffffffffu, cmax1, 1));
      cmax1 = fmaxf(cmax1, __shfl_xor_sync(0xffffffffu, cmax1, 2));
      const float mn0 = fmaxf(m0, cmax0), mn1 = fmaxf(m1, cmax1);
      const float corr0 = __expf(m0 - mn0), corr1 = __expf(m1 - mn1);
      float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
      for (int j = 0; j < CHUNK / 8; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float sv = s[j][e];
          float p = sv > 0.5f * NEG_BIG ? __expf(sv - (e < 2 ? mn0 : mn1)) : 0.f;
          s[j][e] = p;
          if (e < 2) ps0 += p; else ps1 += p;
        }
      }
      ps0 += __shfl_xor_sync(0xffffffffu, ps0, 1);
      ps0 += __shfl_xor_sync(0xffffffffu, ps0, 2);
      ps1 += __shfl_xor_sync(0xffffffffu, ps1, 1);
      ps1 += __shfl_xor_sync(0xffffffffu, ps1, 2);
      l0 = l0 * corr0 + ps0;
      l1 = l1 * corr1 + ps1;
      m0 = mn0;
      m1 = mn1;
#pragma unroll
      for (int j = 0; j < NT_D; ++j) { o[j][0] *= corr0; o[j][1] *= corr0; o[j][2] *= corr1; o[j][3] *= corr1; }
      // ---- O += P V, probabilities as an exact hi + lo bf16 pair
#pragma unroll
      for (int ks = 0; ks < CHUNK / 16; ++ks) {
        uint32_t ph[4], pl[4];
        split_pack(s[2 * ks][0], s[2 * ks][1], ph[0], pl[0]);
        split_pack(s[2 * ks][2], s[2 * ks][3], ph[1], pl[1]);
        split_pack(s[2 * ks + 1][0], s[2 * ks + 1][1], ph[2], pl[2]);
        split_pack(s[2 * ks + 1][2], s[2 * ks + 1][3], ph[3], pl[3]);
#pragma unroll
        for (int jd = 0; jd < NT_D; jd += 2) {
          uint32_t b0, b1, b2, b3;
          uint32_t addr = smem_u32(vd + (ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LD + (jd + (lane >> 4)) * 8);
          ldmatrix_x4_trans(addr, b0, b1, b2, b3);
          mma_bf16(o[jd], ph, b0, b1);
          mma_bf16(o[jd + 1], ph, b2, b3);
          mma_bf16(o[jd], pl, b0, b1);
          mma_bf16(o[jd + 1], pl, b2, b3);
        }
      }
      // last chunk of a split (but not of the block): hand the split's partial over and start afresh
      if (a.n_splits > 1 && (c + 1) % chunks_per_split == 0 && c + 1 < n_chunks) {
        write_partial(split0 + c / chunks_per_split);
        m0 = m1 = NEG_BIG;
        l0 = l1 = 0.f;
#pragma unroll
        for (int j = 0; j < NT_D; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
      }
    }
    __syncthreads();          // the stage is overwritten by the load issued in the next iteration
  }

  POSS_TRACE_POINT(2);
  if (!warp_active) return;
  if (a.n_splits == 1) {
    const float inv0 = 1.f / l0, inv1 = 1.f / l1;
#pragma unroll
    for (int j = 0; j < NT_D; ++j) {
      int dcol = j * 8 + tq * 2;
      if (v0) {
        __nv_bfloat162 w = __floats2bfloat162_rn(o[j][0] * inv0, o[j][1] * inv0);
        *reinterpret_cast<__nv_bfloat162*>(out + ((size_t)r0 * a.Hq + kvh * G + qi0 % G) * D + dcol) = w;
      }
      if (v1) {
        __nv_bfloat162 w = __floats2bfloat162_rn(o[j][2] * inv1, o[j][3] * inv1);
        *reinterpret_cast<__nv_bfloat162*>(out + ((size_t)r1 * a.Hq + kvh * G + qi1 % G) * D + dcol) = w;
      }
    }
    return;
  }
  write_partial(split0 + (n_chunks - 1) / chunks_per_split);
}

// One warp per (row, head), four warps per block.  Lane s loads split s's (m, l) (at most 32 splits); the
// maximum comes from a warp reduction, the normaliser and the outputs are added over the splits in split
// order.  A lane owns D/32 output elements as pairs (2*lane, 2*lane+1) (+64 for the second pair of D = 128):
// 8-byte loads, eight splits in flight at once.
template <int D>
__global__ void __launch_bounds__(128) k_attn_combine_bf16(int n_splits, int n_rh, const float* part, bf16* out) {
  constexpr int NP = D / 64;             // pairs per lane
  pdl_enter(POSS_K_ATTN_COMBINE_BF16);
  const int lane = threadIdx.x & 31;
  const int rh = blockIdx.x * 4 + (threadIdx.x >> 5);       // row * Hq + head
  if (rh >= n_rh) return;
  const float* pp = part + (size_t)rh * n_splits * (D + 2);
  float pm = NEG_BIG, pl = 0.f;
  if (lane < n_splits) {
    float2 ml = __ldcg(reinterpret_cast<const float2*>(pp + lane * (D + 2)));
    pm = ml.x;
    pl = ml.y;
  }
  float mm = pm;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, o));
  const float c_lane = lane < n_splits ? __expf(pm - mm) : 0.f;
  const float lc_lane = pl * c_lane;
  float ll = 0.f;
  float2 oo[NP];
#pragma unroll
  for (int h = 0; h < NP; ++h) oo[h] = make_float2(0.f, 0.f);
  const float* pe = pp + 2 + 2 * lane;
  for (int base = 0; base < n_splits; base += 8) {
    float2 po[8][NP];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (base + u < n_splits) {
#pragma unroll
        for (int h = 0; h < NP; ++h) po[u][h] = __ldcg(reinterpret_cast<const float2*>(pe + (base + u) * (D + 2) + 64 * h));
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (base + u < n_splits) {
        const float c = __shfl_sync(0xffffffffu, c_lane, base + u);
        ll += __shfl_sync(0xffffffffu, lc_lane, base + u);
#pragma unroll
        for (int h = 0; h < NP; ++h) { oo[h].x += po[u][h].x * c; oo[h].y += po[u][h].y * c; }
      }
    }
  }
#pragma unroll
  for (int h = 0; h < NP; ++h)
    *reinterpret_cast<__nv_bfloat162*>(out + (size_t)rh * D + 2 * lane + 64 * h) = __floats2bfloat162_rn(oo[h].x / ll, oo[h].y / ll);
}

template <int D, int NW>
void launch_dn(Launcher& L, const AttnArgs& a, const bf16* q, const bf16* kc, const bf16* vc, float* part, bf16* out) {
  constexpr size_t smem = (size_t)2 * 2 * CHUNK * (D + 8) * sizeof(bf16);
  static PerDeviceFlags attr_done;             // one per instantiation; the opt-in is per device
  bool* attr = attr_done.current();
  if (!attr || !*attr) {
    if (cudaFuncSetAttribute(k_attn_mma<D, NW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
      L.err = POSS_E_CUDA;
      return;
    }
    if (attr) *attr = true;
  }
  int G = a.Hq / a.Hkv;
  int q_tiles = (a.rows * G + 16 * NW - 1) / (16 * NW);
  int spb = a.splits_per_block < 1 ? 1 : a.splits_per_block;
  launch_pdl(L, k_attn_mma<D, NW>, dim3((a.n_splits + spb - 1) / spb, a.Hkv, q_tiles), dim3(32 * NW), smem, a, q, kc, vc,
             part, out);
  if (a.n_splits > 1)
    launch_pdl(L, k_attn_combine_bf16<D>, dim3((a.rows * a.Hq + 3) / 4), dim3(128), 0, a.n_splits, a.rows * a.Hq,
               (const float*)part, out);
}
template <int D>
void launch_d(Launcher& L, const AttnArgs& a, const bf16* q, const bf16* kc, const bf16* vc, float* part, bf16* out) {
  // few query rows per KV head (multi-head attention with a short row batch): one-warp blocks, so that the
  // grid has more, shorter blocks instead of blocks with three idle warps
  if (a.rows * (a.Hq / a.Hkv) <= 16) launch_dn<D, 1>(L, a, q, kc, vc, part, out);
  else launch_dn<D, 4>(L, a, q, kc, vc, part, out);
}

}  // namespace

bool tree_attention_mma_supported(const AttnArgs& a) {
  return (a.d == 64 || a.d == 128) && a.mask_words <= 2 && a.n_tree <= 128 && a.Hq % a.Hkv == 0;
}

void plan_attention_splits_mma(int rows, int Hq, int Hkv, int total_keys, int max_splits, int* n_splits,
                               int* keys_per_split, int* splits_per_block) {
  // The key range is cut into whole 64-key chunks, as many splits as the partial buffer allows.  The cut
  // depends on the key count alone, never on the rows or heads: a token's attention is then summed in the
  // same grouping whether it is verified as one of 61 tree rows or decoded alone, which is what lets the
  // speculative stream reproduce the plain decode bit for bit while the accepted path is the root.
  // (Short blocks also finish sooner: a block's work is a chain of dependent MMAs.)
  int chunks = (total_keys + CHUNK - 1) / CHUNK;
  int ns = chunks;
  if (ns > max_splits) ns = max_splits;
  if (ns > 32) ns = 32;                             // the combine kernel keeps one split per lane
  if (ns < 1) ns = 1;
  int cps = (chunks + ns - 1) / ns;
  int kps = cps * CHUNK;
  ns = (total_keys + kps - 1) / kps;
  if (ns < 1) ns = 1;
  *n_splits = ns;
  *keys_per_split = kps;
  // scheduling only: consecutive splits per block so that about two blocks land on every SM
  int nq = rows * (Hq / Hkv);
  int q_tiles = nq <= 16 ? 1 : (nq + QROWS - 1) / QROWS;
  int per_sm = nq <= 16 ? 3 : 2;                    // blocks that fit an SM at once
  int spb = (ns * Hkv * q_tiles + 74 * per_sm) / (148 * per_sm);
  if (spb < 1) spb = 1;
  *splits_per_block = spb;
}

void launch_tree_attention_mma(Launcher& L, const AttnArgs& a, const bf16* q, const bf16* kc, const bf16* vc,
                               float* part, bf16* out) {
  if (a.rows <= 0) return;
  if (a.d == 128) launch_d<128>(L, a, q, kc, vc, part, out);
  else if (a.d == 64) launch_d<64>(L, a, q, kc, vc, part, out);
  else L.err = POSS_E_SHAPE;
}
