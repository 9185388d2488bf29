// Split-KV tree attention (decode style).
//
// A query row sees every cache slot in [0, n_all) and the slots n_all + j whose bit j is set in the
// row's packed ancestor mask.  Work is split over (key range, KV head, row): a block owns one row and
// one KV head, handles all G = Hq/Hkv query heads of that KV head together (every key/value is loaded
// once per block), and walks its key range 128 keys at a time (4 warps x 32 keys, one key per lane for
// the scores; one slice of the head dimension per lane for the weighted sum).  Each block writes an
// online-softmax partial (m, l, o[d]); a second kernel merges the partials in split order, so the
// result does not depend on scheduling.
#include "poss_internal.cuh"

POSS_TRACE_REGISTER()

#define NEG_BIG (-1.0e30f)

template <typename T, int D> struct KeyLoad;
template <int D> struct KeyLoad<bf16, D> {
  // dot products of one key (D bf16, 16-byte loads) with G query vectors held in shared memory
  template <int G>
  static __device__ __forceinline__ void dots(const bf16* k, const float* qs, float* s) {
#pragma unroll
    for (int c = 0; c < D / 8; ++c) {
      uint4 raw = *reinterpret_cast<const uint4*>(k + c * 8);
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
      float kv[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) { float2 f = __bfloat1622float2(h[i]); kv[2 * i] = f.x; kv[2 * i + 1] = f.y; }
#pragma unroll
      for (int g = 0; g < G; ++g) {
#pragma unroll
        for (int e = 0; e < 8; ++e) s[g] = fmaf(kv[e], qs[g * D + c * 8 + e], s[g]);
      }
    }
  }
};
template <int D> struct KeyLoad<float, D> {
  template <int G>
  static __device__ __forceinline__ void dots(const float* k, const float* qs, float* s) {
#pragma unroll
    for (int c = 0; c < D / 4; ++c) {
      float4 raw = *reinterpret_cast<const float4*>(k + c * 4);
      float kv[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int g = 0; g < G; ++g) {
#pragma unroll
        for (int e = 0; e < 4; ++e) s[g] = fmaf(kv[e], qs[g * D + c * 4 + e], s[g]);
      }
    }
  }
};

template <typename T, int D, int G>
__global__ void __launch_bounds__(128) k_attn_partial(AttnArgs a, const T* q,
                                                      const T* kcache, const T* vcache,
                                                      float* part) {
  constexpr int PER = D / 32;                 // head-dim elements owned by a lane in the PV phase
  __shared__ float qs[G * D];
  __shared__ float sm_m[4][G], sm_l[4][G];
  __shared__ float sm_o[4][G][D];
  pdl_enter(POSS_K_ATTN_PARTIAL);
  int split = blockIdx.x, kvh = blockIdx.y, row = blockIdx.z;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = threadIdx.x; i < G * D; i += 128)
    qs[i] = to_f(q[((size_t)row * a.Hq + kvh * G) * D + i]);
  __syncthreads();
  const T* kb = kcache + (size_t)kvh * a.cap * D;
  const T* vb = vcache + (size_t)kvh * a.cap * D;
  int total = a.n_all + a.n_tree;
  int k_begin = split * a.keys_per_split;
  int k_end = min(total, k_begin + a.keys_per_split);
  const uint64_t* mrow = a.mask + (size_t)row * a.mask_words;

  float m[G], l[G], o[G][PER];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m[g] = NEG_BIG; l[g] = 0.f;
#pragma unroll
    for (int e = 0; e < PER; ++e) o[g][e] = 0.f;
  }
  for (int base = k_begin + warp * 32; base < k_end; base += 128) {
    int j = base + lane;
    bool vis = j < k_end;
    if (vis && j >= a.n_all) {
      int t = j - a.n_all;
      vis = (mrow[t >> 6] >> (t & 63)) & 1ull;
    }
    float s[G];
#pragma unroll
    for (int g = 0; g < G; ++g) s[g] = 0.f;
    if (vis) KeyLoad<T, D>::template dots<G>(kb + (size_t)j * D, qs, s);
    float p[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float sv = vis ? s[g] * a.scale : NEG_BIG;
      float mx = sv;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
      float mn = fmaxf(m[g], mx);
      float corr = __expf(m[g] - mn);
      p[g] = vis ? __expf(sv - mn) : 0.f;
      float ps = p[g];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, off);
      l[g] = l[g] * corr + ps;
      m[g] = mn;
#pragma unroll
      for (int e = 0; e < PER; ++e) o[g][e] *= corr;
    }
    int cnt = min(32, k_end - base);
    for (int jj = 0; jj < cnt; ++jj) {
      float pj[G];
      bool any = false;
#pragma unroll
      for (int g = 0; g < G; ++g) { pj[g] = __shfl_sync(0xffffffffu, p[g], jj); any |= pj[g] != 0.f; }
      if (!any) continue;
      const T* vp = vb + (size_t)(base + jj) * D + lane * PER;
      float vv[PER];
#pragma unroll
      for (int e = 0; e < PER; ++e) vv[e] = to_f(vp[e]);
#pragma unroll
      for (int g = 0; g < G; ++g)
#pragma unroll
        for (int e = 0; e < PER; ++e) o[g][e] = fmaf(pj[g], vv[e], o[g][e]);
    }
  }
  // merge the four warps in warp order
#pragma unroll
  for (int g = 0; g < G; ++g) {
    if (lane == 0) { sm_m[warp][g] = m[g]; sm_l[warp][g] = l[g]; }
#pragma unroll
    for (int e = 0; e < PER; ++e) sm_o[warp][g][lane * PER + e] = o[g][e];
  }
  __syncthreads();
  for (int i = threadIdx.x; i < G * D; i += 128) {
    int g = i / D, e = i % D;
    float mm = fmaxf(fmaxf(sm_m[0][g], sm_m[1][g]), fmaxf(sm_m[2][g], sm_m[3][g]));
    float ll = 0.f, oo = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      float c = __expf(sm_m[w][g] - mm);
      ll += sm_l[w][g] * c;
      oo += sm_o[w][g][e] * c;
    }
    size_t pidx = ((size_t)row * a.Hq + kvh * G + g) * a.n_splits + split;
    float* pp = part + pidx * (D + 2);
    if (e == 0) { pp[0] = mm; pp[1] = ll; }
    pp[2 + e] = oo;
  }
}

template <typename T, int D>
__global__ void k_attn_combine(int n_splits, const float* part, T* out) {
  pdl_enter(POSS_K_ATTN_COMBINE);
  int rh = blockIdx.x;       // row * Hq + head
  int e = threadIdx.x;
  const float* pp = part + (size_t)rh * n_splits * (D + 2);
  float mm = NEG_BIG;
  for (int s = 0; s < n_splits; ++s) mm = fmaxf(mm, pp[s * (D + 2)]);
  float ll = 0.f, oo = 0.f;
  for (int s = 0; s < n_splits; ++s) {
    float c = __expf(pp[s * (D + 2)] - mm);
    ll += pp[s * (D + 2) + 1] * c;
    oo += pp[s * (D + 2) + 2 + e] * c;
  }
  out[(size_t)rh * D + e] = from_f<T>(oo / ll);
}

size_t attn_partial_floats(int rows, int Hq, int d, int n_splits) {
  return (size_t)rows * Hq * n_splits * (d + 2);
}

void plan_attention_splits(int rows, int Hkv, int total_keys, int max_splits, int* n_splits, int* keys_per_split) {
  // enough blocks for ~4 per SM, at least 128 keys per block, whole 128-key steps per split
  int want = (148 * 4 + rows * Hkv - 1) / (rows * Hkv);
  int by_keys = (total_keys + 127) / 128;
  int ns = want < 1 ? 1 : want;
  if (ns > by_keys) ns = by_keys;
  if (ns > max_splits) ns = max_splits;
  if (ns < 1) ns = 1;
  int kps = (total_keys + ns - 1) / ns;
  kps = (kps + 127) / 128 * 128;
  ns = (total_keys + kps - 1) / kps;
  if (ns < 1) ns = 1;
  *n_splits = ns;
  *keys_per_split = kps;
}

template <typename T, int D, int G>
static void launch_attn_g(Launcher& L, const AttnArgs& a, const T* q, const T* kc, const T* vc, float* part, T* out) {
  dim3 grid(a.n_splits, a.Hkv, a.rows);
  launch_pdl(L, k_attn_partial<T, D, G>, grid, dim3(128), 0, a, q, kc, vc, part);
  launch_pdl(L, k_attn_combine<T, D>, dim3(a.rows * a.Hq), dim3(D), 0, a.n_splits, (const float*)part, out);
}
template <typename T, int D>
static void launch_attn_d(Launcher& L, const AttnArgs& a, const T* q, const T* kc, const T* vc, float* part, T* out) {
  switch (a.Hq / a.Hkv) {
    case 1: launch_attn_g<T, D, 1>(L, a, q, kc, vc, part, out); break;
    case 2: launch_attn_g<T, D, 2>(L, a, q, kc, vc, part, out); break;
    case 3: launch_attn_g<T, D, 3>(L, a, q, kc, vc, part, out); break;
    case 4: launch_attn_g<T, D, 4>(L, a, q, kc, vc, part, out); break;
    case 8: launch_attn_g<T, D, 8>(L, a, q, kc, vc, part, out); break;
    default: L.err = POSS_E_SHAPE;
  }
}
template <typename T>
void launch_tree_attention(Launcher& L, const AttnArgs& a, const T* q, const T* kc, const T* vc, float* part,
                           T* out) {
  if (a.rows <= 0) return;
  switch (a.d) {
    case 32: launch_attn_d<T, 32>(L, a, q, kc, vc, part, out); break;
    case 64: launch_attn_d<T, 64>(L, a, q, kc, vc, part, out); break;
    case 128: launch_attn_d<T, 128>(L, a, q, kc, vc, part, out); break;
    default: L.err = POSS_E_SHAPE;
  }
}
template void launch_tree_attention<float>(Launcher&, const AttnArgs&, const float*, const float*, const float*,
                                           float*, float*);
template void launch_tree_attention<bf16>(Launcher&, const AttnArgs&, const bf16*, const bf16*, const bf16*, float*,
                                          bf16*);

template <>
void run_tree_attention<float>(Launcher& L, AttnArgs a, int max_splits, const float* q, const float* kc,
                               const float* vc, float* part, float* out) {
  a.splits_per_block = 1;
  plan_attention_splits(a.rows, a.Hkv, a.n_all + a.n_tree, max_splits, &a.n_splits, &a.keys_per_split);
  launch_tree_attention<float>(L, a, q, kc, vc, part, out);
}
template <>
void run_tree_attention<bf16>(Launcher& L, AttnArgs a, int max_splits, const bf16* q, const bf16* kc, const bf16* vc,
                              float* part, bf16* out) {
  a.splits_per_block = 1;
  if (tree_attention_mma_supported(a)) {
    plan_attention_splits_mma(a.rows, a.Hq, a.Hkv, a.n_all + a.n_tree, max_splits, &a.n_splits, &a.keys_per_split,
                              &a.splits_per_block);
    launch_tree_attention_mma(L, a, q, kc, vc, part, out);
    return;
  }
  plan_attention_splits(a.rows, a.Hkv, a.n_all + a.n_tree, max_splits, &a.n_splits, &a.keys_per_split);
  launch_tree_attention<bf16>(L, a, q, kc, vc, part, out);
}
