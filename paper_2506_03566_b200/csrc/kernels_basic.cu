// Element-wise stages and the SIMT skinny matrix product (check mode and odd shapes).
#include "poss_internal.cuh"

POSS_TRACE_REGISTER()

// ------------------------------------------------------------------ SIMT skinny GEMM
// out[m][n] = sum_k X[m][k] * W[n][k] (+ bias[n]) (+ residual[m][n]).  One warp per output column n,
// eight rows of X at a time in registers.  The reduction order of an output element depends only on
// K, never on M or on the row's place in the batch.
template <typename T> struct Vec8 { };
template <> struct Vec8<float> {
  float v[8];
  __device__ __forceinline__ void load(const float* p) {
    float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
};
template <> struct Vec8<bf16> {
  float v[8];
  __device__ __forceinline__ void load(const bf16* p) {
    uint4 a = *reinterpret_cast<const uint4*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&a);
#pragma unroll
    for (int i = 0; i < 4; ++i) { float2 f = __bfloat1622float2(h[i]); v[2 * i] = f.x; v[2 * i + 1] = f.y; }
  }
};

template <typename T>
__global__ void __launch_bounds__(256) k_gemm_simt(const T* X, int ldx, int M, GemmSegs segs, int N,
                                                   int K, const T* bias,
                                                   const float* residual, int ldr,
                                                   float* out, int ldo) {
  pdl_enter(POSS_K_GEMM_SIMT);
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int n = blockIdx.x * 8 + warp;
  if (n >= N) return;
  const T* wrow;
  {
    int nn = n, s = 0;
    while (s < segs.n - 1 && nn >= segs.rows[s]) { nn -= segs.rows[s]; ++s; }
    wrow = reinterpret_cast<const T*>(segs.w[s]) + (size_t)nn * K;
  }
  for (int m0 = 0; m0 < M; m0 += 8) {
    float acc[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) acc[r] = 0.f;
    for (int k0 = lane * 8; k0 < K; k0 += 256) {
      Vec8<T> wv;
      wv.load(wrow + k0);
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        if (m0 + r < M) {
          Vec8<T> xv;
          xv.load(X + (size_t)(m0 + r) * ldx + k0);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[r] = fmaf(xv.v[e], wv.v[e], acc[r]);
        }
      }
    }
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      float v = acc[r];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0 && m0 + r < M) {
        if (bias) v += to_f(bias[n]);
        if (residual) v += residual[(size_t)(m0 + r) * ldr + n];
        out[(size_t)(m0 + r) * ldo + n] = v;
      }
    }
  }
}

template <typename T>
void launch_gemm_simt(Launcher& L, const T* X, int ldx, int M, const GemmSegs& segs, int K, const T* bias,
                      const float* residual, int ldr, float* out, int ldo) {
  int N = 0;
  for (int i = 0; i < segs.n; ++i) N += segs.rows[i];
  if (M <= 0 || N <= 0) return;
  launch_pdl(L, k_gemm_simt<T>, dim3((N + 7) / 8), dim3(256), 0, X, ldx, M, segs, N, K, bias, residual, ldr, out, ldo);
}
template void launch_gemm_simt<float>(Launcher&, const float*, int, int, const GemmSegs&, int, const float*,
                                      const float*, int, float*, int);
template void launch_gemm_simt<bf16>(Launcher&, const bf16*, int, int, const GemmSegs&, int, const bf16*,
                                     const float*, int, float*, int);

// ------------------------------------------------------------------ layer-input pairs [E[tok] ; feature]
template <typename T>
__global__ void __launch_bounds__(256) k_gather_x(BatchRows s, const int32_t* new_tokens,
                                                  const T* new_features, TreeState ts, int Kmax,
                                                  const T* fb, int level_rows, const T* embed, int H,
                                                  T* X) {
  pdl_enter(POSS_K_GATHER_X);
  int m = blockIdx.x;
  RowRef r = batch_row(s, m);
  int tok;
  const T* feat;
  if (r.level == 0) {
    const int at = s.tok_off[r.seq] + r.j;
    tok = new_tokens[at];
    feat = new_features + (size_t)at * H;
  } else {
    const TreeState t = tree_of(ts, r.seq);
    tok = t.node_tok[r.level * Kmax + r.j];
    int prow = t.node_prow[r.level * Kmax + r.j];
    const int pmc = r.level == 1 ? 1 : s.K;                  // expanded rows per sequence at the parent's level
    feat = fb + ((size_t)(r.level - 1) * level_rows + r.seq * pmc + prow) * H;   // the parent's output feature
  }
  const T* e = embed + (size_t)tok * H;
  T* x = X + (size_t)m * 2 * H;
  constexpr int PER = 16 / sizeof(T);                        // elements per 16-byte piece
  bool vec = (H % PER) == 0 &&
             ((reinterpret_cast<uintptr_t>(e) | reinterpret_cast<uintptr_t>(feat) | reinterpret_cast<uintptr_t>(x)) & 15) == 0;
  if (vec) {
    int n = H / PER;
    const uint4* e4 = reinterpret_cast<const uint4*>(e);
    const uint4* f4 = reinterpret_cast<const uint4*>(feat);
    uint4* x4 = reinterpret_cast<uint4*>(x);
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      x4[i] = e4[i];
      x4[n + i] = f4[i];
    }
  } else {
    for (int i = threadIdx.x; i < H; i += blockDim.x) {
      x[i] = e[i];
      x[H + i] = feat[i];
    }
  }
}
template <typename T>
void launch_gather_x(Launcher& L, const BatchRows& s, const int32_t* new_tokens, const T* new_features,
                     const TreeState& ts, int Kmax, const T* fb, int level_rows, const T* embed, int H, T* X) {
  if (s.M <= 0) return;
  launch_pdl(L, k_gather_x<T>, dim3(s.M), dim3(256), 0, s, new_tokens, new_features, ts, Kmax, fb, level_rows, embed, H,
             X);
}
template void launch_gather_x<float>(Launcher&, const BatchRows&, const int32_t*, const float*, const TreeState&, int,
                                     const float*, int, const float*, int, float*);
template void launch_gather_x<bf16>(Launcher&, const BatchRows&, const int32_t*, const bf16*, const TreeState&, int,
                                    const bf16*, int, const bf16*, int, bf16*);

// ------------------------------------------------------------------ RMSNorm: out = T(gain * x / sqrt(mean x^2 + eps))
template <typename T>
__global__ void __launch_bounds__(256) k_rmsnorm(const float* x, int H, const T* gain,
                                                 float eps, T* out) {
  __shared__ float red[8];
  __shared__ float inv_s;
  pdl_enter(POSS_K_RMSNORM);
  const float* xr = x + (size_t)blockIdx.x * H;
  T* o = out + (size_t)blockIdx.x * H;
  if (gain == nullptr) {
    for (int i = threadIdx.x; i < H; i += 256) o[i] = from_f<T>(xr[i]);
    return;
  }
  // the row is summed in a fixed order: thread-strided partial sums, warp tree, then the eight warps
  const bool vec = (H & 3) == 0 && (reinterpret_cast<uintptr_t>(xr) & 15) == 0;
  float ss = 0.f;
  if (vec) {
    const float4* x4 = reinterpret_cast<const float4*>(xr);
    for (int i = threadIdx.x; i < H / 4; i += 256) {
      float4 v = x4[i];
      ss = fmaf(v.x, v.x, ss); ss = fmaf(v.y, v.y, ss); ss = fmaf(v.z, v.z, ss); ss = fmaf(v.w, v.w, ss);
    }
  } else {
    for (int i = threadIdx.x; i < H; i += 256) { float v = xr[i]; ss = fmaf(v, v, ss); }
  }
  for (int o2 = 16; o2 > 0; o2 >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o2);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < 8; ++w) t += red[w];
    inv_s = rsqrtf(t / (float)H + eps);
  }
  __syncthreads();
  float inv = inv_s;
  if (vec) {
    const float4* x4 = reinterpret_cast<const float4*>(xr);
    for (int i = threadIdx.x; i < H / 4; i += 256) {
      float4 v = x4[i];
      o[4 * i] = from_f<T>(v.x * inv * to_f(gain[4 * i]));
      o[4 * i + 1] = from_f<T>(v.y * inv * to_f(gain[4 * i + 1]));
      o[4 * i + 2] = from_f<T>(v.z * inv * to_f(gain[4 * i + 2]));
      o[4 * i + 3] = from_f<T>(v.w * inv * to_f(gain[4 * i + 3]));
    }
  } else {
    for (int i = threadIdx.x; i < H; i += 256) o[i] = from_f<T>(xr[i] * inv * to_f(gain[i]));
  }
}
template <typename T>
void launch_rmsnorm(Launcher& L, const float* x, int rows, int H, const T* gain, float eps, T* out) {
  if (rows <= 0) return;
  launch_pdl(L, k_rmsnorm<T>, dim3(rows), dim3(256), 0, x, H, gain, eps, out);
}
template void launch_rmsnorm<float>(Launcher&, const float*, int, int, const float*, float, float*);
template void launch_rmsnorm<bf16>(Launcher&, const float*, int, int, const bf16*, float, bf16*);

template <typename T>
__global__ void k_cast(const float* x, size_t n, T* out) {
  pdl_enter(POSS_K_CAST);
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = from_f<T>(x[i]);
}
template <typename T>
void launch_cast_rows(Launcher& L, const float* x, size_t n, T* out) {
  if (n == 0) return;
  launch_pdl(L, k_cast<T>, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, x, n, out);
}
template void launch_cast_rows<float>(Launcher&, const float*, size_t, float*);
template void launch_cast_rows<bf16>(Launcher&, const float*, size_t, bf16*);

// act = T(silu(gate) * up), gate/up stored side by side: gu[row][0..F) gate, [F..2F) up
template <typename T>
__global__ void k_silu_mul(const float* gu, int F, T* out) {
  pdl_enter(POSS_K_SILU_MUL);
  int row = blockIdx.y;
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= F) return;
  float g = gu[(size_t)row * 2 * F + i], u = gu[(size_t)row * 2 * F + F + i];
  out[(size_t)row * F + i] = from_f<T>(silu_f(g) * u);
}
template <typename T>
void launch_silu_mul(Launcher& L, const float* gu, int rows, int F, T* out) {
  if (rows <= 0) return;
  dim3 grid((F + 255) / 256, rows);
  launch_pdl(L, k_silu_mul<T>, grid, dim3(256), 0, gu, F, out);
}
template void launch_silu_mul<float>(Launcher&, const float*, int, int, float*);
template void launch_silu_mul<bf16>(Launcher&, const float*, int, int, bf16*);

// ------------------------------------------------------------------ consumers of a (possibly split-K) product
// Contributors of every tile, computed once per block.
__device__ __forceinline__ void fill_tile_table(const SplitKView& v, TileContrib* tab) {
  if (v.deferred)
    for (int t = threadIdx.x; t < v.n_tiles; t += blockDim.x) tab[t] = splitk_tile_contrib(v, t);
}
// four consecutive columns of row m starting at n (a multiple of 4); N = row length
__device__ __forceinline__ float4 product4(const SplitKView& v, const TileContrib* tab, int m, int n, int N) {
  if (v.deferred) {
    int tile, t;
    splitk_locate(v, n, &tile, &t);
    return splitk_load4(v, m, n, tab[tile], t);
  }
  const float* p = v.direct + (size_t)m * v.ld + n;
  if ((v.ld & 3) == 0 && n + 3 < N && (reinterpret_cast<uintptr_t>(v.direct) & 15) == 0)
    return *reinterpret_cast<const float4*>(p);
  float4 r;
  r.x = p[0];
  r.y = n + 1 < N ? p[1] : 0.f;
  r.z = n + 2 < N ? p[2] : 0.f;
  r.w = n + 3 < N ? p[3] : 0.f;
  return r;
}

// four consecutive elements at a 4-element-aligned position, as one access
template <typename T> __device__ __forceinline__ void load4(const T* p, float* o);
template <> __device__ __forceinline__ void load4<float>(const float* p, float* o) {
  float4 v = *reinterpret_cast<const float4*>(p);
  o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
}
template <> __device__ __forceinline__ void load4<bf16>(const bf16* p, float* o) {
  uint2 raw = *reinterpret_cast<const uint2*>(p);
  float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
  float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
  o[0] = a.x; o[1] = a.y; o[2] = b.x; o[3] = b.y;
}
template <typename T> __device__ __forceinline__ void store4(T* p, const float* v);
template <> __device__ __forceinline__ void store4<float>(float* p, const float* v) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
template <> __device__ __forceinline__ void store4<bf16>(bf16* p, const float* v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
  uint2 raw;
  raw.x = *reinterpret_cast<uint32_t*>(&a);
  raw.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = raw;
}
__device__ __forceinline__ bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// ------------------------------------------------------------------ embedding rows as fp32 (the target pass's input)
template <typename T>
__global__ void k_embed_rows(const int32_t* tokens, const T* embed, int H,
                             float* out) {
  pdl_enter(POSS_K_EMBED_ROWS);
  int m = blockIdx.x;
  const T* e = embed + (size_t)tokens[m] * H;
  float* o = out + (size_t)m * H;
  // four elements per access where the row allows it (the rows are cold: few, wide loads in flight together)
  if ((H & 3) == 0 && aligned16(o) && (reinterpret_cast<uintptr_t>(e) & (4 * sizeof(T) - 1)) == 0) {
    for (int i = threadIdx.x * 4; i < H; i += blockDim.x * 4) {
      float v[4];
      load4<T>(e + i, v);
      store4<float>(o + i, v);
    }
    return;
  }
  for (int i = threadIdx.x; i < H; i += blockDim.x) o[i] = to_f(e[i]);
}
template <typename T>
void launch_embed_rows(Launcher& L, const int32_t* tokens, int rows, const T* embed, int H, float* out) {
  if (rows <= 0) return;
  launch_pdl(L, k_embed_rows<T>, dim3(rows), dim3(256), 0, tokens, embed, H, out);
}
template void launch_embed_rows<float>(Launcher&, const int32_t*, int, const float*, int, float*);
template void launch_embed_rows<bf16>(Launcher&, const int32_t*, int, const bf16*, int, float*);


// four consecutive entries of a weight vector (bias, gain) as floats; `fill` where there is none
template <typename T>
__device__ __forceinline__ void load_w4(const T* w, int n, int N, bool vec, float fill, float* o) {
  o[0] = o[1] = o[2] = o[3] = fill;
  if (!w) return;
  if (vec) { load4<T>(w + n, o); return; }
#pragma unroll
  for (int q = 0; q < 4; ++q) if (n + q < N) o[q] = to_f(w[n + q]);
}

// ---- h = product + bias + residual (fp32, stored);  xn = T(gain * h / rms(h))
// One block per row.  The sum of squares is formed in a fixed order (per-thread partial sums over the
// thread's column groups, a warp tree, then the warps in order), so a row's result does not depend on
// the batch around it.  bias and gain are weights (no kernel writes them): they are read, and the
// contributors of every tile worked out, before the predecessor is awaited.
#define NORM_THREADS 1024
#define NORM_KEEP 2
template <typename T>
__global__ void __launch_bounds__(NORM_THREADS) k_reduce_norm(SplitKView prod, int H, const T* bias,
                                                               const float* residual, const T* gain, float eps,
                                                               float* h, T* xn) {
  __shared__ TileContrib tab[512];
  __shared__ float red[NORM_THREADS / 32];
  __shared__ float inv_s;
  pdl_begin();
  fill_tile_table(prod, tab);
  const int m = blockIdx.x;
  const int n_groups = (H + 3) / 4;
  // whole 16-byte (fp32) / 8-byte (bf16) accesses when the row length and every base pointer allow it
  const bool vec = (H & 3) == 0 && aligned16(h) && aligned16(xn) && (!residual || aligned16(residual)) &&
                   (!bias || aligned16(bias)) && (!gain || aligned16(gain));
  float kb[NORM_KEEP][4], kg[NORM_KEEP][4];
#pragma unroll
  for (int k = 0; k < NORM_KEEP; ++k) {
    const int g = threadIdx.x + k * NORM_THREADS;
    if (g < n_groups) {
      load_w4<T>(bias, g * 4, H, vec, 0.f, kb[k]);
      load_w4<T>(gain, g * 4, H, vec, 1.f, kg[k]);
    }
  }
  __syncthreads();
  pdl_sync(POSS_K_REDUCE_NORM);
  POSS_TRACE_POINT(1);
  float ss = 0.f;
  // value of one group of four columns: product + (residual + bias), stored to h, squares added to ss
  auto group_value = [&](int g, const float* b4) {
    const int n = g * 4;
    float add[4] = {0.f, 0.f, 0.f, 0.f};
    if (residual) {
      if (vec) load4<float>(residual + (size_t)m * H + n, add);
      else {
#pragma unroll
        for (int q = 0; q < 4; ++q) if (n + q < H) add[q] = residual[(size_t)m * H + n + q];
      }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) add[q] += b4[q];
    float4 v = product4(prod, tab, m, n, H);
    float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (n + q < H) {
        e[q] += add[q];
        ss = fmaf(e[q], e[q], ss);
      } else {
        e[q] = 0.f;
      }
    }
    if (vec) store4<float>(h + (size_t)m * H + n, e);
    else {
#pragma unroll
      for (int q = 0; q < 4; ++q) if (n + q < H) h[(size_t)m * H + n + q] = e[q];
    }
    return make_float4(e[0], e[1], e[2], e[3]);
  };
  auto group_store = [&](int g, float4 v, float inv, const float* g4) {
    const int n = g * 4;
    float e[4] = {v.x, v.y, v.z, v.w};
    if (gain) {
#pragma unroll
      for (int q = 0; q < 4; ++q) e[q] = e[q] * inv * g4[q];
    }
    if (vec) store4<T>(xn + (size_t)m * H + n, e);
    else {
#pragma unroll
      for (int q = 0; q < 4; ++q) if (n + q < H) xn[(size_t)m * H + n + q] = from_f<T>(e[q]);
    }
  };
  float4 keep[NORM_KEEP];
#pragma unroll
  for (int k = 0; k < NORM_KEEP; ++k) {
    int g = threadIdx.x + k * NORM_THREADS;
    keep[k] = g < n_groups ? group_value(g, kb[k]) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (int g = threadIdx.x + NORM_KEEP * NORM_THREADS; g < n_groups; g += NORM_THREADS) {
    float b4[4];
    load_w4<T>(bias, g * 4, H, vec, 0.f, b4);
    group_value(g, b4);
  }
  POSS_TRACE_POINT(2);
  for (int o2 = 16; o2 > 0; o2 >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o2);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < NORM_THREADS / 32; ++w) t += red[w];
    inv_s = gain ? rsqrtf(t / (float)H + eps) : 1.f;
  }
  __syncthreads();
  const float inv = inv_s;
#pragma unroll
  for (int k = 0; k < NORM_KEEP; ++k) {
    int g = threadIdx.x + k * NORM_THREADS;
    if (g < n_groups) group_store(g, keep[k], inv, kg[k]);
  }
  for (int g = threadIdx.x + NORM_KEEP * NORM_THREADS; g < n_groups; g += NORM_THREADS) {
    const int n = g * 4;                                    // wider rows: re-read this thread's own stores
    float4 v;
    v.x = h[(size_t)m * H + n];
    v.y = n + 1 < H ? h[(size_t)m * H + n + 1] : 0.f;
    v.z = n + 2 < H ? h[(size_t)m * H + n + 2] : 0.f;
    v.w = n + 3 < H ? h[(size_t)m * H + n + 3] : 0.f;
    float g4[4];
    load_w4<T>(gain, n, H, vec, 1.f, g4);
    group_store(g, v, inv, g4);
  }
}
template <typename T>
void launch_reduce_norm(Launcher& L, const SplitKView& prod, int rows, int H, const T* bias, const float* residual,
                        const T* gain, float eps, float* h, T* xn) {
  if (rows <= 0) return;
  launch_pdl(L, k_reduce_norm<T>, dim3(rows), dim3(NORM_THREADS), 0, prod, H, bias, residual, gain, eps, h, xn);
}
template void launch_reduce_norm<float>(Launcher&, const SplitKView&, int, int, const float*, const float*,
                                        const float*, float, float*, float*);
template void launch_reduce_norm<bf16>(Launcher&, const SplitKView&, int, int, const bf16*, const float*, const bf16*,
                                       float, float*, bf16*);

// ---- out = product + bias + residual, optionally also in the activation dtype
template <typename T>
__global__ void __launch_bounds__(256) k_splitk_reduce(SplitKView prod, int N, const T* bias, const float* residual,
                                                       int ldr, float* out, int ldo, T* out_act) {
  pdl_enter(POSS_K_SPLITK_REDUCE);
  const int m = blockIdx.y;
  const int n = (blockIdx.x * 256 + threadIdx.x) * 4;
  if (n >= N) return;
  float4 v;
  if (prod.deferred) {
    int tile, t;
    splitk_locate(prod, n, &tile, &t);
    TileContrib tc = splitk_tile_contrib(prod, tile);
    v = splitk_load4(prod, m, n, tc, t);
  } else {
    v = product4(prod, nullptr, m, n, N);
  }
  float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    if (n + q < N) {
      if (bias) e[q] += to_f(bias[n + q]);
      if (residual) e[q] += residual[(size_t)m * ldr + n + q];
      if (out) out[(size_t)m * ldo + n + q] = e[q];
      if (out_act) out_act[(size_t)m * ldo + n + q] = from_f<T>(e[q]);
    }
  }
}
template <typename T>
void launch_splitk_reduce(Launcher& L, const SplitKView& prod, int rows, int N, const T* bias, const float* residual,
                          int ldr, float* out, int ldo, T* out_act) {
  if (rows <= 0) return;
  launch_pdl(L, k_splitk_reduce<T>, dim3((N + 1023) / 1024, rows), dim3(256), 0, prod, N, bias, residual, ldr, out, ldo,
             out_act);
}
template void launch_splitk_reduce<float>(Launcher&, const SplitKView&, int, int, const float*, const float*, int,
                                          float*, int, float*);
template void launch_splitk_reduce<bf16>(Launcher&, const SplitKView&, int, int, const bf16*, const float*, int, float*,
                                         int, bf16*);

// ---- act = T(silu(gate) * up) from the parked partials of a SwiGLU product
// One block per (tile of 64 ffn columns, 32 rows): 16 threads across the tile's columns (four each), two
// rows per thread.  The tile, and with it the contributor list, is the same for the whole block.
template <typename T>
__global__ void __launch_bounds__(256) k_splitk_swiglu(SplitKView prod, int M, int F, T* act) {
  pdl_begin();
  const TileContrib tc = splitk_tile_contrib(prod, blockIdx.x);
  const int cg = (threadIdx.x & 15) * 4;
  const int f = blockIdx.x * 64 + cg;
  const int m0 = blockIdx.y * 32 + (threadIdx.x >> 4), m1 = m0 + 16;
  const int l0 = m0 < M ? m0 : M - 1, l1 = m1 < M ? m1 : M - 1;      // rows loaded (clamped), stored if < M
  const int off[4] = {l0 * 128 + cg, l0 * 128 + cg + 64, l1 * 128 + cg, l1 * 128 + cg + 64};
  const bool vec = (F & 3) == 0 && (reinterpret_cast<uintptr_t>(act) & 15) == 0;
  pdl_sync(POSS_K_SPLITK_SWIGLU);
  if (f >= F || m0 >= M) return;
  float4 x[4];
  splitk_sum<4>(prod, tc, off, x);
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int m = r ? m1 : m0;
    if (m >= M) break;
    const float gv[4] = {x[2 * r].x, x[2 * r].y, x[2 * r].z, x[2 * r].w};
    const float uv[4] = {x[2 * r + 1].x, x[2 * r + 1].y, x[2 * r + 1].z, x[2 * r + 1].w};
    float e[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) e[q] = silu_f(gv[q]) * uv[q];
    if (vec) store4<T>(act + (size_t)m * F + f, e);
    else {
#pragma unroll
      for (int q = 0; q < 4; ++q) if (f + q < F) act[(size_t)m * F + f + q] = from_f<T>(e[q]);
    }
  }
}
template <typename T>
void launch_splitk_swiglu(Launcher& L, const SplitKView& prod, int rows, int F, T* act) {
  if (rows <= 0) return;
  launch_pdl(L, k_splitk_swiglu<T>, dim3(prod.n_tiles, (rows + 31) / 32), dim3(256), 0, prod, rows, F, act);
}
template void launch_splitk_swiglu<float>(Launcher&, const SplitKView&, int, int, float*);
template void launch_splitk_swiglu<bf16>(Launcher&, const SplitKView&, int, int, bf16*);

// ------------------------------------------------------------------ rotary embedding + KV append + q
// The product's row layout is [Hq*d q | Hkv*d k | Hkv*d v] fp32.  Rotate-half pairing (j, j + d/2).
// The angle pos * theta^(-2j/d) is formed in double from a table of the d/2 inverse frequencies and
// reduced to [-pi, pi] in double (2 pi split in two terms), so long positions lose nothing; sine and
// cosine of the reduced angle are then taken in fp32.
// A block serves one row and ROPE_ITEMS work items (an item: four neighbouring pairs of one head, i.e. two
// 16-byte groups of the product, or four values of v).  Its last two warps form the row's cos/sin table
// while the item threads have their loads of the product in flight.  Item decoding and the contributors
// of every tile need only the launch parameters and are done before the predecessor is awaited.
#define ROPE_ITEMS 256
template <typename T>
__global__ void __launch_bounds__(ROPE_ITEMS + 64) k_rope_append(RopeArgs a, SplitKView qkv, CachePtrs caches,
                                                                  T* qout) {
  __shared__ TileContrib tab[512];
  __shared__ __align__(16) float cs[64], sn[64];
  pdl_begin();
  fill_tile_table(qkv, tab);
  const int m = blockIdx.x;
  const int half = a.d / 2;
  const int qd = a.Hq * a.d, kd = a.Hkv * a.d, N = qd + 2 * kd;
  const int q0 = a.rows - a.q_rows;
  const bool with_q = m >= q0;
  const int per_head = half / 4;                         // items per rotated head (d is a multiple of 8)
  const int n_qitems = with_q ? a.Hq * per_head : 0;
  const int n_kitems = a.Hkv * per_head;
  const int n_items = n_qitems + n_kitems + kd / 4;
  const bool item_thread = threadIdx.x < ROPE_ITEMS;
  const int i = blockIdx.y * ROPE_ITEMS + threadIdx.x;
  const bool active = item_thread && i < n_items;
  // kind 0 = q, 1 = k (rotated), 2 = v; hh = head, j = first of the four elements inside the head
  int kind = 2, hh = 0, j = 0, col = 0;
  if (active) {
    if (i < n_qitems + n_kitems) {
      kind = i < n_qitems ? 0 : 1;
      const int ii = kind == 0 ? i : i - n_qitems;
      hh = ii / per_head;
      j = (ii - hh * per_head) * 4;
      col = (kind == 0 ? 0 : qd) + hh * a.d + j;
    } else {
      const int ii = (i - n_qitems - n_kitems) * 4;
      hh = ii / a.d;
      j = ii - hh * a.d;
      col = qd + kd + ii;
    }
  }
  int tile_lo = 0, t_lo = 0, tile_hi = 0, t_hi = 0;
  if (active && qkv.deferred) {
    splitk_locate(qkv, col, &tile_lo, &t_lo);
    if (kind != 2) splitk_locate(qkv, col + half, &tile_hi, &t_hi);
  }
  int slot, pos, seq = 0;
  if (a.mode == 0) {
    RowRef r = batch_row(a.s, m);
    seq = r.seq;
    slot = row_slot(a.s, r);
    pos = row_pos(a.s, r);
  } else {
    slot = a.base + m;
  }
  T* kcache = reinterpret_cast<T*>(caches.k[seq]);
  T* vcache = reinterpret_cast<T*>(caches.v[seq]);
  const bool vec = aligned16(kcache) && aligned16(vcache) && (a.q_rows == 0 || aligned16(qout));
  __syncthreads();
  pdl_sync(POSS_K_ROPE_APPEND);
  if (a.mode != 0) pos = a.base + a.depth[m];
  float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
  if (!item_thread) {
    const int jj = threadIdx.x - ROPE_ITEMS;
    if (jj < half) {
      const double two_pi_hi = 6.283185307179586, two_pi_lo = 2.4492935982947064e-16;
      double x = (double)pos * a.inv_freq[jj];
      double k = rint(x * 0.15915494309189535);
      double r = fma(-k, two_pi_hi, x);
      r = fma(-k, two_pi_lo, r);
      float sv, cv;
      sincosf((float)r, &sv, &cv);
      cs[jj] = cv;
      sn[jj] = sv;
    }
  } else if (active) {
    if (!qkv.deferred) {
      lo = product4(qkv, tab, m, col, N);
      if (kind != 2) hi = product4(qkv, tab, m, col + half, N);
    } else if (kind == 2) {
      lo = splitk_load4(qkv, m, col, tab[tile_lo], t_lo);
    } else if (tile_lo == tile_hi) {
      const int off[2] = {m * 128 + t_lo, m * 128 + t_hi};
      float4 x[2];
      splitk_sum<2>(qkv, tab[tile_lo], off, x);
      lo = x[0];
      hi = x[1];
    } else {
      lo = splitk_load4(qkv, m, col, tab[tile_lo], t_lo);
      hi = splitk_load4(qkv, m, col + half, tab[tile_hi], t_hi);
    }
  }
  __syncthreads();
  POSS_TRACE_POINT(1);
  if (!active) return;
  if (kind == 2) {
    T* dst = vcache + ((size_t)hh * a.cap + slot) * a.d + j;
    const float e[4] = {lo.x, lo.y, lo.z, lo.w};
    if (vec) store4<T>(dst, e);
    else { dst[0] = from_f<T>(e[0]); dst[1] = from_f<T>(e[1]); dst[2] = from_f<T>(e[2]); dst[3] = from_f<T>(e[3]); }
    return;
  }
  const float x0[4] = {lo.x, lo.y, lo.z, lo.w}, x1[4] = {hi.x, hi.y, hi.z, hi.w};
  float r0[4], r1[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    r0[e] = x0[e] * cs[j + e] - x1[e] * sn[j + e];
    r1[e] = x1[e] * cs[j + e] + x0[e] * sn[j + e];
  }
  T* dst = kind == 0 ? qout + (size_t)(m - q0) * qd + hh * a.d : kcache + ((size_t)hh * a.cap + slot) * a.d;
  if (vec) {
    store4<T>(dst + j, r0);
    store4<T>(dst + j + half, r1);
  } else {
#pragma unroll
    for (int e = 0; e < 4; ++e) { dst[j + e] = from_f<T>(r0[e]); dst[j + e + half] = from_f<T>(r1[e]); }
  }
  POSS_TRACE_POINT(2);
}
template <typename T>
void launch_rope_append(Launcher& L, const RopeArgs& a, const SplitKView& qkv, const CachePtrs& caches, T* qout) {
  if (a.rows <= 0) return;
  const int per_head = a.d / 8;
  const int n_items = (a.q_rows > 0 ? a.Hq * per_head : 0) + a.Hkv * per_head + a.Hkv * a.d / 4;
  launch_pdl(L, k_rope_append<T>, dim3(a.rows, (n_items + ROPE_ITEMS - 1) / ROPE_ITEMS), dim3(ROPE_ITEMS + 64), 0, a, qkv,
             caches, qout);
}
template void launch_rope_append<float>(Launcher&, const RopeArgs&, const SplitKView&, const CachePtrs&, float*);
template void launch_rope_append<bf16>(Launcher&, const RopeArgs&, const SplitKView&, const CachePtrs&, bf16*);

// chain mask / depth for causal prefill chunks: row r sees rows 0..r of its chunk
__global__ void k_chain_mask(uint64_t* mask, int32_t* depth, int rows) {
  pdl_enter(POSS_K_CHAIN_MASK);
  int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= rows) return;
  depth[r] = r;
  uint64_t lo, hi;
  if (r < 63) { lo = (2ull << r) - 1ull; hi = 0; }
  else if (r == 63) { lo = ~0ull; hi = 0; }
  else { lo = ~0ull; hi = (r - 64 == 63) ? ~0ull : ((2ull << (r - 64)) - 1ull); }
  mask[2 * r] = lo;
  mask[2 * r + 1] = hi;
}
void launch_chain_mask(Launcher& L, uint64_t* mask, int32_t* depth, int rows) {
  launch_pdl(L, k_chain_mask, dim3((rows + 127) / 128), dim3(128), 0, mask, depth, rows);
}
