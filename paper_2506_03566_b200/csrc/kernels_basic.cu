// Element-wise stages and the SIMT skinny matrix product (check mode and odd shapes).
#include "poss_internal.cuh"

#define LAUNCH_CHECK(L)                                         \
  do {                                                          \
    ++*(L).launches;                                            \
    if (cudaGetLastError() != cudaSuccess) (L).err = POSS_E_CUDA; \
  } while (0)

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
__global__ void __launch_bounds__(256) k_gemm_simt(const T* __restrict__ X, int ldx, int M, GemmSegs segs, int N,
                                                   int K, const T* __restrict__ bias,
                                                   const float* __restrict__ residual, int ldr,
                                                   float* __restrict__ out, int ldo) {
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
  k_gemm_simt<T><<<(N + 7) / 8, 256, 0, L.stream>>>(X, ldx, M, segs, N, K, bias, residual, ldr, out, ldo);
  LAUNCH_CHECK(L);
}
template void launch_gemm_simt<float>(Launcher&, const float*, int, int, const GemmSegs&, int, const float*,
                                      const float*, int, float*, int);
template void launch_gemm_simt<bf16>(Launcher&, const bf16*, int, int, const GemmSegs&, int, const bf16*,
                                     const float*, int, float*, int);

// ------------------------------------------------------------------ layer-input pairs [E[tok] ; feature]
template <typename T>
__global__ void k_gather_x(StepRows s, const int32_t* __restrict__ new_tokens, const T* __restrict__ new_features,
                           const int32_t* __restrict__ node_tok, const int32_t* __restrict__ node_prow, int Kmax,
                           const T* __restrict__ fb, const T* __restrict__ embed, int H, T* __restrict__ X) {
  int m = blockIdx.x;
  RowInfo r = row_info(s, m);
  int tok;
  const T* feat;
  if (r.level == 0) {
    tok = new_tokens[r.j];
    feat = new_features + (size_t)r.j * H;
  } else {
    tok = node_tok[r.level * Kmax + r.j];
    int prow = node_prow[r.level * Kmax + r.j];
    feat = fb + ((size_t)(r.level - 1) * Kmax + prow) * H;   // the parent's output feature
  }
  const T* e = embed + (size_t)tok * H;
  T* x = X + (size_t)m * 2 * H;
  for (int i = threadIdx.x; i < H; i += blockDim.x) {
    x[i] = e[i];
    x[H + i] = feat[i];
  }
}
template <typename T>
void launch_gather_x(Launcher& L, StepRows s, const int32_t* new_tokens, const T* new_features,
                     const TreeState& ts, int Kmax, const T* fb, const T* embed, int H, T* X) {
  if (s.M <= 0) return;
  k_gather_x<T><<<s.M, 256, 0, L.stream>>>(s, new_tokens, new_features, ts.node_tok, ts.node_prow, Kmax, fb, embed,
                                           H, X);
  LAUNCH_CHECK(L);
}
template void launch_gather_x<float>(Launcher&, StepRows, const int32_t*, const float*, const TreeState&, int,
                                     const float*, const float*, int, float*);
template void launch_gather_x<bf16>(Launcher&, StepRows, const int32_t*, const bf16*, const TreeState&, int,
                                    const bf16*, const bf16*, int, bf16*);

template <typename T>
__global__ void k_embed_rows(const int32_t* __restrict__ tokens, const T* __restrict__ embed, int H,
                             float* __restrict__ out) {
  int m = blockIdx.x;
  const T* e = embed + (size_t)tokens[m] * H;
  for (int i = threadIdx.x; i < H; i += blockDim.x) out[(size_t)m * H + i] = to_f(e[i]);
}
template <typename T>
void launch_embed_rows(Launcher& L, const int32_t* tokens, int rows, const T* embed, int H, float* out) {
  if (rows <= 0) return;
  k_embed_rows<T><<<rows, 256, 0, L.stream>>>(tokens, embed, H, out);
  LAUNCH_CHECK(L);
}
template void launch_embed_rows<float>(Launcher&, const int32_t*, int, const float*, int, float*);
template void launch_embed_rows<bf16>(Launcher&, const int32_t*, int, const bf16*, int, float*);

// ------------------------------------------------------------------ RMSNorm: out = T(gain * x / sqrt(mean x^2 + eps))
template <typename T>
__global__ void __launch_bounds__(256) k_rmsnorm(const float* __restrict__ x, int H, const T* __restrict__ gain,
                                                 float eps, T* __restrict__ out) {
  __shared__ float red[8];
  __shared__ float inv_s;
  const float* xr = x + (size_t)blockIdx.x * H;
  T* o = out + (size_t)blockIdx.x * H;
  if (gain == nullptr) {
    for (int i = threadIdx.x; i < H; i += 256) o[i] = from_f<T>(xr[i]);
    return;
  }
  float ss = 0.f;
  for (int i = threadIdx.x; i < H; i += 256) { float v = xr[i]; ss = fmaf(v, v, ss); }
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
  for (int i = threadIdx.x; i < H; i += 256) o[i] = from_f<T>(xr[i] * inv * to_f(gain[i]));
}
template <typename T>
void launch_rmsnorm(Launcher& L, const float* x, int rows, int H, const T* gain, float eps, T* out) {
  if (rows <= 0) return;
  k_rmsnorm<T><<<rows, 256, 0, L.stream>>>(x, H, gain, eps, out);
  LAUNCH_CHECK(L);
}
template void launch_rmsnorm<float>(Launcher&, const float*, int, int, const float*, float, float*);
template void launch_rmsnorm<bf16>(Launcher&, const float*, int, int, const bf16*, float, bf16*);

template <typename T>
__global__ void k_cast(const float* __restrict__ x, size_t n, T* __restrict__ out) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = from_f<T>(x[i]);
}
template <typename T>
void launch_cast_rows(Launcher& L, const float* x, size_t n, T* out) {
  if (n == 0) return;
  k_cast<T><<<(unsigned)((n + 255) / 256), 256, 0, L.stream>>>(x, n, out);
  LAUNCH_CHECK(L);
}
template void launch_cast_rows<float>(Launcher&, const float*, size_t, float*);
template void launch_cast_rows<bf16>(Launcher&, const float*, size_t, bf16*);

__global__ void k_widen_bf16(const bf16* __restrict__ x, size_t n, float* __restrict__ out) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = __bfloat162float(x[i]);
}
void launch_widen_bf16(Launcher& L, const bf16* x, size_t n, float* out) {
  if (n == 0) return;
  k_widen_bf16<<<(unsigned)((n + 255) / 256), 256, 0, L.stream>>>(x, n, out);
  LAUNCH_CHECK(L);
}

// act = T(silu(gate) * up), gate/up stored side by side: gu[row][0..F) gate, [F..2F) up
template <typename T>
__global__ void k_silu_mul(const float* __restrict__ gu, int F, T* __restrict__ out) {
  int row = blockIdx.y;
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= F) return;
  float g = gu[(size_t)row * 2 * F + i], u = gu[(size_t)row * 2 * F + F + i];
  float s = g / (1.f + expf(-g));
  out[(size_t)row * F + i] = from_f<T>(s * u);
}
template <typename T>
void launch_silu_mul(Launcher& L, const float* gu, int rows, int F, T* out) {
  if (rows <= 0) return;
  dim3 grid((F + 255) / 256, rows);
  k_silu_mul<T><<<grid, 256, 0, L.stream>>>(gu, F, out);
  LAUNCH_CHECK(L);
}
template void launch_silu_mul<float>(Launcher&, const float*, int, int, float*);
template void launch_silu_mul<bf16>(Launcher&, const float*, int, int, bf16*);

// ------------------------------------------------------------------ rotary embedding + KV append + q
// qkv row layout: [Hq*d q | Hkv*d k | Hkv*d v] fp32.  Rotate-half pairing (j, j + d/2), angle
// pos * theta^(-2j/d) evaluated in double so that long positions lose nothing.
template <typename T>
__global__ void __launch_bounds__(128) k_rope_append(RopeArgs a, const float* __restrict__ qkv,
                                                     T* __restrict__ kcache, T* __restrict__ vcache,
                                                     T* __restrict__ qout) {
  __shared__ float cs[64], sn[64];
  int m = blockIdx.x;
  int slot, pos;
  if (a.mode == 0) {
    RowInfo r = row_info(a.s, m);
    slot = row_slot(a.s, r);
    pos = row_pos(a.s, r);
  } else {
    slot = a.base + m;
    pos = a.base + a.depth[m];
  }
  int half = a.d / 2;
  if ((int)threadIdx.x < half) {
    double inv = exp2(-2.0 * (double)threadIdx.x / (double)a.d * log2((double)a.theta));
    double s, c;
    sincos((double)pos * inv, &s, &c);
    cs[threadIdx.x] = (float)c;
    sn[threadIdx.x] = (float)s;
  }
  __syncthreads();
  int qd = a.Hq * a.d, kd = a.Hkv * a.d;
  const float* row = qkv + (size_t)m * (qd + 2 * kd);
  // keys
  for (int i = threadIdx.x; i < a.Hkv * half; i += blockDim.x) {
    int h = i / half, j = i % half;
    float x0 = row[qd + h * a.d + j], x1 = row[qd + h * a.d + j + half];
    T* dst = kcache + ((size_t)h * a.cap + slot) * a.d;
    dst[j] = from_f<T>(x0 * cs[j] - x1 * sn[j]);
    dst[j + half] = from_f<T>(x1 * cs[j] + x0 * sn[j]);
  }
  // values
  for (int i = threadIdx.x; i < kd; i += blockDim.x) {
    int h = i / a.d, j = i % a.d;
    vcache[((size_t)h * a.cap + slot) * a.d + j] = from_f<T>(row[qd + kd + i]);
  }
  // queries of the current rows
  int q0 = a.rows - a.q_rows;
  if (m >= q0) {
    T* qo = qout + (size_t)(m - q0) * qd;
    for (int i = threadIdx.x; i < a.Hq * half; i += blockDim.x) {
      int h = i / half, j = i % half;
      float x0 = row[h * a.d + j], x1 = row[h * a.d + j + half];
      qo[h * a.d + j] = from_f<T>(x0 * cs[j] - x1 * sn[j]);
      qo[h * a.d + j + half] = from_f<T>(x1 * cs[j] + x0 * sn[j]);
    }
  }
}
template <typename T>
void launch_rope_append(Launcher& L, const RopeArgs& a, const float* qkv, T* kcache, T* vcache, T* qout) {
  if (a.rows <= 0) return;
  k_rope_append<T><<<a.rows, 128, 0, L.stream>>>(a, qkv, kcache, vcache, qout);
  LAUNCH_CHECK(L);
}
template void launch_rope_append<float>(Launcher&, const RopeArgs&, const float*, float*, float*, float*);
template void launch_rope_append<bf16>(Launcher&, const RopeArgs&, const float*, bf16*, bf16*, bf16*);

// chain mask / depth for causal prefill chunks: row r sees rows 0..r of its chunk
__global__ void k_chain_mask(uint64_t* mask, int32_t* depth, int rows) {
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
  k_chain_mask<<<(rows + 127) / 128, 128, 0, L.stream>>>(mask, depth, rows);
  LAUNCH_CHECK(L);
}
