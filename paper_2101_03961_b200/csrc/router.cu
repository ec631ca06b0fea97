// Router kernels of the Switch FFN layer, float32 throughout (Section 2.4, selective precision):
//   forward : h = x W_r (+ b), p = softmax(h) (Eq. 1), e_t = argmax_i p[t,i], g_t = p[t,e_t] (Switch routing, k = 1),
//             per-block partial sums of p for P_i (Eq. 6)
//   backward: G = d_aux.alpha.E.f_i/T + [i = e_t, kept].dgate_t ; dh = p (G - <p,G>) ; dW_r = x^T dh ; dx += dh W_r^T
// The logits are a [T,d]x[d,E] product with E flop per byte of x: FP32-FMA bound, so the kernels are register-tiled
// FFMA loops with the softmax / argmax done by warp shuffles on the accumulators.
#include "switch_common.cuh"

namespace swmoe {
namespace {

constexpr int kKC = 32;                      // contraction chunk staged in shared memory
constexpr int kTokPerWarp = 8;
constexpr int kFwdThreads = 256;             // 8 warps x 8 tokens = kRouterBlockTokens

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename XT> struct Vec16;
template <> struct Vec16<float> { static constexpr int n = 4; };
template <> struct Vec16<__nv_bfloat16> { static constexpr int n = 8; };

// Loads 16 bytes of row `src` (may be null = zero fill) and writes them as floats to dst.
template <typename XT>
__device__ __forceinline__ void load16_as_f32(const XT* src, float* dst) {
  if constexpr (sizeof(XT) == 4) {
    float4 v = src ? *reinterpret_cast<const float4*>(src) : make_float4(0.f, 0.f, 0.f, 0.f);
    *reinterpret_cast<float4*>(dst) = v;
  } else {
    uint4 raw = src ? *reinterpret_cast<const uint4*>(src) : make_uint4(0, 0, 0, 0);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
    float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
    float2 c = __bfloat1622float2(h[2]), e = __bfloat1622float2(h[3]);
    *reinterpret_cast<float4*>(dst) = make_float4(a.x, a.y, b.x, b.y);
    *reinterpret_cast<float4*>(dst + 4) = make_float4(c.x, c.y, e.x, e.y);
  }
}

// ------------------------------------------------------------------------------------------------ forward
template <typename XT, int NE>
__global__ void __launch_bounds__(kFwdThreads)
router_fwd_kernel(const XT* __restrict__ x, const float* __restrict__ W_r, const float* __restrict__ bias,
                  const float* __restrict__ noise, int T, int d,
                  int E, float* __restrict__ probs, int* __restrict__ expert_index, float* __restrict__ gate,
                  float* __restrict__ psum_partial) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int EP = 32 * NE;
  constexpr int XS = kKC + 4;                               // padded row of the x tile (floats)
  constexpr int VEC = Vec16<XT>::n;
  __shared__ __align__(16) float xs[kRouterBlockTokens * XS];
  __shared__ __align__(16) float wsm[kKC * EP];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tok0 = blockIdx.x * kRouterBlockTokens;

  float acc[kTokPerWarp][NE];
#pragma unroll
  for (int j = 0; j < kTokPerWarp; ++j)
#pragma unroll
    for (int n = 0; n < NE; ++n) acc[j][n] = 0.f;

  for (int k0 = 0; k0 < d; k0 += kKC) {
    __syncthreads();
    for (int c = tid; c < kRouterBlockTokens * (kKC / VEC); c += kFwdThreads) {
      const int r = c / (kKC / VEC), kc = (c % (kKC / VEC)) * VEC;
      const int t = tok0 + r, k = k0 + kc;
      const XT* src = (t < T && k < d) ? x + (size_t)t * d + k : nullptr;
      load16_as_f32<XT>(src, &xs[r * XS + kc]);
    }
    for (int c = tid; c < kKC * EP; c += kFwdThreads) {
      const int kk = c / EP, e = c % EP, k = k0 + kk;
      wsm[c] = (k < d && e < E) ? W_r[(size_t)k * E + e] : 0.f;
    }
    __syncthreads();
#pragma unroll 2
    for (int kk = 0; kk < kKC; kk += 4) {
      float4 xv[kTokPerWarp];
#pragma unroll
      for (int j = 0; j < kTokPerWarp; ++j)
        xv[j] = *reinterpret_cast<const float4*>(&xs[(warp * kTokPerWarp + j) * XS + kk]);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float wv[NE];
        if constexpr (NE >= 4) {
#pragma unroll
          for (int n = 0; n < NE; n += 4) {
            float4 w4 = *reinterpret_cast<const float4*>(&wsm[(kk + q) * EP + lane * NE + n]);
            wv[n] = w4.x; wv[n + 1] = w4.y; wv[n + 2] = w4.z; wv[n + 3] = w4.w;
          }
        } else {
#pragma unroll
          for (int n = 0; n < NE; ++n) wv[n] = wsm[(kk + q) * EP + lane * NE + n];
        }
#pragma unroll
        for (int j = 0; j < kTokPerWarp; ++j) {
          const float xq = q == 0 ? xv[j].x : q == 1 ? xv[j].y : q == 2 ? xv[j].z : xv[j].w;
#pragma unroll
          for (int n = 0; n < NE; ++n) acc[j][n] = fmaf(xq, wv[n], acc[j][n]);
        }
      }
    }
  }

  // Softmax (Eq. 1), top-1 and gate per token; one warp owns all E logits of a token.
  float bv[NE];
#pragma unroll
  for (int n = 0; n < NE; ++n) {
    const int e = lane * NE + n;
    bv[n] = (bias != nullptr && e < E) ? bias[e] : 0.f;
  }
  float pacc[NE];
#pragma unroll
  for (int n = 0; n < NE; ++n) pacc[n] = 0.f;

#pragma unroll
  for (int j = 0; j < kTokPerWarp; ++j) {
    const int t = tok0 + warp * kTokPerWarp + j;
    float m = -INFINITY;
    int am = 0x7fffffff;
#pragma unroll
    for (int n = 0; n < NE; ++n) {
      const int e = lane * NE + n;
      float h = e < E ? acc[j][n] + bv[n] : -INFINITY;
      if (noise != nullptr && e < E && t < T) h += noise[(size_t)t * E + e];   // exploration noise on the logits
      acc[j][n] = h;
      if (h > m) { m = h; am = e; }                          // ascending e: first maximum wins
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float om = __shfl_xor_sync(0xffffffffu, m, off);
      const int oa = __shfl_xor_sync(0xffffffffu, am, off);
      if (om > m || (om == m && oa < am)) { m = om; am = oa; }
    }
    float ex[NE], sum = 0.f;
#pragma unroll
    for (int n = 0; n < NE; ++n) {
      ex[n] = (lane * NE + n) < E ? expf(acc[j][n] - m) : 0.f;
      sum += ex[n];
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    const float inv = 1.f / sum;
    if (t < T) {
#pragma unroll
      for (int n = 0; n < NE; ++n) {
        const int e = lane * NE + n;
        const float p = ex[n] * inv;
        if (e < E) probs[(size_t)t * E + e] = p;
        pacc[n] += p;
      }
      if (lane == 0) { expert_index[t] = am; gate[t] = inv; }    // exp(h_max - h_max) = 1, so p_max = 1 / sum
    }
  }

  // Per-block partial of sum_t p[t,i] (Eq. 6), reduced over the 8 warps in a fixed order.
  __syncthreads();
  float* red = wsm;                                           // [8][EP]
#pragma unroll
  for (int n = 0; n < NE; ++n) red[warp * EP + lane * NE + n] = pacc[n];
  __syncthreads();
  for (int e = tid; e < E; e += kFwdThreads) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kFwdThreads / 32; ++w) s += red[w * EP + e];
    psum_partial[(size_t)blockIdx.x * E + e] = s;
  }
}

// ------------------------------------------------------------------------------------------------ backward
template <int N> struct BfVec;                               // N consecutive bfloat16 as one store
template <> struct BfVec<1> { using type = unsigned short; };
template <> struct BfVec<2> { using type = unsigned int; };
template <> struct BfVec<4> { using type = uint2; };
template <> struct BfVec<8> { using type = uint4; };

// Router input under multiplicative jitter (Appendix C): xr = x . u element by element, rounded to the activation type.
template <typename XT>
__global__ void __launch_bounds__(256)
router_jitter_kernel(const uint4* __restrict__ x, const uint4* __restrict__ u, size_t n_vec, uint4* __restrict__ xr) {
  pdl_launch_dependents();
  pdl_wait();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += (size_t)gridDim.x * blockDim.x) {
    const uint4 a = x[i], b = u[i];
    uint4 o;
    if constexpr (sizeof(XT) == 2) {
      const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
      const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
      __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float2 fa = __bfloat1622float2(pa[q]), fb = __bfloat1622float2(pb[q]);
        po[q] = __floats2bfloat162_rn(fa.x * fb.x, fa.y * fb.y);      // the float32 product of two bf16 is exact
      }
    } else {
      const float* fa = reinterpret_cast<const float*>(&a);
      const float* fb = reinterpret_cast<const float*>(&b);
      float* fo = reinterpret_cast<float*>(&o);
#pragma unroll
      for (int q = 0; q < 4; ++q) fo[q] = fa[q] * fb[q];
    }
    xr[i] = o;
  }
}

// dh[t,i] = p[t,i] (G[t,i] - sum_j p[t,j] G[t,j]),  G[t,i] = cG.count_gi + [i = e_t and t kept].dgate_t,
// count_gi counted inside the token's own routing group g = t / Tg.  Top-2 routing (second > 0): the token's second
// assignment T + t adds its own gate gradient at its own expert.
template <int NE>
__global__ void __launch_bounds__(256)
router_dlogits_kernel(const float* __restrict__ probs, const int* __restrict__ expert_index,
                      const int* __restrict__ slot, const int* __restrict__ count, const float* __restrict__ dgate,
                      float cG, int T, int Tg, int E, int second, float* __restrict__ dlogits,
                      __nv_bfloat16* __restrict__ dhsplit, int Epad64) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= T) return;
  const int et = expert_index[t];
  const float dg = slot[t] >= 0 ? dgate[t] : 0.f;
  const int et2 = second ? expert_index[T + t] : -1;
  const float dg2 = (second && slot[T + t] >= 0) ? dgate[T + t] : 0.f;
  count += (size_t)(t / Tg) * E;
  float p[NE], G[NE], s = 0.f;
#pragma unroll
  for (int n = 0; n < NE; ++n) {
    const int e = lane * NE + n;
    p[n] = e < E ? probs[(size_t)t * E + e] : 0.f;
    G[n] = e < E ? cG * (float)count[e] + (e == et ? dg : 0.f) + (e == et2 ? dg2 : 0.f) : 0.f;
    s = fmaf(p[n], G[n], s);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
#pragma unroll
  for (int n = 0; n < NE; ++n) {
    const int e = lane * NE + n;
    const float dh = p[n] * (G[n] - s);
    if (dlogits != nullptr && e < E) dlogits[(size_t)t * E + e] = dh;
    G[n] = e < E ? dh : 0.f;
  }
  if (dhsplit != nullptr && lane * NE < Epad64) {             // bf16 hi / mid parts for the tensor-core products
    __align__(16) __nv_bfloat16 hi[NE], mid[NE], lo[NE];
#pragma unroll
    for (int n = 0; n < NE; ++n) split3(G[n], &hi[n], &mid[n], &lo[n]);
    const size_t plane = (size_t)T * Epad64, at = (size_t)t * Epad64 + lane * NE;    // NE consecutive experts per lane
    using Vec = typename BfVec<NE>::type;
    *reinterpret_cast<Vec*>(dhsplit + at) = *reinterpret_cast<const Vec*>(hi);
    *reinterpret_cast<Vec*>(dhsplit + plane + at) = *reinterpret_cast<const Vec*>(mid);
  }
  if (dhsplit != nullptr) {                                   // padding columns beyond the lanes' experts
    const __nv_bfloat16 z = __float2bfloat16(0.f);
    const size_t plane = (size_t)T * Epad64;
    for (int e = 32 * NE + lane; e < Epad64; e += 32) {
      const size_t at = (size_t)t * Epad64 + e;
      dhsplit[at] = z; dhsplit[plane + at] = z;
    }
  }
}

// partial[chunk][k][e] = sum over the chunk's tokens of x[t,k] dh[t,e]; block = 64 k-rows x all experts.
constexpr int kDwrK = 64, kDwrTok = 32;
template <typename XT, int NE>
__global__ void __launch_bounds__(256)
router_dwr_partial_kernel(const XT* __restrict__ x, const float* __restrict__ dlogits, int T, int d, int E,
                          float* __restrict__ partial) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int EP = 32 * NE;
  constexpr int VEC = Vec16<XT>::n;
  __shared__ __align__(16) float xs[kDwrTok * kDwrK];
  __shared__ __align__(16) float dhs[kDwrTok * EP];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int k0 = blockIdx.x * kDwrK;
  const int tbeg = blockIdx.y * kDwrChunkTokens;
  const int tend = min(T, tbeg + kDwrChunkTokens);

  float acc[8][NE];
#pragma unroll
  for (int j = 0; j < 8; ++j)
#pragma unroll
    for (int n = 0; n < NE; ++n) acc[j][n] = 0.f;

  for (int t0 = tbeg; t0 < tend; t0 += kDwrTok) {
    __syncthreads();
    for (int c = tid; c < kDwrTok * (kDwrK / VEC); c += 256) {
      const int r = c / (kDwrK / VEC), kc = (c % (kDwrK / VEC)) * VEC;
      const int t = t0 + r, k = k0 + kc;
      const XT* src = (t < tend && k < d) ? x + (size_t)t * d + k : nullptr;
      load16_as_f32<XT>(src, &xs[r * kDwrK + kc]);
    }
    for (int c = tid; c < kDwrTok * EP; c += 256) {
      const int r = c / EP, e = c % EP, t = t0 + r;
      dhs[c] = (t < tend && e < E) ? dlogits[(size_t)t * E + e] : 0.f;
    }
    __syncthreads();
#pragma unroll 4
    for (int r = 0; r < kDwrTok; ++r) {
      const float4 xa = *reinterpret_cast<const float4*>(&xs[r * kDwrK + warp * 8]);
      const float4 xb = *reinterpret_cast<const float4*>(&xs[r * kDwrK + warp * 8 + 4]);
      const float xv[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
      float dv[NE];
      if constexpr (NE >= 4) {
#pragma unroll
        for (int n = 0; n < NE; n += 4) {
          float4 v = *reinterpret_cast<const float4*>(&dhs[r * EP + lane * NE + n]);
          dv[n] = v.x; dv[n + 1] = v.y; dv[n + 2] = v.z; dv[n + 3] = v.w;
        }
      } else {
#pragma unroll
        for (int n = 0; n < NE; ++n) dv[n] = dhs[r * EP + lane * NE + n];
      }
#pragma unroll
      for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int n = 0; n < NE; ++n) acc[j][n] = fmaf(xv[j], dv[n], acc[j][n]);
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int k = k0 + warp * 8 + j;
    if (k >= d) continue;
#pragma unroll
    for (int n = 0; n < NE; ++n) {
      const int e = lane * NE + n;
      if (e < E) partial[((size_t)blockIdx.y * d + k) * E + e] = acc[j][n];
    }
  }
}

__global__ void router_dwr_reduce_kernel(const float* __restrict__ partial, int chunks, size_t n,
                                         float* __restrict__ dW_r) {
  pdl_launch_dependents();
  pdl_wait();
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float s = 0.f;
  for (int c = 0; c < chunks; ++c) s += partial[(size_t)c * n + i];   // fixed order: deterministic
  dW_r[i] = s;
}

// dx[t,k] = (accumulate and t kept ? dx[t,k] : 0) + sum_i dh[t,i] W_r[k,i]; block = 64 tokens x 64 k per step.
// accumulate = 2 adds to every token's row (the layer's own skip path has already put dy into the dropped ones).
template <typename XT, int NE>
__global__ void __launch_bounds__(256)
router_dx_kernel(const float* __restrict__ dlogits, const float* __restrict__ W_r, const int* __restrict__ slot,
                 int T, int d, int E, int accumulate, const XT* __restrict__ jitter_u, XT* __restrict__ dx) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int EP = 32 * NE;
  constexpr int ES = EP + 4;
  extern __shared__ __align__(16) float smem[];
  float* dhs = smem;                 // [64][ES]
  float* wrs = smem + 64 * ES;       // [64][ES]
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int tok0 = blockIdx.x * 64;

  for (int c = tid; c < 64 * EP; c += 256) {
    const int r = c / EP, e = c % EP, t = tok0 + r;
    dhs[r * ES + e] = (t < T && e < E) ? dlogits[(size_t)t * E + e] : 0.f;
  }
  for (int k0 = 0; k0 < d; k0 += 64) {
    __syncthreads();
    for (int c = tid; c < 64 * EP; c += 256) {
      const int r = c / EP, e = c % EP, k = k0 + r;
      wrs[r * ES + e] = (k < d && e < E) ? W_r[(size_t)k * E + e] : 0.f;
    }
    __syncthreads();
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
#pragma unroll 4
    for (int e = 0; e < EP; e += 4) {
      float4 dv[4], wv[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) dv[a] = *reinterpret_cast<const float4*>(&dhs[(ty * 4 + a) * ES + e]);
#pragma unroll
      for (int b = 0; b < 4; ++b) wv[b] = *reinterpret_cast<const float4*>(&wrs[(tx + 16 * b) * ES + e]);
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          acc[a][b] = fmaf(dv[a].x, wv[b].x, acc[a][b]);
          acc[a][b] = fmaf(dv[a].y, wv[b].y, acc[a][b]);
          acc[a][b] = fmaf(dv[a].z, wv[b].z, acc[a][b]);
          acc[a][b] = fmaf(dv[a].w, wv[b].w, acc[a][b]);
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const int t = tok0 + ty * 4 + a;
      if (t >= T) continue;
      const bool add = accumulate == 2 || (accumulate && slot[t] >= 0);
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int k = k0 + tx + 16 * b;
        if (k >= d) continue;
        XT* o = dx + (size_t)t * d + k;
        float v = acc[a][b];
        if (jitter_u != nullptr) v *= to_f32(jitter_u[(size_t)t * d + k]);     // d(x . u)/dx = u
        if (add) v += to_f32(*o);
        if constexpr (sizeof(XT) == 4) *o = v; else *o = __float2bfloat16(v);
      }
    }
  }
}

template <typename XT, int NE>
int router_fwd_t(const Shape& s, const Plan& p, const void* x, const float* W_r, const float* bias,
                 const float* noise, void* ws,
                 cudaStream_t st) {
  launch_k(router_fwd_kernel<XT, NE>, dim3(s.router_blocks), dim3(kFwdThreads), 0, st, 
      static_cast<const XT*>(x), W_r, bias, noise, s.T, s.d, s.E, ws_ptr<float>(ws, p.probs),
      ws_ptr<int>(ws, p.expert_index), ws_ptr<float>(ws, p.gate), ws_ptr<float>(ws, p.psum_partial));
  return launch_status();
}

template <typename XT, int NE>
int router_bwd_t(const Shape& s, const Plan& p, const void* x, const float* W_r, const float* dgate, float d_aux,
                 void* ws, void* dx, bool accumulate_dx, float* dW_r, cudaStream_t st) {
  // G's auxiliary-loss term: d_aux . alpha . E . f_gi / T with f_gi = count_gi / Tg  (Eq. 4-6; f is a constant;
  // the loss is the mean over the routing groups, and T = G . Tg)
  const float cG = (float)((double)d_aux * (double)s.alpha * (double)s.E / ((double)s.T * (double)s.Tg));
  float* dlogits = ws_ptr<float>(ws, p.dlogits);
  // The float32 logit gradients are an output of the staged call (and the operand of the FP32-FMA products); the
  // whole-layer backward pass on the tensor cores only needs their bfloat16 parts.
  const bool tc_products = s.router_tc && sizeof(XT) == 2;
  launch_k(router_dlogits_kernel<NE>, dim3((s.T + 7) / 8), dim3(256), 0, st, ws_ptr<float>(ws, p.probs),
                                                            ws_ptr<int>(ws, p.expert_proc), ws_ptr<int>(ws, p.slot),
                                                            ws_ptr<int>(ws, p.count_g), dgate, cG, s.T, s.Tg, s.E, s.top2,
                                                            (tc_products && accumulate_dx) ? nullptr : dlogits,
                                                            (s.router_tc && sizeof(XT) == 2)
                                                                ? ws_ptr<__nv_bfloat16>(ws, p.dhsplit) : nullptr,
                                                            s.Epad64);
  float* partial = ws_ptr<float>(ws, p.dwr_partial);
  const size_t n = (size_t)s.d * s.E;
  if (s.jitter) {                                             // the router's input was x . u (left by the forward pass)
    if (s.jitter_u == nullptr || !aligned16(s.jitter_u)) return SWITCH_MOE_INVALID_ARGUMENT;
    x = ws_ptr<char>(ws, p.xr);
  }
  if constexpr (sizeof(XT) == 2) {
    if (s.router_tc) {
      // tensor-core products (bf16-split operands), then the same fixed-order reduction of the token splits
      int rc = launch_router_tc_bwd(s, p, x, W_r, ws, dx, accumulate_dx, st);
      if (rc != SWITCH_MOE_OK) return rc;
      launch_k(router_dwr_reduce_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st, partial, s.dwr_chunks, n, dW_r);
      return launch_status();
    }
  }
  dim3 grid((s.d + kDwrK - 1) / kDwrK, s.dwr_chunks);
  launch_k(router_dwr_partial_kernel<XT, NE>, dim3(grid), dim3(256), 0, st, static_cast<const XT*>(x), dlogits, s.T, s.d, s.E, partial);
  launch_k(router_dwr_reduce_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st, partial, s.dwr_chunks, n, dW_r);
  constexpr int ES = 32 * NE + 4;
  const size_t smem = 2 * 64 * ES * sizeof(float);
  if (cudaFuncSetAttribute(router_dx_kernel<XT, NE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
      cudaSuccess)
    return SWITCH_MOE_CUDA_ERROR;
  launch_k(router_dx_kernel<XT, NE>, dim3((s.T + 63) / 64), dim3(256), smem, st, dlogits, W_r, ws_ptr<int>(ws, p.slot), s.T, s.d, s.E,
                                                              accumulate_dx ? ((s.residual || s.top2) ? 2 : 1) : 0,
                                                              static_cast<const XT*>(s.jitter_u), static_cast<XT*>(dx));
  return launch_status();
}

}  // namespace

#define SWMOE_DISPATCH_NE(FN, ...)                                                        \
  switch (s.Epad / 32) {                                                                  \
    case 1: return s.dtype == SWITCH_MOE_BF16 ? FN<__nv_bfloat16, 1>(__VA_ARGS__) : FN<float, 1>(__VA_ARGS__); \
    case 2: return s.dtype == SWITCH_MOE_BF16 ? FN<__nv_bfloat16, 2>(__VA_ARGS__) : FN<float, 2>(__VA_ARGS__); \
    case 4: return s.dtype == SWITCH_MOE_BF16 ? FN<__nv_bfloat16, 4>(__VA_ARGS__) : FN<float, 4>(__VA_ARGS__); \
    case 8: return s.dtype == SWITCH_MOE_BF16 ? FN<__nv_bfloat16, 8>(__VA_ARGS__) : FN<float, 8>(__VA_ARGS__); \
    default: return SWITCH_MOE_UNSUPPORTED_SHAPE;                                         \
  }

int launch_router_fwd(const Shape& s, const Plan& p, const void* x, const float* W_r, const float* bias,
                      const float* noise, void* ws,
                      cudaStream_t st) {
  if (s.jitter) {
    if (s.jitter_u == nullptr || !aligned16(s.jitter_u)) return SWITCH_MOE_INVALID_ARGUMENT;
    const size_t n_vec = (size_t)s.T * s.d * s.elt / 16;
    uint4* xr = ws_ptr<uint4>(ws, p.xr);
    const unsigned blocks = (unsigned)((n_vec + 255) / 256 < 148 * 16 ? (n_vec + 255) / 256 : 148 * 16);
    if (s.dtype == SWITCH_MOE_BF16)
      launch_k(router_jitter_kernel<__nv_bfloat16>, dim3(blocks), dim3(256), 0, st, static_cast<const uint4*>(x),
               static_cast<const uint4*>(s.jitter_u), n_vec, xr);
    else
      launch_k(router_jitter_kernel<float>, dim3(blocks), dim3(256), 0, st, static_cast<const uint4*>(x),
               static_cast<const uint4*>(s.jitter_u), n_vec, xr);
    x = xr;
  }
  if (s.router_tc && s.dtype == SWITCH_MOE_BF16) return launch_router_tc_fwd(s, p, x, W_r, bias, noise, ws, st);
  SWMOE_DISPATCH_NE(router_fwd_t, s, p, x, W_r, bias, noise, ws, st)
}

int launch_router_bwd(const Shape& s, const Plan& p, const void* x, const float* W_r, const float* dgate, float d_aux,
                      void* ws, void* dx, bool accumulate_dx, float* dW_r, cudaStream_t st) {
  SWMOE_DISPATCH_NE(router_bwd_t, s, p, x, W_r, dgate, d_aux, ws, dx, accumulate_dx, dW_r, st)
}

}  // namespace swmoe
