// GEGLU gating of the expert FFN (Table 9: the expansion matrix is replaced by two sets of weights that are combined
// non-linearly): hidden = GELU(a) . b with [a | b] = X_d [W_0 | W_1] computed by the grouped GEMM, GELU(z) = z Phi(z)
// (exact form), and the derivative d a = dH . b . GELU'(a), d b = dH . GELU(a).  Element-wise over the rows the
// grouped GEMMs read: an expert's kept rows rounded up to the MMA's token granularity of 16 (those extra rows are
// zero: GELU(0) . 0 = 0).  One warp per slot row, 16-byte accesses.
#include "switch_common.cuh"

namespace swmoe {
namespace {

__device__ __forceinline__ float gelu_f(float z) { return gelu_exact(z); }

template <typename ET> struct Pack;
template <> struct Pack<__nv_bfloat16> {
  static constexpr int n = 8;
  static __device__ __forceinline__ void load(const uint4& v, float* f) {
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) { const float2 t = __bfloat1622float2(p[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
  }
  static __device__ __forceinline__ uint4 store(const float* f) {
    uint4 v;
    __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) p[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    return v;
  }
};
template <> struct Pack<float> {
  static constexpr int n = 4;
  static __device__ __forceinline__ void load(const uint4& v, float* f) {
    const float* p = reinterpret_cast<const float*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) f[i] = p[i];
  }
  static __device__ __forceinline__ uint4 store(const float* f) {
    uint4 v;
    float* p = reinterpret_cast<float*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) p[i] = f[i];
    return v;
  }
};

// kBackward = false: h[row][j] = GELU(ab[row][j]) . ab[row][f + j]
// kBackward = true : dab[row][j] = dh[row][j] . b . GELU'(a),  dab[row][f + j] = dh[row][j] . GELU(a)
template <typename ET, bool kBackward>
__global__ void __launch_bounds__(256)
geglu_kernel(const uint4* __restrict__ ab, const int* __restrict__ kept, int E, int C, int f_vec,
             uint4* __restrict__ h_or_dh, uint4* __restrict__ dab) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int N = Pack<ET>::n;
  const int lane = threadIdx.x & 31;
  const int s = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (s >= E * C) return;
  const int ex = s / C, pos = s - ex * C;
  if (pos >= min(C, (kept[ex] + 15) / 16 * 16)) return;
  const uint4* arow = ab + (size_t)s * 2 * f_vec;
  const uint4* brow = arow + f_vec;
  uint4* hrow = h_or_dh + (size_t)s * f_vec;
  for (int v = lane; v < f_vec; v += 32) {
    float a[N], b[N], o[N];
    Pack<ET>::load(arow[v], a);
    Pack<ET>::load(brow[v], b);
    if (!kBackward) {
#pragma unroll
      for (int i = 0; i < N; ++i) o[i] = gelu_f(a[i]) * b[i];
      hrow[v] = Pack<ET>::store(o);
    } else {
      float g[N], o2[N];
      Pack<ET>::load(hrow[v], g);
#pragma unroll
      for (int i = 0; i < N; ++i) {
        // one evaluation of Phi and phi serves GELU(a) = a Phi(a) and GELU'(a) = Phi(a) + a phi(a)
        float cdf, pdf;
        gelu_cdf_pdf(a[i], &cdf, &pdf);
        o[i] = g[i] * b[i] * fmaf(a[i], pdf, cdf);
        o2[i] = g[i] * (a[i] * cdf);
      }
      uint4* drow = dab + (size_t)s * 2 * f_vec;
      drow[v] = Pack<ET>::store(o);
      drow[f_vec + v] = Pack<ET>::store(o2);
    }
  }
}

// Expert dropout: one warp per slot row, consecutive lanes on consecutive 16-byte pieces of the row; a piece's keep
// bits are one byte (bf16: 8 hidden units) or half a byte (fp32: 4) of the row's mask words.
template <typename ET>
__global__ void __launch_bounds__(256)
expert_dropout_kernel(const uint32_t* __restrict__ keep_bits, const int* __restrict__ kept, int E, int C, int f,
                      float scale, ET* __restrict__ rows) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int N = Pack<ET>::n;                             // elements per 16 bytes
  const int lane = threadIdx.x & 31;
  const int s = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (s >= E * C) return;
  const int ex = s / C, pos = s - ex * C;
  if (pos >= min(C, (kept[ex] + 15) / 16 * 16)) return;
  const uint32_t* words = keep_bits + (size_t)s * (f / 32);
  uint4* row = reinterpret_cast<uint4*>(rows + (size_t)s * f);
  for (int v = lane; v < f / N; v += 32) {
    const int first = v * N;                                   // first hidden unit of this piece
    const uint32_t bits = words[first >> 5] >> (first & 31);
    float x[N];
    Pack<ET>::load(row[v], x);
#pragma unroll
    for (int i = 0; i < N; ++i) x[i] = ((bits >> i) & 1u) ? x[i] * scale : 0.f;
    row[v] = Pack<ET>::store(x);
  }
}

template <bool kBackward>
int launch(const Shape& s, const Plan& p, void* ws, cudaStream_t st) {
  const int f_vec = (int)((size_t)s.f * s.elt / 16);
  const int blocks = (s.E * s.C + 7) / 8;
  const uint4* ab = ws_ptr<uint4>(ws, p.ab);
  uint4* hh = ws_ptr<uint4>(ws, kBackward ? p.dh : p.h);
  uint4* dab = ws_ptr<uint4>(ws, p.dab);
  if (s.dtype == SWITCH_MOE_BF16)
    launch_k(geglu_kernel<__nv_bfloat16, kBackward>, dim3(blocks), dim3(256), 0, st, ab, ws_ptr<int>(ws, p.kept), s.E, s.C,
             f_vec, hh, dab);
  else
    launch_k(geglu_kernel<float, kBackward>, dim3(blocks), dim3(256), 0, st, ab, ws_ptr<int>(ws, p.kept), s.E, s.C, f_vec,
             hh, dab);
  return launch_status();
}

}  // namespace

int launch_geglu_fwd(const Shape& s, const Plan& p, void* ws, cudaStream_t st) { return launch<false>(s, p, ws, st); }
int launch_geglu_bwd(const Shape& s, const Plan& p, void* ws, cudaStream_t st) { return launch<true>(s, p, ws, st); }

int launch_expert_dropout(const Shape& s, const Plan& p, bool backward, void* ws, cudaStream_t st) {
  if (s.keep_bits == nullptr || (reinterpret_cast<uintptr_t>(s.keep_bits) & 3u) != 0) return SWITCH_MOE_INVALID_ARGUMENT;
  const int blocks = (s.E * s.C + 7) / 8;
  void* rows = ws_ptr<char>(ws, backward ? p.dh : p.h);
  if (s.dtype == SWITCH_MOE_BF16)
    launch_k(expert_dropout_kernel<__nv_bfloat16>, dim3(blocks), dim3(256), 0, st, s.keep_bits, ws_ptr<int>(ws, p.kept), s.E,
             s.C, s.f, s.keep_scale, static_cast<__nv_bfloat16*>(rows));
  else
    launch_k(expert_dropout_kernel<float>, dim3(blocks), dim3(256), 0, st, s.keep_bits, ws_ptr<int>(ws, p.kept), s.E, s.C,
             s.f, s.keep_scale, static_cast<float*>(rows));
  return launch_status();
}

}  // namespace swmoe
