// Grouped expert GEMMs on the plain FP32 FMA pipes (no tensor cores): the expert FFN h = x W_in, y = ReLU(h) W_out
// (Section 5, FFN review) and its derivatives, one problem per expert, with the same fused epilogues as the
// tensor-core path.  This is the arithmetic path of the all-float32 configuration (tensor cores have no exact
// float32 mode) and a validation path for bfloat16 inputs; accumulation is float32 in both.
#include "switch_common.cuh"

namespace swmoe {
namespace {

constexpr int kBM = 64, kBN = 64, kBK = 16;

struct SimtProblem {
  const void* A; long long a_es, a_ms, a_ks;   // A(e, m, k) element strides
  const void* B; long long b_es, b_ks, b_ns;   // B(e, k, n) element strides
  int M, K, N;                                  // M < 0: M_e = kept[e];  K < 0: K_e = kept[e]
  int C;                                        // expert capacity (rows per expert of the slot buffers)
  const int* kept; const int* token_of_slot; const float* gate;
  void* out; const void* mask_src; int ld_out;
  const void* res;   // combine / scatter with the skip path inside the layer: row added to the output (x or dy)
  void* out2;        // combine with the skip path: second copy of the output without it
  int plain;         // GEMM1 / dgrad2 without ReLU and mask (GEGLU experts gate elsewhere)
};

__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float* p, float v) { *p = v; }
__device__ __forceinline__ void stf(__nv_bfloat16* p, float v) { *p = __float2bfloat16(v); }
__device__ __forceinline__ float rnd(const float*, float v) { return v; }
__device__ __forceinline__ float rnd(const __nv_bfloat16*, float v) { return __bfloat162float(__float2bfloat16(v)); }

template <typename ET, int OP>
__global__ void __launch_bounds__(256) simt_grouped_gemm_kernel(SimtProblem pr) {
  __shared__ float As[kBK][kBM + 4];
  __shared__ float Bs[kBK][kBN + 4];
  const int e = blockIdx.z;
  const int kept_e = pr.kept[e];
  const int M = pr.M < 0 ? kept_e : pr.M;
  const int K = pr.K < 0 ? kept_e : pr.K;
  const int m0 = blockIdx.y * kBM, n0 = blockIdx.x * kBN;
  if (m0 >= M) return;
  const ET* A = static_cast<const ET*>(pr.A) + (long long)e * pr.a_es;
  const ET* B = static_cast<const ET*>(pr.B) + (long long)e * pr.b_es;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const bool a_k_fast = pr.a_ks == 1, b_n_fast = pr.b_ns == 1;

  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < K; k0 += kBK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = tid + i * 256;
      const int am = a_k_fast ? idx / kBK : idx % kBM, ak = a_k_fast ? idx % kBK : idx / kBM;
      const int gm = m0 + am, gk = k0 + ak;
      As[ak][am] = (gm < M && gk < K) ? ldf(A + (long long)gm * pr.a_ms + (long long)gk * pr.a_ks) : 0.f;
      const int bn = b_n_fast ? idx % kBN : idx / kBK, bk = b_n_fast ? idx / kBN : idx % kBK;
      const int gn = n0 + bn, gk2 = k0 + bk;
      Bs[bk][bn] = (gn < pr.N && gk2 < K) ? ldf(B + (long long)gk2 * pr.b_ks + (long long)gn * pr.b_ns) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kBK; ++kk) {
      const float4 a4 = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float4 b4 = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float av[4] = {a4.x, a4.y, a4.z, a4.w}, bv[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }

#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
    long long row;
    float scale = 1.f;
    if (OP == kGemm2Combine || OP == kDgrad1Scatter) {
      const int tok = pr.token_of_slot[(long long)e * pr.C + m];
      row = (long long)tok * pr.ld_out;
      if (OP == kGemm2Combine) scale = pr.gate[tok];                 // Eq. 2: y = p_i(x) E_i(x)
    } else if (OP == kGemm1Relu || OP == kDgrad2Mask) {
      row = ((long long)e * pr.C + m) * pr.ld_out;
    } else {
      row = ((long long)e * M + m) * pr.ld_out;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= pr.N) continue;
      float v = acc[i][j] * scale;
      if (OP == kGemm1Relu && !pr.plain) v = fmaxf(v, 0.f);
      if (OP == kDgrad2Mask && !pr.plain) v = ldf(static_cast<const ET*>(pr.mask_src) + row + n) > 0.f ? v : 0.f;
      if (OP == kGemm2Combine && pr.out2 != nullptr) stf(static_cast<ET*>(pr.out2) + row + n, v);
      if ((OP == kGemm2Combine || OP == kDgrad1Scatter) && pr.res != nullptr)   // the expert term is rounded first
        v = rnd(static_cast<const ET*>(nullptr), v) + ldf(static_cast<const ET*>(pr.res) + row + n);
      stf(static_cast<ET*>(pr.out) + row + n, v);
    }
  }
}

template <typename ET>
int launch_t(GemmOp op, const Shape& s, const Plan& p, const GemmArgs& a, void* ws, cudaStream_t st) {
  SimtProblem pr{};
  const long long C = s.C, d = s.d, f = s.f;
  pr.C = s.C;
  pr.kept = ws_ptr<int>(ws, p.kept);
  pr.token_of_slot = ws_ptr<int>(ws, p.token_of_slot);
  pr.gate = ws_ptr<float>(ws, p.gate);
  void* xd = ws_ptr<char>(ws, p.xd); void* h = ws_ptr<char>(ws, p.h);
  void* dyd = ws_ptr<char>(ws, p.dyd); void* dh = ws_ptr<char>(ws, p.dh);
  const long long fin = s.fin;                               // columns of W_in: f, or 2 f for GEGLU experts
  void* ab = ws_ptr<char>(ws, p.ab);
  void* du = s.geglu ? ws_ptr<char>(ws, p.dab) : dh;         // gradient of the pre-activation(s)
  int max_m;
  switch (op) {
    case kGemm1Relu:      // H[e] (C x f) = ReLU(X_d[e] (C x d) . W_in[e] (d x f));  GEGLU: [a | b] (C x 2f), no ReLU
      pr = SimtProblem{xd, C * d, d, 1, a.W_in, d * fin, fin, 1, -1, s.d, s.fin, s.C, pr.kept, pr.token_of_slot,
                       pr.gate, s.geglu ? ab : h, nullptr, s.fin};
      pr.plain = s.geglu;
      max_m = s.C; break;
    case kGemm2Combine:   // y[token] = g . (H[e] (C x f) . W_out[e] (f x d))
      pr = SimtProblem{h, C * f, f, 1, a.W_out, f * d, d, 1, -1, s.f, s.d, s.C, pr.kept, pr.token_of_slot, pr.gate,
                       a.y, nullptr, s.d};
      max_m = s.C; break;
    case kDgrad2Mask:     // dH[e] = (dY_d[e] (C x d) . W_out[e]^T (d x f)) * [H > 0];  GEGLU: no mask
      pr = SimtProblem{dyd, C * d, d, 1, a.W_out, f * d, 1, d, -1, s.d, s.f, s.C, pr.kept, pr.token_of_slot, pr.gate,
                       dh, h, s.f};
      pr.plain = s.geglu;
      max_m = s.C; break;
    case kDgrad1Scatter:  // dx[token] = dH[e] (C x f) . W_in[e]^T (f x d);  GEGLU: d[a | b] (C x 2f)
      pr = SimtProblem{du, C * fin, fin, 1, a.W_in, d * fin, 1, fin, -1, s.fin, s.d, s.C, pr.kept, pr.token_of_slot,
                       pr.gate, a.dx, nullptr, s.d};
      max_m = s.C; break;
    case kWgrad2:         // dW_out[e] (f x d) = H[e]^T (f x kept) . dY_d[e] (kept x d)
      pr = SimtProblem{h, C * f, 1, f, dyd, C * d, d, 1, s.f, -1, s.d, s.C, pr.kept, pr.token_of_slot, pr.gate,
                       a.dW_out, nullptr, s.d};
      max_m = s.f; break;
    case kWgrad1:         // dW_in[e] (d x f) = X_d[e]^T (d x kept) . dH[e] (kept x f);  GEGLU: d[a | b], 2f columns
      pr = SimtProblem{xd, C * d, 1, d, du, C * fin, fin, 1, s.d, -1, s.fin, s.C, pr.kept, pr.token_of_slot, pr.gate,
                       a.dW_in, nullptr, s.fin};
      max_m = s.d; break;
    default: return SWITCH_MOE_INVALID_ARGUMENT;
  }
  // (top-2 routing adds the skip path where the two assignments' rows are summed, not here)
  if (s.residual && !s.top2 && op == kGemm2Combine) { pr.res = a.x; pr.out2 = ws_ptr<char>(ws, p.layer_y); }
  if (s.residual && !s.top2 && op == kDgrad1Scatter) pr.res = a.dy;
  dim3 grid((pr.N + kBN - 1) / kBN, (max_m + kBM - 1) / kBM, s.E);
  switch (op) {
    case kGemm1Relu: simt_grouped_gemm_kernel<ET, kGemm1Relu><<<grid, 256, 0, st>>>(pr); break;
    case kGemm2Combine: simt_grouped_gemm_kernel<ET, kGemm2Combine><<<grid, 256, 0, st>>>(pr); break;
    case kDgrad2Mask: simt_grouped_gemm_kernel<ET, kDgrad2Mask><<<grid, 256, 0, st>>>(pr); break;
    case kDgrad1Scatter: simt_grouped_gemm_kernel<ET, kDgrad1Scatter><<<grid, 256, 0, st>>>(pr); break;
    case kWgrad2: simt_grouped_gemm_kernel<ET, kWgrad2><<<grid, 256, 0, st>>>(pr); break;
    case kWgrad1: simt_grouped_gemm_kernel<ET, kWgrad1><<<grid, 256, 0, st>>>(pr); break;
  }
  return launch_status();
}

}  // namespace

int launch_simt_gemm(GemmOp op, const Shape& s, const Plan& p, const GemmArgs& a, void* ws, cudaStream_t st) {
  return s.dtype == SWITCH_MOE_BF16 ? launch_t<__nv_bfloat16>(op, s, p, a, ws, st)
                                    : launch_t<float>(op, s, p, a, ws, st);
}

}  // namespace swmoe
