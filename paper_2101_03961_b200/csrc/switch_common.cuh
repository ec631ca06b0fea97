// Shared host-side plumbing of the Switch FFN library: shape derivation, workspace layout, launch checks.
// Nothing here is shared with the CPU oracle.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "switch_moe.h"

namespace swmoe {

constexpr int kMaxExperts = 256;        // router kernels keep ceil(E/32) <= 8 experts per lane
constexpr int kRouterBlockTokens = 64;  // tokens per router-forward block (one partial P-sum row each)
constexpr int kPlanBlockTokens = 256;   // tokens per dispatch-plan block (one histogram row each)
constexpr int kTileM = 128;             // token rows per tensor-core tile; tails are zero-filled to this
constexpr int kPairTileTokens = 320;    // widest token tile of the paired-CTA GEMM (tokens on the MMA's N side, two
                                        // column segments above 256): an expert within the capacity of the paper's
                                        // layers (capacity factor 1.25 at 256 tokens per expert) is one tile
constexpr int kDwrChunkTokens = 512;    // tokens per split of the dW_r reduction
constexpr int kMaxGroups = 64;          // routing groups per call

struct Shape {
  int T, d, f, E;
  int C;            // rows per expert in the slot buffers: groups x capacity
  int G, Tg, Cg;    // routing groups, tokens per group, capacity of one expert for one group (Eq. 3)
  int dtype;        // switch_moe_dtype
  int gemm_path;    // resolved: 0 = tcgen05 on CTA pairs, 1 = SIMT, 2 = single-CTA tcgen05
  float alpha;
  size_t elt;       // bytes per activation / expert-weight element
  int Epad;         // E rounded up to 32 * {1,2,4,8}
  int Epad64;       // E rounded up to a multiple of 64 (tensor-core router operands)
  int router_tc;    // 1: router on the tensor cores (bf16 x, bf16 split of fp32 operands); 0: FP32 FMA
  int router_hist;  // 1: the router's forward kernel also writes the dispatch plan's block histograms
  int router_blocks, plan_blocks, max_mtiles, dwr_chunks;
  int residual;     // 1: y = x + layer(x), dx = dy + d layer / dx (SWITCH_MOE_FLAG_RESIDUAL)
  int reroute;      // 1: overflowed tokens are offered to their second-choice expert (SWITCH_MOE_FLAG_REROUTE)
  int reroute_stages;   // stages after the first (0 without the flag): stage k + 1 offers the k-th next choice
  int geglu;        // 1: GEGLU experts: W_in is [E, d, 2 f] (SWITCH_MOE_FLAG_GEGLU)
  int fin;          // columns of W_in per expert: f, or 2 f for GEGLU
  int dropout;      // 1: expert dropout on the hidden activations (SWITCH_MOE_FLAG_EXPERT_DROPOUT)
  const uint32_t* keep_bits;   // device [E C][f / 32] keep mask; may be null when only sizes are asked for
  float keep_scale;            // 1 / (1 - rate)
  int top2;         // 1: top-2 routing (SWITCH_MOE_FLAG_TOP2)
  int Tv;           // assignments the dispatch plan places: T, or 2 T for top-2 routing (first choices, then second)
  int jitter;       // 1: the router's input is x . u (SWITCH_MOE_FLAG_INPUT_JITTER)
  const void* jitter_u;   // device [T, d] factors u (activation dtype); may be null when only sizes are asked for
};

// Workspace layout: byte offsets from the (1024-byte aligned) workspace base.
struct Plan {
  size_t status, expert_index, gate, slot, token_of_slot, count, kept, count_g, group_base, psum, psum_partial, hist, hist_base,
      tile_expert, tile_row0, ntile, probs, dlogits, xd, h, dyd, dh, dgate, dwr_partial, wsplit, dhsplit, hmask, layer_y, alt, expert_proc, xr, ab, dab, yv, dxv, total;
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline int resolve_shape(const switch_moe_config* cfg, Shape* s) {
  if (!cfg) return SWITCH_MOE_INVALID_ARGUMENT;
  if (cfg->T <= 0 || cfg->d_model <= 0 || cfg->d_ff <= 0 || cfg->E <= 0) return SWITCH_MOE_INVALID_ARGUMENT;
  if (cfg->capacity_override < 0) return SWITCH_MOE_INVALID_ARGUMENT;
  if (cfg->capacity_override == 0 && !(cfg->capacity_factor > 0.f)) return SWITCH_MOE_INVALID_ARGUMENT;
  if (cfg->dtype != SWITCH_MOE_BF16 && cfg->dtype != SWITCH_MOE_F32) return SWITCH_MOE_INVALID_ARGUMENT;
  if (cfg->gemm_path != SWITCH_MOE_GEMM_DEFAULT && cfg->gemm_path != SWITCH_MOE_GEMM_SIMT &&
      cfg->gemm_path != SWITCH_MOE_GEMM_TC_1CTA)
    return SWITCH_MOE_INVALID_ARGUMENT;
  for (int i = 0; i < 2; ++i)
    if (cfg->reserved[i] != 0) return SWITCH_MOE_INVALID_ARGUMENT;
  if (cfg->reroute_stages < 0 || cfg->reroute_stages > 16) return SWITCH_MOE_INVALID_ARGUMENT;
  if (cfg->groups < 0) return SWITCH_MOE_INVALID_ARGUMENT;
  const int G = cfg->groups > 1 ? cfg->groups : 1;
  if (cfg->T % G != 0) return SWITCH_MOE_INVALID_ARGUMENT;
  if (G > 1 && ((cfg->T / G) % kPlanBlockTokens != 0 || cfg->T > 65536 || G > kMaxGroups))
    return SWITCH_MOE_UNSUPPORTED_SHAPE;
  if ((cfg->flags & ~(SWITCH_MOE_FLAG_RESIDUAL | SWITCH_MOE_FLAG_REROUTE | SWITCH_MOE_FLAG_INPUT_JITTER |
                      SWITCH_MOE_FLAG_GEGLU | SWITCH_MOE_FLAG_TOP2 | SWITCH_MOE_FLAG_EXPERT_DROPOUT)) != 0)
    return SWITCH_MOE_INVALID_ARGUMENT;
  if (cfg->E > kMaxExperts) return SWITCH_MOE_UNSUPPORTED_SHAPE;
  if (cfg->d_model % 8 != 0 || cfg->d_ff % 8 != 0) return SWITCH_MOE_UNSUPPORTED_SHAPE;
  s->T = cfg->T; s->d = cfg->d_model; s->f = cfg->d_ff; s->E = cfg->E;
  s->dtype = cfg->dtype; s->alpha = cfg->alpha;
  long long C;
  if (cfg->capacity_override > 0) {
    C = cfg->capacity_override;
  } else {
    double c = (double)(cfg->T / G) * (double)cfg->capacity_factor / (double)cfg->E;   // Eq. 3, floored
    C = (long long)c;
  }
  if (C > cfg->T / G) C = cfg->T / G;
  if (C <= 0) return SWITCH_MOE_INVALID_ARGUMENT;
  if ((long long)cfg->E * C * G > 0x7fffffffLL) return SWITCH_MOE_UNSUPPORTED_SHAPE;
  s->G = G; s->Tg = cfg->T / G; s->Cg = (int)C;
  s->C = (int)C * G;
  s->elt = cfg->dtype == SWITCH_MOE_BF16 ? 2 : 4;
  s->gemm_path = (cfg->dtype == SWITCH_MOE_F32 || cfg->gemm_path == SWITCH_MOE_GEMM_SIMT) ? 1 : cfg->gemm_path;
  if (s->gemm_path != 1 && (cfg->d_model % 64 != 0 || cfg->d_ff % 64 != 0)) return SWITCH_MOE_UNSUPPORTED_SHAPE;
  s->residual = (cfg->flags & SWITCH_MOE_FLAG_RESIDUAL) ? 1 : 0;
  if (s->residual && s->gemm_path == SWITCH_MOE_GEMM_TC_1CTA) return SWITCH_MOE_UNSUPPORTED_SHAPE;
  s->geglu = (cfg->flags & SWITCH_MOE_FLAG_GEGLU) ? 1 : 0;
  s->fin = s->geglu ? 2 * cfg->d_ff : cfg->d_ff;
  if (s->geglu && s->gemm_path == SWITCH_MOE_GEMM_TC_1CTA) return SWITCH_MOE_UNSUPPORTED_SHAPE;
  s->dropout = (cfg->flags & SWITCH_MOE_FLAG_EXPERT_DROPOUT) ? 1 : 0;
  s->keep_bits = s->dropout ? cfg->expert_keep : nullptr;
  s->keep_scale = 1.f;
  if (s->dropout) {
    if (!(cfg->expert_dropout >= 0.f) || !(cfg->expert_dropout < 1.f)) return SWITCH_MOE_INVALID_ARGUMENT;
    if (cfg->d_ff % 32 != 0) return SWITCH_MOE_UNSUPPORTED_SHAPE;
    if (G > 1) return SWITCH_MOE_UNSUPPORTED_SHAPE;          // built and checked for one routing group
    s->keep_scale = 1.f / (1.f - cfg->expert_dropout);
  }
  s->top2 = (cfg->flags & SWITCH_MOE_FLAG_TOP2) ? 1 : 0;
  // top-2 routing is built and checked for the plain ReLU layer (with or without the skip path) only
  if (s->top2 && ((cfg->flags & (SWITCH_MOE_FLAG_REROUTE | SWITCH_MOE_FLAG_GEGLU | SWITCH_MOE_FLAG_EXPERT_DROPOUT |
                                 SWITCH_MOE_FLAG_INPUT_JITTER)) ||
                  cfg->router_noise != nullptr || G > 1 || cfg->T % kPlanBlockTokens != 0))
    return SWITCH_MOE_UNSUPPORTED_SHAPE;
  s->Tv = s->top2 ? 2 * cfg->T : cfg->T;
  s->jitter = (cfg->flags & SWITCH_MOE_FLAG_INPUT_JITTER) ? 1 : 0;
  s->jitter_u = s->jitter ? cfg->router_jitter : nullptr;
  s->reroute = (cfg->flags & SWITCH_MOE_FLAG_REROUTE) ? 1 : 0;
  s->reroute_stages = s->reroute ? (cfg->reroute_stages > 1 ? cfg->reroute_stages : 1) : 0;
  if (s->reroute && G > 1) return SWITCH_MOE_UNSUPPORTED_SHAPE;
  int ne = (cfg->E + 31) / 32;
  int ne_pow2 = 1;
  while (ne_pow2 < ne) ne_pow2 *= 2;
  s->Epad = 32 * ne_pow2;
  s->Epad64 = (cfg->E + 63) / 64 * 64;
  s->router_tc = s->gemm_path != 1 ? 1 : 0;
  s->router_hist = (s->router_tc && s->Epad64 <= 128 && !s->top2) ? 1 : 0;
  s->plan_blocks = (s->Tv + kPlanBlockTokens - 1) / kPlanBlockTokens;
  s->max_mtiles = cfg->E * ((s->C + kTileM - 1) / kTileM);
  if (s->router_tc) {
    // dW_r split so that tiles x splits fills the GPU
    s->router_blocks = (cfg->T + 255) / 256;                 // one partial P-sum row per block of 256 tokens
    const int m_tiles = (cfg->d_model + kTileM - 1) / kTileM;
    const int k_blocks = (cfg->T + 63) / 64;
    int splits = 144 / m_tiles;
    if (splits < 1) splits = 1;
    if (splits > 64) splits = 64;
    if (splits > k_blocks) splits = k_blocks;
    s->dwr_chunks = splits;
  } else {
    s->router_blocks = (cfg->T + kRouterBlockTokens - 1) / kRouterBlockTokens;
    s->dwr_chunks = (cfg->T + kDwrChunkTokens - 1) / kDwrChunkTokens;
  }
  return SWITCH_MOE_OK;
}

inline void make_plan(const Shape& s, Plan* p) {
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; };
  const size_t T = s.T, E = s.E, C = s.C, d = s.d, f = s.f, Tv = s.Tv;
  p->status = take(16 * sizeof(int32_t));
  p->expert_index = take(Tv * 4);
  p->gate = take(Tv * 4);
  p->slot = take(Tv * 4);
  p->token_of_slot = take(E * C * 4);
  p->count = take(E * 4);
  p->kept = take(E * 4);
  p->count_g = take((size_t)s.G * E * 4);                  // per group: tokens whose argmax is expert i
  p->group_base = take((size_t)s.G * E * 4);               // per group: kept tokens of expert i in earlier groups
  p->psum = take(E * 4);
  p->psum_partial = take((size_t)s.router_blocks * E * 4);
  p->hist = take((size_t)s.plan_blocks * E * 4);
  p->hist_base = take((size_t)s.plan_blocks * E * 4);
  p->tile_expert = take(((size_t)s.max_mtiles + 4) * 4);   // [0] = number of token tiles, then one entry per tile
  p->tile_row0 = take(((size_t)s.max_mtiles + 4) * 4);
  p->ntile = take(((size_t)s.max_mtiles + 4) * 16);        // int4 {expert, first row, rows}; [0].x = count
  p->probs = take(T * E * 4);
  p->dlogits = take(T * E * 4);
  p->xd = take(E * C * d * s.elt);
  p->h = take(E * C * f * s.elt);
  p->dyd = take(E * C * d * s.elt);
  p->dh = take(E * C * f * s.elt);
  p->dgate = take(Tv * 4);
  p->dwr_partial = take((size_t)s.dwr_chunks * d * E * 4);
  p->wsplit = take(3 * d * (size_t)s.Epad64 * 2);
  p->dhsplit = take(3 * T * (size_t)s.Epad64 * 2);
  p->hmask = take(E * C * ((f + 31) / 32) * 4);            // one bit per element of H: [H > 0]
  p->layer_y = s.residual ? take(T * d * s.elt) : 0;       // g . E(x) without the skip path (for the gate's gradient)
  p->alt = s.reroute ? take(T * 4 * (size_t)s.reroute_stages) : 0;   // per stage: next choice of the tokens without a slot, -1 for the others
  p->expert_proc = s.reroute ? take(T * 4) : p->expert_index;   // the expert that processes each token
  p->xr = s.jitter ? take(T * d * s.elt) : 0;               // the router's input x . u, rounded to the activation dtype
  p->ab = s.geglu ? take(E * C * 2 * f * s.elt) : 0;        // GEGLU: [a | b] = X_d [W_0 | W_1] per slot
  p->dab = s.geglu ? take(E * C * 2 * f * s.elt) : 0;       // GEGLU: gradient of [a | b] per slot
  p->yv = s.top2 ? take(Tv * d * s.elt) : 0;                // top-2: weighted expert output per assignment
  p->dxv = s.top2 ? take(Tv * d * s.elt) : 0;               // top-2: input gradient per assignment
  p->total = off;
}

// w = hi + mid + lo with hi, mid, lo bfloat16 (round to nearest); exact to about 2^-24 relative.
__device__ __forceinline__ void split3(float w, __nv_bfloat16* hi, __nv_bfloat16* mid, __nv_bfloat16* lo) {
  const __nv_bfloat16 h = __float2bfloat16(w);
  const float r1 = w - __bfloat162float(h);
  const __nv_bfloat16 m = __float2bfloat16(r1);
  const float r2 = r1 - __bfloat162float(m);
  *hi = h; *mid = m; *lo = __float2bfloat16(r2);
}

template <typename T>
inline T* ws_ptr(void* ws, size_t off) { return reinterpret_cast<T*>(static_cast<char*>(ws) + off); }

// ---- programmatic dependent launch --------------------------------------------------------------------------
// Every kernel of the layer is launched with programmatic stream serialization: it may be scheduled (and run its
// prologue: barrier init, tensor-memory allocation) while the previous kernel of the stream is still draining.
// The contract inside the kernels: call pdl_launch_dependents() first, and pdl_wait() before the first access to
// global memory; pdl_wait() returns once the previous kernel has completed and its writes are visible.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

inline bool& launch_failed_flag() { static thread_local bool failed = false; return failed; }

template <typename Kern, typename... Args>
inline void launch_k(Kern kernel, dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, kernel, args...) != cudaSuccess) launch_failed_flag() = true;
}

inline int launch_status() {
  const bool failed = launch_failed_flag();
  launch_failed_flag() = false;
  return (cudaGetLastError() == cudaSuccess && !failed) ? SWITCH_MOE_OK : SWITCH_MOE_CUDA_ERROR;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- kernels' host launchers (each returns a switch_moe_status) ----------------------------------------
int launch_router_fwd(const Shape& s, const Plan& p, const void* x, const float* W_r, const float* bias,
                      const float* noise, void* ws, cudaStream_t st);
int launch_dispatch_plan(const Shape& s, const Plan& p, const int32_t* expert_index, float* aux_loss, void* ws,
                         cudaStream_t st);
int launch_gather_x(const Shape& s, const Plan& p, const void* x, void* y, void* ws, cudaStream_t st);
// Top-2 routing: second choices (expert and weight) of every token; sums of the two assignments' rows.
int launch_top2_choice(const Shape& s, const Plan& p, void* ws, cudaStream_t st);
// `skip` (may be null): rows added to the sum, the layer's input (forward) or dy (backward) when the layer carries its
// own residual connection.
int launch_top2_sum(const Shape& s, const Plan& p, const void* per_assignment, const void* skip, void* out, void* ws,
                    cudaStream_t st);
int launch_gather_dy(const Shape& s, const Plan& p, const void* dy, const void* y, void* dx, void* ws, cudaStream_t st);
int launch_router_bwd(const Shape& s, const Plan& p, const void* x, const float* W_r, const float* dgate, float d_aux,
                      void* ws, void* dx, bool accumulate_dx, float* dW_r, cudaStream_t st);

// Tensor-core router (bf16 x): forward (logits, softmax, top-1, gate, P-sum partials) and the two backward products.
int launch_router_tc_fwd(const Shape& s, const Plan& p, const void* x, const float* W_r, const float* bias,
                         const float* noise, void* ws, cudaStream_t st);
int launch_router_tc_bwd(const Shape& s, const Plan& p, const void* x, const float* W_r, void* ws, void* dx,
                         bool accumulate_dx, cudaStream_t st);

// GELU(z) = z Phi(z), the exact form (GEGLU experts), and what its derivative needs.  Phi(z) = (1 + erf(z / sqrt 2)) / 2
// with the rational approximation 7.1.26 of Abramowitz and Stegun for erf (absolute error below 1.5e-7, i.e. the
// resolution of a float32 near 1): erf(x) = 1 - (a1 t + .. + a5 t^5) exp(-x^2), t = 1 / (1 + p x), x >= 0.  Its
// exponential exp(-z^2 / 2) is the one the density phi(z) needs, so one exp2 and one reciprocal serve the value
// and the derivative; the library erff costs about three times the instructions, and the gating is bound by the
// number of instructions it issues.  One definition for the element-wise kernels and the GEMM epilogue that gates:
// both must round identically.
__device__ __forceinline__ void gelu_cdf_pdf(float z, float* cdf, float* pdf) {
  const float az = fabsf(z);
  const float e = __expf(-0.5f * z * z);
  float t;                                                    // the hardware's approximate reciprocal (1 ulp)
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(0.3275911f * 0.70710678118654752f, az, 1.f)));
  float poly = fmaf(1.061405429f, t, -1.453152027f);
  poly = fmaf(poly, t, 1.421413741f);
  poly = fmaf(poly, t, -0.284496736f);
  poly = fmaf(poly, t, 0.254829592f);
  const float tail = 0.5f * poly * t * e;                     // Phi(-|z|)
  *cdf = z >= 0.f ? 1.f - tail : tail;
  *pdf = 0.3989422804014327f * e;
}
__device__ __forceinline__ float gelu_exact(float z) {
  float cdf, pdf;
  gelu_cdf_pdf(z, &cdf, &pdf);
  return z * cdf;
}

// The six expert GEMMs (Section 5: h = x W_in, y = ReLU(h) W_out, and their derivatives).
enum GemmOp {
  kGemm1Relu = 0,     // H = ReLU(X_d W_in)
  kGemm2Combine = 1,  // y[token] = g . (H W_out)[slot]
  kDgrad2Mask = 2,    // dH = (dY_d W_out^T) * [H > 0]
  kDgrad1Scatter = 3, // dx[token] = (dH W_in^T)[slot]
  kWgrad2 = 4,        // dW_out = H^T dY_d
  kWgrad1 = 5         // dW_in = X_d^T dH
};
struct GemmArgs {
  const void* W_in; const void* W_out;   // expert weights
  void* y; void* dx; void* dW_in; void* dW_out;
  const void* x; const void* dy;         // skip-path sources (residual configuration only): y += x, dx += dy
};
int launch_simt_gemm(GemmOp op, const Shape& s, const Plan& p, const GemmArgs& a, void* ws, cudaStream_t st);
int launch_tc_gemm(GemmOp op, const Shape& s, const Plan& p, const GemmArgs& a, void* ws, cudaStream_t st);
int launch_pair_gemm(GemmOp op, const Shape& s, const Plan& p, const GemmArgs& a, void* ws, cudaStream_t st);
int launch_pair_dgrad1_wgrad1(const Shape& s, const Plan& p, const GemmArgs& a, void* ws, cudaStream_t st);
// GEGLU gating over the kept rows: H = GELU(a) . b, and its derivative d[a | b] from dH (element-wise).
int launch_geglu_fwd(const Shape& s, const Plan& p, void* ws, cudaStream_t st);
int launch_geglu_bwd(const Shape& s, const Plan& p, void* ws, cudaStream_t st);
// Expert dropout: rows[slot][j] *= keep bit / (1 - rate) over the kept rows of the hidden activations (forward) or of
// their gradient (backward).
int launch_expert_dropout(const Shape& s, const Plan& p, bool backward, void* ws, cudaStream_t st);

}  // namespace swmoe
