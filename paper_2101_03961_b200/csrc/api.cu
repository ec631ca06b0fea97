// C ABI of the Switch FFN library: argument checks, workspace planning and the launch sequences of the forward and
// backward passes.  Every step of the layer runs in this library's own kernels; nothing here allocates device memory.
#include <cstring>

#include "switch_common.cuh"

using namespace swmoe;

namespace {

struct Ctx {
  Shape s;
  Plan p;
};

int prepare(const switch_moe_config* cfg, const void* workspace, size_t workspace_bytes, bool need_ws, Ctx* c) {
  int rc = resolve_shape(cfg, &c->s);
  if (rc != SWITCH_MOE_OK) return rc;
  make_plan(c->s, &c->p);
  if (need_ws) {
    if (workspace == nullptr) return SWITCH_MOE_INVALID_ARGUMENT;
    if ((reinterpret_cast<uintptr_t>(workspace) & 1023u) != 0) return SWITCH_MOE_UNSUPPORTED_SHAPE;
    if (workspace_bytes < c->p.total) return SWITCH_MOE_WORKSPACE_TOO_SMALL;
  }
  return SWITCH_MOE_OK;
}

int run_gemm(GemmOp op, const Ctx& c, const GemmArgs& a, void* ws, cudaStream_t st) {
  if (c.s.gemm_path == 0) return launch_pair_gemm(op, c.s, c.p, a, ws, st);
  if (c.s.gemm_path == 2) return launch_tc_gemm(op, c.s, c.p, a, ws, st);
  return launch_simt_gemm(op, c.s, c.p, a, ws, st);
}

// Optional per-stage timing: records the caller's event `i` on the stream (see switch_moe_config::stage_events).
int mark(const switch_moe_config* cfg, int i, cudaStream_t st) {
  if (cfg->stage_events == nullptr) return SWITCH_MOE_OK;
  return cudaEventRecord(static_cast<cudaEvent_t>(cfg->stage_events[i]), st) == cudaSuccess ? SWITCH_MOE_OK
                                                                                             : SWITCH_MOE_CUDA_ERROR;
}

#define SWMOE_TRY(expr)                    \
  do {                                     \
    int rc__ = (expr);                     \
    if (rc__ != SWITCH_MOE_OK) return rc__; \
  } while (0)

}  // namespace

extern "C" {

int switch_moe_capacity(const switch_moe_config* cfg, int32_t* C_out) {
  if (C_out == nullptr) return SWITCH_MOE_INVALID_ARGUMENT;
  Shape s;
  SWMOE_TRY(resolve_shape(cfg, &s));
  *C_out = s.Cg;
  return SWITCH_MOE_OK;
}

int switch_moe_workspace_bytes(const switch_moe_config* cfg, size_t* bytes_out) {
  if (bytes_out == nullptr) return SWITCH_MOE_INVALID_ARGUMENT;
  Ctx c;
  SWMOE_TRY(prepare(cfg, nullptr, 0, false, &c));
  *bytes_out = c.p.total;
  return SWITCH_MOE_OK;
}

int switch_moe_workspace_view(const switch_moe_config* cfg, void* workspace, int32_t region, void** ptr_out,
                              size_t* bytes_out) {
  if (ptr_out == nullptr || bytes_out == nullptr || workspace == nullptr) return SWITCH_MOE_INVALID_ARGUMENT;
  Ctx c;
  SWMOE_TRY(prepare(cfg, nullptr, 0, false, &c));
  const Shape& s = c.s;
  const Plan& p = c.p;
  const size_t T = s.T, E = s.E, C = s.C;
  size_t off, bytes;
  switch (region) {
    case SWITCH_MOE_WS_STATUS: off = p.status; bytes = 16 * 4; break;
    case SWITCH_MOE_WS_EXPERT_INDEX: off = p.expert_index; bytes = (size_t)s.Tv * 4; break;
    case SWITCH_MOE_WS_GATE: off = p.gate; bytes = (size_t)s.Tv * 4; break;
    case SWITCH_MOE_WS_SLOT: off = p.slot; bytes = (size_t)s.Tv * 4; break;
    case SWITCH_MOE_WS_TOKEN_OF_SLOT: off = p.token_of_slot; bytes = E * C * 4; break;
    case SWITCH_MOE_WS_COUNT: off = p.count; bytes = E * 4; break;
    case SWITCH_MOE_WS_KEPT: off = p.kept; bytes = E * 4; break;
    case SWITCH_MOE_WS_PSUM: off = p.psum; bytes = E * 4; break;
    case SWITCH_MOE_WS_PROBS: off = p.probs; bytes = T * E * 4; break;
    case SWITCH_MOE_WS_XD: off = p.xd; bytes = E * C * s.d * s.elt; break;
    case SWITCH_MOE_WS_H: off = p.h; bytes = E * C * s.f * s.elt; break;
    case SWITCH_MOE_WS_DYD: off = p.dyd; bytes = E * C * s.d * s.elt; break;
    case SWITCH_MOE_WS_DH: off = p.dh; bytes = E * C * s.f * s.elt; break;
    case SWITCH_MOE_WS_DGATE: off = p.dgate; bytes = (size_t)s.Tv * 4; break;
    case SWITCH_MOE_WS_DLOGITS: off = p.dlogits; bytes = T * E * 4; break;
    case SWITCH_MOE_WS_EXPERT_PROC:
      if (!s.reroute) return SWITCH_MOE_INVALID_ARGUMENT;
      off = p.expert_proc; bytes = T * 4; break;
    case SWITCH_MOE_WS_SECOND_CHOICE:
      if (!s.reroute) return SWITCH_MOE_INVALID_ARGUMENT;
      off = p.alt; bytes = T * 4 * (size_t)s.reroute_stages; break;
    case SWITCH_MOE_WS_LAYER_Y:
      if (!s.residual) return SWITCH_MOE_INVALID_ARGUMENT;
      off = p.layer_y; bytes = T * s.d * s.elt; break;
    default: return SWITCH_MOE_INVALID_ARGUMENT;
  }
  *ptr_out = static_cast<char*>(workspace) + off;
  *bytes_out = bytes;
  return SWITCH_MOE_OK;
}

int switch_moe_router_fwd(const switch_moe_config* cfg, const void* x, const float* W_r, const float* router_bias,
                          void* workspace, size_t workspace_bytes, void* stream) {
  Ctx c;
  SWMOE_TRY(prepare(cfg, workspace, workspace_bytes, true, &c));
  if (x == nullptr || W_r == nullptr) return SWITCH_MOE_INVALID_ARGUMENT;
  if (!aligned16(x) || !aligned16(W_r)) return SWITCH_MOE_UNSUPPORTED_SHAPE;
  return launch_router_fwd(c.s, c.p, x, W_r, router_bias, cfg->router_noise, workspace,
                           static_cast<cudaStream_t>(stream));
}

int switch_moe_dispatch_plan(const switch_moe_config* cfg, const int32_t* expert_index, float* aux_loss,
                             void* workspace, size_t workspace_bytes, void* stream) {
  Ctx c;
  SWMOE_TRY(prepare(cfg, workspace, workspace_bytes, true, &c));
  return launch_dispatch_plan(c.s, c.p, expert_index, aux_loss, workspace, static_cast<cudaStream_t>(stream));
}

int switch_moe_fwd(const switch_moe_config* cfg, const void* x, const float* W_r, const float* router_bias,
                   const void* W_in, const void* W_out, void* y, float* aux_loss, void* workspace,
                   size_t workspace_bytes, void* stream) {
  Ctx c;
  SWMOE_TRY(prepare(cfg, workspace, workspace_bytes, true, &c));
  if (!x || !W_r || !W_in || !W_out || !y || !aux_loss) return SWITCH_MOE_INVALID_ARGUMENT;
  if (!aligned16(x) || !aligned16(W_r) || !aligned16(W_in) || !aligned16(W_out) || !aligned16(y))
    return SWITCH_MOE_UNSUPPORTED_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(ws_ptr<char>(workspace, c.p.status), 0, 16 * 4, st) != cudaSuccess) return SWITCH_MOE_CUDA_ERROR;
  SWMOE_TRY(mark(cfg, 0, st));
  SWMOE_TRY(launch_router_fwd(c.s, c.p, x, W_r, router_bias, cfg->router_noise, workspace, st));
  if (c.s.top2) SWMOE_TRY(launch_top2_choice(c.s, c.p, workspace, st));     // assignments T .. 2T - 1
  SWMOE_TRY(mark(cfg, 1, st));
  SWMOE_TRY(launch_dispatch_plan(c.s, c.p, nullptr, aux_loss, workspace, st));
  SWMOE_TRY(mark(cfg, 2, st));
  // top-2 routing: the experts write one weighted output row per assignment; the two rows of a token are summed last
  void* y_rows = c.s.top2 ? ws_ptr<void>(workspace, c.p.yv) : y;
  SWMOE_TRY(launch_gather_x(c.s, c.p, x, y_rows, workspace, st));
  GemmArgs a{};
  a.W_in = W_in; a.W_out = W_out; a.y = y_rows; a.x = x;
  SWMOE_TRY(mark(cfg, 3, st));
  SWMOE_TRY(run_gemm(kGemm1Relu, c, a, workspace, st));
  // hidden = GELU(a) . b: inside GEMM1's epilogue on the CTA-pair path, an element-wise kernel otherwise
  if (c.s.geglu && c.s.gemm_path != 0) SWMOE_TRY(launch_geglu_fwd(c.s, c.p, workspace, st));
  // expert dropout: in GEMM1's epilogue on the CTA-pair path, an element-wise kernel otherwise
  if (c.s.dropout && c.s.gemm_path != 0) SWMOE_TRY(launch_expert_dropout(c.s, c.p, false, workspace, st));
  SWMOE_TRY(mark(cfg, 4, st));
  SWMOE_TRY(run_gemm(kGemm2Combine, c, a, workspace, st));
  if (c.s.top2)                                                                   // Eq. 2: sum over the two experts
    SWMOE_TRY(launch_top2_sum(c.s, c.p, y_rows, c.s.residual ? x : nullptr, y, workspace, st));
  SWMOE_TRY(mark(cfg, 5, st));
  return SWITCH_MOE_OK;
}

int switch_moe_bwd(const switch_moe_config* cfg, const void* dy, float d_aux, const void* x, const float* W_r,
                   const void* W_in, const void* W_out, const void* y, void* workspace, size_t workspace_bytes,
                   void* dx, float* dW_r, void* dW_in, void* dW_out, void* stream) {
  Ctx c;
  SWMOE_TRY(prepare(cfg, workspace, workspace_bytes, true, &c));
  if (!dy || !x || !W_r || !W_in || !W_out || !y || !dx || !dW_r || !dW_in || !dW_out)
    return SWITCH_MOE_INVALID_ARGUMENT;
  if (!aligned16(dy) || !aligned16(x) || !aligned16(W_r) || !aligned16(W_in) || !aligned16(W_out) || !aligned16(y) ||
      !aligned16(dx) || !aligned16(dW_r) || !aligned16(dW_in) || !aligned16(dW_out))
    return SWITCH_MOE_UNSUPPORTED_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  GemmArgs a{};
  // top-2 routing: gradients are formed per assignment (the gate's from the per-assignment outputs the forward pass
  // left in the workspace) and the two input-gradient rows of a token are summed before the router adds its part
  void* dx_rows = c.s.top2 ? ws_ptr<void>(workspace, c.p.dxv) : dx;
  a.W_in = W_in; a.W_out = W_out; a.dx = dx_rows; a.dW_in = dW_in; a.dW_out = dW_out; a.dy = dy;
  SWMOE_TRY(mark(cfg, 6, st));
  SWMOE_TRY(launch_gather_dy(c.s, c.p, dy, c.s.top2 ? ws_ptr<void>(workspace, c.p.yv) : y, dx, workspace, st));
  SWMOE_TRY(mark(cfg, 7, st));
  SWMOE_TRY(run_gemm(kDgrad2Mask, c, a, workspace, st));
  // the dropout factors on the way back and d[a | b] from dH: inside dgrad2's epilogue on the CTA-pair path,
  // element-wise kernels otherwise
  if (c.s.dropout && c.s.gemm_path != 0) SWMOE_TRY(launch_expert_dropout(c.s, c.p, true, workspace, st));
  if (c.s.geglu && c.s.gemm_path != 0) SWMOE_TRY(launch_geglu_bwd(c.s, c.p, workspace, st));
  SWMOE_TRY(mark(cfg, 8, st));
  SWMOE_TRY(run_gemm(kWgrad2, c, a, workspace, st));
  SWMOE_TRY(mark(cfg, 9, st));
  if (c.s.gemm_path == 0) {
    // both products of dH in one launch (they share its rows through L2); the stage event between them falls after both
    SWMOE_TRY(launch_pair_dgrad1_wgrad1(c.s, c.p, a, workspace, st));
    SWMOE_TRY(mark(cfg, 10, st));
  } else {
    SWMOE_TRY(run_gemm(kDgrad1Scatter, c, a, workspace, st));
    SWMOE_TRY(mark(cfg, 10, st));
    SWMOE_TRY(run_gemm(kWgrad1, c, a, workspace, st));
  }
  if (c.s.top2) SWMOE_TRY(launch_top2_sum(c.s, c.p, dx_rows, c.s.residual ? dy : nullptr, dx, workspace, st));
  SWMOE_TRY(mark(cfg, 11, st));
  SWMOE_TRY(launch_router_bwd(c.s, c.p, x, W_r, ws_ptr<float>(workspace, c.p.dgate), d_aux, workspace, dx, true, dW_r,
                              st));
  SWMOE_TRY(mark(cfg, 12, st));
  return SWITCH_MOE_OK;
}

int switch_moe_router_bwd(const switch_moe_config* cfg, const void* x, const float* W_r, const float* dgate,
                          float d_aux, void* workspace, size_t workspace_bytes, void* dx_router, float* dW_r,
                          void* stream) {
  Ctx c;
  SWMOE_TRY(prepare(cfg, workspace, workspace_bytes, true, &c));
  if (!x || !W_r || !dgate || !dx_router || !dW_r) return SWITCH_MOE_INVALID_ARGUMENT;
  if (!aligned16(x) || !aligned16(W_r) || !aligned16(dx_router) || !aligned16(dW_r))
    return SWITCH_MOE_UNSUPPORTED_SHAPE;
  return launch_router_bwd(c.s, c.p, x, W_r, dgate, d_aux, workspace, dx_router, false, dW_r,
                           static_cast<cudaStream_t>(stream));
}

namespace {
// Shared body of the two host-activation entry points.  `slot_free` (may be null): event the uploads wait for instead
// of the work already enqueued on `stream`; `step_done` (may be null): recorded on the download stream after the last
// copy.  Returns with everything enqueued; nothing is synchronised here.
int step_host_enqueue(const switch_moe_config* cfg, const void* x_host, const void* dy_host, float d_aux,
                      const float* W_r, const float* router_bias, const void* W_in, const void* W_out, void* x_dev,
                      void* dy_dev, void* y_dev, void* dx_dev, float* aux_dev, float* dW_r, void* dW_in, void* dW_out,
                      void* y_host, void* dx_host, float* aux_host, void* workspace, size_t workspace_bytes,
                      cudaStream_t st, cudaStream_t up, cudaStream_t down, cudaEvent_t slot_free,
                      cudaEvent_t step_done) {
  Ctx c;
  SWMOE_TRY(prepare(cfg, workspace, workspace_bytes, true, &c));
  if (!x_host || !dy_host || !x_dev || !dy_dev || !y_dev || !dx_dev || !aux_dev || !y_host || !dx_host || !aux_host)
    return SWITCH_MOE_INVALID_ARGUMENT;
  const size_t act = (size_t)c.s.T * c.s.d * c.s.elt;
  cudaEvent_t ev[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};   // start, x up, dy up, fwd done, bwd done
  int rc = SWITCH_MOE_OK;
  auto ck = [&](cudaError_t e) { if (e != cudaSuccess && rc == SWITCH_MOE_OK) rc = SWITCH_MOE_CUDA_ERROR; };
  for (int i = 0; i < 5; ++i) ck(cudaEventCreateWithFlags(&ev[i], cudaEventDisableTiming));
  if (rc == SWITCH_MOE_OK) {
    if (slot_free != nullptr) {
      ck(cudaStreamWaitEvent(up, slot_free, 0));               // the staging buffers' previous user has finished
    } else {
      ck(cudaEventRecord(ev[0], st));                          // copies start after earlier work on `stream`
      if (up != st) ck(cudaStreamWaitEvent(up, ev[0], 0));
    }
    ck(cudaMemcpyAsync(x_dev, x_host, act, cudaMemcpyHostToDevice, up));
    ck(cudaEventRecord(ev[1], up));
    ck(cudaMemcpyAsync(dy_dev, dy_host, act, cudaMemcpyHostToDevice, up));
    ck(cudaEventRecord(ev[2], up));
    if (up != st) ck(cudaStreamWaitEvent(st, ev[1], 0));
  }
  if (rc == SWITCH_MOE_OK)
    rc = switch_moe_fwd(cfg, x_dev, W_r, router_bias, W_in, W_out, y_dev, aux_dev, workspace, workspace_bytes, st);
  if (rc == SWITCH_MOE_OK) {
    ck(cudaEventRecord(ev[3], st));
    if (down != st) ck(cudaStreamWaitEvent(down, ev[3], 0));
    ck(cudaMemcpyAsync(y_host, y_dev, act, cudaMemcpyDeviceToHost, down));
    ck(cudaMemcpyAsync(aux_host, aux_dev, sizeof(float), cudaMemcpyDeviceToHost, down));
    if (up != st) ck(cudaStreamWaitEvent(st, ev[2], 0));
  }
  if (rc == SWITCH_MOE_OK)
    rc = switch_moe_bwd(cfg, dy_dev, d_aux, x_dev, W_r, W_in, W_out, y_dev, workspace, workspace_bytes, dx_dev, dW_r,
                        dW_in, dW_out, st);
  if (rc == SWITCH_MOE_OK) {
    ck(cudaEventRecord(ev[4], st));
    if (down != st) ck(cudaStreamWaitEvent(down, ev[4], 0));
    ck(cudaMemcpyAsync(dx_host, dx_dev, act, cudaMemcpyDeviceToHost, down));
    if (step_done != nullptr) ck(cudaEventRecord(step_done, down));
  }
  // an event that has been recorded but not reached yet is released when it completes
  for (int i = 0; i < 5; ++i)
    if (ev[i] != nullptr) cudaEventDestroy(ev[i]);
  return rc;
}
}  // namespace

int switch_moe_step_host(const switch_moe_config* cfg, const void* x_host, const void* dy_host, float d_aux,
                         const float* W_r, const float* router_bias, const void* W_in, const void* W_out,
                         void* x_dev, void* dy_dev, void* y_dev, void* dx_dev, float* aux_dev, float* dW_r,
                         void* dW_in, void* dW_out, void* y_host, void* dx_host, float* aux_host, void* workspace,
                         size_t workspace_bytes, void* stream, void* h2d_stream, void* d2h_stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // Optional copy streams let dy travel to the device during the forward pass and y travel back during the
  // backward pass.  Without them (NULL) every copy is ordered on `stream`.
  cudaStream_t up = h2d_stream ? static_cast<cudaStream_t>(h2d_stream) : st;
  cudaStream_t down = d2h_stream ? static_cast<cudaStream_t>(d2h_stream) : st;
  int rc = step_host_enqueue(cfg, x_host, dy_host, d_aux, W_r, router_bias, W_in, W_out, x_dev, dy_dev, y_dev, dx_dev,
                             aux_dev, dW_r, dW_in, dW_out, y_host, dx_host, aux_host, workspace, workspace_bytes, st,
                             up, down, nullptr, nullptr);
  // always drain what was enqueued, also after an error
  if (cudaStreamSynchronize(up) != cudaSuccess && rc == SWITCH_MOE_OK) rc = SWITCH_MOE_CUDA_ERROR;
  if (cudaStreamSynchronize(st) != cudaSuccess && rc == SWITCH_MOE_OK) rc = SWITCH_MOE_CUDA_ERROR;
  if (cudaStreamSynchronize(down) != cudaSuccess && rc == SWITCH_MOE_OK) rc = SWITCH_MOE_CUDA_ERROR;
  return rc;
}

int switch_moe_step_host_enqueue(const switch_moe_config* cfg, const void* x_host, const void* dy_host, float d_aux,
                                 const float* W_r, const float* router_bias, const void* W_in, const void* W_out,
                                 void* x_dev, void* dy_dev, void* y_dev, void* dx_dev, float* aux_dev, float* dW_r,
                                 void* dW_in, void* dW_out, void* y_host, void* dx_host, float* aux_host,
                                 void* workspace, size_t workspace_bytes, void* stream, void* h2d_stream,
                                 void* d2h_stream, void* slot_free_event, void* step_done_event) {
  if (h2d_stream == nullptr || d2h_stream == nullptr || step_done_event == nullptr) return SWITCH_MOE_INVALID_ARGUMENT;
  return step_host_enqueue(cfg, x_host, dy_host, d_aux, W_r, router_bias, W_in, W_out, x_dev, dy_dev, y_dev, dx_dev,
                           aux_dev, dW_r, dW_in, dW_out, y_host, dx_host, aux_host, workspace, workspace_bytes,
                           static_cast<cudaStream_t>(stream), static_cast<cudaStream_t>(h2d_stream),
                           static_cast<cudaStream_t>(d2h_stream), static_cast<cudaEvent_t>(slot_free_event),
                           static_cast<cudaEvent_t>(step_done_event));
}

int switch_moe_check_device_status(const switch_moe_config* cfg, void* workspace, int32_t* info_out, void* stream) {
  Ctx c;
  SWMOE_TRY(prepare(cfg, workspace, ~(size_t)0, true, &c));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t host[16];
  if (cudaMemcpyAsync(host, ws_ptr<char>(workspace, c.p.status), sizeof(host), cudaMemcpyDeviceToHost, st) !=
      cudaSuccess)
    return SWITCH_MOE_CUDA_ERROR;
  if (cudaStreamSynchronize(st) != cudaSuccess) return SWITCH_MOE_CUDA_ERROR;
  if (info_out != nullptr) std::memcpy(info_out, host, sizeof(host));
  return host[0] != 0 ? SWITCH_MOE_DEVICE_TIMEOUT : SWITCH_MOE_OK;
}

int switch_moe_stage_launches(const switch_moe_config* cfg, int32_t* launches_out) {
  if (launches_out == nullptr) return SWITCH_MOE_INVALID_ARGUMENT;
  Shape s;
  SWMOE_TRY(resolve_shape(cfg, &s));
  int32_t* n = launches_out;
  for (int i = 0; i < SWITCH_MOE_STAGE_EVENTS - 1; ++i) n[i] = 0;
  // forward.  Router: the kernel itself; on the tensor cores also the bf16 split of W_r and, with more than 128
  // experts, the column sums of the probabilities (up to 128 experts the router kernel's epilogue leaves them, and
  // the plan's block histograms too); input jitter adds the element-wise product, top-2 routing the second-choice kernel.
  n[0] = (s.router_tc ? (s.Epad64 <= 128 ? 2 : 3) : 1) + (s.jitter ? 1 : 0) + (s.top2 ? 1 : 0);
  // plan: one fused kernel when the router left the histograms and there is one routing group; else (histogram,)
  // scan, assign; stage 2 of rerouting adds four
  n[1] = (s.router_hist ? (s.G == 1 ? 1 : 2) : 3) + 4 * s.reroute_stages;
  n[2] = 1;                                           // gather
  const int slow = s.gemm_path != 0 ? 1 : 0;   // gating and dropout are element-wise kernels off the CTA-pair path
  n[3] = 1 + (s.geglu ? slow : 0) + (s.dropout ? slow : 0);   // GEMM1 (+ GEGLU gating kernel, + expert dropout kernel)
  n[4] = 1 + (s.top2 ? 1 : 0);                        // GEMM2 + combine (+ sum of the two assignments' rows)
  // backward.  With the paired-CTA path the two products of dH are one launch (stage 9).
  n[6] = 1;
  n[7] = 1 + (s.dropout ? slow : 0) + (s.geglu ? slow : 0);
  n[8] = 1;
  n[9] = 1;
  n[10] = (s.gemm_path == 0 ? 0 : 1) + (s.top2 ? 1 : 0);
  n[11] = 4;                                          // logit gradients, x^T dh partials, their reduction, dx += dh W_r^T
  return SWITCH_MOE_OK;
}

int switch_moe_launches_per_step(const switch_moe_config* cfg, int32_t* launches_out) {
  if (launches_out == nullptr) return SWITCH_MOE_INVALID_ARGUMENT;
  int32_t n[SWITCH_MOE_STAGE_EVENTS];
  SWMOE_TRY(switch_moe_stage_launches(cfg, n));
  int total = 0;
  for (int i = 0; i < SWITCH_MOE_STAGE_EVENTS - 1; ++i) total += n[i];
  *launches_out = total;
  return SWITCH_MOE_OK;
}

const char* switch_moe_status_string(int status) {
  switch (status) {
    case SWITCH_MOE_OK: return "ok";
    case SWITCH_MOE_INVALID_ARGUMENT: return "invalid argument (null pointer, non-positive size, or capacity 0)";
    case SWITCH_MOE_UNSUPPORTED_SHAPE: return "unsupported shape or misaligned pointer";
    case SWITCH_MOE_WORKSPACE_TOO_SMALL: return "workspace too small";
    case SWITCH_MOE_CUDA_ERROR: return "CUDA error";
    case SWITCH_MOE_DEVICE_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

}  // extern "C"
