/*
 * switch_moe.h -- C ABI of the Switch FFN layer (Switch Transformer, arxiv 2101.03961) for one NVIDIA B200.
 *
 * One call = one routing group of T tokens (rows of x, in token order).  The layer is
 *   router      h = x . W_r (+ b), p = softmax(h) in float32          (Section 2.1, Eq. 1; Section 2.4 selective precision)
 *   top-1       e_t = argmax_i p[t,i], gate g_t = p[t,e_t]            (Section 2.1, "Switch Routing")
 *   capacity    C = floor(T * capacity_factor / E)                    (Section 2.2, Eq. 3)
 *   dispatch    expert i keeps its first C tokens in token order, later ones are dropped (Section 2.2, Fig. 3)
 *   expert FFN  o_t = ReLU(x_t W_in[e_t]) W_out[e_t], no bias         (Section 5, FFN review)
 *   combine     y_t = g_t . o_t ; y_t = 0 for a dropped token         (Section 2.1, Eq. 2 with k = 1; Fig. 2)
 *   aux loss    alpha . E . sum_i f_i . P_i                           (Section 2.2, Eq. 4-6)
 * and its backward pass (derivative of the above; f carries no gradient, Section 2.2).
 *
 * Conventions for every entry point
 *   - Plain C, no exceptions.  Return value: SWITCH_MOE_OK (0) or a negative switch_moe_status.
 *   - Unless a parameter says HOST, every data pointer is a DEVICE pointer owned by the caller; the library
 *     never allocates or frees device memory and keeps no state between calls other than what it writes into
 *     the caller's workspace.  All tensors are dense, row-major, 16-byte aligned.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only enqueue work; they do
 *     not synchronise unless stated.  Calls sharing one workspace must be ordered on one stream.
 *   - dtype SWITCH_MOE_BF16: x, W_in, W_out, y, dy, dx, dW_in, dW_out are bfloat16; the router (W_r, bias, probs,
 *     gate, dW_r, aux loss) is float32.  dtype SWITCH_MOE_F32: everything is float32.
 *   - Gradients are overwritten, not accumulated.
 *   - Limits: 1 <= E <= 256; d_model and d_ff multiples of 8 (bf16: multiples of 64 for the tensor-core path);
 *     T * capacity_factor / E >= 1.
 */
#ifndef SWITCH_MOE_H_
#define SWITCH_MOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum switch_moe_dtype { SWITCH_MOE_BF16 = 0, SWITCH_MOE_F32 = 1 };

enum switch_moe_gemm_path {
  SWITCH_MOE_GEMM_DEFAULT = 0, /* bf16: tcgen05 grouped GEMM on CTA pairs (tokens on the MMA N side) and tensor-core
                                  router; f32: plain FP32 FMA grouped GEMM and router */
  SWITCH_MOE_GEMM_SIMT = 1,    /* validation only: FP32-FMA grouped GEMM and router for either dtype */
  SWITCH_MOE_GEMM_TC_1CTA = 2  /* validation only: single-CTA tcgen05 grouped GEMM with 128-token tiles (bf16) */
};

/* SWITCH_MOE_FLAG_RESIDUAL: the layer adds its own input to its output, y_t = x_t + g_t E_{e_t}(x_t): the residual
   connection around the Switch FFN layer (Fig. 2), fused into the combine step.  A dropped token's row is then its
   input row (Section 2.2: it reaches the next layer through the residual connection).  The backward pass adds dy to
   dx accordingly.  bf16: the expert term is rounded to bf16 before the addition and the sum is rounded again.  The
   forward pass also keeps the output without the skip path in the workspace (SWITCH_MOE_WS_LAYER_Y): the gate's
   gradient <dy_t, E(x_t)> cannot be recovered from a bf16 y_t - x_t.  Not available on SWITCH_MOE_GEMM_TC_1CTA.
   SWITCH_MOE_FLAG_REROUTE: stage 2 of No-Token-Left-Behind routing (Appendix B): after the Switch routing of
   Section 2.2, every token that overflowed its expert is offered, in token order, to the expert with its
   second-highest probability and takes that expert's next free slot if one is left; its gate is that expert's
   probability.  Tokens kept by the first stage keep their slots, and f in the auxiliary loss still counts the
   argmax.  switch_moe_config.reroute_stages repeats the step with the third, fourth, .. choices (the figure's
   caption: the process can be iterated); equal probabilities are ranked by index, lowest first.  One routing group
   only.
   SWITCH_MOE_FLAG_INPUT_JITTER: the router's input is x . u, element by element, with u = router_jitter (input
   jitter as the text describes it, Appendix C); the experts still see x.  The product
   is rounded to the activation dtype (the router's input is a tensor of that type) and kept in the workspace for
   the backward pass, where dW_r uses it and the router's part of dx is multiplied by u.
   SWITCH_MOE_FLAG_GEGLU: the experts are GEGLU FFNs (Table 9: two expansion matrices whose outputs are combined
   non-linearly): W_in is [E, d_model, 2 d_ff] = [W_0 | W_1] per expert (and dW_in likewise), hidden = GELU(x W_0) . (x W_1) with the exact form GELU(z) = z Phi(z) (not the tanh fit; Phi is evaluated to about 3e-7 absolute), y = hidden W_out.  The two products are
   one grouped GEMM with 2 d_ff output columns.  On the default path its epilogue also gates (a CTA multiplies 64
   columns of W_0 and the same 64 columns of W_1, the two epilogue warps that hold a and b of a hidden unit exchange
   them through shared memory): it writes the hidden activations and, for the backward pass, the two factors
   GELU(a) and b GELU'(a) of every hidden unit (rounded to the activation dtype) instead of a and b; dgrad2's
   epilogue multiplies dH by them and writes d[a | b] directly.  On the other paths the gating and its derivative
   are element-wise kernels over the kept rows.  Not available on SWITCH_MOE_GEMM_TC_1CTA.
   SWITCH_MOE_FLAG_TOP2: top-2 routing, the Mixture-of-Experts layer the paper compares with (Eq. 1-2 with the two
   highest-probability experts): y_t = p_a E_a(x_t) + p_b E_b(x_t) with the softmax probabilities of Eq. 1 as they
   are.  Every token's first choice is placed before any second choice (token order within each round), all against
   the capacity of Eq. 3; f in the auxiliary loss counts the first choice.  The library numbers the 2T assignments
   v = t (first choice of token t) and v = T + t (second choice): the workspace regions EXPERT_INDEX, GATE, SLOT and
   DGATE then have 2T entries and TOKEN_OF_SLOT holds v.  Needs T to be a multiple of 256; not together with
   REROUTE, several routing groups, GEGLU experts, expert dropout, input jitter or logit noise (UNSUPPORTED_SHAPE).  With RESIDUAL the input row is added where the two assignments' rows are
   summed (one rounding of the three-term sum), and dy likewise on the way back.
   SWITCH_MOE_FLAG_EXPERT_DROPOUT: expert dropout (the fine-tuning regularisation of Section 2.4: a larger dropout
   rate on the hidden activations inside every expert): the experts' hidden activations are
   multiplied by keep / (1 - expert_dropout), and so is their gradient on the way back.  The keep mask is an input
   (expert_keep), one bit per hidden unit of every slot row; the caller draws it.  On the default path both happen in
   GEMM epilogues (GEMM1 applies the factor before it rounds; the ReLU mask bits it saves then say "kept and
   positive", so dgrad2 only multiplies by 1 / (1 - rate); with GEGLU experts the factors saved for the backward pass
   carry it), on the other paths in element-wise kernels.  One routing group only. */
enum switch_moe_flags {
  SWITCH_MOE_FLAG_RESIDUAL = 1, SWITCH_MOE_FLAG_REROUTE = 2, SWITCH_MOE_FLAG_INPUT_JITTER = 4, SWITCH_MOE_FLAG_GEGLU = 8,
  SWITCH_MOE_FLAG_TOP2 = 16, SWITCH_MOE_FLAG_EXPERT_DROPOUT = 32
};

typedef enum switch_moe_status {
  SWITCH_MOE_OK = 0,
  SWITCH_MOE_INVALID_ARGUMENT = -1,    /* null pointer, non-positive size, capacity 0 */
  SWITCH_MOE_UNSUPPORTED_SHAPE = -2,   /* E > 256, d_model / d_ff not a supported multiple, misaligned pointer */
  SWITCH_MOE_WORKSPACE_TOO_SMALL = -3,
  SWITCH_MOE_CUDA_ERROR = -4,          /* a CUDA runtime / driver call or a kernel launch failed */
  SWITCH_MOE_DEVICE_TIMEOUT = -5       /* a bounded device-side wait gave up (see switch_moe_check_device_status) */
} switch_moe_status;

typedef struct switch_moe_config {
  int32_t T;                 /* tokens in this routing group */
  int32_t d_model;
  int32_t d_ff;
  int32_t E;                 /* number of experts (the paper's N) */
  float capacity_factor;     /* Eq. 3 */
  float alpha;               /* Eq. 4 coefficient */
  int32_t capacity_override; /* 0: use Eq. 3; > 0: use this expert capacity instead */
  int32_t dtype;             /* switch_moe_dtype */
  int32_t gemm_path;         /* switch_moe_gemm_path */
  int32_t flags;             /* bitwise OR of switch_moe_flags */
  int32_t groups;            /* routing groups G in this call (0 or 1: one group).  The pseudo-code's leading cores
                                dimension: group g is rows [g T/G, (g+1) T/G) of x and is routed on its own -- own
                                capacity floor((T/G) capacity_factor / E) by Eq. 3, own f and P in Eq. 5-6 -- while
                                the experts are shared; the auxiliary loss is the mean of the groups' losses.  An
                                expert's rows in the slot buffers are numbered group by group, each group's kept
                                tokens in token order, G x capacity rows per expert.  G > 1 needs T / G to be a
                                multiple of 256, T <= 65536 and G <= 64. */
  int32_t reroute_stages;    /* SWITCH_MOE_FLAG_REROUTE: how many further stages follow stage 1 (0 or 1: the figure's
                                stage 2 alone; n: stages 2 .. n + 1, stage k offering the tokens still without a slot
                                to the expert with their k-th highest probability; at most 16).  Ignored without
                                the flag.  SWITCH_MOE_WS_SECOND_CHOICE then holds one int32[T] array per stage. */
  int32_t reserved[2];       /* must be 0 */
  void* const* stage_events; /* HOST array of SWITCH_MOE_STAGE_EVENTS cudaEvent_t handles, or NULL (default).
                                When set, fwd records event i on the stream before its stage i (0 router, 1 dispatch
                                plan, 2 gather, 3 GEMM1+ReLU, 4 GEMM2+combine) and event 5 after the last one; bwd
                                records events 6..11 before (6 gather dy, 7 dgrad2, 8 wgrad2, 9 dgrad1, 10 wgrad1,
                                11 router backward) and event 12 after.  With gemm_path 0 dgrad1 and wgrad1 are one
                                launch: event 10 follows it, so stage 9 spans both products and stage 10 is empty.
                                For per-kernel timing only. */
  const float* router_noise; /* DEVICE float[T, E] added to the router logits before the softmax, or NULL (default).
                                The router pseudo-code of the appendix adds uniform(1 - eps, 1 + eps) noise to the
                                logits in training (the text instead speaks of multiplicative jitter on the router's
                                input; this field follows the pseudo-code).  The noise is an input, drawn by the
                                caller; it is a constant of the backward pass. */
  const void* router_jitter; /* DEVICE [T, d_model] in the activation dtype: the factors u of SWITCH_MOE_FLAG_INPUT_JITTER
                                (e.g. uniform(1 - eps, 1 + eps), drawn by the caller); must be set, 16-byte aligned,
                                when the flag is, and is ignored otherwise.  Needed by fwd, router_fwd, bwd and
                                router_bwd alike. */
  const uint32_t* expert_keep; /* DEVICE uint32[E * G * C][d_ff / 32]: bit i of word [row][w] = keep hidden unit 32 w + i
                                  of slot row `row` (SWITCH_MOE_FLAG_EXPERT_DROPOUT; d_ff a multiple of 32) */
  float expert_dropout;        /* the dropout rate of that flag, in [0, 1) */
} switch_moe_config;

#define SWITCH_MOE_STAGE_EVENTS 13

/* Regions of the workspace that switch_moe_workspace_view can expose (all written by the library). */
enum switch_moe_ws_region {
  SWITCH_MOE_WS_STATUS = 0,         /* int32[16]; [0] != 0 after a device-side timeout ([0] = code of the wait that gave
                                       up, [1] = its block, [2] = the barrier phase) */
  SWITCH_MOE_WS_EXPERT_INDEX = 1,   /* int32[T]   e_t */
  SWITCH_MOE_WS_GATE = 2,           /* float[T]   g_t (the un-masked top-1 probability, also for dropped tokens) */
  SWITCH_MOE_WS_SLOT = 3,           /* int32[T]   row of the token in the slot buffers: e_t * (G C) + (kept tokens of
                                       e_t in earlier groups) + pos_t, or -1 if dropped */
  SWITCH_MOE_WS_TOKEN_OF_SLOT = 4,  /* int32[E*G*C] token stored in each slot, or -1 */
  SWITCH_MOE_WS_COUNT = 5,          /* int32[E]   tokens whose argmax is expert i, before the capacity cut */
  SWITCH_MOE_WS_KEPT = 6,           /* int32[E]   kept tokens: sum over groups of min(count in the group, C) */
  SWITCH_MOE_WS_PSUM = 7,           /* float[E]   sum_t p[t,i] */
  SWITCH_MOE_WS_PROBS = 8,          /* float[T,E] router probabilities */
  SWITCH_MOE_WS_XD = 9,             /* [E,G*C,d_model] dispatched tokens (dtype of x); likewise the next three */
  SWITCH_MOE_WS_H = 10,             /* [E,C,d_ff]    ReLU(x W_in) per slot */
  SWITCH_MOE_WS_DYD = 11,           /* [E,C,d_model] g . dy per slot (backward) */
  SWITCH_MOE_WS_DH = 12,            /* [E,C,d_ff]    gradient of the pre-activation per slot (backward) */
  SWITCH_MOE_WS_DGATE = 13,         /* float[T]   <dy_t, o_t> for kept tokens (backward) */
  SWITCH_MOE_WS_DLOGITS = 14,       /* float[T,E] gradient of the router logits: written by switch_moe_router_bwd, and
                                       by switch_moe_bwd only where the router runs on the FP32 FMA path (the
                                       tensor-core path keeps just the bfloat16 parts it multiplies) */
  SWITCH_MOE_WS_LAYER_Y = 15,       /* [T,d_model] g_t E(x_t) without the skip path (only with SWITCH_MOE_FLAG_RESIDUAL;
                                       rows of dropped tokens are not written) */
  SWITCH_MOE_WS_EXPERT_PROC = 16,   /* int32[T] the expert that processes the token: e_t unless stage 2 rerouted it
                                       (only with SWITCH_MOE_FLAG_REROUTE) */
  SWITCH_MOE_WS_SECOND_CHOICE = 17, /* int32[T] second-choice expert of a token that overflowed in stage 1, -1 for the
                                       others (only with SWITCH_MOE_FLAG_REROUTE) */
  SWITCH_MOE_WS_REGION_COUNT = 18
};

/* Eq. 3.  HOST call.  *C_out = capacity_override if > 0, else floor((T / G) * capacity_factor / E) capped at T / G:
   the capacity of one expert for one routing group (the slot buffers hold G * C rows per expert).
 * Errors: INVALID_ARGUMENT for null pointers, non-positive sizes or a resulting capacity of 0. */
int switch_moe_capacity(const switch_moe_config* cfg, int32_t* C_out);

/* HOST call.  Bytes of device workspace that fwd/bwd need for this config (a few hundred MB at Switch-Base
 * shapes: the per-slot buffers X_d, H, dY_d, dH dominate).  The workspace must be 1024-byte aligned. */
int switch_moe_workspace_bytes(const switch_moe_config* cfg, size_t* bytes_out);

/* HOST call.  Device address and size of one workspace region (switch_moe_ws_region), for diagnostics and
 * staged tests.  Nothing is copied. */
int switch_moe_workspace_view(const switch_moe_config* cfg, void* workspace, int32_t region, void** ptr_out,
                              size_t* bytes_out);

/* Forward of the whole layer (all of: router, Eq. 1; top-1; Eq. 3 capacity and token-order dispatch, Fig. 3;
 * expert FFN; gate-scaled combine, Eq. 2; auxiliary loss, Eq. 4-6).
 *   x [T,d_model]; W_r [d_model,E] float32; router_bias float32[E] or NULL (constant added to the logits; the
 *   paper's router has none); W_in [E,d_model,d_ff]; W_out [E,d_ff,d_model];
 *   y [T,d_model] (out; rows of dropped tokens are written as 0); aux_loss device float[1] (out).
 * The workspace keeps what backward needs (probs, expert index, gate, slots, X_d, H). */
int switch_moe_fwd(const switch_moe_config* cfg, const void* x, const float* W_r, const float* router_bias,
                   const void* W_in, const void* W_out, void* y, float* aux_loss, void* workspace,
                   size_t workspace_bytes, void* stream);

/* Backward of the whole layer, for upstream gradients dy [T,d_model] of y and the scalar d_aux of the auxiliary
 * loss (1.0 when that loss is simply added to the model loss, Section 2.2).  `workspace` must be the one the
 * matching switch_moe_fwd call filled, and x, W_r, W_in, W_out, y the same buffers with unchanged contents.
 *   dx [T,d_model], dW_r [d_model,E] float32, dW_in [E,d_model,d_ff], dW_out [E,d_ff,d_model] (all out).
 * The gate gradient uses o_t = y_t / g_t (g_t >= 1/E > 0).  f carries no gradient (Section 2.2). */
int switch_moe_bwd(const switch_moe_config* cfg, const void* dy, float d_aux, const void* x, const float* W_r,
                   const void* W_in, const void* W_out, const void* y, void* workspace, size_t workspace_bytes,
                   void* dx, float* dW_r, void* dW_in, void* dW_out, void* stream);

/* Staged: the router alone (Eq. 1, top-1, the P-sums of Eq. 6).  Fills the workspace regions PROBS, EXPERT_INDEX,
 * GATE and the per-block partial sums that the dispatch plan reduces into PSUM. */
int switch_moe_router_fwd(const switch_moe_config* cfg, const void* x, const float* W_r, const float* router_bias,
                          void* workspace, size_t workspace_bytes, void* stream);

/* Staged: the dispatch plan alone (Eq. 3, Fig. 3, Eq. 4-6) for a caller-supplied expert index (device int32[T],
 * e.g. the oracle's).  If expert_index is NULL the workspace's EXPERT_INDEX is used.  Fills COUNT, KEPT, SLOT,
 * TOKEN_OF_SLOT, PSUM (from whatever partial sums the workspace holds) and, if aux_loss != NULL, the loss. */
int switch_moe_dispatch_plan(const switch_moe_config* cfg, const int32_t* expert_index, float* aux_loss,
                             void* workspace, size_t workspace_bytes, void* stream);

/* Staged: the router's backward alone for a caller-supplied gate gradient (device float[T]; entries of dropped
 * tokens are ignored).  The paper states no backward pass; this is the derivative of its forward definitions: the
 * gate value p_i(x) of Eq. 2 carries the gradient into the router (Section 2.1: the gate keeps the router
 * differentiable), the softmax of Eq. 1 is differentiated as usual, and the auxiliary loss of Eq. 4 contributes
 * through P_i only, because f_i (Eq. 5) is not differentiable (Section 2.2):
 * G = d_aux.alpha.E.f_i/T + [i = e_t, kept].dgate_t, dh = p (G - <p,G>), dW_r = x^T dh,
 * dx_router = dh W_r^T.  Uses PROBS, EXPERT_INDEX, SLOT, COUNT of the workspace.  dx_router [T,d_model] is written
 * in the config's dtype (not accumulated). */
int switch_moe_router_bwd(const switch_moe_config* cfg, const void* x, const float* W_r, const float* dgate,
                          float d_aux, void* workspace, size_t workspace_bytes, void* dx_router, float* dW_r,
                          void* stream);

/* The dispatch plan for callers that cannot allocate device memory and have no workspace to pass.  (The paper has
 * no counterpart: this is a packaging variant of switch_moe_dispatch_plan, not a step of the method.)
 * Meant for a process whose device heap is owned entirely by another allocator (a serving arena, a framework's
 * caching pool), or a call site where cudaMalloc's device-wide synchronisation cannot be tolerated.  The only
 * scratch the plan needs -- per-block expert histograms and their scan -- is a 512 KiB array compiled into the
 * library, resident on every GPU that loads it until the process exits; the call itself allocates and frees
 * nothing (no cudaMalloc / cudaFree, no allocating library routine).
 *   expert_index device int32[T] (in; an entry that is negative or >= E means "no expert" and takes no slot).
 *   Outputs, all caller-owned device buffers: count int32[E], kept int32[E], slot int32[T] (e*C + position, or -1
 *   if dropped), token_of_slot int32[E*C] (-1 for empty slots) -- the same values switch_moe_dispatch_plan leaves
 *   in its workspace regions of those names.
 * Limits: T <= SWITCH_MOE_STATIC_PLAN_MAX_TOKENS, E <= 256, one routing group, and the top-1 plan of Section 2.2
 * only: a config with SWITCH_MOE_FLAG_TOP2 or SWITCH_MOE_FLAG_REROUTE is refused like an oversized one
 * (SWITCH_MOE_UNSUPPORTED_SHAPE), since those plans place more assignments than the array is sized for.
 * The first call on each device looks up the array's device address (with that device current); make that first
 * call before starting any stream capture.  All calls on a device share the one array: nothing in it needs
 * clearing between calls (every word read is written earlier in the same call), but two calls whose kernels
 * overlap on the GPU (different streams, or several host threads) race on it -- serialise them. */
#define SWITCH_MOE_STATIC_PLAN_MAX_TOKENS 65536
int switch_moe_dispatch_plan_static(const switch_moe_config* cfg, const int32_t* expert_index, int32_t* count,
                                    int32_t* kept, int32_t* slot, int32_t* token_of_slot, void* stream);

/* One training step with HOST activations: copies x_host and dy_host (pinned host memory, [T,d_model]) to the
 * device buffers x_dev / dy_dev, runs switch_moe_fwd and switch_moe_bwd, and copies y, dx and the auxiliary loss
 * back to y_host, dx_host, aux_host.  Weights and weight gradients stay on the device.  x_dev, dy_dev, y_dev, dx_dev,
 * aux_dev are caller-owned device staging buffers.  h2d_stream / d2h_stream (cudaStream_t, may be NULL) are
 * optional extra streams: with them dy is uploaded during the forward pass and y downloaded during the backward
 * pass; with NULL every copy runs on `stream`.  The call creates and destroys a few CUDA events (no device
 * memory) and synchronises all the streams it used before returning. */
int switch_moe_step_host(const switch_moe_config* cfg, const void* x_host, const void* dy_host, float d_aux,
                         const float* W_r, const float* router_bias, const void* W_in, const void* W_out,
                         void* x_dev, void* dy_dev, void* y_dev, void* dx_dev, float* aux_dev, float* dW_r,
                         void* dW_in, void* dW_out, void* y_host, void* dx_host, float* aux_host, void* workspace,
                         size_t workspace_bytes, void* stream, void* h2d_stream, void* d2h_stream);

/* The same step without the final synchronisation, for callers that keep several steps in flight: everything is
 * enqueued and the call returns.  h2d_stream and d2h_stream are required.  slot_free_event (cudaEvent_t, may be NULL):
 * the uploads into x_dev / dy_dev wait for it instead of for the work already enqueued on `stream` -- pass the
 * step_done_event of the step that last used these staging buffers.  step_done_event (cudaEvent_t, required) is
 * recorded on d2h_stream after the last download: y_host, dx_host and aux_host are valid, and the host inputs and all
 * staging buffers reusable, once it has completed.  The kernels of all steps share `stream`, so one workspace and one
 * set of weight-gradient buffers serve every step in flight; only the five staging buffers (and the host result
 * buffers) need one copy per step in flight. */
int switch_moe_step_host_enqueue(const switch_moe_config* cfg, const void* x_host, const void* dy_host, float d_aux,
                                 const float* W_r, const float* router_bias, const void* W_in, const void* W_out,
                                 void* x_dev, void* dy_dev, void* y_dev, void* dx_dev, float* aux_dev, float* dW_r,
                                 void* dW_in, void* dW_out, void* y_host, void* dx_host, float* aux_host,
                                 void* workspace, size_t workspace_bytes, void* stream, void* h2d_stream,
                                 void* d2h_stream, void* slot_free_event, void* step_done_event);

/* Synchronises `stream`, reads the workspace's status word and returns SWITCH_MOE_DEVICE_TIMEOUT if a kernel
 * gave up on a bounded wait (its results are then invalid), SWITCH_MOE_CUDA_ERROR if the stream reports an
 * error, else SWITCH_MOE_OK.  info_out (HOST int32[16], may be NULL) receives the raw status words. */
int switch_moe_check_device_status(const switch_moe_config* cfg, void* workspace, int32_t* info_out, void* stream);

/* HOST call.  Number of this library's kernels that one switch_moe_fwd plus one switch_moe_bwd launch. */
int switch_moe_launches_per_step(const switch_moe_config* cfg, int32_t* launches_out);

/* HOST call.  The same count per stage: launches_out (HOST int32[SWITCH_MOE_STAGE_EVENTS - 1]) entry i is the number
 * of kernels launched between stage event i and stage event i + 1 (see switch_moe_config::stage_events; entry 5, the
 * gap between the forward and the backward pass, is 0). */
int switch_moe_stage_launches(const switch_moe_config* cfg, int32_t* launches_out);

/* HOST call.  Static description of a status code. */
const char* switch_moe_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* SWITCH_MOE_H_ */
