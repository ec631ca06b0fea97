// Capacity-limited dispatch of the Switch FFN layer (Section 2.2, Eq. 3 and Fig. 3) and the load-balancing loss
// (Eq. 4-6), as integer index work: no one-hot dispatch / combine tensor is ever built.
//   plan   : count_i, pos_t = number of earlier tokens with the same expert, keep_t = pos_t < C,
//            slot_t = e_t * C + pos_t, token_of_slot, kept_i = min(count_i, C), token-tile list for the grouped GEMMs,
//            P-sums and aux = alpha . E . sum_i (count_i / T)(Psum_i / T)
//   gather : X_d[slot] = x[token]   (forward)        dY_d[slot] = g_token . dy[token], dgate_token (backward)
// Positions are deterministic (token order): block histograms -> column scan -> stable in-block rank. No atomics
// decide a position.
#include "switch_common.cuh"

namespace swmoe {
namespace {

// hist[b][e] = number of tokens of block b routed to expert e
__global__ void __launch_bounds__(kPlanBlockTokens)
plan_hist_kernel(const int* __restrict__ expert_index, int T, int E, int* __restrict__ hist) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int h[kMaxExperts];
  for (int e = threadIdx.x; e < E; e += blockDim.x) h[e] = 0;
  __syncthreads();
  const int t = blockIdx.x * kPlanBlockTokens + threadIdx.x;
  const int e = t < T ? expert_index[t] : -1;
  if ((unsigned)e < (unsigned)E) atomicAdd(&h[e], 1);        // integer counts: order-independent; negative or >= E: no vote
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) hist[(size_t)blockIdx.x * E + e] = h[e];
}

// Tile lists, shared by both scan kernels: 128-row token tiles (single-CTA GEMM) and, for the paired-CTA GEMM, each
// expert's kept rows cut into the fewest pieces of at most kPairTileTokens rows, equal up to rounding each piece to a
// multiple of 16 (the MMA's N granularity).  Thread 0 adds the loss terms and scans the per-expert tile counts; the first E
// threads write their expert's entries.  `term` and `kept_s` are shared-memory arrays filled before the call.
__device__ __forceinline__ void write_tile_lists(const float* term, const int* kept_s, int E, float loss_scale,
                                                 float* __restrict__ aux_loss, int* __restrict__ tile_expert,
                                                 int* __restrict__ tile_row0, int4* __restrict__ ntile) {
  // Everything here is a sum or a running sum over the experts, done by the first kMaxExperts threads in log2 steps
  // (a fixed tree, so the loss is the same number on every run): the loss terms, and the number of tiles before
  // each expert in the two lists.
  __shared__ int start128[kMaxExperts], startn[kMaxExperts];
  __shared__ float lsum[kMaxExperts];
  const int e = threadIdx.x;
  __syncthreads();
  int n128 = 0, npair = 0;
  if (e < kMaxExperts) {
    const int k = e < E ? kept_s[e] : 0;
    n128 = (k + kTileM - 1) / kTileM;
    npair = (k + kPairTileTokens - 1) / kPairTileTokens;
    start128[e] = n128; startn[e] = npair;
    lsum[e] = e < E ? term[e] : 0.f;
  }
  __syncthreads();
  for (int off = 1; off < kMaxExperts; off <<= 1) {            // inclusive scans (counts), pairwise tree (loss)
    int a = 0, b = 0;
    float c = 0.f;
    const bool scan = e < kMaxExperts && e >= off;
    const bool tree = e < kMaxExperts && (e & (2 * off - 1)) == 0 && e + off < kMaxExperts;
    if (scan) { a = start128[e - off]; b = startn[e - off]; }
    if (tree) c = lsum[e + off];
    __syncthreads();
    if (scan) { start128[e] += a; startn[e] += b; }
    if (tree) lsum[e] += c;
    __syncthreads();
  }
  if (e == 0) {
    if (aux_loss != nullptr) *aux_loss = loss_scale * lsum[0];                        // Eq. 4
    const int n = start128[kMaxExperts - 1], m = startn[kMaxExperts - 1];
    tile_expert[0] = n;
    tile_row0[0] = n;
    ntile[0] = make_int4(m, 0, 0, 0);
  }
  if (e < E) {
    const int k = kept_s[e];
    int n = start128[e] - n128;                                // tiles of earlier experts
    for (int r = 0; r < k; r += kTileM, ++n) { tile_expert[1 + n] = e; tile_row0[1 + n] = r; }
    if (k > 0) {
      const int pieces = npair;
      const int rows = ((k + pieces - 1) / pieces + 15) / 16 * 16;
      int m = startn[e] - npair;
      for (int r = 0; r < k; r += rows, ++m) ntile[1 + m] = make_int4(e, r, min(rows, (k - r + 15) / 16 * 16), 0);
    }
  }
}

// One block of 1024 threads = G groups x Ew columns (Ew = E rounded up to a power of two, at least 32; G = 1024 / Ew):
// thread (g, e) owns slice g of the rows of column e.  Column scan of the histograms, counts, kept, P-sums (all in a
// fixed order), the auxiliary loss and the token-tile list.  A thread's rows are loaded once, all loads in flight
// together, and kept in registers for the scan (up to kScanRows rows per thread; longer slices are re-read).
constexpr int kScanThreads = 1024;
constexpr int kScanRows = 16;
__global__ void __launch_bounds__(kScanThreads)
plan_scan_kernel(const int* __restrict__ hist, int plan_blocks, int loss_blocks, const float* __restrict__ psum_partial,
                 int router_blocks, int T, int E, int Ew, int C, float alpha, int* __restrict__ hist_base,
                 int* __restrict__ count, int* __restrict__ kept, float* __restrict__ psum,
                 float* __restrict__ aux_loss, int* __restrict__ tile_expert, int* __restrict__ tile_row0,
                 int4* __restrict__ ntile, int* __restrict__ count_g, int* __restrict__ group_base) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int qsum[kScanThreads];                         // [g][e], Ew columns per row
  __shared__ int qfirst[kScanThreads];                       // the same over rows < loss_blocks (top-2: first choices)
  __shared__ float qps[kScanThreads];
  __shared__ float term[kMaxExperts];
  __shared__ int kept_s[kMaxExperts];
  const int G = kScanThreads / Ew;
  const int e = threadIdx.x % Ew, g = threadIdx.x / Ew;
  const int hq = (plan_blocks + G - 1) / G, h0 = g * hq, h1 = min(plan_blocks, h0 + hq);
  const int rq = (router_blocks + G - 1) / G, r0 = g * rq, r1 = min(router_blocks, r0 + rq);
  int hv[kScanRows];
  if (e < E) {
#pragma unroll
    for (int j = 0; j < kScanRows; ++j) hv[j] = h0 + j < h1 ? hist[(size_t)(h0 + j) * E + e] : 0;
    float pv[kScanRows];
#pragma unroll
    for (int j = 0; j < kScanRows; ++j) pv[j] = r0 + j < r1 ? psum_partial[(size_t)(r0 + j) * E + e] : 0.f;
    int sum = 0, first = 0;
#pragma unroll
    for (int j = 0; j < kScanRows; ++j) { sum += hv[j]; if (h0 + j < loss_blocks) first += hv[j]; }
    for (int b = h0 + kScanRows; b < h1; ++b) {
      const int v = hist[(size_t)b * E + e];
      sum += v;
      if (b < loss_blocks) first += v;
    }
    float ps = 0.f;
#pragma unroll
    for (int j = 0; j < kScanRows; ++j) ps += pv[j];                                   // fixed order
    for (int b = r0 + kScanRows; b < r1; ++b) ps += psum_partial[(size_t)b * E + e];
    qsum[g * Ew + e] = sum;
    qfirst[g * Ew + e] = first;
    qps[g * Ew + e] = ps;
  }
  __syncthreads();
  if (e < E) {
    int run = 0;
    for (int q = 0; q < g; ++q) run += qsum[q * Ew + e];
#pragma unroll
    for (int j = 0; j < kScanRows; ++j)
      if (h0 + j < h1) { hist_base[(size_t)(h0 + j) * E + e] = run; run += hv[j]; }
    for (int b = h0 + kScanRows; b < h1; ++b) { hist_base[(size_t)b * E + e] = run; run += hist[(size_t)b * E + e]; }
    if (g == 0) {
      int total = 0, first = 0;
      float ps = 0.f;
      for (int q = 0; q < G; ++q) { total += qsum[q * Ew + e]; first += qfirst[q * Ew + e]; ps += qps[q * Ew + e]; }
      count[e] = first;                                                                // f counts the argmax (Eq. 5)
      count_g[e] = first;                                                              // one routing group
      group_base[e] = 0;
      const int k = min(total, C);
      kept[e] = k;
      kept_s[e] = k;
      psum[e] = ps;
      term[e] = ((float)first / (float)T) * (ps / (float)T);                           // f_i . P_i  (Eq. 5, 6)
    }
  }
  write_tile_lists(term, kept_s, E, alpha * (float)E, aux_loss, tile_expert, tile_row0, ntile);
}

// Several routing groups (the pseudo-code's leading cores dimension): every group has its own counts, its own
// capacity cut and its own f and P; an expert's rows are numbered group by group.  One block of 1024 threads;
// thread (q, e) handles groups q, q + Q, ... of column e (Q = 1024 / Ew).  hist_base[b][e] is the position base of
// block b inside its own group; group_base[g][e] = kept tokens of expert e in groups before g; the loss is the mean
// of the groups' losses: (alpha E / G) sum_g sum_i (count_gi / Tg)(Psum_gi / Tg).
constexpr int kScanGroupCells = 8192;                        // G x Ew counters kept in shared memory
__global__ void __launch_bounds__(kScanThreads)
plan_scan_groups_kernel(const int* __restrict__ hist, int blocks_per_group, const float* __restrict__ psum_partial,
                        int rows_per_group, int NG, int Tg, int E, int Ew, int Cg, float alpha,
                        int* __restrict__ hist_base, int* __restrict__ count, int* __restrict__ kept,
                        float* __restrict__ psum, float* __restrict__ aux_loss, int* __restrict__ tile_expert,
                        int* __restrict__ tile_row0, int4* __restrict__ ntile, int* __restrict__ count_g,
                        int* __restrict__ group_base) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int cnt_s[kScanGroupCells];                     // [g][e], Ew columns per row
  __shared__ float qps[kScanThreads], qterm[kScanThreads];   // [q][e]
  __shared__ float term[kMaxExperts];
  __shared__ int kept_s[kMaxExperts];
  const int Q = kScanThreads / Ew;
  const int e = threadIdx.x % Ew, q = threadIdx.x / Ew;
  float ps_tot = 0.f, t_tot = 0.f;
  if (e < E) {
    for (int g = q; g < NG; g += Q) {
      int run = 0;
      for (int b = g * blocks_per_group; b < (g + 1) * blocks_per_group; ++b) {
        hist_base[(size_t)b * E + e] = run;
        run += hist[(size_t)b * E + e];
      }
      float ps = 0.f;
      for (int r = g * rows_per_group; r < (g + 1) * rows_per_group; ++r) ps += psum_partial[(size_t)r * E + e];
      cnt_s[g * Ew + e] = run;
      count_g[(size_t)g * E + e] = run;
      ps_tot += ps;                                                                    // fixed order
      t_tot += ((float)run / (float)Tg) * (ps / (float)Tg);                            // f_gi . P_gi  (Eq. 5, 6)
    }
  }
  qps[threadIdx.x] = ps_tot;
  qterm[threadIdx.x] = t_tot;
  __syncthreads();
  if (q == 0 && e < E) {
    int base = 0, total = 0;
    for (int g = 0; g < NG; ++g) {
      const int c = cnt_s[g * Ew + e];
      group_base[(size_t)g * E + e] = base;
      base += min(c, Cg);
      total += c;
    }
    float ps = 0.f, tm = 0.f;
    for (int k = 0; k < Q; ++k) { ps += qps[k * Ew + e]; tm += qterm[k * Ew + e]; }
    count[e] = total;
    kept[e] = base;
    kept_s[e] = base;
    psum[e] = ps;
    term[e] = tm;
  }
  write_tile_lists(term, kept_s, E, alpha * (float)E / (float)NG, aux_loss, tile_expert, tile_row0, ntile);
}

// pos_t = base[block][e] + (tokens of earlier warps with e) + (earlier lanes with e); slot, token_of_slot.
__global__ void __launch_bounds__(kPlanBlockTokens)
plan_assign_kernel(const int* __restrict__ expert_index, const int* __restrict__ hist_base,
                   const int* __restrict__ kept, const int* __restrict__ group_base, int blocks_per_group, int T,
                   int E, int C, int Cg, int* __restrict__ slot, int* __restrict__ token_of_slot) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int warp_cnt[kPlanBlockTokens / 32][kMaxExperts];
  constexpr int kWarps = kPlanBlockTokens / 32;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int i = tid; i < kWarps * kMaxExperts; i += blockDim.x) (&warp_cnt[0][0])[i] = 0;
  __syncthreads();
  const int t = blockIdx.x * kPlanBlockTokens + tid;
  int e = t < T ? expert_index[t] : -1;                       // negative: no expert (takes no slot)
  if (e >= E) e = -1;                                         // an index no expert has is treated the same way
  const unsigned same = __match_any_sync(0xffffffffu, e >= 0 ? e : -1 - lane);   // distinct dummies for those lanes
  const int rank = __popc(same & ((1u << lane) - 1u));
  if (e >= 0 && rank == 0) warp_cnt[warp][e] = __popc(same);
  __syncthreads();
  if (t < T && e < 0) slot[t] = -1;
  if (e >= 0) {
    int pos = hist_base[(size_t)blockIdx.x * E + e] + rank;                  // position inside the token's own group
    for (int w = 0; w < warp; ++w) pos += warp_cnt[w][e];
    const int grp = blockIdx.x / blocks_per_group;
    const int s = pos < Cg ? e * C + group_base[(size_t)grp * E + e] + pos : -1;
    slot[t] = s;
    if (s >= 0) token_of_slot[s] = t;
  }
  // empty slots of every expert: -1 (disjoint from the kept slots written above)
  const int total = E * C;
  for (int s = blockIdx.x * blockDim.x + tid; s < total; s += gridDim.x * blockDim.x) {
    const int ex = s / C, pos = s - ex * C;
    if (pos >= kept[ex]) token_of_slot[s] = -1;
  }
}

// The whole plan in one launch, for one routing group whose block histograms already exist (the tensor-core router's
// forward kernel leaves hist[r][e] = tokens of the r-th block of 256 tokens routed to expert e).  Every block of 1024
// tokens adds up the histogram columns itself -- all rows for the totals (kept_i = min(count_i, C), Eq. 3), the rows
// before its own tokens for its position base -- instead of waiting for a scan kernel: the table is small (64 KB at
// 128 x 128) and stays in L2.  Then, as in plan_assign_kernel, pos_t = base + (tokens of earlier warps with the same
// expert) + (earlier lanes with it), in token order, with no atomics deciding a position.  One extra block writes the
// counts, the P-sums, the auxiliary loss (Eq. 4-6) and the tile lists.
constexpr int kFusedTokens = 1024;
__global__ void __launch_bounds__(kFusedTokens)
plan_fused_kernel(const int* __restrict__ expert_index, const int* __restrict__ hist, int hist_rows,
                  const float* __restrict__ psum_partial, int router_blocks, int T, int E, int Ew, int C, float alpha,
                  int* __restrict__ slot, int* __restrict__ token_of_slot, int* __restrict__ count,
                  int* __restrict__ kept, float* __restrict__ psum, float* __restrict__ aux_loss,
                  int* __restrict__ tile_expert, int* __restrict__ tile_row0, int4* __restrict__ ntile,
                  int* __restrict__ count_g, int* __restrict__ group_base) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int part_pre[kFusedTokens], part_tot[kFusedTokens];    // [slice][column]; the extra block keeps floats here
  __shared__ int base_s[kMaxExperts], kept_s[kMaxExperts];
  __shared__ float term[kMaxExperts];
  constexpr int kWarps = kFusedTokens / 32;
  __shared__ int warp_cnt[kMaxExperts][kWarps];                // [expert][warp of the block]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_token_blocks = (int)gridDim.x - 1;
  const bool summary = (int)blockIdx.x == n_token_blocks;
  const int Q = kFusedTokens / Ew, q = tid / Ew, e = tid % Ew;
  const int row_end = summary ? hist_rows : min(hist_rows, (int)blockIdx.x * (kFusedTokens / kPlanBlockTokens));
  int pre = 0, tot = 0;
  if (e < E) {
    for (int r0 = q; r0 < hist_rows; r0 += 8 * Q) {
      int v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = r0 + j * Q < hist_rows ? hist[(size_t)(r0 + j * Q) * E + e] : 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { tot += v[j]; if (r0 + j * Q < row_end) pre += v[j]; }
    }
  }
  part_pre[tid] = pre;
  part_tot[tid] = tot;
  for (int i = tid; i < kWarps * kMaxExperts; i += kFusedTokens) (&warp_cnt[0][0])[i] = 0;
  __syncthreads();
  int total = 0;
  if (tid < E) {
    int b = 0;
    for (int k = 0; k < Q; ++k) { b += part_pre[k * Ew + tid]; total += part_tot[k * Ew + tid]; }
    base_s[tid] = b;
    kept_s[tid] = min(total, C);
  }
  __syncthreads();
  if (summary) {
    // P-sums in a fixed order (slice by slice, rows ascending inside a slice), then the loss and the tile lists
    float* part_ps = reinterpret_cast<float*>(part_pre);
    float ps = 0.f;
    if (e < E) {
      for (int r0 = q; r0 < router_blocks; r0 += 16 * Q) {      // 16 rows in flight, added in row order
        float v[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = r0 + j * Q < router_blocks ? psum_partial[(size_t)(r0 + j * Q) * E + e] : 0.f;
#pragma unroll
        for (int j = 0; j < 16; ++j) ps += v[j];
      }
    }
    __syncthreads();
    part_ps[tid] = ps;
    __syncthreads();
    if (tid < E) {
      float sum = 0.f;
      for (int k = 0; k < Q; ++k) sum += part_ps[k * Ew + tid];
      count[tid] = total;                                                              // f counts the argmax (Eq. 5)
      count_g[tid] = total;
      group_base[tid] = 0;
      kept[tid] = kept_s[tid];
      psum[tid] = sum;
      term[tid] = ((float)total / (float)T) * (sum / (float)T);                        // f_i . P_i  (Eq. 5, 6)
    }
    write_tile_lists(term, kept_s, E, alpha * (float)E, aux_loss, tile_expert, tile_row0, ntile);
    return;
  }
  const int t = (int)blockIdx.x * kFusedTokens + tid;
  int et = t < T ? expert_index[t] : -1;                      // negative: no expert (takes no slot)
  if (et >= E) et = -1;
  const unsigned same = __match_any_sync(0xffffffffu, et >= 0 ? et : -1 - lane);   // distinct dummies for those lanes
  const int rank = __popc(same & ((1u << lane) - 1u));
  if (et >= 0 && rank == 0) warp_cnt[et][warp] = __popc(same);
  __syncthreads();
  for (int ex = warp; ex < E; ex += kWarps) {                  // exclusive scan over the block's warps, per expert
    const int c = warp_cnt[ex][lane];
    int incl = c;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += up;
    }
    warp_cnt[ex][lane] = incl - c;
  }
  __syncthreads();
  if (t < T) {
    int sl = -1;
    if (et >= 0) {
      const int pos = base_s[et] + warp_cnt[et][warp] + rank;
      if (pos < C) { sl = et * C + pos; token_of_slot[sl] = t; }
    }
    slot[t] = sl;
  }
  // empty slots of every expert: -1 (disjoint from the kept slots written above)
  const int total_slots = E * C;
  for (int sidx = (int)blockIdx.x * kFusedTokens + tid; sidx < total_slots; sidx += n_token_blocks * kFusedTokens) {
    const int ex = sidx / C, pos = sidx - ex * C;
    if (pos >= kept_s[ex]) token_of_slot[sidx] = -1;
  }
}

// ---- further stages of No-Token-Left-Behind routing (Appendix B) ---------------------------------------------
// alt[t] = the expert that follows prev[t] in the token's ranking of the experts (probability, highest first; equal
// probabilities by index, lowest first) for a token that has no slot yet; -1 for a token that has one, and when no
// expert is left.  With prev = the argmax this is the second choice (stage 2), with prev = the previous stage's
// choices the third, and so on.  One warp per token.
__global__ void __launch_bounds__(256)
reroute_choice_kernel(const float* __restrict__ probs, const int* __restrict__ prev, const int* __restrict__ slot,
                      int T, int E, int* __restrict__ alt) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (t >= T) return;
  const int e1 = prev[t];
  if (slot[t] >= 0 || e1 < 0 || e1 >= E) {
    if (lane == 0) alt[t] = -1;
    return;
  }
  const float v1 = probs[(size_t)t * E + e1];
  float best = -1.f;
  int arg = 0x7fffffff;
  for (int e = lane; e < E; e += 32) {
    const float v = probs[(size_t)t * E + e];
    const bool later = v < v1 || (v == v1 && e > e1);         // ranked after prev[t]
    if (later && v > best) { best = v; arg = e; }             // ascending e: the first maximum wins
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float ob = __shfl_xor_sync(0xffffffffu, best, off);
    const int oa = __shfl_xor_sync(0xffffffffu, arg, off);
    if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
  }
  if (lane == 0) alt[t] = arg < E ? arg : -1;                  // nothing ranked after prev[t]
}

// Position bases of a further stage: the rerouted tokens of expert e queue up behind the kept[e] tokens it has so far.
// One thread per expert; also rewrites kept[] and the tile lists for the grown experts.
__global__ void __launch_bounds__(kMaxExperts)
reroute_scan_kernel(const int* __restrict__ hist, int plan_blocks, int E, int C, int* __restrict__ hist_base,
                    int* __restrict__ kept, int* __restrict__ tile_expert, int* __restrict__ tile_row0,
                    int4* __restrict__ ntile) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ float term[kMaxExperts];
  __shared__ int kept_s[kMaxExperts];
  const int e = threadIdx.x;
  if (e < E) {
    int run = kept[e];
    for (int b0 = 0; b0 < plan_blocks; b0 += 8) {
      int v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = b0 + j < plan_blocks ? hist[(size_t)(b0 + j) * E + e] : 0;
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (b0 + j < plan_blocks) { hist_base[(size_t)(b0 + j) * E + e] = run; run += v[j]; }
    }
    const int k = min(run, C);
    kept[e] = k;
    kept_s[e] = k;
    term[e] = 0.f;
  }
  write_tile_lists(term, kept_s, E, 0.f, nullptr, tile_expert, tile_row0, ntile);
}

// Slots of the rerouted tokens (same stable in-block rank as the first stage), their gate (the probability of the
// expert that now processes them, Eq. 2) and, for every token, the expert that processes it.
__global__ void __launch_bounds__(kPlanBlockTokens)
reroute_assign_kernel(const int* __restrict__ alt, const int* __restrict__ expert_index,
                      const int* __restrict__ hist_base, const float* __restrict__ probs, int T, int E, int C,
                      int* __restrict__ slot, int* __restrict__ token_of_slot, float* __restrict__ gate,
                      int* __restrict__ expert_proc, int first_stage) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int warp_cnt[kPlanBlockTokens / 32][kMaxExperts];
  constexpr int kWarps = kPlanBlockTokens / 32;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int i = tid; i < kWarps * kMaxExperts; i += blockDim.x) (&warp_cnt[0][0])[i] = 0;
  __syncthreads();
  const int t = blockIdx.x * kPlanBlockTokens + tid;
  int a = t < T ? alt[t] : -1;
  if (a >= E) a = -1;
  const int key = a >= 0 ? a : -1 - lane;                     // distinct dummies for tokens that do not move
  const unsigned same = __match_any_sync(0xffffffffu, key);
  const int rank = __popc(same & ((1u << lane) - 1u));
  if (a >= 0 && rank == 0) warp_cnt[warp][a] = __popc(same);
  __syncthreads();
  if (t < T) {
    bool moved = false;
    if (a >= 0) {
      int pos = hist_base[(size_t)blockIdx.x * E + a] + rank;
      for (int w = 0; w < warp; ++w) pos += warp_cnt[w][a];
      if (pos < C) {
        const int s = a * C + pos;
        slot[t] = s;
        token_of_slot[s] = t;
        gate[t] = probs[(size_t)t * E + a];
        moved = true;
      }
    }
    // the expert that processes the token: its first choice until a stage moves it
    if (moved) expert_proc[t] = a;
    else if (first_stage) expert_proc[t] = expert_index[t];
  }
}

// ---- top-2 routing ------------------------------------------------------------------------------------------
// Second choice of every token: the expert with the second-highest probability (lowest index on ties) and its
// probability, stored as assignment T + t.  One warp per token.
__global__ void __launch_bounds__(256)
top2_choice_kernel(const float* __restrict__ probs, int T, int E, int* __restrict__ expert_index,
                   float* __restrict__ gate) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (t >= T) return;
  const int e1 = expert_index[t];
  float best = -1.f;
  int arg = 0x7fffffff;
  for (int e = lane; e < E; e += 32) {
    const float v = probs[(size_t)t * E + e];
    if (e != e1 && v > best) { best = v; arg = e; }          // ascending e: the first maximum wins
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float ob = __shfl_xor_sync(0xffffffffu, best, off);
    const int oa = __shfl_xor_sync(0xffffffffu, arg, off);
    if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
  }
  if (lane == 0) {
    expert_index[T + t] = arg < E ? arg : -1;                 // E == 1: no second choice (a negative index takes no slot)
    gate[T + t] = arg < E ? best : 0.f;
  }
}

// out[t] = rows[t] + rows[T + t] (+ skip[t]), a dropped assignment (slot < 0) counting as zero: y from the weighted
// expert outputs of the two choices, dx from their input gradients; `skip` is the layer's input (or dy) when the
// layer carries its own residual connection.  One warp per token, float32 sum, one rounding.
template <bool kBf16>
__global__ void __launch_bounds__(256)
top2_sum_kernel(const uint4* __restrict__ rows, const uint4* __restrict__ skip, const int* __restrict__ slot, int T,
                int row_vec, uint4* __restrict__ out) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (t >= T) return;
  const bool k1 = slot[t] >= 0, k2 = slot[T + t] >= 0;
  const uint4* r1 = rows + (size_t)t * row_vec;
  const uint4* r2 = rows + (size_t)(T + t) * row_vec;
  const uint4* r3 = skip != nullptr ? skip + (size_t)t * row_vec : nullptr;
  uint4* dst = out + (size_t)t * row_vec;
  const uint4 zero = make_uint4(0, 0, 0, 0);
  for (int v = lane; v < row_vec; v += 32) {
    const uint4 a = k1 ? r1[v] : zero, b = k2 ? r2[v] : zero, c = r3 != nullptr ? r3[v] : zero;
    uint4 o;
    if (kBf16) {
      const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
      const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
      const __nv_bfloat162* pc = reinterpret_cast<const __nv_bfloat162*>(&c);
      __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 fa = __bfloat1622float2(pa[i]), fb = __bfloat1622float2(pb[i]), fc = __bfloat1622float2(pc[i]);
        po[i] = __floats2bfloat162_rn((fa.x + fb.x) + fc.x, (fa.y + fb.y) + fc.y);
      }
    } else {
      const float* fa = reinterpret_cast<const float*>(&a);
      const float* fb = reinterpret_cast<const float*>(&b);
      const float* fc = reinterpret_cast<const float*>(&c);
      float* fo = reinterpret_cast<float*>(&o);
#pragma unroll
      for (int i = 0; i < 4; ++i) fo[i] = (fa[i] + fb[i]) + fc[i];
    }
    dst[v] = o;
  }
}

// Forward gather.  Part 1 (blockIdx.x < slot_blocks): one warp per slot row; kept slots copy the token's row
// with 128-bit loads and stores, slots in [kept_i, roundup(kept_i, kTileM)) are zero-filled so that tensor-core
// tiles never read stale rows.  Part 2: one warp per token; dropped tokens get a zero output row (their
// representation reaches the next layer only through the residual connection, Section 2.2), or, when the layer
// itself adds the skip path (`residual`), their input row.
__global__ void __launch_bounds__(256)
gather_x_kernel(const uint4* __restrict__ x, const int* __restrict__ token_of_slot, const int* __restrict__ kept,
                const int* __restrict__ slot, int T, int E, int C, int row_vec, int slot_blocks, int residual,
                uint4* __restrict__ xd, uint4* __restrict__ y) {
  // top-2 routing: slot s may hold assignment T + t (the second choice of token t): its source row is still x[t]
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  if ((int)blockIdx.x < slot_blocks) {
    const int s = blockIdx.x * 8 + wib;
    if (s >= E * C) return;
    const int ex = s / C, pos = s - ex * C, k = kept[ex];
    uint4* dst = xd + (size_t)s * row_vec;
    if (pos < k) {
      int tok = token_of_slot[s];
      if (tok >= T) tok -= T;
      const uint4* src = x + (size_t)tok * row_vec;
      for (int v = lane; v < row_vec; v += 32) dst[v] = src[v];
    } else if (pos < (k + kTileM - 1) / kTileM * kTileM) {
      for (int v = lane; v < row_vec; v += 32) dst[v] = make_uint4(0, 0, 0, 0);
    }
  } else {
    const int t = (blockIdx.x - slot_blocks) * 8 + wib;
    if (t >= T || slot[t] >= 0) return;
    uint4* dst = y + (size_t)t * row_vec;
    const uint4* src = x + (size_t)t * row_vec;
    for (int v = lane; v < row_vec; v += 32) dst[v] = residual ? src[v] : make_uint4(0, 0, 0, 0);
  }
}

__device__ __forceinline__ float dot_scale8(const uint4& a, const uint4& b, float g, uint4* out) {
  const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
  const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
  __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(out);
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 fa = __bfloat1622float2(pa[i]), fb = __bfloat1622float2(pb[i]);
    s = fmaf(fa.x, fb.x, s);
    s = fmaf(fa.y, fb.y, s);
    po[i] = __floats2bfloat162_rn(g * fa.x, g * fa.y);
  }
  return s;
}
__device__ __forceinline__ float dot_scale4(const uint4& a, const uint4& b, float g, uint4* out) {
  const float* fa = reinterpret_cast<const float*>(&a);
  const float* fb = reinterpret_cast<const float*>(&b);
  float* fo = reinterpret_cast<float*>(out);
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) { s = fmaf(fa[i], fb[i], s); fo[i] = g * fa[i]; }
  return s;
}

// Backward gather: dY_d[slot] = g . dy[token] (derivative of Eq. 2 w.r.t. the expert output) and
// dgate[token] = <dy, o> with o = y / g (derivative w.r.t. the gate).  Tail rows are zero-filled as in forward.
// With the skip path inside the layer, blocks past `slot_blocks` (one warp per token) start the dropped tokens'
// dx rows at dy: the router's gradient is added to them later, and no expert ever writes them.
template <bool kBf16>
__global__ void __launch_bounds__(256)
gather_dy_kernel(const uint4* __restrict__ dy, const uint4* __restrict__ y, const float* __restrict__ gate,
                 const int* __restrict__ token_of_slot, const int* __restrict__ kept, const int* __restrict__ slot,
                 int T, int E, int C, int row_vec, int slot_blocks, uint4* __restrict__ dyd,
                 float* __restrict__ dgate, uint4* __restrict__ dx) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  if ((int)blockIdx.x >= slot_blocks) {
    const int t = (blockIdx.x - slot_blocks) * 8 + wib;
    if (t >= T || slot[t] >= 0) return;
    const uint4* src = dy + (size_t)t * row_vec;
    uint4* dst = dx + (size_t)t * row_vec;
    for (int v = lane; v < row_vec; v += 32) dst[v] = src[v];
    return;
  }
  const int s = blockIdx.x * 8 + wib;
  if (s >= E * C) return;
  const int ex = s / C, pos = s - ex * C, k = kept[ex];
  uint4* dst = dyd + (size_t)s * row_vec;
  if (pos < k) {
    const int t = token_of_slot[s];                           // top-2 routing: assignment t or T + t of token t mod T
    const float g = gate[t];
    const uint4* src = dy + (size_t)(t >= T ? t - T : t) * row_vec;
    const uint4* ysrc = y + (size_t)t * row_vec;
    float dot = 0.f;
    for (int v = lane; v < row_vec; v += 32) {
      uint4 o;
      dot += kBf16 ? dot_scale8(src[v], ysrc[v], g, &o) : dot_scale4(src[v], ysrc[v], g, &o);
      dst[v] = o;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
    if (lane == 0) dgate[t] = dot / g;
  } else if (pos < (k + kTileM - 1) / kTileM * kTileM) {
    for (int v = lane; v < row_vec; v += 32) dst[v] = make_uint4(0, 0, 0, 0);
  }
}

}  // namespace

int launch_reroute(const Shape& s, const Plan& p, void* ws, cudaStream_t st);

int launch_dispatch_plan(const Shape& s, const Plan& p, const int32_t* expert_index, float* aux_loss, void* ws,
                         cudaStream_t st) {
  int* ei = ws_ptr<int>(ws, p.expert_index);
  if (expert_index != nullptr && expert_index != ei) {
    if (cudaMemcpyAsync(ei, expert_index, (size_t)s.Tv * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
      return SWITCH_MOE_CUDA_ERROR;
  }
  // the tensor-core router's forward kernel leaves the histograms of its own expert choices in the workspace
  const bool have_hist = expert_index == nullptr && s.router_hist;
  if (have_hist && s.G == 1) {
    int Ewf = 32;
    while (Ewf < s.E) Ewf *= 2;
    const int token_blocks = (s.T + kFusedTokens - 1) / kFusedTokens;
    launch_k(plan_fused_kernel, dim3(token_blocks + 1), dim3(kFusedTokens), 0, st, ei, ws_ptr<int>(ws, p.hist),
             s.plan_blocks, ws_ptr<float>(ws, p.psum_partial), s.router_blocks, s.T, s.E, Ewf, s.Cg, s.alpha,
             ws_ptr<int>(ws, p.slot), ws_ptr<int>(ws, p.token_of_slot), ws_ptr<int>(ws, p.count),
             ws_ptr<int>(ws, p.kept), ws_ptr<float>(ws, p.psum), aux_loss, ws_ptr<int>(ws, p.tile_expert),
             ws_ptr<int>(ws, p.tile_row0), ws_ptr<int4>(ws, p.ntile), ws_ptr<int>(ws, p.count_g),
             ws_ptr<int>(ws, p.group_base));
    return launch_reroute(s, p, ws, st);
  }
  if (!have_hist)
    launch_k(plan_hist_kernel, dim3(s.plan_blocks), dim3(kPlanBlockTokens), 0, st, ei, s.Tv, s.E, ws_ptr<int>(ws, p.hist));
  int Ew = 32;
  while (Ew < s.E) Ew *= 2;
  const int blocks_per_group = s.plan_blocks / s.G;
  int* count_g = ws_ptr<int>(ws, p.count_g);
  int* group_base = ws_ptr<int>(ws, p.group_base);
  if (s.G == 1) {
    launch_k(plan_scan_kernel, dim3(1), dim3(kScanThreads), 0, st, ws_ptr<int>(ws, p.hist), s.plan_blocks,
             s.top2 ? s.plan_blocks / 2 : s.plan_blocks, ws_ptr<float>(ws, p.psum_partial), s.router_blocks, s.T, s.E, Ew,
             s.Cg, s.alpha,
             ws_ptr<int>(ws, p.hist_base), ws_ptr<int>(ws, p.count), ws_ptr<int>(ws, p.kept),
             ws_ptr<float>(ws, p.psum), aux_loss, ws_ptr<int>(ws, p.tile_expert), ws_ptr<int>(ws, p.tile_row0),
             ws_ptr<int4>(ws, p.ntile), count_g, group_base);
  } else {
    if (s.G * Ew > kScanGroupCells || s.router_blocks % s.G != 0) return SWITCH_MOE_UNSUPPORTED_SHAPE;
    launch_k(plan_scan_groups_kernel, dim3(1), dim3(kScanThreads), 0, st, ws_ptr<int>(ws, p.hist), blocks_per_group,
             ws_ptr<float>(ws, p.psum_partial), s.router_blocks / s.G, s.G, s.Tg, s.E, Ew, s.Cg, s.alpha,
             ws_ptr<int>(ws, p.hist_base), ws_ptr<int>(ws, p.count), ws_ptr<int>(ws, p.kept),
             ws_ptr<float>(ws, p.psum), aux_loss, ws_ptr<int>(ws, p.tile_expert), ws_ptr<int>(ws, p.tile_row0),
             ws_ptr<int4>(ws, p.ntile), count_g, group_base);
  }
  launch_k(plan_assign_kernel, dim3(s.plan_blocks), dim3(kPlanBlockTokens), 0, st, ei, ws_ptr<int>(ws, p.hist_base),
           ws_ptr<int>(ws, p.kept), group_base, blocks_per_group, s.Tv, s.E, s.C, s.Cg, ws_ptr<int>(ws, p.slot),
           ws_ptr<int>(ws, p.token_of_slot));
  return launch_reroute(s, p, ws, st);
}

// The further stages of No-Token-Left-Behind routing, after either form of the first-stage plan: per stage the next
// choices of the tokens still without a slot, their block histograms, the position bases behind the rows every
// expert already holds, and the slots.
int launch_reroute(const Shape& s, const Plan& p, void* ws, cudaStream_t st) {
  int* ei = ws_ptr<int>(ws, p.expert_index);
  for (int stage = 0; stage < s.reroute_stages; ++stage) {
    int* alt = ws_ptr<int>(ws, p.alt) + (size_t)stage * s.T;
    const int* prev = stage == 0 ? ei : alt - s.T;
    launch_k(reroute_choice_kernel, dim3((s.T + 7) / 8), dim3(256), 0, st, ws_ptr<float>(ws, p.probs), prev,
             ws_ptr<int>(ws, p.slot), s.T, s.E, alt);
    launch_k(plan_hist_kernel, dim3(s.plan_blocks), dim3(kPlanBlockTokens), 0, st, alt, s.T, s.E,
             ws_ptr<int>(ws, p.hist));
    launch_k(reroute_scan_kernel, dim3(1), dim3(kMaxExperts), 0, st, ws_ptr<int>(ws, p.hist), s.plan_blocks, s.E, s.C,
             ws_ptr<int>(ws, p.hist_base), ws_ptr<int>(ws, p.kept), ws_ptr<int>(ws, p.tile_expert),
             ws_ptr<int>(ws, p.tile_row0), ws_ptr<int4>(ws, p.ntile));
    launch_k(reroute_assign_kernel, dim3(s.plan_blocks), dim3(kPlanBlockTokens), 0, st, alt, ei,
             ws_ptr<int>(ws, p.hist_base), ws_ptr<float>(ws, p.probs), s.T, s.E, s.C, ws_ptr<int>(ws, p.slot),
             ws_ptr<int>(ws, p.token_of_slot), ws_ptr<float>(ws, p.gate), ws_ptr<int>(ws, p.expert_proc),
             stage == 0 ? 1 : 0);
  }
  return launch_status();
}

int launch_gather_x(const Shape& s, const Plan& p, const void* x, void* y, void* ws, cudaStream_t st) {
  const int row_vec = (int)((size_t)s.d * s.elt / 16);
  // top-2 routing: the output rows of dropped assignments are skipped by the kernel that sums the two choices
  const int slot_blocks = (s.E * s.C + 7) / 8, tok_blocks = s.top2 ? 0 : (s.T + 7) / 8;
  launch_k(gather_x_kernel, dim3(slot_blocks + tok_blocks), dim3(256), 0, st, 
      static_cast<const uint4*>(x), ws_ptr<int>(ws, p.token_of_slot), ws_ptr<int>(ws, p.kept),
      ws_ptr<int>(ws, p.slot), s.T, s.E, s.C, row_vec, slot_blocks, s.residual, ws_ptr<uint4>(ws, p.xd),
      static_cast<uint4*>(y));
  return launch_status();
}

int launch_gather_dy(const Shape& s, const Plan& p, const void* dy, const void* y, void* dx, void* ws, cudaStream_t st) {
  const int row_vec = (int)((size_t)s.d * s.elt / 16);
  const int slot_blocks = (s.E * s.C + 7) / 8;
  // (top-2 routing: dx rows are formed by the kernel that sums the two assignments, and `y` is the per-assignment
  // output buffer already)
  const int blocks = slot_blocks + ((s.residual && !s.top2) ? (s.T + 7) / 8 : 0);
  // with the skip path inside the layer, y holds x + g . E(x): the gate's gradient needs the copy without x
  const void* ysrc = (s.residual && !s.top2) ? ws_ptr<char>(ws, p.layer_y) : y;
  if (s.dtype == SWITCH_MOE_BF16)
    launch_k(gather_dy_kernel<true>, dim3(blocks), dim3(256), 0, st, static_cast<const uint4*>(dy),
             static_cast<const uint4*>(ysrc), ws_ptr<float>(ws, p.gate), ws_ptr<int>(ws, p.token_of_slot),
             ws_ptr<int>(ws, p.kept), ws_ptr<int>(ws, p.slot), s.T, s.E, s.C, row_vec, slot_blocks,
             ws_ptr<uint4>(ws, p.dyd), ws_ptr<float>(ws, p.dgate), static_cast<uint4*>(dx));
  else
    launch_k(gather_dy_kernel<false>, dim3(blocks), dim3(256), 0, st, static_cast<const uint4*>(dy),
             static_cast<const uint4*>(ysrc), ws_ptr<float>(ws, p.gate), ws_ptr<int>(ws, p.token_of_slot),
             ws_ptr<int>(ws, p.kept), ws_ptr<int>(ws, p.slot), s.T, s.E, s.C, row_vec, slot_blocks,
             ws_ptr<uint4>(ws, p.dyd), ws_ptr<float>(ws, p.dgate), static_cast<uint4*>(dx));
  return launch_status();
}

int launch_top2_choice(const Shape& s, const Plan& p, void* ws, cudaStream_t st) {
  launch_k(top2_choice_kernel, dim3((s.T + 7) / 8), dim3(256), 0, st, ws_ptr<float>(ws, p.probs), s.T, s.E,
           ws_ptr<int>(ws, p.expert_index), ws_ptr<float>(ws, p.gate));
  return launch_status();
}

int launch_top2_sum(const Shape& s, const Plan& p, const void* per_assignment, const void* skip, void* out, void* ws,
                    cudaStream_t st) {
  const int row_vec = (int)((size_t)s.d * s.elt / 16);
  if (s.dtype == SWITCH_MOE_BF16)
    launch_k(top2_sum_kernel<true>, dim3((s.T + 7) / 8), dim3(256), 0, st, static_cast<const uint4*>(per_assignment),
             static_cast<const uint4*>(skip), ws_ptr<int>(ws, p.slot), s.T, row_vec, static_cast<uint4*>(out));
  else
    launch_k(top2_sum_kernel<false>, dim3((s.T + 7) / 8), dim3(256), 0, st, static_cast<const uint4*>(per_assignment),
             static_cast<const uint4*>(skip), ws_ptr<int>(ws, p.slot), s.T, row_vec, static_cast<uint4*>(out));
  return launch_status();
}

}  // namespace swmoe
