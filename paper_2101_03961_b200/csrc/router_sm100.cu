// Router of the Switch FFN layer on the B200 tensor cores with float32-grade accuracy (Section 2.4: the router is the
// part of the layer that must not run in bfloat16).
//
// x is bfloat16, hence exact in float32.  A float32 operand w is written as the sum of two bfloat16 numbers
// (w = hi + mid up to 2^-18 relative: each part carries 8 significant bits and a third part would add what the 1e-5
// tolerance of the router never sees), every bf16 x bf16 product is exact in float32, and tcgen05 accumulates in
// float32.  So
//   logits   h = x W_r            = x (W_hi + W_mid)                              (Section 2.1; Eq. 1 follows in the epilogue)
//   dW_r       = x^T dh           = x^T (dh_hi + dh_mid)                          (contraction over tokens, split over CTAs)
//   dx_router  = dh W_r^T         ~ dh_hi W_hi^T + dh_hi W_mid^T + dh_mid W_hi^T  (the output is bfloat16: 2^-16 suffices)
// are bfloat16 tensor-core products whose results agree with the float32 definition to a few 1e-6 relative, and the
// router stops being bound by the FP32 FMA pipes (E flop per byte of x) and becomes a streaming kernel.
//
// The forward epilogue keeps one token per thread (a TMEM lane holds all E logits of a token): softmax, top-1 with
// lowest-index ties and the gate need no cross-thread traffic; the column sums of p for Eq. 6 use warp shuffles.
#include "tc_common.cuh"

namespace swmoe {
using namespace tc;
namespace {

constexpr int kRTcThreads = 320;                     // generic kernel: TMA warp, MMA warp, 8 epilogue warps
constexpr int kRTcOutStageBytes = 8 * 32 * 128;
constexpr int kRTcSmemBytes = 1024 + kStages * kStageBytes + kRTcOutStageBytes + 128;

// kRDxRes: dx with the two parts of one 256-row block of W_r resident in shared memory for the CTA's whole life
// (up to 128 experts): only the logit gradients stream, and every staged block of them meets the W_r parts it pairs
// with in the three cross terms without a reload.
enum RouterOp { kRFwd = 0, kRDwr = 1, kRDx = 2, kRDxRes = 3 };

struct RouterTcParams {
  int T, d, E, Epad64;
  int mma_n;                 // MMA N: Epad64 (fwd, dwr) or 256 (dx)
  int n_mtiles, n_ntiles;
  int splits, chunk_kblocks, total_kblocks;   // dwr: split of the token contraction
  int wrap;                  // k-blocks per part: d/64 (fwd), Epad64/64 (dx); dwr derives it per tile
  int both_parts;            // dwr: 1 = a stage holds the x block and both parts of dh (2 x mma_n columns <= 256)
  const float* bias; const float* noise; float* probs; int* expert_index; float* gate;   // fwd
  float* partial;                                                                         // dwr
  __nv_bfloat16* dx; const int* slot; int accumulate; const __nv_bfloat16* jitter_u;      // dx
  int* status;
};

struct RTile {
  int m0, n0, split, k_base, wrap, k_blocks;
};

template <int OP>
__device__ __forceinline__ int r_total_tiles(const RouterTcParams& p) {
  if (OP == kRFwd) return p.n_mtiles;
  if (OP == kRDwr) return p.n_mtiles * p.splits;
  if (OP == kRDxRes) return p.n_mtiles;
  return p.n_mtiles * p.n_ntiles;
}

template <int OP>
__device__ __forceinline__ RTile r_decode(const RouterTcParams& p, int id) {
  RTile t;
  t.split = 0; t.k_base = 0; t.n0 = 0;
  if (OP == kRFwd) {
    t.m0 = id * kTileM; t.wrap = p.wrap;
  } else if (OP == kRDwr) {
    const int mt = id / p.splits;
    t.split = id - mt * p.splits;
    t.m0 = mt * kTileM;
    t.k_base = t.split * p.chunk_kblocks;
    t.wrap = max(0, min(p.chunk_kblocks, p.total_kblocks - t.k_base));
  } else if (OP == kRDxRes) {                         // id = token tile; the CTA's block of W_r rows is fixed
    t.m0 = id * kTileM;
    t.n0 = (int)(blockIdx.x % (unsigned)p.n_ntiles) * kBN;
    t.wrap = p.wrap;
  } else {
    const int mt = id / p.n_ntiles;
    t.m0 = mt * kTileM;
    t.n0 = (id - mt * p.n_ntiles) * kBN;
    t.wrap = p.wrap;
  }
  // forward: W_r = hi + mid, one part after the other; dW_r: dh = hi + mid, both parts staged with the x block they
  // multiply when they fit (up to 128 experts), else one after the other; dx: three cross terms
  t.k_blocks = (OP == kRDx ? 3 : (OP == kRDwr && p.both_parts) ? 1 : 2) * t.wrap;   // kRDxRes: hi and mid of dh
  return t;
}

template <int OP>
__global__ void __launch_bounds__(kRTcThreads, 1)
router_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const RouterTcParams p) {
  constexpr bool kAMn = (OP == kRDwr);                 // x^T: token rows are the contraction, d contiguous
  constexpr bool kDx = (OP == kRDx || OP == kRDxRes);
  constexpr bool kBMn = !kDx;                          // fwd: W [d][E]; dwr: dh [T][E]; dx: W as [d rows][E contiguous]
  pdl_launch_dependents();
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kStages * kStageBytes + kRTcOutStageBytes;
  uint8_t* bar_gen = smem_gen + kStages * kStageBytes + kRTcOutStageBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };
  volatile uint32_t* tmem_ptr_s = reinterpret_cast<volatile uint32_t*>(bar_gen + 8 * (2 * kStages + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_gen + 8 * (2 * kStages + 4) + 4);
  const uint32_t wfull_bar = bar_base + 8u * (2 * kStages + 5);     // kRDxRes: the resident W_r parts have landed
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // kRDxRes: the operand ring's first 64 KB are four 16 KB stages of logit-gradient blocks, the rest holds the
  // resident W_r parts: [part][k-block] blocks of 256 rows x 64 experts (32 KB each)
  const uint32_t w_res = smem_base + kStages * kABytes;
  // tiles of this CTA: kRDxRes deals token tiles out among the CTAs that share a block of W_r rows
  const int tile_first = OP == kRDxRes ? (int)(blockIdx.x / (unsigned)p.n_ntiles) : (int)blockIdx.x;
  const int tile_step = OP == kRDxRes ? (int)(gridDim.x / (unsigned)p.n_ntiles) : (int)gridDim.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 8); }
    mbar_init(wfull_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(const_cast<uint32_t*>(tmem_ptr_s))), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_s;
  pdl_wait();                                                 // the previous kernel's results are needed from here on
  const int n_tiles = r_total_tiles<OP>(p);
  const int b_atoms = (p.mma_n + 63) / 64;
  const bool both = OP == kRDwr && p.both_parts;
  const uint32_t stage_tx = kABytes + (kBMn ? (uint32_t)(both ? 2 : 1) * b_atoms * kAtomBytes : (uint32_t)kBBytes);

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      if (OP == kRDxRes) {                                    // W_r parts hi, mid of this CTA's 256 rows, once
        const int n0 = (int)(blockIdx.x % (unsigned)p.n_ntiles) * kBN;
        mbar_arrive_expect_tx(wfull_bar, 2u * (uint32_t)p.wrap * kBBytes);
        for (int part = 0; part < 2; ++part)
          for (int kk = 0; kk < p.wrap; ++kk)
            tma_load_3d(w_res + (uint32_t)(part * p.wrap + kk) * kBBytes, &tmB, wfull_bar, kk * kBK, n0, part);
      }
      for (int id = tile_first; id < n_tiles && ok; id += tile_step) {
        const RTile t = r_decode<OP>(p, id);
        for (int kb = 0; kb < t.k_blocks; ++kb) {
          const int part = kb / t.wrap, kblk = t.k_base + (kb - part * t.wrap);
          ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 11);
          if (!ok) break;
          if (OP == kRDxRes) {                                // dh part [128 tok][64 e] only
            mbar_arrive_expect_tx(full_bar(stage), kABytes);
            tma_load_3d(smem_base + stage * kABytes, &tmA, full_bar(stage), kblk * kBK, t.m0, part);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
            continue;
          }
          const uint32_t a_dst = smem_base + stage * kStageBytes, b_dst = a_dst + kABytes;
          mbar_arrive_expect_tx(full_bar(stage), stage_tx);
          if (OP == kRFwd) {
            tma_load_3d(a_dst, &tmA, full_bar(stage), kblk * kBK, t.m0, 0);                 // x tile [128 tok][64 k]
            for (int j = 0; j < b_atoms; ++j)                                                // W part [64 k][64 e]
              tma_load_3d(b_dst + j * kAtomBytes, &tmB, full_bar(stage), 64 * j, kblk * kBK, part);
          } else if (OP == kRDwr) {
            tma_load_3d(a_dst, &tmA, full_bar(stage), t.m0, kblk * kBK, 0);                 // x^T: [64 tok][64 k-of-d]
            tma_load_3d(a_dst + kAtomBytes, &tmA, full_bar(stage), t.m0 + 64, kblk * kBK, 0);
            for (int j = 0; j < b_atoms; ++j)                                                // dh part [64 tok][64 e]
              tma_load_3d(b_dst + j * kAtomBytes, &tmB, full_bar(stage), 64 * j, kblk * kBK, part);
            if (both)                                                                        // the other part, behind it
              for (int j = 0; j < b_atoms; ++j)
                tma_load_3d(b_dst + (b_atoms + j) * kAtomBytes, &tmB, full_bar(stage), 64 * j, kblk * kBK, 1);
          } else {
            const int a_part = part == 2 ? 1 : 0, b_part = part == 1 ? 1 : 0;               // (hi,hi) (hi,mid) (mid,hi)
            tma_load_3d(a_dst, &tmA, full_bar(stage), kblk * kBK, t.m0, a_part);            // dh part [128 tok][64 e]
            tma_load_3d(b_dst, &tmB, full_bar(stage), kblk * kBK, t.n0, b_part);            // W part [256 k-of-d][64 e]
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (*abort_flag != 0) {
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 2000000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)kAMn << 15) | ((uint32_t)kBMn << 16) |
                             ((uint32_t)(p.mma_n >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
      const uint32_t a_lbo = kAMn ? kAtomBytes : 16u, b_lbo = kBMn ? kAtomBytes : 16u;
      const uint32_t a_kstep = kAMn ? kUmmaK * 128u : kUmmaK * 2u;
      const uint32_t b_kstep = kBMn ? kUmmaK * 128u : kUmmaK * 2u;
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      if (OP == kRDxRes) ok = mbar_wait(wfull_bar, 0u, abort_flag, p.status, 15);
      for (int id = tile_first; id < n_tiles && ok; id += tile_step) {
        const RTile t = r_decode<OP>(p, id);
        ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status, 12);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * kBN;
        for (int kb = 0; kb < t.k_blocks; ++kb) {
          ok = mbar_wait(full_bar(stage), phase, abort_flag, p.status, 13);
          if (!ok) break;
          tc_fence_after();
          if (OP == kRDxRes) {
            // staged block: part `dpart` of dh, experts 64 kk .. 64 kk + 63.  dh_hi meets W_hi and W_mid, dh_mid meets W_hi.
            const int dpart = kb / t.wrap, kk = kb - dpart * t.wrap;
            const uint32_t a_src = smem_base + stage * kABytes;
            const int n_w = dpart == 0 ? 2 : 1;
            for (int wp = 0; wp < n_w; ++wp) {
              const uint32_t b_src = w_res + (uint32_t)(wp * t.wrap + kk) * kBBytes;
#pragma unroll
              for (int ks = 0; ks < kBK / kUmmaK; ++ks) {
                const uint64_t ad = make_smem_desc(a_src + ks * a_kstep, a_lbo, 1024u);
                const uint64_t bd = make_smem_desc(b_src + ks * b_kstep, b_lbo, 1024u);
                tc_mma_bf16(d_tmem, ad, bd, idesc, (kb > 0 || wp > 0 || ks > 0) ? 1u : 0u);
              }
            }
            tc_commit(empty_bar(stage));
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
            continue;
          }
          const uint32_t a_src = smem_base + stage * kStageBytes, b_src = a_src + kABytes;
#pragma unroll
          for (int ks = 0; ks < kBK / kUmmaK; ++ks) {
            const uint64_t ad = make_smem_desc(a_src + ks * a_kstep, a_lbo, 1024u);
            const uint64_t bd = make_smem_desc(b_src + ks * b_kstep, b_lbo, 1024u);
            tc_mma_bf16(d_tmem, ad, bd, idesc, (kb > 0 || ks > 0) ? 1u : 0u);
          }
          if (both) {
#pragma unroll
            for (int ks = 0; ks < kBK / kUmmaK; ++ks) {
              const uint64_t ad = make_smem_desc(a_src + ks * a_kstep, a_lbo, 1024u);
              const uint64_t bd = make_smem_desc(b_src + (uint32_t)b_atoms * kAtomBytes + ks * b_kstep, b_lbo, 1024u);
              tc_mma_bf16(d_tmem, ad, bd, idesc, 1u);
            }
          }
          tc_commit(empty_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (t.k_blocks > 0) tc_commit(tfull_bar(acc));
        else mbar_arrive(tfull_bar(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    const int lg = warp & 3;
    const int half = (warp - 2) >> 2;                         // second warp of the lane group: other half of the columns
    uint8_t* my_stage_gen = smem_gen + kStages * kStageBytes + (warp - 2) * 4096;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int id = tile_first; id < n_tiles && ok; id += tile_step) {
      const RTile t = r_decode<OP>(p, id);
      const int r = lg * 32 + lane;
      // dx: previous contents of the rows this thread will write (prefetched before the accumulator is ready)
      long long offs[8];
      unsigned add_mask = 0;
      if (kDx) {
        const int tok = t.m0 + r;
        const long long row_off = tok < p.T ? (long long)tok * p.d : -1;
        const int add = (p.accumulate && tok < p.T && (p.accumulate == 2 || p.slot[tok] >= 0)) ? 1 : 0;
#pragma unroll
        for (int it = 0; it < 8; ++it) {
          offs[it] = __shfl_sync(0xffffffffu, row_off, it * 4 + (lane >> 3));
          add_mask |= (unsigned)__shfl_sync(0xffffffffu, add, it * 4 + (lane >> 3)) << it;
        }
      }
      ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status, 14);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_addr = tmem_base + ((uint32_t)(lg * 32) << 16) + (uint32_t)acc * kBN;
      const bool have_acc = t.k_blocks > 0;

      if (OP == kRFwd && half == 1) {                         // one token per thread needs all columns: first warp only
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(acc));
      } else if (OP == kRFwd) {
        // ---- Eq. 1 softmax, top-1 (lowest index on ties) and gate for token m0 + r; all E logits are in this lane
        const int tok = t.m0 + r;
        const int nch = p.mma_n / 32;
        const float* nrow = (p.noise != nullptr && tok < p.T) ? p.noise + (size_t)tok * p.E : nullptr;
        auto addend = [&](int e) { return (p.bias ? p.bias[e] : 0.f) + (nrow ? nrow[e] : 0.f); };
        float m = -INFINITY;
        int am = 0;
        for (int c = 0; c < nch; ++c) {
          uint32_t v[32];
          tc_ld32(t_addr + c * 32, v);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int e = c * 32 + i;
            if (e < p.E) {
              const float h = __uint_as_float(v[i]) + addend(e);
              if (h > m) { m = h; am = e; }
            }
          }
        }
        float sum = 0.f;
        for (int c = 0; c < nch; ++c) {
          uint32_t v[32];
          tc_ld32(t_addr + c * 32, v);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int e = c * 32 + i;
            if (e < p.E) sum += expf(__uint_as_float(v[i]) + addend(e) - m);
          }
        }
        const float inv = 1.f / sum;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          if (c >= nch) break;
          uint32_t v[32];
          tc_ld32(t_addr + c * 32, v);
          tc_wait_ld();
          if (c == nch - 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
          }
          float pr[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int e = c * 32 + i;
            pr[i] = (e < p.E && tok < p.T)
                        ? expf(__uint_as_float(v[i]) + addend(e) - m) * inv : 0.f;
          }
          if (tok < p.T) {
            float* dst = p.probs + (size_t)tok * p.E + c * 32;
            if ((p.E & 3) == 0) {
#pragma unroll
              for (int i = 0; i < 32; i += 4)
                if (c * 32 + i < p.E) *reinterpret_cast<float4*>(dst + i) = make_float4(pr[i], pr[i + 1], pr[i + 2], pr[i + 3]);
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (c * 32 + i < p.E) dst[i] = pr[i];
            }
          }
        }
        if (tok < p.T) { p.expert_index[tok] = am; p.gate[tok] = inv; }
      } else if (OP == kRDwr) {
        // ---- float32 partial of x^T dh for this token split: row = m0 + r (an index into d_model)
        const int row = t.m0 + r;
        const int nch = p.mma_n / 32;
        bool released = false;
        for (int c = half; c < nch; c += 2) {
          uint32_t v[32];
          if (have_acc) {
            tc_ld32(t_addr + c * 32, v);
            tc_wait_ld();
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = 0u;
          }
          if (c + 2 >= nch) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
            released = true;
          }
          if (row < p.d) {
            float* dst = p.partial + ((size_t)t.split * p.d + row) * p.E + c * 32;
            if ((p.E & 3) == 0) {
#pragma unroll
              for (int i = 0; i < 32; i += 4)
                if (c * 32 + i < p.E)
                  *reinterpret_cast<float4*>(dst + i) = make_float4(__uint_as_float(v[i]), __uint_as_float(v[i + 1]),
                                                                    __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (c * 32 + i < p.E) dst[i] = __uint_as_float(v[i]);
            }
          }
        }
        if (!released) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(tempty_bar(acc));
        }
      } else {
        // ---- dx[token] = (accumulate and kept ? dx[token] : 0) + dh W_r^T, 64 columns at a time
#pragma unroll 1
        for (int c = 2 * half; c < 2 * half + 2; ++c) {
          const int col = t.n0 + c * 64 + (lane & 7) * 8;
          uint4 prev[8];
#pragma unroll
          for (int it = 0; it < 8; ++it)
            prev[it] = (((add_mask >> it) & 1u) && col < p.d) ? *reinterpret_cast<const uint4*>(p.dx + offs[it] + col)
                                                             : make_uint4(0, 0, 0, 0);
          uint4 uu[8];                                        // jitter factors of the same elements, fetched early too
          if (p.jitter_u != nullptr) {
#pragma unroll
            for (int it = 0; it < 8; ++it)
              uu[it] = (offs[it] >= 0 && col < p.d) ? *reinterpret_cast<const uint4*>(p.jitter_u + offs[it] + col)
                                                    : make_uint4(0, 0, 0, 0);
          }
          uint32_t v[64];
          tc_ld32(t_addr + c * 64, v);
          tc_ld32(t_addr + c * 64 + 32, v + 32);
          tc_wait_ld();
          if (c == 2 * half + 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
          }
          // stage the float32 values as two bf16-pair planes?  No: keep float32 accuracy of the sum by staging
          // bf16(acc) only when nothing is added; otherwise add in float32 after the transpose (values are bf16
          // on both sides, so staging bf16(acc) costs one extra rounding of the small router term only).
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            uint32_t w[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(v[j * 8 + 2 * q]),
                                                        __uint_as_float(v[j * 8 + 2 * q + 1]));
              w[q] = *reinterpret_cast<uint32_t*>(&h2);
            }
            *reinterpret_cast<uint4*>(my_stage_gen + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                make_uint4(w[0], w[1], w[2], w[3]);
          }
          __syncwarp();
          if (col < p.d) {
#pragma unroll
            for (int it = 0; it < 8; ++it) {
              const int rr = it * 4 + (lane >> 3);
              uint4 val = *reinterpret_cast<const uint4*>(my_stage_gen + rr * 128 + (((lane & 7) ^ (rr & 7)) << 4));
              if (p.jitter_u != nullptr && offs[it] >= 0) {      // d(x . u)/dx = u
                __nv_bfloat162* vp = reinterpret_cast<__nv_bfloat162*>(&val);
                const __nv_bfloat162* up = reinterpret_cast<const __nv_bfloat162*>(&uu[it]);
                if ((add_mask >> it) & 1u) {                     // one rounding for (router term . u) + dx
                  const __nv_bfloat162* pp = reinterpret_cast<const __nv_bfloat162*>(&prev[it]);
#pragma unroll
                  for (int q = 0; q < 4; ++q) {
                    const float2 a = __bfloat1622float2(vp[q]), b = __bfloat1622float2(pp[q]), c2 = __bfloat1622float2(up[q]);
                    vp[q] = __floats2bfloat162_rn(fmaf(a.x, c2.x, b.x), fmaf(a.y, c2.y, b.y));
                  }
                } else {
#pragma unroll
                  for (int q = 0; q < 4; ++q) {
                    const float2 a = __bfloat1622float2(vp[q]), c2 = __bfloat1622float2(up[q]);
                    vp[q] = __floats2bfloat162_rn(a.x * c2.x, a.y * c2.y);
                  }
                }
              } else if ((add_mask >> it) & 1u) {
                __nv_bfloat162* vp = reinterpret_cast<__nv_bfloat162*>(&val);
                const __nv_bfloat162* pp = reinterpret_cast<const __nv_bfloat162*>(&prev[it]);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  const float2 a = __bfloat1622float2(vp[q]), b = __bfloat1622float2(pp[q]);
                  vp[q] = __floats2bfloat162_rn(a.x + b.x, a.y + b.y);
                }
              }
              if (offs[it] >= 0) *reinterpret_cast<uint4*>(p.dx + offs[it] + col) = val;
            }
          }
          __syncwarp();
        }
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------------------------
// Forward router for E <= 128.  A CTA works on 256 consecutive tokens at a time -- two 128-token tiles that share every
// staged k-block of W_r, so the weight parts cross shared memory once per 256 tokens -- and those 256 tokens are
// exactly one block of the dispatch plan.  The epilogue (one token per thread: a TMEM lane holds all E logits of a
// token) therefore also produces what the plan needs from the router: the block's histogram of expert choices
// (Section 2.2: the counts behind Eq. 3's capacity cut and Eq. 5's f) and the block's column sums of the
// probabilities (Eq. 6's P), both in a fixed order.
struct RouterFwdParams {
  int T, d, E, Epad64, n_ptiles, k_blocks, b_atoms, stages, stage_bytes;
  const float* bias; const float* noise; float* probs; int* expert_index; float* gate;
  float* psum_partial;       // [n_ptiles][E]: column sums of p over each block of 256 tokens
  int* hist;                 // [n_ptiles][E]: tokens of each 256-token block per expert
  int* status;
};
constexpr int kRFParts = 2;                                    // W_r = hi + mid (bfloat16 each): exact to 2^-18 relative
constexpr int kRFThreads = 320;                                // TMA warp, MMA warp, 8 epilogue warps (4 per token tile)
constexpr int kRFRingBytes = kStages * kStageBytes;            // 192 KB of operand stages
constexpr int kRFOutBytes = 8 * 128 * 4;                       // the eight epilogue warps' column sums (E <= 128 floats each)
constexpr int kRFTailBytes = 2048;                             // barriers, TMEM pointer, abort flag, the block's histogram
constexpr int kRFSmemBytes = 1024 + kRFRingBytes + kRFOutBytes + kRFTailBytes;

template <int NCH>                                             // 32-logit chunks per token: 2 (E <= 64) or 4 (E <= 128)
__global__ void __launch_bounds__(kRFThreads, 1)
router_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                     const RouterFwdParams p) {
  pdl_launch_dependents();
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kRFRingBytes + kRFOutBytes;
  uint8_t* bar_gen = smem_gen + kRFRingBytes + kRFOutBytes;
  const uint32_t full0 = bar_base, empty0 = bar_base + 8u * kStages;
  const uint32_t tfull0 = bar_base + 16u * kStages, tempty0 = tfull0 + 16u;
  volatile uint32_t* tmem_ptr_s = reinterpret_cast<volatile uint32_t*>(bar_gen + 8 * (2 * kStages + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_gen + 8 * (2 * kStages + 4) + 4);
  volatile int* fail_s = reinterpret_cast<volatile int*>(bar_gen + 8 * (2 * kStages + 4) + 8);   // an epilogue warp gave up
  int* hist_s = reinterpret_cast<int*>(bar_gen + 1024);        // kMaxExperts counters
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full0 + 8u * s, 1); mbar_init(empty0 + 8u * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull0 + 8u * a, 1); mbar_init(tempty0 + 8u * a, 8); }
    *abort_flag = 0;
    *fail_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(const_cast<uint32_t*>(tmem_ptr_s))), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int i = threadIdx.x; i < kMaxExperts; i += kRFThreads) hist_s[i] = 0;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_s;
  pdl_wait();                                                 // the previous kernel's results are needed from here on
  const int n_tiles = p.n_ptiles, kbs = p.k_blocks, b_atoms = p.b_atoms;
  const uint32_t n_stages = (uint32_t)p.stages, stage_bytes = (uint32_t)p.stage_bytes;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int id = blockIdx.x; id < n_tiles && ok; id += gridDim.x) {
        const int m0 = id * 2 * kTileM;
#pragma unroll 1
        for (int kb = 0; kb < kbs; ++kb) {
          ok = mbar_wait(empty0 + 8u * stage, phase ^ 1u, abort_flag, p.status, 31);
          if (!ok) break;
          const uint32_t a_dst = smem_base + stage * stage_bytes, fb = full0 + 8u * stage;
          mbar_arrive_expect_tx(fb, stage_bytes);
          // CTAs walk the contraction in rotated order (the sum does not care): otherwise all of them would ask
          // the same L2 lines of W_r at the same moment
          int kr = kb + (int)(blockIdx.x % (unsigned)kbs);
          if (kr >= kbs) kr -= kbs;
          tma_load_3d(a_dst, &tmA, fb, kr * kBK, m0, 0);                              // x tiles [128 tok][64 k]
          tma_load_3d(a_dst + kABytes, &tmA, fb, kr * kBK, m0 + kTileM, 0);
          uint32_t b_dst = a_dst + 2 * kABytes;
          for (int part = 0; part < kRFParts; ++part)
            for (int j = 0; j < b_atoms; ++j, b_dst += kAtomBytes)                     // W part [64 k][64 e]
              tma_load_3d(b_dst, &tmB, fb, 64 * j, kr * kBK, part);
          if (++stage == n_stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (*abort_flag != 0) {
        const long long t0 = clock64();
        while (clock64() - t0 < 4000000ll) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(p.Epad64 >> 3) << 17) |
                             ((uint32_t)(kTileM >> 4) << 24);
      const uint64_t a_desc0 = make_smem_desc(smem_base, 16u, 1024u);
      const uint64_t b_desc0 = make_smem_desc(smem_base + 2 * kABytes, kAtomBytes, 1024u);
      const uint32_t part_step = (uint32_t)(b_atoms * kAtomBytes) >> 4;
      uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
      bool ok = true;
      for (int id = blockIdx.x; id < n_tiles && ok; id += gridDim.x) {
        ok = mbar_wait(tempty0 + 8u * acc, acc_phase ^ 1u, abort_flag, p.status, 32);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * (uint32_t)kBN;      // tile 0: 128 columns here, tile 1: the next 128
#pragma unroll 1
        for (int kb = 0; kb < kbs; ++kb) {
          ok = mbar_wait(full0 + 8u * stage, phase, abort_flag, p.status, 33);
          if (!ok) break;
          tc_fence_after();
          const uint64_t ad = a_desc0 + (uint64_t)(stage * (stage_bytes >> 4));
          const uint64_t bd0 = b_desc0 + (uint64_t)(stage * (stage_bytes >> 4));
#pragma unroll
          for (int tile = 0; tile < 2; ++tile) {
            uint64_t bd = bd0;
#pragma unroll
            for (int part = 0; part < kRFParts; ++part, bd += part_step) {
#pragma unroll
              for (int ks = 0; ks < kBK / kUmmaK; ++ks)
                tc_mma_bf16(d_tmem + tile * 128u, ad + (uint64_t)(tile * (kABytes >> 4) + ks * ((kUmmaK * 2) >> 4)),
                            bd + (uint64_t)(ks * ((kUmmaK * 128) >> 4)), idesc, (kb > 0 || part > 0 || ks > 0) ? 1u : 0u);
            }
          }
          tc_commit(empty0 + 8u * stage);
          if (++stage == n_stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(tfull0 + 8u * acc);
        acc ^= 1u;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    const int lg = warp & 3, ti = (warp - 2) >> 2;            // TMEM lane group; which of the two token tiles
    const int et = threadIdx.x - 64;                          // 0..255 over the epilogue warps
    uint32_t acc = 0, acc_phase = 0;
    bool ok = true;
    for (int id = blockIdx.x; id < n_tiles; id += gridDim.x) {
      const int tok0 = id * 2 * kTileM + ti * kTileM + lg * 32;
      const int tok = tok0 + lane;                            // the token whose logits this lane holds
      ok = mbar_wait(tfull0 + 8u * acc, acc_phase, abort_flag, p.status, 34);
      ok = __all_sync(0xffffffffu, ok);
      // the eight warps meet at barriers below: all of them leave together if the bounded wait of any gave up
      if (!ok && lane == 0) *fail_s = 1;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (*fail_s != 0) break;
      tc_fence_after();
      const uint32_t t_addr = tmem_base + ((uint32_t)(lg * 32) << 16) + acc * (uint32_t)kBN + (uint32_t)ti * 128u;
      float h[NCH * 32];
      {
        uint32_t v[NCH * 32];
#pragma unroll
        for (int c = 0; c < NCH; ++c) tc_ld32(t_addr + c * 32, v + c * 32);       // all loads in flight together
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < NCH * 32; ++i) h[i] = __uint_as_float(v[i]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty0 + 8u * acc);         // logits are in registers: the accumulator is free
      // Eq. 1 and top-1 (first maximum wins), all within this lane.  Few warps run here, so every dependent chain is
      // paid in full: the maximum and the sum are kept as four interleaved chains, and the exponential is the
      // hardware exp2 of a pre-scaled argument (relative error below 1e-6 for |h - m| < 10, inside the 1e-5 the
      // router is held to).
      if (p.bias != nullptr) {
#pragma unroll
        for (int e = 0; e < NCH * 32; ++e)
          if (e < p.E) h[e] += p.bias[e];
      }
      if (p.noise != nullptr && tok < p.T) {                  // exploration noise on the logits (an input)
        const float* nrow = p.noise + (size_t)tok * p.E;
#pragma unroll
        for (int e = 0; e < NCH * 32; ++e)
          if (e < p.E) h[e] += nrow[e];
      }
      float mq[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      int aq[4] = {0, 1, 2, 3};
#pragma unroll
      for (int e = 0; e < NCH * 32; e += 4) {
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (e + u < p.E && h[e + u] > mq[u]) { mq[u] = h[e + u]; aq[u] = e + u; }      // ascending: first maximum wins
      }
      float m = mq[0];
      int am = aq[0];
#pragma unroll
      for (int u = 1; u < 4; ++u)
        if (mq[u] > m || (mq[u] == m && aq[u] < am)) { m = mq[u]; am = aq[u]; }
      const float kLog2e = 1.4426950408889634f;
      const float ms = m * kLog2e;
      float sq[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int e = 0; e < NCH * 32; e += 4) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          float ex = 0.f;
          if (e + u < p.E) {
            const float arg = fmaf(h[e + u], kLog2e, -ms);
            asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(ex) : "f"(arg));
          }
          h[e + u] = ex;
          sq[u] += ex;
        }
      }
      const float sum = (sq[0] + sq[1]) + (sq[2] + sq[3]);
      const float inv = 1.f / sum;
      const bool live = tok < p.T;
      if (live) {
        p.expert_index[tok] = am;
        p.gate[tok] = inv;
        atomicAdd(&hist_s[am], 1);                            // integer counts: the order does not matter
      }
      // Probabilities: every thread writes its own token's row, 16 bytes at a time (no transposition: the few warps
      // of this kernel are bound by the number of memory instructions they issue, not by how the bytes coalesce).
      // Column sums over the warp's 32 tokens (Eq. 6's sum over tokens) by a halving exchange: in each of five steps
      // a lane hands half of its values to the lane whose index differs in one bit and adds what it receives, so that
      // lane l ends with column 32 c + l summed over all lanes in a fixed (tree) order.
      float* prow = p.probs + (size_t)(live ? tok : 0) * p.E;
      float colsum[NCH];
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        float w[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) w[i] = h[c * 32 + i] * inv;
        if (live) {
          if ((p.E & 3) == 0) {
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              if (c * 32 + i < p.E) *reinterpret_cast<float4*>(prow + c * 32 + i) = make_float4(w[i], w[i + 1], w[i + 2], w[i + 3]);
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (c * 32 + i < p.E) prow[c * 32 + i] = w[i];
          }
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) w[i] = 0.f;             // rows past the last token add nothing to the sums
        }
#pragma unroll
        for (int half = 16; half >= 1; half >>= 1) {
          const bool upper = (lane & half) != 0;
#pragma unroll
          for (int j = 0; j < half; ++j) {
            const float send = upper ? w[j] : w[j + half];
            const float keep = upper ? w[j + half] : w[j];
            w[j] = keep + __shfl_xor_sync(0xffffffffu, send, half);
          }
        }
        colsum[c] = w[0];
      }
      float* sums = reinterpret_cast<float*>(smem_gen + kRFRingBytes) + (warp - 2) * (NCH * 32);
#pragma unroll
      for (int c = 0; c < NCH; ++c) sums[c * 32 + lane] = colsum[c];
      asm volatile("bar.sync 1, 256;" ::: "memory");          // the eight epilogue warps: histogram and column sums complete
      if (warp == 2) {                                        // the eight warps' sums, added in warp order
        const float* t0 = reinterpret_cast<const float*>(smem_gen + kRFRingBytes);
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
          const int e = c * 32 + lane;
          float v = t0[e];
#pragma unroll
          for (int w = 1; w < 8; ++w) v += t0[w * (NCH * 32) + e];
          if (e < p.E) p.psum_partial[(size_t)id * p.E + e] = v;
        }
      }
      if (et < p.E) {
        p.hist[(size_t)id * p.E + et] = hist_s[et];
        hist_s[et] = 0;
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");          // before the next round reuses the tiles and the counters
      acc ^= 1u;
      if (acc == 0) acc_phase ^= 1u;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// partial[b][e] = sum of p[t][e] over the rows of block b (Eq. 6), in a fixed order: 4 row groups per column, each
// summed sequentially, then added in order.
__global__ void __launch_bounds__(1024)
probs_colsum_kernel(const float* __restrict__ probs, int T, int E, int rows_per_block, float* __restrict__ partial) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ float part[4][kMaxExperts];
  const int e = threadIdx.x % kMaxExperts, g = threadIdx.x / kMaxExperts;
  const int r0 = blockIdx.x * rows_per_block, r1 = min(T, r0 + rows_per_block);
  const int q = (r1 - r0 + 3) / 4, a = r0 + g * q, b = min(r1, a + q);
  if (e < E) {
    float s = 0.f;
    for (int t0 = a; t0 < b; t0 += 8) {
      float v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = t0 + j < b ? probs[(size_t)(t0 + j) * E + e] : 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) s += v[j];
    }
    part[g][e] = s;
  }
  __syncthreads();
  if (g == 0 && e < E) partial[(size_t)blockIdx.x * E + e] = ((part[0][e] + part[1][e]) + part[2][e]) + part[3][e];
}

// wsplit[part][k][e] for e < Epad64 (zero beyond E): W_r = hi + mid + (a remainder below 2^-18 relative that no
// product uses: the forward logits and the backward dx both stop at hi + mid)
__global__ void split_w_kernel(const float* __restrict__ W_r, int d, int E, int Epad64,
                               __nv_bfloat16* __restrict__ wsplit) {
  pdl_launch_dependents();
  pdl_wait();
  const size_t n = (size_t)d * Epad64;
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int k = (int)(i / Epad64), e = (int)(i - (size_t)k * Epad64);
  __nv_bfloat16 h, m, l;
  split3(e < E ? W_r[(size_t)k * E + e] : 0.f, &h, &m, &l);
  wsplit[i] = h; wsplit[n + i] = m;
}

int sm_count_or_default() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
  return n;
}

template <int OP>
int launch_op(const CUtensorMap& tmA, const CUtensorMap& tmB, const RouterTcParams& q, cudaStream_t st, int grid = 0) {
  if (cudaFuncSetAttribute(router_tc_kernel<OP>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRTcSmemBytes) !=
      cudaSuccess)
    return SWITCH_MOE_CUDA_ERROR;
  launch_k(router_tc_kernel<OP>, dim3(grid > 0 ? grid : sm_count_or_default()), dim3(kRTcThreads), kRTcSmemBytes, st,
           tmA, tmB, q);
  return launch_status();
}

}  // namespace

int launch_router_tc_fwd(const Shape& s, const Plan& p, const void* x, const float* W_r, const float* bias,
                         const float* noise, void* ws,
                         cudaStream_t st) {
  __nv_bfloat16* wsplit = ws_ptr<__nv_bfloat16>(ws, p.wsplit);
  const size_t n = (size_t)s.d * s.Epad64;
  launch_k(split_w_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st, W_r, s.d, s.E, s.Epad64, wsplit);
  CUtensorMap tmA, tmB;
  if (make_map(&tmA, x, 1, s.T, s.d, kTileM) != SWITCH_MOE_OK) return SWITCH_MOE_CUDA_ERROR;
  if (make_map(&tmB, wsplit, 3, s.d, s.Epad64, 64) != SWITCH_MOE_OK) return SWITCH_MOE_CUDA_ERROR;
  if (s.Epad64 <= 128) {
    // 256 tokens per CTA and round; the epilogue also leaves the plan's histogram and the P-sum partials
    RouterFwdParams q{};
    q.T = s.T; q.d = s.d; q.E = s.E; q.Epad64 = s.Epad64; q.n_ptiles = (s.T + 2 * kTileM - 1) / (2 * kTileM);
    q.k_blocks = s.d / kBK;
    q.b_atoms = s.Epad64 / 64;
    q.stage_bytes = 2 * kABytes + kRFParts * q.b_atoms * kAtomBytes;
    q.stages = kRFRingBytes / q.stage_bytes < kStages ? kRFRingBytes / q.stage_bytes : kStages;
    q.bias = bias; q.noise = noise; q.probs = ws_ptr<float>(ws, p.probs); q.expert_index = ws_ptr<int>(ws, p.expert_index);
    q.gate = ws_ptr<float>(ws, p.gate); q.status = ws_ptr<int>(ws, p.status);
    q.psum_partial = ws_ptr<float>(ws, p.psum_partial); q.hist = ws_ptr<int>(ws, p.hist);
    const int grid = q.n_ptiles < sm_count_or_default() ? q.n_ptiles : sm_count_or_default();
    if (s.Epad64 == 64) {
      if (cudaFuncSetAttribute(router_fwd_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRFSmemBytes) !=
          cudaSuccess)
        return SWITCH_MOE_CUDA_ERROR;
      launch_k(router_fwd_tc_kernel<2>, dim3(grid), dim3(kRFThreads), kRFSmemBytes, st, tmA, tmB, q);
    } else {
      if (cudaFuncSetAttribute(router_fwd_tc_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRFSmemBytes) !=
          cudaSuccess)
        return SWITCH_MOE_CUDA_ERROR;
      launch_k(router_fwd_tc_kernel<4>, dim3(grid), dim3(kRFThreads), kRFSmemBytes, st, tmA, tmB, q);
    }
    return launch_status();
  }
  const int n_mtiles = (s.T + kTileM - 1) / kTileM;
  RouterTcParams q{};
  q.T = s.T; q.d = s.d; q.E = s.E; q.Epad64 = s.Epad64; q.mma_n = s.Epad64;
  q.n_mtiles = n_mtiles; q.n_ntiles = 1; q.wrap = s.d / kBK;
  q.bias = bias; q.noise = noise; q.probs = ws_ptr<float>(ws, p.probs); q.expert_index = ws_ptr<int>(ws, p.expert_index);
  q.gate = ws_ptr<float>(ws, p.gate); q.status = ws_ptr<int>(ws, p.status);
  const int rc = launch_op<kRFwd>(tmA, tmB, q, st);
  if (rc != SWITCH_MOE_OK) return rc;
  // Eq. 6 partial sums: one row per 256 tokens, reduced in a fixed order by the dispatch plan
  launch_k(probs_colsum_kernel, dim3(s.router_blocks), dim3(1024), 0, st, ws_ptr<float>(ws, p.probs), s.T, s.E, 2 * kTileM,
           ws_ptr<float>(ws, p.psum_partial));
  return launch_status();
}

int launch_router_tc_bwd(const Shape& s, const Plan& p, const void* x, const float* W_r, void* ws, void* dx,
                         bool accumulate_dx, cudaStream_t st) {
  __nv_bfloat16* wsplit = ws_ptr<__nv_bfloat16>(ws, p.wsplit);
  __nv_bfloat16* dhsplit = ws_ptr<__nv_bfloat16>(ws, p.dhsplit);
  if (!accumulate_dx) {
    // staged call: split W_r here.  The whole-layer backward (accumulate_dx) reuses the parts its forward pass left
    // in the workspace: W_r must be unchanged between the two calls anyway.
    const size_t nw = (size_t)s.d * s.Epad64;
    launch_k(split_w_kernel, dim3((unsigned)((nw + 255) / 256)), dim3(256), 0, st, W_r, s.d, s.E, s.Epad64, wsplit);
  }
  RouterTcParams q{};
  q.T = s.T; q.d = s.d; q.E = s.E; q.Epad64 = s.Epad64;
  q.status = ws_ptr<int>(ws, p.status);
  CUtensorMap tmA, tmB;
  // dW_r partials: A = x^T (MN-major view of x [T][d]), B = dh parts [3][T][Epad64] (MN-major)
  if (make_map(&tmA, x, 1, s.T, s.d, 64) != SWITCH_MOE_OK) return SWITCH_MOE_CUDA_ERROR;
  if (make_map(&tmB, dhsplit, 3, s.T, s.Epad64, 64) != SWITCH_MOE_OK) return SWITCH_MOE_CUDA_ERROR;
  q.mma_n = s.Epad64;
  q.both_parts = s.Epad64 <= 128 ? 1 : 0;
  q.n_mtiles = (s.d + kTileM - 1) / kTileM; q.n_ntiles = 1;
  q.splits = s.dwr_chunks;
  q.total_kblocks = (s.T + kBK - 1) / kBK;
  q.chunk_kblocks = (q.total_kblocks + q.splits - 1) / q.splits;
  q.partial = ws_ptr<float>(ws, p.dwr_partial);
  int rc = launch_op<kRDwr>(tmA, tmB, q, st);
  if (rc != SWITCH_MOE_OK) return rc;
  // dx: A = dh parts (K-major), B = W parts [3][d][Epad64] (K-major: rows are d_model indices)
  if (make_map(&tmA, dhsplit, 3, s.T, s.Epad64, kTileM) != SWITCH_MOE_OK) return SWITCH_MOE_CUDA_ERROR;
  if (make_map(&tmB, wsplit, 3, s.d, s.Epad64, kBN) != SWITCH_MOE_OK) return SWITCH_MOE_CUDA_ERROR;
  q.mma_n = kBN;
  q.n_mtiles = (s.T + kTileM - 1) / kTileM; q.n_ntiles = (s.d + kBN - 1) / kBN;
  q.wrap = s.Epad64 / kBK;
  q.dx = static_cast<__nv_bfloat16*>(dx); q.slot = ws_ptr<int>(ws, p.slot); q.accumulate = accumulate_dx ? ((s.residual || s.top2) ? 2 : 1) : 0;   // 2: every row already holds a value
  q.jitter_u = static_cast<const __nv_bfloat16*>(s.jitter_u);
  // up to 128 experts the two parts of a 256-row block of W_r (at most 128 KB) stay in shared memory: the CTAs are
  // dealt out evenly over the row blocks and each walks its share of the token tiles
  const int sms = sm_count_or_default();
  if (s.Epad64 <= 128 && sms >= q.n_ntiles) return launch_op<kRDxRes>(tmA, tmB, q, st, sms / q.n_ntiles * q.n_ntiles);
  return launch_op<kRDx>(tmA, tmB, q, st);
}

}  // namespace swmoe
