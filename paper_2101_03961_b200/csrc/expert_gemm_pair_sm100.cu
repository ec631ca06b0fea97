// Grouped expert GEMMs on pairs of SMs (tcgen05 cta_group::2, M = 256), bfloat16 in, float32 accumulate, bfloat16
// out: the expert FFN h = x W_in, y = ReLU(h) W_out (Section 5, FFN review) and its derivatives, with the layer's
// element-wise steps fused into the epilogues (ReLU, the gate of Eq. 2 with the scatter back to token order, the
// ReLU mask of the backward pass; for GEGLU experts the gating GELU(a) . b in GEMM1's epilogue and its derivative in
// dgrad2's, two more instantiations of the same kernel).
//
// Orientation.  An expert has about 256 tokens but thousands of weight rows, so the weight matrix sits on the MMA's
// M side (256 rows per CTA pair, 128 per CTA) and the expert's tokens on the N side, whose granularity is 16:
//   H^T  [f, tok] = W_in^T  [f, d] . X_d^T  [d, tok]      y^T  [d, tok] = W_out^T [d, f] . H^T  [f, tok]
//   dH^T [f, tok] = W_out   [f, d] . dY_d^T [d, tok]      dx^T [d, tok] = W_in    [d, f] . dH^T [f, tok]
// so no 128-row token tile is padded, every weight element enters shared memory exactly once, and the epilogue
// transposes 32x32 blocks through shared memory to write token-major rows.  The weight gradients keep the natural
// orientation (dW_out = H^T dY_d, dW_in = X_d^T dH: M = weight rows, N = weight columns, contraction over tokens).
//
// A CTA pair shares the B operand: each CTA stages its own 128 A rows and half of B per 64-deep k-block, the leader
// CTA's single MMA thread issues M=256 instructions that read both CTAs' shared memory, and tcgen05.commit with a
// cluster mask releases stages and publishes accumulators in both CTAs.  TMA loads carry no multicast.  Each CTA
// drains its own 128 TMEM lanes with 8 epilogue warps while the next tile's MMAs run.
//
// One pass per expert.  A token tile holds up to 320 tokens (the capacity of the paper's layers at capacity factor
// 1.25), so an expert's weights cross shared memory once; a tile wider than the MMA's N limit of 256 is two column
// segments, i.e. two MMAs per k-step that read the same A block.  The token operand's TMA box is exactly the rows
// the tile has (one tensor map per box height), so no byte enters shared memory that no MMA reads.
// Two accumulators of up to 320 columns do not fit 512 TMEM columns side by side, so they overlap in the middle:
// even tiles of a CTA pair use columns [0, n), odd tiles [512 - n, 512).  The epilogue drains a tile starting from
// the middle columns and tells the MMA thread (barrier `tmid`) once the columns the next tile also uses have been
// read; the next tile's MMAs then start while the rest of the tile is still being drained.
//
// Every mbarrier wait is bounded in time (status word + abort flag); both CTAs always reach the final cluster
// barrier, so tensor memory is freed and no CTA exits while its peer can still address its shared memory.
#include "tc_common.cuh"

namespace swmoe {
using namespace tc;
namespace {

constexpr int kPStages = 6;                            // weight gradients: six stages of A (16 KB) + half of B (16 KB)
constexpr int kPMaxStages = 8;                         // token products: as many stages as fit, at most this
constexpr int kPHalfBytes = 16384;                     // A tile (128 x 64) and B half tile (<= 128 x 64)
constexpr int kPStageBytes = 2 * kPHalfBytes;
constexpr int kPRingBytes = kPStages * kPStageBytes;   // 192 KB of operand stages
constexpr int kPTransWarp = 16 * 144;                  // per epilogue warp: 16 token pairs x (32 weight rows x 4 B, padded
                                                       // to 144 B so that 16-byte reads of 8 rows do not collide)
constexpr int kPTransBytes = 8 * kPTransWarp;
constexpr int kPAuxBytes = 8 * 128;                    // 8 epilogue warps x 32 gates
constexpr int kPKeptCache = kMaxExperts;                 // kept[e] for every expert
constexpr int kPTileCache = 448;                        // first token tiles of the list ({expert, row, rows})
constexpr int kPCacheBytes = kPKeptCache * 4 + kPTileCache * 16;
constexpr int kPSmemBytes = 1024 + kPRingBytes + kPTransBytes + kPAuxBytes + 256 + kPCacheBytes;
constexpr int kPThreads = 320;
constexpr uint32_t kPeerMask = 0xFEFFFFFFu;            // clears the CTA-rank bit of a shared::cluster address
// GEMM1 of GEGLU experts with the gating in its epilogue (a seventh instantiation beside the six GemmOp products):
// a CTA's 128 weight rows are 64 columns of W_0 and the same 64 columns of W_1, so a_j and b_j of one hidden unit sit
// in TMEM lanes j and 64 + j of one CTA, i.e. with epilogue warps two lane groups apart.
constexpr int kGemm1Gated = 6;
// dgrad2 of GEGLU experts with the derivative of the gating in its epilogue: d a = dH . (b GELU'(a)), d b = dH . GELU(a),
// the two factors read back from what the gated GEMM1 saved.
constexpr int kDgrad2Gated = 7;

struct PairParams {
  int op;                  // GemmOp
  int token_op;            // 1: tokens on N (transposed epilogue); 0: weight gradient (contraction over tokens)
  int a_mn_major;
  int Mw;                  // rows of the M-side operand per expert (d_ff or d_model)
  int Nfix;                // weight gradients: output columns
  int k_blocks_fixed;      // token ops: K / 64
  int n_mpairs, n_ntiles_fixed;
  int C, E;
  const int4* ntile;       // [0].x = number of token tiles; then {expert, first slot row, rows (multiple of 16)}
  const int* kept;
  const int* token_of_slot;
  const float* gate;
  __nv_bfloat16* out;
  uint32_t* hmask;          // [d_ff/32][E*C]: bit i of word [w][row]: H[row][32w + i] > 0 (written by GEMM1, read by
                            // dgrad2); rows are contiguous so that 32 token rows are one 128-byte store / load
  long long hmask_rows;     // E*C
  long long ld_out;
  int* status;
  const __nv_bfloat16* res;   // combine / scatter with the skip path inside the layer: rows added to the output (x or dy)
  __nv_bfloat16* out2;        // combine with the skip path: second copy of the output without it
  int plain;                  // GEMM1 / dgrad2 without ReLU and without the ReLU mask (GEGLU experts)
  int gate_f;                 // gated products: d_ff.  Gated GEMM1: W_in has 2 d_ff columns [W_0 | W_1]; out = the saved
                              // factors, one 32-bit word {GELU(a), b GELU'(a)} per hidden unit and slot row; out2 = hidden.
                              // Gated dgrad2: out = d[a | b] (2 d_ff columns), gate_in = those words.
  const uint32_t* gate_in;
  // expert dropout (Section 2.4) in the epilogues: GEMM1 multiplies the hidden activations by keep / (1 - rate) before
  // it rounds them and takes the mask bits (the gated GEMM1: the hidden activations and both saved factors); dgrad2
  // multiplies by 1 / (1 - rate), its mask bits already say "kept and positive".
  const uint32_t* keep_bits;  // [E * C][d_ff / 32]: bit i of word [row][w] = keep hidden unit 32 w + i; or null
  int keep_words;             // d_ff / 32
  float keep_scale;           // 1 / (1 - rate); 1 without dropout
  int stages, stage_bytes;    // operand ring: token products size a stage for the widest tile the capacity allows
  // ceil(2^32 / divisor) for the three divisions of the tile decode (n_mpairs; n_mpairs * n_ntiles_fixed;
  // n_ntiles_fixed): id / d = umulhi(id, magic) as long as id * d < 2^32
  uint32_t magic_mpairs, magic_per_e, magic_nt;
};

__device__ __forceinline__ int fast_div(int id, uint32_t magic, int divisor) {
  return divisor == 1 ? id : (int)__umulhi((uint32_t)id, magic);
}

// Token products: the token operand's TMA box is exactly this CTA's share of the tile (n / 2 rows, a multiple of 8):
// one tensor map per height 8, 16, .., 128.  Weight gradients use entry 0 (a 64-row box of the token contraction).
constexpr int kBMaps = 16;
struct BMapSet {
  CUtensorMap m[kBMaps];
};

struct PTile {
  int e, m0, n0, row0, n, n1, k_blocks, last_mmas;   // n1: columns of the first segment (n if n <= 256)
};

// Tile decode reads the plan through shared-memory copies made at kernel start: a dependent global load per tile
// would stall the single-thread producer for longer than a short tile's whole k-loop.
__device__ __forceinline__ PTile p_decode(const PairParams& p, int id, const int* kept_s, const int4* tile_s) {
  PTile t;
  if (p.token_op) {
    const int nt = fast_div(id, p.magic_mpairs, p.n_mpairs);
    const int4 q = nt < kPTileCache ? tile_s[nt] : p.ntile[1 + nt];
    t.e = q.x; t.row0 = q.y; t.n = q.z; t.n0 = 0;
    t.n1 = t.n <= 256 ? t.n : ((t.n >> 1) + 15) & ~15;         // two segments: both multiples of 16, both <= 256
    t.m0 = (id - nt * p.n_mpairs) * 256;
    t.k_blocks = p.k_blocks_fixed;
    t.last_mmas = kBK / kUmmaK;
  } else {
    const int per_e = p.n_mpairs * p.n_ntiles_fixed;
    t.e = fast_div(id, p.magic_per_e, per_e);
    const int rem = id - t.e * per_e;
    const int mp = fast_div(rem, p.magic_nt, p.n_ntiles_fixed);
    t.m0 = mp * 256;
    t.n0 = (rem - mp * p.n_ntiles_fixed) * 256;
    t.row0 = 0; t.n = 256; t.n1 = 256;
    const int k = kept_s[t.e];
    t.k_blocks = (k + kBK - 1) / kBK;
    const int rem_rows = k - (t.k_blocks - 1) * kBK;          // rows of the last k-block that hold tokens
    t.last_mmas = (rem_rows + kUmmaK - 1) / kUmmaK;            // rows beyond them are never multiplied
  }
  return t;
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t local_bar, uint32_t cta) {
  asm volatile(
      "{\n\t.reg .b32 ra;\n\t"
      "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
      "mbarrier.arrive.shared::cluster.b64 _, [ra];\n\t}"
      ::"r"(local_bar), "r"(cta)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* tm, uint32_t leader_bar, int c0,
                                                 int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(leader_bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((uint16_t)3)
      : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// One instantiation per product (OP is a GemmOp): each kernel carries only its own epilogue, and the operand
// orientations are compile-time constants, which keeps the code footprint of every role small.
//
// `pair` of `n_pairs` is this CTA pair's place among the pairs that work on this product: the whole grid for a
// launch of one product, a share of it when two products run side by side in one launch (below).
template <int OP, bool DROP = false>                          // DROP: expert dropout in this product's epilogue
__device__ __forceinline__ void pair_body(const CUtensorMap& tmA, const BMapSet& bm, const PairParams& p,
                                          const int pair, const int n_pairs) {
  constexpr bool kGated = OP == kGemm1Gated, kDGated = OP == kDgrad2Gated;
  constexpr bool kTok = OP <= kDgrad1Scatter || kGated || kDGated;   // tokens on N, transposed epilogue
  constexpr bool kAMn = (OP == kGemm1Relu || kGated || OP == kGemm2Combine || OP == kWgrad2 || OP == kWgrad1);
  constexpr bool kBMn = !kTok;
  pdl_launch_dependents();
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  uint8_t* trans_gen = smem_gen + kPRingBytes;
  uint8_t* aux_gen = trans_gen + kPTransBytes;
  uint8_t* bar_gen = aux_gen + kPAuxBytes;
  const uint32_t bar_base = smem_base + kPRingBytes + kPTransBytes + kPAuxBytes;
  // barrier block: full[S] | empty[S] | tmem_full[2] | tmem_empty[2] | tmem_mid[2] | tmem_ptr | abort | gate[4]
  // (S = kPMaxStages; gate[i] at byte 192 + 8 i: the handshake of the two epilogue warps that hold a and b of the
  // same hidden units, gated GEMM1 only)
  const uint32_t full0 = bar_base, empty0 = bar_base + 8u * kPMaxStages;
  const uint32_t tfull0 = bar_base + 16u * kPMaxStages, tempty0 = tfull0 + 16u, tmid0 = tfull0 + 32u;
  const uint32_t gate0 = bar_base + 192u;
  volatile uint32_t* tmem_ptr_s = reinterpret_cast<volatile uint32_t*>(bar_gen + 8 * (2 * kPMaxStages + 6));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_gen + 8 * (2 * kPMaxStages + 6) + 4);
  int* kept_s = reinterpret_cast<int*>(bar_gen + 256);
  int4* tile_s = reinterpret_cast<int4*>(bar_gen + 256 + kPKeptCache * 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();                   // 0 = leader (issues the MMAs)
  const uint32_t n_stages = kTok ? (uint32_t)p.stages : (uint32_t)kPStages;
  const uint32_t stage_bytes = kTok ? (uint32_t)p.stage_bytes : (uint32_t)kPStageBytes;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kPMaxStages; ++s) { mbar_init(full0 + 8u * s, 1); mbar_init(empty0 + 8u * s, 1); }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull0 + 8u * a, 1); mbar_init(tempty0 + 8u * a, 16); mbar_init(tmid0 + 8u * a, 16);
    }
    if (kGated)
      for (int a = 0; a < 4; ++a) mbar_init(gate0 + 8u * a, 2);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(const_cast<uint32_t*>(tmem_ptr_s))), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  pdl_wait();                                                 // the previous kernel's results are needed from here on
  const int n_ntiles_listed = kTok ? p.ntile[0].x : 0;
  for (int i = threadIdx.x; i < p.E; i += kPThreads) kept_s[i] = p.kept[i];
  for (int i = threadIdx.x; i < min(n_ntiles_listed, kPTileCache); i += kPThreads) tile_s[i] = p.ntile[1 + i];
  tc_fence_before();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_s;
  const int n_tiles = kTok ? n_ntiles_listed * p.n_mpairs : p.E * p.n_mpairs * p.n_ntiles_fixed;

  // Accumulator columns of this pair's `it`-th tile: even tiles [0, n), odd tiles [512 - n, 512).  Consecutive tiles
  // share the middle columns when n + n_next > 512.
  if (warp == 0) {
    // ------------------------------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int id = pair; id < n_tiles && ok; id += n_pairs) {
        const PTile t = p_decode(p, id, kept_s, tile_s);
        // coordinates of this CTA's boxes; only the contraction coordinate moves inside the tile
        // gated GEMM1: 64 columns of W_0 and the same 64 columns of W_1 (a pair covers 128 hidden units)
        const int a_m = kGated ? (t.m0 >> 1) + 64 * (int)rank : t.m0 + 128 * (int)rank;
        const int a_m2 = kGated ? p.gate_f + a_m : a_m + 64;
        const int e = t.e, kbs = t.k_blocks;
        // token products: this CTA's half of each column segment's token rows, in boxes of exactly that height;
        // weight gradients: this CTA's 128 of the 256 output columns
        const int h1 = t.n1 >> 1, h2 = (t.n - t.n1) >> 1;
        const int b_r = kTok ? t.row0 + (int)rank * h1 : t.n0 + 128 * (int)rank;
        const int b_r2 = t.row0 + t.n1 + (int)rank * h2;
        const CUtensorMap* tmB = kTok ? &bm.m[(h1 >> 3) - 1] : &bm.m[0];
        const CUtensorMap* tmB2 = (kTok && h2 > 0) ? &bm.m[(h2 >> 3) - 1] : tmB;
        // both CTAs' bytes land on the leader's barrier
        const uint32_t tx_bytes = kTok ? 2u * (uint32_t)(kPHalfBytes + (t.n >> 1) * 128) : 2u * (uint32_t)kPStageBytes;
#pragma unroll 1
        for (int kb = 0; kb < kbs; ++kb) {
          const uint32_t eb = empty0 + 8u * stage;
          ok = mbar_wait(eb, phase ^ 1u, abort_flag, p.status, 21);
          if (!ok) break;
          const uint32_t a_dst = smem_base + stage * stage_bytes, b_dst = a_dst + kPHalfBytes;
          const uint32_t fb = full0 + 8u * stage;
          const uint32_t lead_full = fb & kPeerMask;
          const int k0 = kb * kBK;
          if (rank == 0) mbar_arrive_expect_tx(fb, tx_bytes);
          if (kAMn) {
            tma_load_3d_pair(a_dst, &tmA, lead_full, a_m, k0, e);
            tma_load_3d_pair(a_dst + kAtomBytes, &tmA, lead_full, a_m2, k0, e);
          } else {
            tma_load_3d_pair(a_dst, &tmA, lead_full, k0, a_m, e);
          }
          if (kBMn) {
            tma_load_3d_pair(b_dst, tmB, lead_full, b_r, k0, e);
            tma_load_3d_pair(b_dst + kAtomBytes, tmB, lead_full, b_r + 64, k0, e);
          } else {
            tma_load_3d_pair(b_dst, tmB, lead_full, k0, b_r, e);
            if (h2 > 0) tma_load_3d_pair(b_dst + (uint32_t)h1 * 128u, tmB2, lead_full, k0, b_r2, e);
          }
          if (++stage == n_stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (*abort_flag != 0) {
        const long long t0 = clock64();
        while (clock64() - t0 < 4000000ll) __nanosleep(1000);  // let copies in flight land (about 2 ms)
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------------------------ MMA issuer (leader CTA)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc_base = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)kAMn << 15) |
                                      ((uint32_t)kBMn << 16) | ((uint32_t)(256 >> 4) << 24);
      // descriptors differ between stages and k-steps only in the start-address field (units of 16 bytes)
      constexpr uint32_t a_kstep = (kAMn ? kUmmaK * 128u : kUmmaK * 2u) >> 4;
      constexpr uint32_t b_kstep = (kBMn ? kUmmaK * 128u : kUmmaK * 2u) >> 4;
      const uint64_t a_desc0 = make_smem_desc(smem_base, kAMn ? kAtomBytes : 16u, 1024u);
      const uint64_t b_desc0 = make_smem_desc(smem_base + kPHalfBytes, kBMn ? kAtomBytes : 16u, 1024u);
      uint32_t stage = 0, phase = 0, it = 0;
      int n_prev = 0;
      bool ok = true;
      for (int id = pair; id < n_tiles && ok; id += n_pairs, ++it) {
        const PTile t = p_decode(p, id, kept_s, tile_s);
        const uint32_t side = it & 1u, use = it >> 1;          // this side's `use`-th tile
        const uint32_t idesc1 = idesc_base | ((uint32_t)(t.n1 >> 3) << 17);
        const int n2 = t.n - t.n1;
        const uint32_t idesc2 = idesc_base | ((uint32_t)(n2 >> 3) << 17);
        const uint32_t b2_off = ((uint32_t)(t.n1 >> 1) * 128u) >> 4;    // second segment's rows in this CTA's half of B
        const int kbs = t.k_blocks, last_mmas = t.last_mmas;
        // the side's previous tile has been read out completely ...
        ok = mbar_wait(tempty0 + 8u * side, (use & 1u) ^ 1u, abort_flag, p.status, 22);
        if (!ok) break;
        // ... and so have the middle columns of the other side's tile, if this tile reaches into them
        if (kTok && it > 0 && n_prev + t.n > kTmemCols) {
          ok = mbar_wait(tmid0 + 8u * (side ^ 1u), ((it - 1u) >> 1) & 1u, abort_flag, p.status, 25);
          if (!ok) break;
        }
        n_prev = t.n;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (side ? (uint32_t)(kTmemCols - t.n) : 0u);
        const uint32_t d_tmem2 = d_tmem + (uint32_t)t.n1;
#pragma unroll 1
        for (int kb = 0; kb < kbs; ++kb) {
          ok = mbar_wait(full0 + 8u * stage, phase, abort_flag, p.status, 23);
          if (!ok) break;
          tc_fence_after();
          const uint64_t ad = a_desc0 + (uint64_t)(stage * (stage_bytes >> 4));
          const uint64_t bd = b_desc0 + (uint64_t)(stage * (stage_bytes >> 4));
          const int n_mma = (!kTok && kb == kbs - 1) ? last_mmas : kBK / kUmmaK;
          const uint32_t acc0 = kb > 0 ? 1u : 0u;
          tc_mma_bf16_pair(d_tmem, ad, bd, idesc1, acc0);
          if (kTok && n2 > 0) tc_mma_bf16_pair(d_tmem2, ad, bd + b2_off, idesc2, acc0);
#pragma unroll
          for (int ks = 1; ks < kBK / kUmmaK; ++ks) {
            if (ks < n_mma) {
              tc_mma_bf16_pair(d_tmem, ad + ks * a_kstep, bd + ks * b_kstep, idesc1, 1u);
              if (kTok && n2 > 0) tc_mma_bf16_pair(d_tmem2, ad + ks * a_kstep, bd + b2_off + ks * b_kstep, idesc2, 1u);
            }
          }
          tc_commit_pair(empty0 + 8u * stage);                // frees this stage in both CTAs
          if (++stage == n_stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (kbs > 0) {
          tc_commit_pair(tfull0 + 8u * side);                 // accumulator complete, in both CTAs
        } else {                                              // nothing to contract: epilogues write zeros
          mbar_arrive(tfull0 + 8u * side);
          mbar_arrive_remote(tfull0 + 8u * side, 1);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------------------------------ epilogue warps (both CTAs)
    const int lg = warp & 3;
    const int half = (warp - 2) >> 2;
    uint8_t* tr = trans_gen + (warp - 2) * kPTransWarp;       // this warp's transpose tile
    float* gate_s = reinterpret_cast<float*>(aux_gen + (warp - 2) * 128);
    uint32_t it = 0;
    bool ok = true;
    // gated GEMM1: lane groups 0, 1 hold a = x W_0, lane groups 2, 3 hold b = x W_1 of the same 32 hidden units
    const int role = lg >> 1;
    const uint8_t* tr_other = trans_gen + (half * 4 + lg) * kPTransWarp;   // the transpose tile of the warp two lane groups away
    const uint32_t gate_bar = gate0 + 8u * (uint32_t)(half * 2 + (lg & 1));
    uint32_t gate_phase = 0;
    for (int id = pair; id < n_tiles && ok; id += n_pairs, ++it) {
      const PTile t = p_decode(p, id, kept_s, tile_s);
      const uint32_t side = it & 1u, use = it >> 1;
      const int unit0 = (t.m0 >> 1) + 64 * (int)rank + 32 * (lg & 1);        // gated GEMM1: first hidden unit of this warp
      // first M row (weight row = output column) this warp holds
      const int m_warp = kGated ? role * p.gate_f + unit0 : t.m0 + 128 * (int)rank + 32 * lg;
      const int n_chunks = kTok ? (t.n + 31) >> 5 : 8;
      const bool have_acc = t.k_blocks > 0;
      const int c0 = side ? kTmemCols - t.n : 0;              // first accumulator column of the tile
      // Token products.  Chunks of 32 accumulator columns are numbered so that chunk j of an even tile holds the
      // tile's tokens [32 j, 32 j + 32) and chunk j of an odd tile its tokens [n - 32 (j + 1), n - 32 j): a chunk is
      // then always inside the 512 columns, and counting j down from the last chunk starts in the middle columns, the
      // ones the next tile may also use.  Lane i describes token column (chunk's first token) + i: the element offset
      // of its output row (or -1) and its gate.  This warp's chunks are j = n_chunks - 1 - half, then every second
      // one down to 0; their descriptions (and ReLU masks) are fetched before the accumulator is awaited.
      constexpr bool kSlotRows = (OP == kGemm1Relu || kGated || OP == kDgrad2Mask || kDGated);
      constexpr int kQueue = 5;                                // (320 / 32) chunks over two warps
      int row_limit = 0;
      long long q_off[kQueue] = {-1, -1, -1, -1, -1};           // head = next chunk to process
      float q_gate[kQueue] = {1.f, 1.f, 1.f, 1.f, 1.f};
      uint32_t q_mw[kQueue] = {0u, 0u, 0u, 0u, 0u};             // dgrad2: ReLU mask bits of weight rows m_warp..+31 per token
      const int mcol = m_warp + (lane & 3) * 8;               // store `it` writes weight rows mcol .. mcol + 7
      const bool col_ok = kGated ? unit0 + (lane & 3) * 8 < p.gate_f : mcol < p.Mw;
      auto chunk_tok0 = [&](int j) { return side ? t.n - 32 * (j + 1) : 32 * j; };
      auto describe = [&](int j, long long* off, float* g) {
        const int col = chunk_tok0(j) + lane, slot_row = t.row0 + col;
        *off = -1;
        *g = 1.f;
        if (j >= 0 && col >= 0 && col < t.n && slot_row < row_limit) {
          if (kSlotRows) {
            *off = ((long long)t.e * p.C + slot_row) * p.ld_out;
          } else {
            const int tok = p.token_of_slot[(long long)t.e * p.C + slot_row];
            *off = (long long)tok * p.ld_out;
            if (OP == kGemm2Combine) *g = p.gate[tok];        // Eq. 2: y = p_i(x) E_i(x)
          }
        }
      };
      int j_mid = 0;                                            // chunks j >= j_mid hold columns the next tile uses too
      if (kTok) {
        const int kept_e = kept_s[t.e];
        row_limit = kSlotRows ? min(p.C, (kept_e + 15) / 16 * 16) : kept_e;
        const int id_next = id + n_pairs;
        const int n_next = id_next < n_tiles ? p_decode(p, id_next, kept_s, tile_s).n : 0;
        j_mid = (t.n - max(0, t.n + n_next - kTmemCols)) >> 5;
        // everything the epilogue needs from global memory is requested here, before the accumulator is awaited
#pragma unroll
        for (int k = 0; k < kQueue; ++k) describe(n_chunks - 1 - half - 2 * k, &q_off[k], &q_gate[k]);
        if (DROP && (OP == kGemm1Relu || kGated) && (kGated ? unit0 < p.gate_f : m_warp < p.Mw)) {
          const int unit_word = (kGated ? unit0 : m_warp) >> 5;   // this warp's 32 hidden units are one word per row
#pragma unroll
          for (int k = 0; k < kQueue; ++k)
            if (q_off[k] >= 0)
              q_mw[k] = p.keep_bits[((long long)t.e * p.C + t.row0 + chunk_tok0(n_chunks - 1 - half - 2 * k) + lane) *
                                        p.keep_words + unit_word];
        }
        if (OP == kDgrad2Mask && !p.plain && m_warp < p.Mw) {
#pragma unroll
          for (int k = 0; k < kQueue; ++k)
            if (q_off[k] >= 0)
              q_mw[k] = p.hmask[(long long)(m_warp >> 5) * p.hmask_rows + (long long)t.e * p.C + t.row0 +
                                chunk_tok0(n_chunks - 1 - half - 2 * k) + lane];
        }
      }
      // gated dgrad2: the saved factors of this lane's hidden unit for the 32 tokens of a chunk, one word per token
      // ({GELU(a), b GELU'(a)} as two bfloat16), fetched one chunk ahead; 0 for columns that hold no token
      uint32_t gg[kDGated ? 32 : 1];
      auto fetch_factors = [&](int j, uint32_t* dst) {
        if constexpr (kDGated) {
          const int tok_first = chunk_tok0(j);
          const bool unit_ok = m_warp < p.Mw;
          const uint32_t* src = p.gate_in + ((long long)t.e * p.C + t.row0 + tok_first) * p.gate_f + m_warp + lane;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int col = tok_first + i;
            const bool valid = unit_ok && j >= 0 && col >= 0 && col < t.n && t.row0 + col < row_limit;
            dst[i] = valid ? src[(long long)i * p.gate_f] : 0u;
          }
        }
      };
      fetch_factors(n_chunks - 1 - half, gg);
      ok = mbar_wait(tfull0 + 8u * side, use & 1u, abort_flag, p.status, 24);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_addr = tmem_base + ((uint32_t)(lg * 32) << 16) + (uint32_t)c0;
      if constexpr (!kTok) {
        // Weight gradients (row = weight row): 64 output columns at a time, so that a row is a whole 128-byte line.
        // The warp's 2 KB of shared memory hold 16 rows x 128 bytes: rows 0-15 and 16-31 of the warp take turns, and
        // every store instruction then writes 4 complete lines (the store path's cost grows with the number of lines
        // an instruction touches).
#pragma unroll 1
        for (int c = half; c < 4; c += 2) {
          uint32_t v[64];
          if (have_acc) {
            tc_ld32(t_addr + c * 64, v);
            tc_ld32(t_addr + c * 64 + 32, v + 32);
            tc_wait_ld();
          } else {
#pragma unroll
            for (int i = 0; i < 64; ++i) v[i] = 0u;
          }
          if (c + 2 >= 4) {                                   // last chunk of this warp: accumulator read out
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(tempty0 + 8u * side, 0);
          }
          uint4 ch[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            uint32_t w[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
              __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(v[q * 8 + 2 * h]),
                                                        __uint_as_float(v[q * 8 + 2 * h + 1]));
              w[h] = *reinterpret_cast<uint32_t*>(&h2);
            }
            ch[q] = make_uint4(w[0], w[1], w[2], w[3]);
          }
          const int chunk = lane & 7;
          const int col = t.n0 + c * 64 + chunk * 8;
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            if ((lane >> 4) == hf) {
#pragma unroll
              for (int q = 0; q < 8; ++q)
                *reinterpret_cast<uint4*>(tr + (lane & 15) * 128 + ((q ^ (lane & 7)) << 4)) = ch[q];
            }
            __syncwarp();
#pragma unroll
            for (int st = 0; st < 4; ++st) {
              const int rr = st * 4 + (lane >> 3);
              const uint4 val = *reinterpret_cast<const uint4*>(tr + rr * 128 + ((chunk ^ (rr & 7)) << 4));
              const int orow = m_warp + hf * 16 + rr;
              if (orow < p.Mw && col < p.Nfix)
                *reinterpret_cast<uint4*>(p.out + ((long long)t.e * p.Mw + orow) * p.ld_out + col) = val;
            }
            __syncwarp();
          }
        }
        continue;
      } else {
        bool released = false, mid_sent = false;
#pragma unroll 1
        for (int j = n_chunks - 1 - half; j >= 0; j -= 2) {
          const int tok0 = chunk_tok0(j);                       // token column of lane 0 (-16 in an odd tile's last chunk)
          uint32_t v[32];
          if (have_acc) {
            tc_ld32(t_addr + (uint32_t)(tok0 + 0), v);
            tc_wait_ld();
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = 0u;
          }
          if (!mid_sent && j - 2 < j_mid) {                     // this warp's share of the middle columns is read out
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(tmid0 + 8u * side, 0);
            mid_sent = true;
          }
          if (j - 2 < 0) {                                      // last chunk of this warp: accumulator read out
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(tempty0 + 8u * side, 0);
            released = true;
          }
          uint32_t gn[kDGated ? 32 : 1];                        // gated dgrad2: the next chunk's factors, in flight meanwhile
          fetch_factors(j - 2, gn);
          {
            // Store `st` of this lane writes weight rows mcol .. mcol + 7 of token column tcol(st) of the chunk:
            // eight lanes' token pairs x four row groups per instruction.
            auto tcol = [&](int st) { return 16 * (st >> 1) + 2 * (lane >> 2) + (st & 1); };
            uint32_t mword[4] = {0u, 0u, 0u, 0u};
            if constexpr (kGated) {
              // GEGLU gating.  Both warps of a pair round their values (a or b of 32 hidden units x 32 tokens) into
              // their transpose tiles; between two handshakes the a warp takes b of the chunk's tokens 0-15 from the
              // other tile and the b warp a of tokens 16-31.  Each then has a and b of one hidden unit per lane for 16
              // tokens and forms GELU(a), b GELU'(a) (saved for the backward pass as one word per unit and row) and the
              // hidden activation GELU(a) b, and transposes both through its own tile.
              uint32_t pk[16];
#pragma unroll
              for (int k = 0; k < 16; ++k) {
                const __nv_bfloat162 t2 = __floats2bfloat162_rn(__uint_as_float(v[2 * k]), __uint_as_float(v[2 * k + 1]));
                pk[k] = *reinterpret_cast<const uint32_t*>(&t2);
                *reinterpret_cast<uint32_t*>(tr + k * 144 + lane * 4) = pk[k];
              }
              __syncwarp();
              if (lane == 0) mbar_arrive(gate_bar);
              ok = mbar_wait(gate_bar, gate_phase, abort_flag, p.status, 26);     // both tiles are written
              gate_phase ^= 1u;
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) break;
              uint32_t other[8];
#pragma unroll
              for (int k = 0; k < 8; ++k)
                other[k] = *reinterpret_cast<const uint32_t*>(tr_other + (8 * role + k) * 144 + lane * 4);
              __syncwarp();
              if (lane == 0) mbar_arrive(gate_bar);
              ok = mbar_wait(gate_bar, gate_phase, abort_flag, p.status, 27);     // both tiles have been read
              gate_phase ^= 1u;
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) break;
              uint32_t hw[8];
#pragma unroll
              for (int k = 0; k < 8; ++k) {                     // this warp's token pair k: tokens 16 role + 2 k, + 1
                const uint32_t mine = role ? pk[8 + k] : pk[k];
                const uint32_t aw = role ? other[k] : mine, bw = role ? mine : other[k];
                const float2 af = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&aw));
                const float2 bf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&bw));
                float cdf0, pdf0, cdf1, pdf1;
                gelu_cdf_pdf(af.x, &cdf0, &pdf0);
                gelu_cdf_pdf(af.y, &cdf1, &pdf1);
                float ga0 = af.x * cdf0, ga1 = af.y * cdf1;
                float gp0 = bf.x * fmaf(af.x, pdf0, cdf0), gp1 = bf.y * fmaf(af.y, pdf1, cdf1);
                if (DROP) {                                     // expert dropout: the hidden unit's factor on all three
                  const uint32_t kw0 = __shfl_sync(0xffffffffu, q_mw[0], 16 * role + 2 * k);
                  const uint32_t kw1 = __shfl_sync(0xffffffffu, q_mw[0], 16 * role + 2 * k + 1);
                  const float f0 = (kw0 >> lane) & 1u ? p.keep_scale : 0.f, f1 = (kw1 >> lane) & 1u ? p.keep_scale : 0.f;
                  ga0 *= f0; gp0 *= f0; ga1 *= f1; gp1 *= f1;
                }
                const __nv_bfloat162 s0 = __floats2bfloat162_rn(ga0, gp0);
                const __nv_bfloat162 s1 = __floats2bfloat162_rn(ga1, gp1);
                const __nv_bfloat162 h2 = __floats2bfloat162_rn(ga0 * bf.x, ga1 * bf.y);
                hw[k] = *reinterpret_cast<const uint32_t*>(&h2);
                // saved factors: tile row = token of this warp (0..15), one word per lane
                *reinterpret_cast<uint32_t*>(tr + (2 * k) * 144 + lane * 4) = *reinterpret_cast<const uint32_t*>(&s0);
                *reinterpret_cast<uint32_t*>(tr + (2 * k + 1) * 144 + lane * 4) = *reinterpret_cast<const uint32_t*>(&s1);
              }
              __syncwarp();
              const bool warp_ok = unit0 < p.gate_f;
#pragma unroll
              for (int pass = 0; pass < 4; ++pass) {            // a store writes 4 tokens x 32 hidden units x 4 bytes
                const int trow = 4 * pass + (lane >> 3);
                const uint4 val = *reinterpret_cast<const uint4*>(tr + trow * 144 + (lane & 7) * 16);
                const long long off = __shfl_sync(0xffffffffu, q_off[0], 16 * role + trow);
                // the saved row has one word (two bfloat16) per hidden unit: d_ff words = the 2 d_ff elements of q_off's row
                if (off >= 0 && warp_ok)
                  *reinterpret_cast<uint4*>(p.out + off + 2 * (unit0 + (lane & 7) * 4)) = val;
              }
              __syncwarp();
#pragma unroll
              for (int k = 0; k < 8; ++k) *reinterpret_cast<uint32_t*>(tr + k * 144 + lane * 4) = hw[k];
              __syncwarp();
              const uint8_t* src = tr + (lane >> 2) * 144 + (lane & 3) * 32;
              const uint4 lo = *reinterpret_cast<const uint4*>(src);
              const uint4 hi = *reinterpret_cast<const uint4*>(src + 16);
#pragma unroll
              for (int tb = 0; tb < 2; ++tb) {
                const uint32_t sel = tb ? 0x7632u : 0x5410u;
                const uint4 val = make_uint4(__byte_perm(lo.x, lo.y, sel), __byte_perm(lo.z, lo.w, sel),
                                             __byte_perm(hi.x, hi.y, sel), __byte_perm(hi.z, hi.w, sel));
                const long long off = __shfl_sync(0xffffffffu, q_off[0], 16 * role + 2 * (lane >> 2) + tb);
                // the saved row has 2 d_ff elements, the hidden row d_ff: half the element offset
                if (off >= 0 && col_ok) *reinterpret_cast<uint4*>(p.out2 + (off >> 1) + unit0 + (lane & 3) * 8) = val;
              }
            } else {
            long long offs[4];
#pragma unroll
            for (int st = 0; st < 4; ++st) offs[st] = __shfl_sync(0xffffffffu, q_off[0], tcol(st));
            if (OP == kGemm2Combine) gate_s[lane] = q_gate[0];
            __syncwarp();
            // gated dgrad2 writes two sets of columns from one accumulator: d a = dH . (b GELU'(a)) at column j, then
            // d b = dH . GELU(a) at column d_ff + j
#pragma unroll
            for (int rnd = 0; rnd < (kDGated ? 2 : 1); ++rnd) {
            if (rnd > 0) __syncwarp();                          // the tile's readers of the first set are done
            const int mcol_r = mcol + rnd * p.gate_f;
            // transpose: this lane holds weight row m_warp + lane for 32 tokens.  Two tokens are packed into one
            // 32-bit word, tr[token pair][lane]: half the shared-memory stores of a 16-bit layout, each a full
            // 128-byte wavefront; a reader takes the words of eight rows (32 bytes) and separates the two tokens.
#pragma unroll
            for (int i4 = 0; i4 < 32; i4 += 4) {
              float g[4] = {1.f, 1.f, 1.f, 1.f};
              if (OP == kGemm2Combine) {
                const float4 g4 = *reinterpret_cast<const float4*>(gate_s + i4);
                g[0] = g4.x; g[1] = g4.y; g[2] = g4.z; g[3] = g4.w;
              }
              float a[4];
#pragma unroll
              for (int u = 0; u < 4; ++u) {
                a[u] = __uint_as_float(v[i4 + u]);
                if (OP == kGemm2Combine) a[u] *= g[u];
                if (OP == kGemm1Relu && !p.plain) a[u] = fmaxf(a[u], 0.f);
                if (DROP && OP == kGemm1Relu) {                 // expert dropout before the rounding and the mask bits
                  const uint32_t kw = __shfl_sync(0xffffffffu, q_mw[0], i4 + u);
                  a[u] = (kw >> lane) & 1u ? a[u] * p.keep_scale : 0.f;
                }
                if (DROP && OP == kDgrad2Mask) a[u] *= p.keep_scale;
                if (kDGated)                                    // high half: b GELU'(a); low half: GELU(a)
                  a[u] *= __uint_as_float(rnd == 0 ? (gg[kDGated ? i4 + u : 0] & 0xFFFF0000u) : (gg[kDGated ? i4 + u : 0] << 16));
              }
              *reinterpret_cast<__nv_bfloat162*>(tr + (i4 >> 1) * 144 + lane * 4) = __floats2bfloat162_rn(a[0], a[1]);
              *reinterpret_cast<__nv_bfloat162*>(tr + ((i4 >> 1) + 1) * 144 + lane * 4) = __floats2bfloat162_rn(a[2], a[3]);
            }
            __syncwarp();
#pragma unroll
            for (int pass = 0; pass < 2; ++pass) {
              const uint8_t* src = tr + (8 * pass + (lane >> 2)) * 144 + (lane & 3) * 32;
              const uint4 lo = *reinterpret_cast<const uint4*>(src);           // rows 8 g .. 8 g + 3, both tokens
              const uint4 hi = *reinterpret_cast<const uint4*>(src + 16);      // rows 8 g + 4 .. 8 g + 7
#pragma unroll
              for (int tb = 0; tb < 2; ++tb) {
                const int st = 2 * pass + tb;
                const uint32_t sel = tb ? 0x7632u : 0x5410u;                   // high halves: the pair's second token
                uint4 val = make_uint4(__byte_perm(lo.x, lo.y, sel), __byte_perm(lo.z, lo.w, sel),
                                       __byte_perm(hi.x, hi.y, sel), __byte_perm(hi.z, hi.w, sel));
                if (OP == kDgrad2Mask && !p.plain) {            // ReLU'(u) = [u > 0]: bits saved by the forward GEMM
                  const uint32_t bits = __shfl_sync(0xffffffffu, q_mw[0], tcol(st)) >> ((lane & 3) * 8);
                  uint32_t* w = reinterpret_cast<uint32_t*>(&val);
#pragma unroll
                  for (int q = 0; q < 4; ++q)
                    w[q] &= ((bits >> (2 * q)) & 1u ? 0x0000FFFFu : 0u) | ((bits >> (2 * q + 1)) & 1u ? 0xFFFF0000u : 0u);
                }
                if (OP == kGemm1Relu && !p.plain) {             // save [H > 0] as one bit per element for the backward pass
                  const uint32_t* w = reinterpret_cast<const uint32_t*>(&val);
                  uint32_t m8 = 0;
#pragma unroll
                  for (int q = 0; q < 4; ++q)
                    m8 |= ((w[q] & 0x00007FFFu) ? 1u << (2 * q) : 0u) | ((w[q] & 0x7FFF0000u) ? 1u << (2 * q + 1) : 0u);
                  uint32_t word = m8 << ((lane & 3) * 8);
                  word |= __shfl_xor_sync(0xffffffffu, word, 1);
                  word |= __shfl_xor_sync(0xffffffffu, word, 2);
                  mword[st] = word;                             // the word of token tcol(st), in all four lanes of its group
                }
                if ((OP == kGemm2Combine || OP == kDgrad1Scatter) && p.res != nullptr && offs[st] >= 0 && col_ok) {
                  // skip path inside the layer: y = x + g E(x), dx = dy + dH W_in^T (the expert term is already bf16)
                  if (OP == kGemm2Combine) *reinterpret_cast<uint4*>(p.out2 + offs[st] + mcol) = val;
                  const uint4 r = *reinterpret_cast<const uint4*>(p.res + offs[st] + mcol);
                  const __nv_bfloat162* rv = reinterpret_cast<const __nv_bfloat162*>(&r);
                  __nv_bfloat162* vv = reinterpret_cast<__nv_bfloat162*>(&val);
#pragma unroll
                  for (int q = 0; q < 4; ++q) {
                    const float2 a2 = __bfloat1622float2(vv[q]), b2 = __bfloat1622float2(rv[q]);
                    vv[q] = __floats2bfloat162_rn(a2.x + b2.x, a2.y + b2.y);
                  }
                }
                if (offs[st] >= 0 && col_ok) *reinterpret_cast<uint4*>(p.out + offs[st] + mcol_r) = val;
              }
            }
            }
            }
            if constexpr (kDGated) {
#pragma unroll
              for (int i = 0; i < 32; ++i) gg[i] = gn[i];
            }
            if (OP == kGemm1Relu && !p.plain) {                 // lane i stores the mask word of token row i: one 128-byte line
              // token `lane` was handled as st = 2 (lane / 16) + (lane & 1) by the four lanes 4 ((lane / 2) & 7) ..
              uint32_t mine = 0;
#pragma unroll
              for (int st = 0; st < 4; ++st) {
                const uint32_t w = __shfl_sync(0xffffffffu, mword[st], 4 * ((lane >> 1) & 7));
                if (2 * (lane >> 4) + (lane & 1) == st) mine = w;
              }
              if (q_off[0] >= 0 && m_warp < p.Mw)
                p.hmask[(long long)(m_warp >> 5) * p.hmask_rows + (long long)t.e * p.C + t.row0 + tok0 + lane] = mine;
            }
#pragma unroll
            for (int k = 0; k < kQueue - 1; ++k) {              // advance the queue
              q_off[k] = q_off[k + 1];
              q_gate[k] = q_gate[k + 1];
              q_mw[k] = q_mw[k + 1];
            }
            __syncwarp();
          }
        }
        if (!mid_sent) {                                        // this warp had no chunk in this tile
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_remote(tmid0 + 8u * side, 0);
        }
        if (!released) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_remote(tempty0 + 8u * side, 0);
        }
      }
    }
  }

  // ---------------------------------------------------------------------------------------------- teardown
  __syncwarp();                                               // single-lane roles rejoin their warps
  tc_fence_before();
  cluster_sync_all();
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

template <int OP, bool DROP = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPThreads, 1)
expert_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ BMapSet bm,
                        const PairParams p) {
  pair_body<OP, DROP>(tmA, bm, p, (int)(blockIdx.x >> 1), (int)(gridDim.x >> 1));
}

// Two products that read the same activations, side by side in one launch: the first `split` CTA pairs work on
// product A, the others on product B, each walking the experts in the same order.  dgrad1 (dx = dH W_in^T) and wgrad1
// (dW_in = X_d^T dH) both read dH and nothing of each other; run one after the other each reads its 0.2 GB from HBM,
// run together the expert's rows that one of them fetched are still in L2 when the other asks for them (whichever
// runs ahead pays the HBM latency and so falls back: the two stay within a few experts of each other).
template <int OPA, int OPB>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPThreads, 1)
expert_gemm_pair_dual_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ BMapSet tmB0,
                             const PairParams p0, const __grid_constant__ CUtensorMap tmA1,
                             const __grid_constant__ BMapSet tmB1, const PairParams p1, const int split) {
  const int cl = (int)(blockIdx.x >> 1), n = (int)(gridDim.x >> 1);
  if (cl < split) pair_body<OPA>(tmA0, tmB0, p0, cl, split);
  else pair_body<OPB>(tmA1, tmB1, p1, cl - split, n - split);
}

// persistent grid: as many CTA pairs as can be resident at once (at most one CTA per SM).  The occupancy query
// costs tens of microseconds of host time, so its answer is kept per device and kernel.
template <typename Kernel>
int pair_grid(Kernel kernel, int* cached_grid, int dev, int sm_count, cudaStream_t st, int* grid_out) {
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPSmemBytes) != cudaSuccess)
    return SWITCH_MOE_CUDA_ERROR;
  int grid = (dev >= 0 && dev < 64) ? cached_grid[dev] : 0;
  if (grid == 0) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)(sm_count & ~1), 1, 1);
    lc.blockDim = dim3(kPThreads, 1, 1);
    lc.dynamicSmemBytes = kPSmemBytes;
    lc.stream = st;
    int max_clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&max_clusters, kernel, &lc) != cudaSuccess || max_clusters < 1) {
      (void)cudaGetLastError();
      max_clusters = sm_count / 2;
    }
    grid = 2 * (max_clusters < sm_count / 2 ? max_clusters : sm_count / 2);
    if (grid < 2) return SWITCH_MOE_CUDA_ERROR;
    if (dev >= 0 && dev < 64) cached_grid[dev] = grid;
  }
  *grid_out = grid;
  return SWITCH_MOE_OK;
}

template <int OP, bool DROP = false>
int launch_pair_op(const CUtensorMap& tmA, const BMapSet& tmB, const PairParams& q, int dev, int sm_count,
                   cudaStream_t st) {
  static int cached_grid[64] = {0};
  int grid = 0;
  const int rc = pair_grid(expert_gemm_pair_kernel<OP, DROP>, cached_grid, dev, sm_count, st, &grid);
  if (rc != SWITCH_MOE_OK) return rc;
  launch_k(expert_gemm_pair_kernel<OP, DROP>, dim3(grid), dim3(kPThreads), kPSmemBytes, st, tmA, tmB, q);
  return launch_status();
}

// Operands, output and tile counts of one product.
// The token operand's maps: one per box height (8 j rows, j = 1..16).
int make_token_maps(BMapSet* bm, const void* base, long long E, long long rows, long long cols) {
  for (int j = 1; j <= kBMaps; ++j)
    if (make_map(&bm->m[j - 1], base, E, rows, cols, 8 * j) != SWITCH_MOE_OK) return SWITCH_MOE_CUDA_ERROR;
  return SWITCH_MOE_OK;
}

int pair_problem(GemmOp op, const Shape& s, const Plan& p, const GemmArgs& a, void* ws, PairParams* out,
                 CUtensorMap* tmA_out, BMapSet* tmB_out) {
  const void* xd = ws_ptr<char>(ws, p.xd);
  const void* h = ws_ptr<char>(ws, p.h);
  const void* dyd = ws_ptr<char>(ws, p.dyd);
  const void* dh = ws_ptr<char>(ws, p.dh);
  const int fin = s.fin;                                      // columns of W_in: f, or 2 f for GEGLU experts
  const void* du = s.geglu ? ws_ptr<char>(ws, p.dab) : dh;    // gradient of the pre-activation(s)

  PairParams q{};
  q.op = (int)op;
  q.C = s.C; q.E = s.E;
  q.ntile = ws_ptr<int4>(ws, p.ntile);
  q.kept = ws_ptr<int>(ws, p.kept);
  q.token_of_slot = ws_ptr<int>(ws, p.token_of_slot);
  q.gate = ws_ptr<float>(ws, p.gate);
  q.status = ws_ptr<int>(ws, p.status);
  q.hmask = ws_ptr<uint32_t>(ws, p.hmask);
  q.hmask_rows = (long long)s.E * s.C;
  q.keep_scale = 1.f;
  CUtensorMap& tmA = *tmA_out;
  BMapSet& bm = *tmB_out;
  CUtensorMap& tmB = bm.m[0];
  int rc = SWITCH_MOE_OK, rc2 = SWITCH_MOE_OK;
  int K = 0;
  switch (op) {
    case kGemm1Relu:       // A = W_in [E][d (k)][f (m)]: m contiguous -> MN-major; B = X_d [E][C][d] K-major
      q.token_op = 1; q.a_mn_major = 1; q.Mw = fin; K = s.d;   // GEGLU: 2 f weight columns [W_0 | W_1], no ReLU
      rc = make_map(&tmA, a.W_in, s.E, s.d, fin, 64); rc2 = make_token_maps(&bm, xd, s.E, s.C, s.d);
      q.out = s.geglu ? ws_ptr<__nv_bfloat16>(ws, p.ab) : ws_ptr<__nv_bfloat16>(ws, p.h); q.ld_out = fin;
      q.plain = s.geglu;
      if (s.geglu) { q.gate_f = s.f; q.out2 = ws_ptr<__nv_bfloat16>(ws, p.h); }   // gating in the epilogue
      if (s.dropout) {
        if (s.keep_bits == nullptr || (reinterpret_cast<uintptr_t>(s.keep_bits) & 3u) != 0) return SWITCH_MOE_INVALID_ARGUMENT;
        q.keep_bits = s.keep_bits; q.keep_words = s.f / 32; q.keep_scale = s.keep_scale;
      }
      break;
    case kGemm2Combine:    // A = W_out [E][f (k)][d (m)] MN-major; B = H [E][C][f] K-major
      q.token_op = 1; q.a_mn_major = 1; q.Mw = s.d; K = s.f;
      rc = make_map(&tmA, a.W_out, s.E, s.f, s.d, 64); rc2 = make_token_maps(&bm, h, s.E, s.C, s.f);
      q.out = static_cast<__nv_bfloat16*>(a.y); q.ld_out = s.d;
      if (s.residual && !s.top2) {   // (top-2 routing adds the skip path where the two assignments' rows are summed)
        q.res = static_cast<const __nv_bfloat16*>(a.x); q.out2 = ws_ptr<__nv_bfloat16>(ws, p.layer_y);
      }
      break;
    case kDgrad2Mask:      // A = W_out [E][f (m)][d (k)] K-major; B = dY_d [E][C][d] K-major
      q.token_op = 1; q.a_mn_major = 0; q.Mw = s.f; K = s.d;
      rc = make_map(&tmA, a.W_out, s.E, s.f, s.d, 128); rc2 = make_token_maps(&bm, dyd, s.E, s.C, s.d);
      q.out = ws_ptr<__nv_bfloat16>(ws, p.dh); q.ld_out = s.f; q.plain = s.geglu;
      if (s.dropout && !s.geglu) q.keep_scale = s.keep_scale;   // (GEGLU: the saved factors carry the dropout factor)
      if (s.geglu) {   // the derivative of the gating in the epilogue: d[a | b] is written, dH never is
        q.out = ws_ptr<__nv_bfloat16>(ws, p.dab); q.ld_out = fin; q.gate_f = s.f;
        q.gate_in = ws_ptr<uint32_t>(ws, p.ab);
      }
      break;
    case kDgrad1Scatter:   // A = W_in [E][d (m)][f (k)] K-major; B = dH [E][C][f] K-major  (GEGLU: d[a | b], K = 2 f)
      q.token_op = 1; q.a_mn_major = 0; q.Mw = s.d; K = fin;
      rc = make_map(&tmA, a.W_in, s.E, s.d, fin, 128); rc2 = make_token_maps(&bm, du, s.E, s.C, fin);
      q.out = static_cast<__nv_bfloat16*>(a.dx); q.ld_out = s.d;
      if (s.residual && !s.top2) q.res = static_cast<const __nv_bfloat16*>(a.dy);
      break;
    case kWgrad2:          // dW_out [f][d] = H^T dY_d: A = H [E][C (k)][f (m)] MN-major; B = dY_d [E][C (k)][d (n)]
      q.token_op = 0; q.a_mn_major = 1; q.Mw = s.f; q.Nfix = s.d;
      rc = make_map(&tmA, h, s.E, s.C, s.f, 64); rc2 = make_map(&tmB, dyd, s.E, s.C, s.d, 64);
      q.out = static_cast<__nv_bfloat16*>(a.dW_out); q.ld_out = s.d; break;
    case kWgrad1:          // dW_in [d][f] = X_d^T dH  (GEGLU: X_d^T d[a | b], 2 f columns)
      q.token_op = 0; q.a_mn_major = 1; q.Mw = s.d; q.Nfix = fin;
      rc = make_map(&tmA, xd, s.E, s.C, s.d, 64); rc2 = make_map(&tmB, du, s.E, s.C, fin, 64);
      q.out = static_cast<__nv_bfloat16*>(a.dW_in); q.ld_out = fin; break;
    default: return SWITCH_MOE_INVALID_ARGUMENT;
  }
  if (rc != SWITCH_MOE_OK || rc2 != SWITCH_MOE_OK) return SWITCH_MOE_CUDA_ERROR;
  q.n_mpairs = (q.Mw + 255) / 256;
  // operand ring of the token products: a stage holds A (16 KB) and this CTA's half of the widest token tile the
  // capacity allows (at most kPairTileTokens / 2 rows of 128 bytes, rounded up to whole 1 KB swizzle atoms)
  const int widest = s.C < kPairTileTokens ? (s.C + 15) / 16 * 16 : kPairTileTokens;
  q.stage_bytes = kPHalfBytes + ((widest / 2) * 128 + 1023) / 1024 * 1024;
  q.stages = kPRingBytes / q.stage_bytes < kPMaxStages ? kPRingBytes / q.stage_bytes : kPMaxStages;
  q.n_ntiles_fixed = q.token_op ? 0 : (q.Nfix + 255) / 256;
  q.k_blocks_fixed = q.token_op ? K / kBK : 0;
  auto magic = [](int d) { return d > 1 ? (uint32_t)((0x100000000ull + (uint64_t)d - 1) / (uint64_t)d) : 0u; };
  q.magic_mpairs = magic(q.n_mpairs);
  q.magic_per_e = magic(q.n_mpairs * (q.n_ntiles_fixed > 0 ? q.n_ntiles_fixed : 1));
  q.magic_nt = magic(q.n_ntiles_fixed > 0 ? q.n_ntiles_fixed : 1);
  // the decode's divisions are exact only while id * divisor < 2^32: ids are below E * 16 * n_mpairs * n_ntiles
  {
    const uint64_t ids = q.token_op ? (uint64_t)s.max_mtiles * q.n_mpairs
                                    : (uint64_t)s.E * q.n_mpairs * (q.n_ntiles_fixed > 0 ? q.n_ntiles_fixed : 1);
    if (ids * (uint64_t)(q.n_mpairs * (q.n_ntiles_fixed > 0 ? q.n_ntiles_fixed : 1)) >= 0x100000000ull)
      return SWITCH_MOE_UNSUPPORTED_SHAPE;
  }
  *out = q;
  return SWITCH_MOE_OK;
}

int device_and_sms(int* dev, int* sm_count) {
  if (cudaGetDevice(dev) != cudaSuccess) return SWITCH_MOE_CUDA_ERROR;
  if (cudaDeviceGetAttribute(sm_count, cudaDevAttrMultiProcessorCount, *dev) != cudaSuccess)
    return SWITCH_MOE_CUDA_ERROR;
  return SWITCH_MOE_OK;
}

}  // namespace

int launch_pair_gemm(GemmOp op, const Shape& s, const Plan& p, const GemmArgs& a, void* ws, cudaStream_t st) {
  int dev = 0, sm_count = 0;
  if (device_and_sms(&dev, &sm_count) != SWITCH_MOE_OK) return SWITCH_MOE_CUDA_ERROR;
  PairParams q;
  CUtensorMap tmA;
  BMapSet tmB;
  const int rc = pair_problem(op, s, p, a, ws, &q, &tmA, &tmB);
  if (rc != SWITCH_MOE_OK) return rc;
  switch (op) {
    case kGemm1Relu:
      if (s.geglu) return s.dropout ? launch_pair_op<kGemm1Gated, true>(tmA, tmB, q, dev, sm_count, st)
                                    : launch_pair_op<kGemm1Gated>(tmA, tmB, q, dev, sm_count, st);
      return s.dropout ? launch_pair_op<kGemm1Relu, true>(tmA, tmB, q, dev, sm_count, st)
                       : launch_pair_op<kGemm1Relu>(tmA, tmB, q, dev, sm_count, st);
    case kGemm2Combine: return launch_pair_op<kGemm2Combine>(tmA, tmB, q, dev, sm_count, st);
    case kDgrad2Mask:
      if (s.geglu) return launch_pair_op<kDgrad2Gated>(tmA, tmB, q, dev, sm_count, st);
      return s.dropout ? launch_pair_op<kDgrad2Mask, true>(tmA, tmB, q, dev, sm_count, st)
                       : launch_pair_op<kDgrad2Mask>(tmA, tmB, q, dev, sm_count, st);
    case kDgrad1Scatter: return launch_pair_op<kDgrad1Scatter>(tmA, tmB, q, dev, sm_count, st);
    case kWgrad2: return launch_pair_op<kWgrad2>(tmA, tmB, q, dev, sm_count, st);
    default: return launch_pair_op<kWgrad1>(tmA, tmB, q, dev, sm_count, st);
  }
}

// dgrad1 and wgrad1 in one launch (see expert_gemm_pair_dual_kernel).  The two products have the same flops; the
// weight gradient's tiles are the slower ones, so it gets the larger share of the CTA pairs (39 of 74 measured best
// on B200 at the bench shape: 1.3% of the step against two launches).
int launch_pair_dgrad1_wgrad1(const Shape& s, const Plan& p, const GemmArgs& a, void* ws, cudaStream_t st) {
  int dev = 0, sm_count = 0;
  if (device_and_sms(&dev, &sm_count) != SWITCH_MOE_OK) return SWITCH_MOE_CUDA_ERROR;
  PairParams q0, q1;
  CUtensorMap tmA0, tmA1;
  BMapSet tmB0, tmB1;
  int rc = pair_problem(kDgrad1Scatter, s, p, a, ws, &q0, &tmA0, &tmB0);
  if (rc != SWITCH_MOE_OK) return rc;
  rc = pair_problem(kWgrad1, s, p, a, ws, &q1, &tmA1, &tmB1);
  if (rc != SWITCH_MOE_OK) return rc;
  static int cached_grid[64] = {0};
  int grid = 0;
  auto kernel = expert_gemm_pair_dual_kernel<kDgrad1Scatter, kWgrad1>;
  rc = pair_grid(kernel, cached_grid, dev, sm_count, st, &grid);
  if (rc != SWITCH_MOE_OK) return rc;
  const int n_pairs = grid / 2;
  if (n_pairs < 2) {                                          // nothing to share a launch with: one after the other
    rc = launch_pair_op<kDgrad1Scatter>(tmA0, tmB0, q0, dev, sm_count, st);
    return rc != SWITCH_MOE_OK ? rc : launch_pair_op<kWgrad1>(tmA1, tmB1, q1, dev, sm_count, st);
  }
  int split = (n_pairs * 35 + 37) / 74;
  if (split < 1) split = 1;
  if (split > n_pairs - 1) split = n_pairs - 1;
  launch_k(kernel, dim3(grid), dim3(kPThreads), kPSmemBytes, st, tmA0, tmB0, q0, tmA1, tmB1, q1, split);
  return launch_status();
}

}  // namespace swmoe
