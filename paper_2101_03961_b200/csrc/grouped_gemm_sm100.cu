// Grouped expert GEMMs on the B200 tensor cores (tcgen05 + TMEM, operands staged by TMA), bfloat16 in, float32
// accumulate, bfloat16 out: the expert FFN h = x W_in, y = ReLU(h) W_out (Section 5, FFN review) for every expert's
// kept tokens, and its four derivative products, each with its element-wise step fused into the epilogue:
//   H  = ReLU(X_d W_in)                      y[token]  = g . (H W_out)[slot]          (Eq. 2: gate-scaled combine)
//   dH = (dY_d W_out^T) * [H > 0]            dx[token] = (dH W_in^T)[slot]
//   dW_out = H^T dY_d                        dW_in     = X_d^T dH                     (contraction over kept tokens)
//
// One persistent CTA per SM, 320 threads: warp 0 issues TMA loads into a 4-stage ring of 128B-swizzled tiles
// (A 128x64, B 256x64 per stage), warp 1 issues tcgen05.mma (M=128, N=256, K=16) into one of two 128x256 float32
// accumulators in tensor memory, warps 2-9 drain the other accumulator (tcgen05.ld; each warp owns one 32-lane group
// and one half of the columns), apply the epilogue and write full 128-byte row segments.  Operands may be K-major or MN-major (the weight matrices are used both ways), chosen
// per product by descriptor bits only.  No TMA multicast is used anywhere.
//
// Every wait on an mbarrier is bounded in time; a wait that gives up records a code in the workspace status word,
// raises a CTA-wide abort flag, lets in-flight copies land, frees tensor memory and returns.
#include "tc_common.cuh"

namespace swmoe {
using namespace tc;
namespace {

constexpr int kOutStageBytes = 8 * 32 * 128;         // 8 epilogue warps x 32 rows x 128 B
constexpr int kBarBytes = 128;
constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kOutStageBytes + kBarBytes;
constexpr int kThreads = 320;                        // TMA warp, MMA warp, 8 epilogue warps

struct TcParams {
  int op;                     // GemmOp
  int a_mn_major, b_mn_major;
  int token_m;                // 1: M runs over an expert's token slots (tile list); 0: M fixed (weight gradients)
  int n_ntiles, n_mtiles_fixed, k_blocks_fixed;
  int M, N;                   // M: rows of the output per expert when !token_m; N: columns
  int C, E;
  const int* tile_expert;     // [0] = number of token tiles, then expert of each tile
  const int* tile_row0;       // [0] unused, then first slot row of each tile
  const int* kept;
  const int* token_of_slot;
  const float* gate;
  __nv_bfloat16* out;
  const __nv_bfloat16* mask_src;
  long long ld_out;
  int* status;
};

struct TileCoord {
  int e, m0, n0, k_blocks;
  bool valid;
};

__device__ __forceinline__ int total_tiles(const TcParams& p) {
  return p.token_m ? p.tile_expert[0] * p.n_ntiles : p.E * p.n_mtiles_fixed * p.n_ntiles;
}

__device__ __forceinline__ TileCoord decode_tile(const TcParams& p, int id) {
  TileCoord t;
  if (p.token_m) {
    const int mt = id / p.n_ntiles;
    t.e = p.tile_expert[1 + mt];
    t.m0 = p.tile_row0[1 + mt];
    t.n0 = (id - mt * p.n_ntiles) * kBN;
    t.k_blocks = p.k_blocks_fixed;
  } else {
    const int per_e = p.n_mtiles_fixed * p.n_ntiles;
    t.e = id / per_e;
    const int rem = id - t.e * per_e;
    const int mt = rem / p.n_ntiles;
    t.m0 = mt * kTileM;
    t.n0 = (rem - mt * p.n_ntiles) * kBN;
    t.k_blocks = (p.kept[t.e] + kBK - 1) / kBK;
  }
  t.valid = true;
  return t;
}

__global__ void __launch_bounds__(kThreads, 1)
grouped_gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                       const TcParams p) {
  pdl_launch_dependents();
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t out_stage_base = smem_base + kStages * kStageBytes;
  const uint32_t bar_base = out_stage_base + kOutStageBytes;
  uint8_t* bar_gen = smem_gen + kStages * kStageBytes + kOutStageBytes;
  // barrier block: full[4] | empty[4] | tmem_full[2] | tmem_empty[2] | tmem_ptr | abort
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };
  volatile uint32_t* tmem_ptr_s = reinterpret_cast<volatile uint32_t*>(bar_gen + 8 * (2 * kStages + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_gen + 8 * (2 * kStages + 4) + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 8); }
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

  const int n_tiles = total_tiles(p);

  if (warp == 0) {
    // ------------------------------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int id = blockIdx.x; id < n_tiles && ok; id += gridDim.x) {
        const TileCoord t = decode_tile(p, id);
        for (int kb = 0; kb < t.k_blocks; ++kb) {
          ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 1);
          if (!ok) break;
          const uint32_t a_dst = smem_base + stage * kStageBytes, b_dst = a_dst + kABytes;
          mbar_arrive_expect_tx(full_bar(stage), kStageBytes);
          if (p.a_mn_major) {
            tma_load_3d(a_dst, &tmA, full_bar(stage), t.m0, kb * kBK, t.e);
            tma_load_3d(a_dst + kAtomBytes, &tmA, full_bar(stage), t.m0 + 64, kb * kBK, t.e);
          } else {
            tma_load_3d(a_dst, &tmA, full_bar(stage), kb * kBK, t.m0, t.e);
          }
          if (p.b_mn_major) {
#pragma unroll
            for (int j = 0; j < kBN / 64; ++j)
              tma_load_3d(b_dst + j * kAtomBytes, &tmB, full_bar(stage), t.n0 + 64 * j, kb * kBK, t.e);
          } else {
            tma_load_3d(b_dst, &tmB, full_bar(stage), kb * kBK, t.n0, t.e);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (*abort_flag != 0) {
        // give copies that are still in flight a bounded time to land before the CTA's shared memory is released
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 2000000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.a_mn_major << 15) |
                             ((uint32_t)p.b_mn_major << 16) | ((uint32_t)(kBN >> 3) << 17) |
                             ((uint32_t)(kTileM >> 4) << 24);
      const uint32_t a_lbo = p.a_mn_major ? kAtomBytes : 16u, b_lbo = p.b_mn_major ? kAtomBytes : 16u;
      const uint32_t a_kstep = p.a_mn_major ? kUmmaK * 128u : kUmmaK * 2u;
      const uint32_t b_kstep = p.b_mn_major ? kUmmaK * 128u : kUmmaK * 2u;
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int id = blockIdx.x; id < n_tiles && ok; id += gridDim.x) {
        const TileCoord t = decode_tile(p, id);
        ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status, 2);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * kBN;
        for (int kb = 0; kb < t.k_blocks; ++kb) {
          ok = mbar_wait(full_bar(stage), phase, abort_flag, p.status, 3);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_src = smem_base + stage * kStageBytes, b_src = a_src + kABytes;
#pragma unroll
          for (int ks = 0; ks < kBK / kUmmaK; ++ks) {
            const uint64_t ad = make_smem_desc(a_src + ks * a_kstep, a_lbo, 1024u);
            const uint64_t bd = make_smem_desc(b_src + ks * b_kstep, b_lbo, 1024u);
            tc_mma_bf16(d_tmem, ad, bd, idesc, (kb > 0 || ks > 0) ? 1u : 0u);
          }
          tc_commit(empty_bar(stage));                        // frees the stage once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (t.k_blocks > 0) tc_commit(tfull_bar(acc));        // accumulator complete
        else mbar_arrive(tfull_bar(acc));                     // nothing to contract: the epilogue writes zeros
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------------------------------ epilogue warps
    const int lg = warp & 3;                                  // TMEM lane group this warp may read
    const int half = (warp - 2) >> 2;                         // which pair of 64-column chunks this warp drains
    uint8_t* my_stage_gen = smem_gen + kStages * kStageBytes + (warp - 2) * 4096;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int id = blockIdx.x; id < n_tiles && ok; id += gridDim.x) {
      const TileCoord t = decode_tile(p, id);
      const int r = lg * 32 + lane;                           // this thread's row of the tile
      // Per-row output base (element offset) and validity.
      long long row_off = -1;
      float scale = 1.f;
      if (p.token_m) {
        const int slot_row = t.m0 + r;
        if (p.op == kGemm1Relu || p.op == kDgrad2Mask) {
          if (slot_row < p.C) row_off = ((long long)t.e * p.C + slot_row) * p.ld_out;
        } else if (slot_row < p.kept[t.e]) {
          const int tok = p.token_of_slot[(long long)t.e * p.C + slot_row];
          row_off = (long long)tok * p.ld_out;
          if (p.op == kGemm2Combine) scale = p.gate[tok];
        }
      } else if (t.m0 + r < p.M) {
        row_off = ((long long)t.e * p.M + t.m0 + r) * p.ld_out;
      }
      // write-out assignment: instruction `it` covers rows it*4 + lane/8, 16-byte column (lane & 7)
      long long offs[8];
#pragma unroll
      for (int it = 0; it < 8; ++it) offs[it] = __shfl_sync(0xffffffffu, row_off, it * 4 + (lane >> 3));
      // ReLU mask of the first chunk, fetched while the accumulator is still being produced
      uint4 hm[8];
      if (p.op == kDgrad2Mask) {
        const int col = t.n0 + (2 * half) * 64 + (lane & 7) * 8;
#pragma unroll
        for (int it = 0; it < 8; ++it)
          hm[it] = (offs[it] >= 0 && col < p.N) ? *reinterpret_cast<const uint4*>(p.mask_src + offs[it] + col)
                                                : make_uint4(0, 0, 0, 0);
      }
      ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status, 4);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_addr = tmem_base + ((uint32_t)(lg * 32) << 16) + (uint32_t)acc * kBN;
#pragma unroll 1
      for (int cc = 0; cc < 2; ++cc) {
        const int c = 2 * half + cc;
        uint32_t v[64];
        if (t.k_blocks > 0) {
          tc_ld32(t_addr + c * 64, v);
          tc_ld32(t_addr + c * 64 + 32, v + 32);
          tc_wait_ld();
        } else {
#pragma unroll
          for (int i = 0; i < 64; ++i) v[i] = 0u;
        }
        if (cc == 1) {                                        // this warp's share is read: hand it back to the MMA warp
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(tempty_bar(acc));
        }
        // float32 -> epilogue -> bfloat16, staged row-wise with a 16-byte XOR swizzle (conflict-free both ways)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          uint32_t w[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            float a = __uint_as_float(v[j * 8 + 2 * q]) * scale;
            float b = __uint_as_float(v[j * 8 + 2 * q + 1]) * scale;
            if (p.op == kGemm1Relu) { a = fmaxf(a, 0.f); b = fmaxf(b, 0.f); }
            __nv_bfloat162 h2 = __floats2bfloat162_rn(a, b);
            w[q] = *reinterpret_cast<uint32_t*>(&h2);
          }
          *reinterpret_cast<uint4*>(my_stage_gen + lane * 128 + ((j ^ (lane & 7)) << 4)) =
              make_uint4(w[0], w[1], w[2], w[3]);
        }
        __syncwarp();
        // coalesced write-out: each instruction covers 4 rows x 128 bytes
        const int col = t.n0 + c * 64 + (lane & 7) * 8;
        uint4 val[8];
#pragma unroll
        for (int it = 0; it < 8; ++it) {
          const int rr = it * 4 + (lane >> 3);
          val[it] = *reinterpret_cast<const uint4*>(my_stage_gen + rr * 128 + (((lane & 7) ^ (rr & 7)) << 4));
        }
        if (p.op == kDgrad2Mask) {                            // ReLU'(u) = [u > 0], read from the saved activation
          const __nv_bfloat16 zero = __float2bfloat16(0.f);
#pragma unroll
          for (int it = 0; it < 8; ++it) {
            const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&hm[it]);
            __nv_bfloat162* vp = reinterpret_cast<__nv_bfloat162*>(&val[it]);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              if (!(__low2float(hp[q]) > 0.f)) vp[q].x = zero;
              if (!(__high2float(hp[q]) > 0.f)) vp[q].y = zero;
            }
          }
          if (cc == 0) {                                      // fetch the second chunk's mask behind this chunk's stores
            const int col2 = col + 64;
#pragma unroll
            for (int it = 0; it < 8; ++it)
              hm[it] = (offs[it] >= 0 && col2 < p.N) ? *reinterpret_cast<const uint4*>(p.mask_src + offs[it] + col2)
                                                     : make_uint4(0, 0, 0, 0);
          }
        }
        if (col < p.N) {
#pragma unroll
          for (int it = 0; it < 8; ++it)
            if (offs[it] >= 0) *reinterpret_cast<uint4*>(p.out + offs[it] + col) = val[it];
        }
        __syncwarp();
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  // ---------------------------------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

}  // namespace

// bf16 tensor [E][rows][cols] (cols contiguous), box {64 cols, box_rows rows, 1}, 128-byte swizzle, zero OOB fill.
int tc::make_map(CUtensorMap* tm, const void* base, long long E, long long rows, long long cols, int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return SWITCH_MOE_CUDA_ERROR;
  cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)E};
  cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)cols * (cuuint64_t)rows * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SWITCH_MOE_OK : SWITCH_MOE_CUDA_ERROR;
}


int launch_tc_gemm(GemmOp op, const Shape& s, const Plan& p, const GemmArgs& a, void* ws, cudaStream_t st) {
  int dev = 0, sm_count = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SWITCH_MOE_CUDA_ERROR;
  if (cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return SWITCH_MOE_CUDA_ERROR;
  if (cudaFuncSetAttribute(grouped_gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) !=
      cudaSuccess)
    return SWITCH_MOE_CUDA_ERROR;
  const void* xd = ws_ptr<char>(ws, p.xd);
  const void* h = ws_ptr<char>(ws, p.h);
  const void* dyd = ws_ptr<char>(ws, p.dyd);
  const void* dh = ws_ptr<char>(ws, p.dh);

  TcParams q{};
  q.op = (int)op;
  q.C = s.C; q.E = s.E;
  q.tile_expert = ws_ptr<int>(ws, p.tile_expert);
  q.tile_row0 = ws_ptr<int>(ws, p.tile_row0);
  q.kept = ws_ptr<int>(ws, p.kept);
  q.token_of_slot = ws_ptr<int>(ws, p.token_of_slot);
  q.gate = ws_ptr<float>(ws, p.gate);
  q.status = ws_ptr<int>(ws, p.status);
  CUtensorMap tmA, tmB;
  int rc = SWITCH_MOE_OK, rc2 = SWITCH_MOE_OK;
  int K = 0;
  switch (op) {
    case kGemm1Relu:       // A = X_d [E,C,d] K-major; B = W_in [E,d,f]: k rows, n contiguous -> MN-major
      q.token_m = 1; q.a_mn_major = 0; q.b_mn_major = 1; q.N = s.f; K = s.d;
      rc = make_map(&tmA, xd, s.E, s.C, s.d, kTileM); rc2 = make_map(&tmB, a.W_in, s.E, s.d, s.f, 64);
      q.out = ws_ptr<__nv_bfloat16>(ws, p.h); q.ld_out = s.f; break;
    case kGemm2Combine:    // A = H [E,C,f] K-major; B = W_out [E,f,d] MN-major
      q.token_m = 1; q.a_mn_major = 0; q.b_mn_major = 1; q.N = s.d; K = s.f;
      rc = make_map(&tmA, h, s.E, s.C, s.f, kTileM); rc2 = make_map(&tmB, a.W_out, s.E, s.f, s.d, 64);
      q.out = static_cast<__nv_bfloat16*>(a.y); q.ld_out = s.d; break;
    case kDgrad2Mask:      // A = dY_d [E,C,d] K-major; B = W_out [E,f,d] as (n = f rows, k = d contiguous) -> K-major
      q.token_m = 1; q.a_mn_major = 0; q.b_mn_major = 0; q.N = s.f; K = s.d;
      rc = make_map(&tmA, dyd, s.E, s.C, s.d, kTileM); rc2 = make_map(&tmB, a.W_out, s.E, s.f, s.d, kBN);
      q.out = ws_ptr<__nv_bfloat16>(ws, p.dh); q.mask_src = ws_ptr<__nv_bfloat16>(ws, p.h); q.ld_out = s.f; break;
    case kDgrad1Scatter:   // A = dH [E,C,f] K-major; B = W_in [E,d,f] as (n = d rows, k = f contiguous) -> K-major
      q.token_m = 1; q.a_mn_major = 0; q.b_mn_major = 0; q.N = s.d; K = s.f;
      rc = make_map(&tmA, dh, s.E, s.C, s.f, kTileM); rc2 = make_map(&tmB, a.W_in, s.E, s.d, s.f, kBN);
      q.out = static_cast<__nv_bfloat16*>(a.dx); q.ld_out = s.d; break;
    case kWgrad2:          // A = H [E,C,f] as (k = slot rows, m = f contiguous) MN-major; B = dY_d [E,C,d] MN-major
      q.token_m = 0; q.a_mn_major = 1; q.b_mn_major = 1; q.M = s.f; q.N = s.d;
      rc = make_map(&tmA, h, s.E, s.C, s.f, 64); rc2 = make_map(&tmB, dyd, s.E, s.C, s.d, 64);
      q.out = static_cast<__nv_bfloat16*>(a.dW_out); q.ld_out = s.d; break;
    case kWgrad1:          // A = X_d [E,C,d] MN-major; B = dH [E,C,f] MN-major
      q.token_m = 0; q.a_mn_major = 1; q.b_mn_major = 1; q.M = s.d; q.N = s.f;
      rc = make_map(&tmA, xd, s.E, s.C, s.d, 64); rc2 = make_map(&tmB, dh, s.E, s.C, s.f, 64);
      q.out = static_cast<__nv_bfloat16*>(a.dW_in); q.ld_out = s.f; break;
    default: return SWITCH_MOE_INVALID_ARGUMENT;
  }
  if (rc != SWITCH_MOE_OK || rc2 != SWITCH_MOE_OK) return SWITCH_MOE_CUDA_ERROR;
  q.n_ntiles = (q.N + kBN - 1) / kBN;
  q.n_mtiles_fixed = q.token_m ? 0 : (q.M + kTileM - 1) / kTileM;
  q.k_blocks_fixed = q.token_m ? K / kBK : 0;
  const int grid = sm_count > 0 ? sm_count : 148;
  launch_k(grouped_gemm_tc_kernel, dim3(grid), dim3(kThreads), kSmemBytes, st, tmA, tmB, q);
  return launch_status();
}

}  // namespace swmoe
