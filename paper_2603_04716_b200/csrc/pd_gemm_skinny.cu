// Decode-mode projections: Y[B, N] = X[B, K] * W[N, K]^T for a small batch B.
//
// With one token per sequence the projections stream every weight once per step and are
// HBM-bound, so the job is to keep all SMs loading weights.  The roles of the operands are
// swapped with respect to the prefill GEMM: a tile is 128 weight rows (the M side of
// tcgen05.mma, so no tensor-core rows are wasted on padding) by the whole batch (the N side,
// rounded up to 16/32/64/128/256), and the K range is split across blocks until every SM has
// work (two blocks per SM, so one block's epilogue overlaps another's main loop).  A block accumulates its K slice in tensor memory and adds it into
// an fp32 [B, N] buffer (red.global.add, L2-resident; plain stores when K is not split).
// Small row-wise kernels then apply the layer's fused operations to the fp32 sums: RoPE and the
// KV-cache append, residual add with the following RMSNorm, SwiGLU, residual add.
//
// The chain of a decode layer is launched with programmatic serialization.  Weights do not depend on
// earlier kernels, so a block fills its whole TMA ring with weight tiles BEFORE it waits for the previous
// kernel; only the activation tiles and the accumulation into the fp32 buffer come after the wait.  The
// weight stream therefore keeps running across kernel boundaries.  (Pulling further weight tiles into L2
// before the wait was measured too: no gain, the ring already covers the gap.)  The fp32 buffer of a K-split
// projection is cleared by a row-wise kernel earlier in the chain instead of a memset.
#include <cstdlib>

#include "pd_common.cuh"
#include "pd_ptx.cuh"

namespace pd {
namespace {

constexpr int SK_BM = 128;  // weight rows per tile
constexpr int SK_BK = 64;
constexpr int SK_THREADS = 192;

template <int BNB, int MT>
struct SkinnyCfg {
  static constexpr int W_BYTES = MT * SK_BM * SK_BK * 2;
  static constexpr int X_BYTES = BNB * SK_BK * 2;
  static constexpr int STAGE_BYTES = W_BYTES + ((X_BYTES + 1023) / 1024) * 1024;  // keep tiles 1024-byte aligned
  static constexpr int STAGES = MT == 2 ? (BNB >= 256 ? 3 : 4) : (BNB >= 256 ? 2 : (BNB >= 128 ? 3 : 4));
  static constexpr int ACC_COLS = BNB < 32 ? 32 : BNB;   // tensor-memory columns per accumulator
  static constexpr int TMEM_COLS = MT * ACC_COLS;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 128;
  static constexpr int BLOCKS_PER_SM = MT == 2 ? 1 : 2;
};

struct SkinnyDev {
  float* acc;  // [B, N] fp32
  int batch, n, k_blocks, splits, tiles_n;
  int* err_word;
  const float* scale_x;  // FP8 operands: per-row scales of X [B] and of W [N]
  const float* scale_w;
  bf16* swiglu_out;      // not NULL (only with splits == 1): W is the gate/up matrix, write silu(gate) * up here
  int swiglu_ld;         // its row pitch (= number of SwiGLU features)
};

// One chunk of CH accumulator columns (batch rows b0 ..) of the thread that owns output feature n -> the fp32
// buffer: vector store when K is not split, vector reduction otherwise; FP8 sums are scaled on the way.
template <int CH, bool F8>
__device__ __forceinline__ void skinny_store_chunk(const SkinnyDev& p, uint32_t (&v)[32], int n, int lane, int b0) {
  // 4 x 4 transposes across groups of four lanes: afterwards lane 4q + r holds, for batch column
  // c0 + 4m + r, the four consecutive features 4q .. 4q + 3 in v[4m .. 4m + 3], i.e. 16 contiguous bytes
  // of the output row, so one vector store / vector reduction replaces four scalar ones (scalar fp32
  // reductions into L2 were measured four times slower per byte).
  const int r4 = lane & 3;
#pragma unroll
  for (int m = 0; m < CH; m += 4) {
#pragma unroll
    for (int s2 = 0; s2 < 4; s2 += 2) {
      const uint32_t send = (r4 & 1) ? v[m + s2] : v[m + s2 + 1];
      const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, 1);
      if (r4 & 1) v[m + s2] = recv; else v[m + s2 + 1] = recv;
    }
#pragma unroll
    for (int s2 = 0; s2 < 2; ++s2) {
      const uint32_t send = (r4 & 2) ? v[m + s2] : v[m + s2 + 2];
      const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, 2);
      if (r4 & 2) v[m + s2] = recv; else v[m + s2 + 2] = recv;
    }
  }
  const int n4 = n - r4;  // first of this lane's four features (n is a multiple of 4 per group of lanes)
  if (n4 < p.n) {
    float4 sw4 = make_float4(1.f, 1.f, 1.f, 1.f);
    if constexpr (F8) sw4 = __ldg(reinterpret_cast<const float4*>(p.scale_w + n4));
#pragma unroll
    for (int m = 0; m < CH; m += 4) {
      const int b = b0 + m + r4;
      if (b < p.batch) {
        if constexpr (F8) {
          const float sx = __ldg(p.scale_x + b);
          v[m] = __float_as_uint(__uint_as_float(v[m]) * (sx * sw4.x));
          v[m + 1] = __float_as_uint(__uint_as_float(v[m + 1]) * (sx * sw4.y));
          v[m + 2] = __float_as_uint(__uint_as_float(v[m + 2]) * (sx * sw4.z));
          v[m + 3] = __float_as_uint(__uint_as_float(v[m + 3]) * (sx * sw4.w));
        }
        float* dst = p.acc + static_cast<size_t>(b) * p.n + n4;
        if (p.splits > 1) ptx::red_add_v4_f32(dst, v[m], v[m + 1], v[m + 2], v[m + 3]);
        else *reinterpret_cast<uint4*>(dst) = make_uint4(v[m], v[m + 1], v[m + 2], v[m + 3]);
      }
    }
  }
}

// Named barrier 1 over the 128 epilogue threads (warps 2-5) and its AND-reduction form.
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ bool epi_all(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 p, %1, 0;\n\t"
      "bar.red.and.pred q, 1, 128, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r) : "r"(static_cast<uint32_t>(pred)) : "memory");
  return r != 0;
}

// SwiGLU straight from the accumulator of an unsplit gate/up tile: its 128 weight rows are 64 gate rows followed by
// the 64 up rows of the same features, i.e. tensor-memory lanes r and r + 64, which belong to different warps.  The
// up warps pass their chunk through shared memory (the operand stages are idle by now; two buffers so one barrier
// per chunk suffices), the gate warps compute silu(gate) * up and store bf16: a warp writes 32 consecutive features
// of one batch row.  Executed by all four epilogue warps; `ok` is made uniform over them first.
template <int BNB, bool F8>
__device__ __forceinline__ void skinny_swiglu_tile(const SkinnyDev& p, uint32_t t_row, int tn, int tb, int lane_group,
                                                   int lane, float* xbuf, bool ok) {
  if (!epi_all(ok)) return;
  constexpr int CH = BNB < 32 ? BNB : 32;
  const int r = lane_group * 32 + lane;   // weight row inside the tile
  const int n = tn * SK_BM + r;
  const int f = tn * 64 + (r & 63);       // SwiGLU feature of this row
  float sw = 1.f;
  if constexpr (F8) sw = n < p.n ? __ldg(p.scale_w + n) : 0.f;
  int it = 0;
#pragma unroll 1
  for (int c0 = 0; c0 < BNB; c0 += CH, ++it) {
    const int b0 = tb * BNB + c0;
    if (b0 >= p.batch) break;  // uniform: the rest of the accumulator is padding
    uint32_t v[32];
    if constexpr (CH == 32) ptx::tmem_ld_32x32(t_row + c0, v);
    else ptx::tmem_ld_32x16(t_row + c0, v);
    ptx::tmem_ld_wait();
    if constexpr (F8) {
#pragma unroll
      for (int j = 0; j < CH; ++j)
        v[j] = __float_as_uint(__uint_as_float(v[j]) * (sw * (b0 + j < p.batch ? __ldg(p.scale_x + b0 + j) : 0.f)));
    }
    float* buf = xbuf + (it & 1) * (64 * 33);
    if (lane_group >= 2) {
#pragma unroll
      for (int j = 0; j < CH; ++j) buf[(r - 64) * 33 + j] = __uint_as_float(v[j]);
    }
    epi_sync();
    if (lane_group < 2 && n < p.n) {
#pragma unroll
      for (int j = 0; j < CH; ++j) {
        if (b0 + j < p.batch) {
          const float g = __uint_as_float(v[j]);
          const float u = buf[r * 33 + j];
          p.swiglu_out[static_cast<size_t>(b0 + j) * p.swiglu_ld + f] = __float2bfloat16(g / (1.f + __expf(-g)) * u);
        }
      }
    }
  }
}

// F8: both operands are E4M3 codes (a 128-byte shared-memory row then holds 128 K elements, one MMA covers 32)
// and every partial sum is multiplied by scale_x[b] * scale_w[n] on its way out.
template <int BNB, int MT, bool F8>
__global__ void __launch_bounds__(SK_THREADS)
gemm_skinny_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x, SkinnyDev p) {
  using Cfg = SkinnyCfg<BNB, MT>;
  constexpr int STAGES = Cfg::STAGES;
  constexpr int KE = F8 ? 2 * SK_BK : SK_BK;  // K elements per stage (128 bytes per row either way)
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * Cfg::STAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar0 = ptx::smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  const uint32_t acc_bar = bar0 + 8u * (2 * STAGES);

  // work unit: (batch tile, weight-row tile, K slice)
  int unit = blockIdx.x;
  const int split = unit % p.splits;
  unit /= p.splits;
  const int tn = unit % p.tiles_n;
  const int tb = unit / p.tiles_n;
  const int kb0 = static_cast<int>(static_cast<long long>(p.k_blocks) * split / p.splits);
  const int kb1 = static_cast<int>(static_cast<long long>(p.k_blocks) * (split + 1) / p.splits);

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    ptx::mbar_init(acc_bar, 1);
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmap_w);
    ptx::prefetch_tensormap(&tmap_x);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_slot), Cfg::TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  ptx::grid_launch_dependents();
  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      // ring prologue: weight tiles first (they depend on no earlier kernel), then the dependency wait,
      // then the activation tiles of the same stages
      const int pre = min(STAGES, kb1 - kb0);
      for (int i = 0; i < pre; ++i) {
        const uint32_t sw = smem_base + i * Cfg::STAGE_BYTES;
        ptx::mbar_arrive_expect_tx(full_bar(i), Cfg::W_BYTES + Cfg::X_BYTES);
        ptx::tma_load_2d(sw, &tmap_w, (kb0 + i) * KE, tn * (MT * SK_BM), full_bar(i));
      }
      ptx::grid_dependency_wait();
      for (int i = 0; i < pre; ++i) {
        const uint32_t sx = smem_base + i * Cfg::STAGE_BYTES + Cfg::W_BYTES;
        ptx::tma_load_2d(sx, &tmap_x, (kb0 + i) * KE, tb * BNB, full_bar(i));
      }
      if (pre == STAGES) phase = 1u;  // the ring has wrapped once
      else stage = pre;
      for (int kb = kb0 + pre; kb < kb1; ++kb) {
        if (!ptx::mbar_wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
        const uint32_t sw = smem_base + stage * Cfg::STAGE_BYTES;
        const uint32_t sx = sw + Cfg::W_BYTES;
        ptx::mbar_arrive_expect_tx(full_bar(stage), Cfg::W_BYTES + Cfg::X_BYTES);
        ptx::tma_load_2d(sw, &tmap_w, kb * KE, tn * (MT * SK_BM), full_bar(stage));  // box of MT * 128 rows
        ptx::tma_load_2d(sx, &tmap_x, kb * KE, tb * BNB, full_bar(stage));
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
      if (!ok) {
#pragma unroll 1
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let loads in flight land before shared memory is released
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = F8 ? ptx::umma_idesc_e4m3(SK_BM, BNB) : ptx::umma_idesc_bf16(SK_BM, BNB);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!ptx::mbar_wait_bounded(full_bar(stage), phase, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t sw = smem_base + stage * Cfg::STAGE_BYTES;
        const uint64_t dw = ptx::umma_desc_sw128(sw);
        const uint64_t dx = ptx::umma_desc_sw128(sw + Cfg::W_BYTES);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {  // 32 bytes along K per instruction
            const uint32_t accum = (kb > kb0 || kk > 0) ? 1u : 0u;
            if constexpr (F8)
              ptx::umma_f8(tmem_base + mt * Cfg::ACC_COLS, dw + mt * (SK_BM * 128 / 16) + 2u * kk, dx + 2u * kk, idesc, accum);
            else
              ptx::umma_bf16(tmem_base + mt * Cfg::ACC_COLS, dw + mt * (SK_BM * 128 / 16) + 2u * kk, dx + 2u * kk, idesc,
                             accum);
          }
        }
        ptx::umma_commit(empty_bar(stage));
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
      if (ok) ptx::umma_commit(acc_bar);
    }
  } else {
    const int lane_group = warp & 3;
    const bool ok = __all_sync(0xffffffffu, ptx::mbar_wait_bounded(acc_bar, 0u, abort_flag));
    ptx::grid_dependency_wait();  // (long since satisfied) orders the sums after the kernel that cleared the buffer
    if (MT == 1 && p.swiglu_out) {  // block-uniform
      ptx::tc_fence_after();
      skinny_swiglu_tile<BNB, F8>(p, tmem_base + (static_cast<uint32_t>(lane_group * 32) << 16), tn, tb, lane_group, lane,
                                  reinterpret_cast<float*>(smem_al), ok && kb1 > kb0);
    } else if (ok && kb1 > kb0) {
      ptx::tc_fence_after();
      constexpr int CH = BNB < 32 ? BNB : 32;
#pragma unroll 1
      for (int mt = 0; mt < MT; ++mt) {
      const int n = (tn * MT + mt) * SK_BM + lane_group * 32 + lane;  // output feature of this thread
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(lane_group * 32) << 16) + mt * Cfg::ACC_COLS;
#pragma unroll 1
      for (int c0 = 0; c0 < BNB; c0 += CH) {
        uint32_t v[32];
        if constexpr (CH == 32) ptx::tmem_ld_32x32(t_row + c0, v);
        else ptx::tmem_ld_32x16(t_row + c0, v);
        ptx::tmem_ld_wait();
        skinny_store_chunk<CH, F8>(p, v, n, lane, tb * BNB + c0);
      }
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0 && p.err_word) atomicExch(p.err_word, 1);
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
  }
}

// ------------------------------------------------------------- CTA-pair variant (batch tiles of 128 and 256)
// A cluster of two CTAs on one TPC owns 256 weight rows x the batch tile for one K slice.  Each CTA loads its own 128
// weight rows and HALF of the activation tile (a stage is 32 KB instead of 48 KB at a 256-wide batch tile, so three
// stages fit where two did and the activations cross from L2 once per pair), the even CTA issues
// tcgen05.mma.cta_group::2 (M = 256) for both, and each CTA adds its 128 output features into the fp32 buffer.
// Barrier protocol as in the prefill pair GEMM: `full` in the even CTA counts both CTAs' bytes, `empty` and the
// accumulator barrier are signalled in both CTAs by one multicast commit; a CTA waits only on its own barriers.
template <int BNB>
struct SkinnyPairCfg {
  static constexpr int W_BYTES = SK_BM * 128;
  static constexpr int XH_BYTES = (BNB / 2) * 128;
  static constexpr int STAGE_BYTES = W_BYTES + XH_BYTES;
  static constexpr int STAGES = BNB >= 256 ? 3 : 4;
  static constexpr int TMEM_COLS = BNB;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 128;
};

template <int BNB, bool F8>
__global__ void __launch_bounds__(SK_THREADS)
gemm_skinny_pair_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x, SkinnyDev p) {
  using Cfg = SkinnyPairCfg<BNB>;
  constexpr int STAGES = Cfg::STAGES;
  constexpr int KE = F8 ? 2 * SK_BK : SK_BK;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * Cfg::STAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();
  const uint32_t bar0 = ptx::smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  const uint32_t acc_bar = bar0 + 8u * (2 * STAGES);

  // work unit of the pair: (batch tile, pair of weight-row tiles, K slice)
  int unit = blockIdx.x >> 1;
  const int split = unit % p.splits;
  unit /= p.splits;
  const int pairs_n = p.tiles_n >> 1;
  const int tp = unit % pairs_n;
  const int tb = unit / pairs_n;
  const int tn = 2 * tp + static_cast<int>(rank);  // this CTA's weight-row tile
  const int kb0 = static_cast<int>(static_cast<long long>(p.k_blocks) * split / p.splits);
  const int kb1 = static_cast<int>(static_cast<long long>(p.k_blocks) * (split + 1) / p.splits);

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    ptx::mbar_init(acc_bar, 1);
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmap_w);
    ptx::prefetch_tensormap(&tmap_x);
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(ptx::smem_u32(tmem_slot), Cfg::TMEM_COLS);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  ptx::grid_launch_dependents();
  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      // ring prologue: weight tiles first (they depend on no earlier kernel), then the dependency wait, then the
      // activation half tiles of the same stages
      const int pre = min(STAGES, kb1 - kb0);
      for (int i = 0; i < pre; ++i) {
        if (rank == 0) ptx::mbar_arrive_expect_tx(full_bar(i), 2 * Cfg::STAGE_BYTES);
        ptx::tma_load_2d_pair(smem_base + i * Cfg::STAGE_BYTES, &tmap_w, (kb0 + i) * KE, tn * SK_BM,
                              ptx::map_to_cta(full_bar(i), 0));
      }
      ptx::grid_dependency_wait();
      for (int i = 0; i < pre; ++i)
        ptx::tma_load_2d_pair(smem_base + i * Cfg::STAGE_BYTES + Cfg::W_BYTES, &tmap_x, (kb0 + i) * KE,
                              tb * BNB + static_cast<int>(rank) * (BNB / 2), ptx::map_to_cta(full_bar(i), 0));
      if (pre == STAGES) phase = 1u;  // the ring has wrapped once
      else stage = pre;
      for (int kb = kb0 + pre; kb < kb1; ++kb) {
        if (!ptx::mbar_wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
        const uint32_t sw = smem_base + stage * Cfg::STAGE_BYTES;
        const uint32_t lead_full = ptx::map_to_cta(full_bar(stage), 0);
        if (rank == 0) ptx::mbar_arrive_expect_tx(full_bar(stage), 2 * Cfg::STAGE_BYTES);
        ptx::tma_load_2d_pair(sw, &tmap_w, kb * KE, tn * SK_BM, lead_full);
        ptx::tma_load_2d_pair(sw + Cfg::W_BYTES, &tmap_x, kb * KE, tb * BNB + static_cast<int>(rank) * (BNB / 2), lead_full);
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
      if (!ok) {
#pragma unroll 1
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let loads in flight land before shared memory is released
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = F8 ? ptx::umma_idesc_e4m3(2 * SK_BM, BNB) : ptx::umma_idesc_bf16(2 * SK_BM, BNB);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!ptx::mbar_wait_bounded(full_bar(stage), phase, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t sw = smem_base + stage * Cfg::STAGE_BYTES;
        const uint64_t dw = ptx::umma_desc_sw128(sw);
        const uint64_t dx = ptx::umma_desc_sw128(sw + Cfg::W_BYTES);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {  // 32 bytes along K per instruction
          const uint32_t accum = (kb > kb0 || kk > 0) ? 1u : 0u;
          if constexpr (F8) ptx::umma_f8_pair(tmem_base, dw + 2u * kk, dx + 2u * kk, idesc, accum);
          else ptx::umma_bf16_pair(tmem_base, dw + 2u * kk, dx + 2u * kk, idesc, accum);
        }
        ptx::umma_commit_pair(empty_bar(stage), 3);
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
      if (ok) ptx::umma_commit_pair(acc_bar, 3);
    }
  } else {
    const int lane_group = warp & 3;
    const bool ok = __all_sync(0xffffffffu, ptx::mbar_wait_bounded(acc_bar, 0u, abort_flag));
    ptx::grid_dependency_wait();  // (long since satisfied) orders the sums after the kernel that cleared the buffer
    if (p.swiglu_out) {  // block-uniform
      ptx::tc_fence_after();
      skinny_swiglu_tile<BNB, F8>(p, tmem_base + (static_cast<uint32_t>(lane_group * 32) << 16), tn, tb, lane_group, lane,
                                  reinterpret_cast<float*>(smem_al), ok && kb1 > kb0);
    } else if (ok && kb1 > kb0) {
      ptx::tc_fence_after();
      const int n = tn * SK_BM + lane_group * 32 + lane;  // output feature of this thread
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(lane_group * 32) << 16);
#pragma unroll 1
      for (int c0 = 0; c0 < BNB; c0 += 32) {
        if (tb * BNB + c0 >= p.batch) break;  // warp-uniform: the rest of the accumulator is padding
        uint32_t v[32];
        ptx::tmem_ld_32x32(t_row + c0, v);
        ptx::tmem_ld_wait();
        skinny_store_chunk<32, F8>(p, v, n, lane, tb * BNB + c0);
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();  // neither CTA leaves (or frees tensor memory) while its peer may still signal it
  if (*abort_flag && threadIdx.x == 0 && p.err_word) atomicExch(p.err_word, 1);
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(tmem_base, Cfg::TMEM_COLS);
  }
}

// K slices per (weight tile, batch tile) unit: fill the resident block slots, each block with at least 8 K-blocks.
int skinny_splits(int units, int k_blocks, int blocks_per_sm) {
  int splits = (blocks_per_sm * 148 + units / 2) / units;
  if (splits > k_blocks / 8) splits = k_blocks / 8;
  return splits < 1 ? 1 : splits;
}

int skinny_bnb(int batch) { return batch <= 16 ? 16 : batch <= 32 ? 32 : batch <= 64 ? 64 : batch <= 128 ? 128 : 256; }

template <int BNB, int MT, bool F8>
pd_status launch_skinny(const SkinnyGemmArgs& g, cudaStream_t stream) {
  using Cfg = SkinnyCfg<BNB, MT>;
  static PerDeviceInt smem_opt_in;
  auto kern = gemm_skinny_kernel<BNB, MT, F8>;
  PD_TRY(opt_in_smem(smem_opt_in, kern, Cfg::SMEM_BYTES));
  CUtensorMap tw, tx;
  if (F8) {
    PD_TRY(make_tmap_u8(&tw, g.w, g.n, g.k, g.k, MT * SK_BM));
    PD_TRY(make_tmap_u8(&tx, g.x, g.batch, g.k, g.ldx, BNB));
  } else {
    PD_TRY(make_tmap_bf16(&tw, g.w, g.n, g.k, g.k, MT * SK_BM));
    PD_TRY(make_tmap_bf16(&tx, g.x, g.batch, g.k, g.ldx, BNB));
  }
  SkinnyDev p{};
  p.scale_x = g.scale_x; p.scale_w = g.scale_w;
  p.acc = g.acc; p.batch = g.batch; p.n = g.n; p.k_blocks = g.k / (F8 ? 2 * SK_BK : SK_BK);
  p.tiles_n = (g.n + MT * SK_BM - 1) / (MT * SK_BM);
  const int tiles_b = (g.batch + BNB - 1) / BNB;
  const int units = p.tiles_n * tiles_b;
  const int splits = skinny_splits(units, p.k_blocks, Cfg::BLOCKS_PER_SM);  // (k_blocks already counts FP8 stages)
  p.splits = splits;
  p.err_word = g.err_word;
  if (g.swiglu_out) {
    if (splits != 1 || tiles_b != 1 || MT != 1 || g.n % SK_BM != 0) return PD_ERR_UNSUPPORTED_SHAPE;
    p.swiglu_out = g.swiglu_out; p.swiglu_ld = g.n / 2;
  }
  if (splits > 1 && !g.acc_zeroed)
    PD_CUDA_TRY(cudaMemsetAsync(g.acc, 0, static_cast<size_t>(g.batch) * g.n * sizeof(float), stream));
  PD_CUDA_TRY(launch_pdl(kern, dim3(units * splits), dim3(SK_THREADS), Cfg::SMEM_BYTES, stream, tw, tx, p));
  count_launch();
  return PD_OK;
}

// CTA-pair launch (cluster of two + programmatic serialization).  Same K-slice count as the single-CTA kernel
// would use, so the callers' decision which buffers need clearing does not depend on the path taken.
template <int BNB, bool F8>
pd_status launch_skinny_pair(const SkinnyGemmArgs& g, cudaStream_t stream) {
  using Cfg = SkinnyPairCfg<BNB>;
  static PerDeviceInt usable_memo;  // per device: -1 unknown, 0 clusters of two cannot be placed, 1 fine
  int usable = usable_memo.get();
  auto kern = gemm_skinny_pair_kernel<BNB, F8>;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.blockDim = dim3(SK_THREADS);
  cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
  cfg.stream = stream;
  cfg.attrs = attr;
  if (usable < 0) {
    usable = 0;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES) == cudaSuccess) {
      cfg.gridDim = dim3(2);
      cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) == cudaSuccess && n > 0) usable = 1;
      else cudaGetLastError();
    }
    usable_memo.set(usable);
  }
  if (!usable) return PD_ERR_UNSUPPORTED_SHAPE;
  CUtensorMap tw, tx;
  if (F8) {
    PD_TRY(make_tmap_u8(&tw, g.w, g.n, g.k, g.k, SK_BM));
    PD_TRY(make_tmap_u8(&tx, g.x, g.batch, g.k, g.ldx, BNB / 2));
  } else {
    PD_TRY(make_tmap_bf16(&tw, g.w, g.n, g.k, g.k, SK_BM));
    PD_TRY(make_tmap_bf16(&tx, g.x, g.batch, g.k, g.ldx, BNB / 2));
  }
  SkinnyDev p{};
  p.scale_x = g.scale_x; p.scale_w = g.scale_w;
  p.acc = g.acc; p.batch = g.batch; p.n = g.n; p.k_blocks = g.k / (F8 ? 2 * SK_BK : SK_BK);
  p.tiles_n = g.n / SK_BM;
  const int tiles_b = (g.batch + BNB - 1) / BNB;
  p.splits = skinny_splits(p.tiles_n * tiles_b, p.k_blocks, 2);
  p.err_word = g.err_word;
  if (g.swiglu_out) {
    if (p.splits != 1 || tiles_b != 1) return PD_ERR_UNSUPPORTED_SHAPE;
    p.swiglu_out = g.swiglu_out; p.swiglu_ld = g.n / 2;
  }
  if (p.splits > 1 && !g.acc_zeroed)
    PD_CUDA_TRY(cudaMemsetAsync(g.acc, 0, static_cast<size_t>(g.batch) * g.n * sizeof(float), stream));
  cfg.gridDim = dim3(static_cast<unsigned>(2 * (p.tiles_n / 2) * tiles_b * p.splits));
  cfg.numAttrs = pdl_enabled() ? 2 : 1;
  PD_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tw, tx, p));
  count_launch();
  return PD_OK;
}

// Batches above 64 (FP8: above 128, where it was measured to pay) run on the CTA-pair kernel; PD_SKINNY_PAIRS=0 in
// the environment keeps them on the single-CTA kernel (for A/B timing).  Measured per 8B layer, bf16: 258 -> 243 us
// at B = 96, 298 -> 277 at 128, 400 -> 374 at 192, 480 -> 463 at 256.
static int skinny_pair_mode() {
  static const int mode = [] {
    const char* v = std::getenv("PD_SKINNY_PAIRS");
    return (v && v[0] == '0') ? 0 : 1;
  }();
  return mode;
}

// ------------------------------------------------------------ row-wise epilogues
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  uint4 o;
  o.x = ptx::pack_bf16(f[0], f[1]);
  o.y = ptx::pack_bf16(f[2], f[3]);
  o.z = ptx::pack_bf16(f[4], f[5]);
  o.w = ptx::pack_bf16(f[6], f[7]);
  return o;
}
__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  f[0] = ptx::bf16_lo(v.x); f[1] = ptx::bf16_hi(v.x);
  f[2] = ptx::bf16_lo(v.y); f[3] = ptx::bf16_hi(v.y);
  f[4] = ptx::bf16_lo(v.z); f[5] = ptx::bf16_hi(v.z);
  f[6] = ptx::bf16_lo(v.w); f[7] = ptx::bf16_hi(v.w);
}
__device__ __forceinline__ void load8(const float* p, float (&f)[8]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  const float4 b = *reinterpret_cast<const float4*>(p + 4);
  f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}

// Clears n floats at p with the threads of one block (p 16-byte aligned, n a multiple of 4).
__device__ __forceinline__ void zero_row(float* p, int n) {
  float4* q = reinterpret_cast<float4*>(p);
  for (int i = threadIdx.x; i < n / 4; i += blockDim.x) q[i] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// RoPE + KV append for one decode token per block: acc[b, Nqkv] -> q (bf16, in the qkv buffer), cache.
__global__ void __launch_bounds__(128) skinny_rope_kv_kernel(const float* __restrict__ acc, bf16* qkv, RopeEpilogue rp,
                                                             int* err_word, float* zero_ptr, int zero_cols) {
  const int b = blockIdx.x;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  if (zero_ptr) zero_row(zero_ptr + static_cast<size_t>(b) * zero_cols, zero_cols);
  const int pos = rp.kv_len[b], slot = b;
  if (pos < 0 || pos >= rp.len_cap || pos >= rp.max_pos || slot >= rp.batch_cap) {
    if (threadIdx.x == 0 && err_word) atomicExch(err_word, 2);
    return;
  }
  const int hd = rp.head_dim, half = hd / 2, per_head = half / 8;
  const int n_heads = rp.n_q_heads + 2 * rp.n_kv_heads;
  const int n_qkv = n_heads * hd;
  const float* row = acc + static_cast<size_t>(b) * n_qkv;
  const float2* tab = rp.rope_tab + static_cast<size_t>(pos) * half;
  for (int w = threadIdx.x; w < n_heads * per_head; w += blockDim.x) {
    const int h = w / per_head, i0 = (w - h * per_head) * 8;
    float lo[8], hi[8];
    load8(row + h * hd + i0, lo);
    load8(row + h * hd + half + i0, hi);
    bf16* dst;
    if (h < rp.n_q_heads) {
      dst = qkv + static_cast<size_t>(b) * n_qkv + h * hd;
    } else if (h < rp.n_q_heads + rp.n_kv_heads) {
      dst = rp.k_cache + ((static_cast<size_t>(slot) * rp.n_kv_heads + (h - rp.n_q_heads)) * rp.len_cap + pos) * hd;
    } else {
      dst = rp.v_cache +
            ((static_cast<size_t>(slot) * rp.n_kv_heads + (h - rp.n_q_heads - rp.n_kv_heads)) * rp.len_cap + pos) * hd;
    }
    if (h < rp.n_q_heads + rp.n_kv_heads) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float2 cs = tab[i0 + e];
        const float a = lo[e], c = hi[e];
        lo[e] = a * cs.x - c * cs.y;
        hi[e] = c * cs.x + a * cs.y;
      }
    }
    *reinterpret_cast<uint4*>(dst + i0) = pack8(lo);
    *reinterpret_cast<uint4*>(dst + half + i0) = pack8(hi);
  }
}

// h = x + acc (stored bf16); optionally n = RMSNorm(h) * gain computed from the stored h.
constexpr int RES_THREADS = 256;
constexpr int RES_MAX_CHUNKS = 8;
template <bool NORM>
__global__ void __launch_bounds__(RES_THREADS) skinny_residual_kernel(const float* __restrict__ acc,
                                                                       const bf16* __restrict__ x, bf16* h,
                                                                       const bf16* __restrict__ gain, bf16* n, int d,
                                                                       float eps, float* zero_ptr, int zero_cols,
                                                                       uint8_t* __restrict__ q_out,
                                                                       float* __restrict__ s_out) {
  const int b = blockIdx.x;
  const int chunks = d / 8;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  if (zero_ptr) zero_row(zero_ptr + static_cast<size_t>(b) * zero_cols, zero_cols);
  uint4 hv[RES_MAX_CHUNKS];
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < RES_MAX_CHUNKS; ++i) {
    const int c = threadIdx.x + i * RES_THREADS;
    if (c < chunks) {
      float f[8], r[8];
      load8(acc + static_cast<size_t>(b) * d + c * 8, f);
      unpack8(*reinterpret_cast<const uint4*>(x + static_cast<size_t>(b) * d + c * 8), r);
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] += r[e];
      hv[i] = pack8(f);
      *reinterpret_cast<uint4*>(h + static_cast<size_t>(b) * d + c * 8) = hv[i];
      if (NORM) {
        unpack8(hv[i], f);  // the norm sees the stored (rounded) residual stream
#pragma unroll
        for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
      }
    }
  }
  if constexpr (NORM) {
  __shared__ float red[RES_THREADS / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < RES_THREADS / 32; ++w) tot += red[w];
  const float scale = rsqrtf(tot / static_cast<float>(d) + eps);
  float amax = 0.f;
#pragma unroll
  for (int i = 0; i < RES_MAX_CHUNKS; ++i) {
    const int c = threadIdx.x + i * RES_THREADS;
    if (c < chunks) {
      float f[8], g[8];
      unpack8(hv[i], f);
      unpack8(reinterpret_cast<const uint4*>(gain)[c], g);
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] = f[e] * scale * g[e];
      hv[i] = pack8(f);
      *reinterpret_cast<uint4*>(n + static_cast<size_t>(b) * d + c * 8) = hv[i];
      if (q_out) {
        unpack8(hv[i], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(f[e]));
      }
    }
  }
  if (q_out) {  // block-uniform: E4M3 codes and scale of the stored n, as the row quantiser would produce them
    __syncthreads();
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
    __syncthreads();
    float mx = 0.f;
#pragma unroll
    for (int w = 0; w < RES_THREADS / 32; ++w) mx = fmaxf(mx, red[w]);
    const float qs = mx > 0.f ? __fdiv_rn(mx, 448.f) : 1.f;
    if (threadIdx.x == 0) s_out[b] = qs;
#pragma unroll
    for (int i = 0; i < RES_MAX_CHUNKS; ++i) {
      const int c = threadIdx.x + i * RES_THREADS;
      if (c < chunks) {
        float f[8];
        unpack8(hv[i], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) f[e] = __fdiv_rn(f[e], qs);
        uint2 o;
        o.x = ptx::cvt_e4m3x2(f[0], f[1]) | (ptx::cvt_e4m3x2(f[2], f[3]) << 16);
        o.y = ptx::cvt_e4m3x2(f[4], f[5]) | (ptx::cvt_e4m3x2(f[6], f[7]) << 16);
        *reinterpret_cast<uint2*>(q_out + static_cast<size_t>(b) * d + c * 8) = o;
      }
    }
  }
  }  // NORM
}

// a[b, f] = silu(gate) * up with the weight rows interleaved 64 gate / 64 up.
__global__ void __launch_bounds__(256) skinny_swiglu_kernel(const float* __restrict__ acc, bf16* __restrict__ out,
                                                             int rows, int f, float* zero_ptr, int zero_cols) {
  const int chunks_per_row = f / 8;
  const size_t total = static_cast<size_t>(rows) * chunks_per_row;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  if (zero_ptr) {
    float4* q = reinterpret_cast<float4*>(zero_ptr);
    const size_t quads = static_cast<size_t>(rows) * zero_cols / 4;
    for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < quads;
         i += static_cast<size_t>(gridDim.x) * blockDim.x)
      q[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (size_t idx = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; idx < total;
       idx += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const size_t r = idx / chunks_per_row;
    const int c = static_cast<int>(idx - r * chunks_per_row);
    const int f0 = c * 8;
    const float* base = acc + r * (2 * static_cast<size_t>(f)) + (f0 >> 6) * 128 + (f0 & 63);
    float g[8], u[8];
    load8(base, g);
    load8(base + 64, u);
#pragma unroll
    for (int e = 0; e < 8; ++e) g[e] = g[e] / (1.f + __expf(-g[e])) * u[e];
    *reinterpret_cast<uint4*>(out + r * f + f0) = pack8(g);
  }
}

}  // namespace

bool gemm_skinny_fuses_swiglu(int batch, int n, int k, bool fp8) {
  static const bool off = [] { const char* v = std::getenv("PD_FUSE_SWIGLU"); return v && v[0] == '0'; }();
  return !off && batch <= 256 && n % SK_BM == 0 && gemm_skinny_splits(batch, n, k, fp8) == 1;
}

int gemm_skinny_splits(int batch, int n, int k, bool fp8) {
  const int bnb = skinny_bnb(batch);
  const int units = ((n + SK_BM - 1) / SK_BM) * ((batch + bnb - 1) / bnb);
  return skinny_splits(units, k / (fp8 ? 2 * SK_BK : SK_BK), 2);
}

pd_status gemm_skinny(const SkinnyGemmArgs& g, cudaStream_t stream) {
  if (!g.x || !g.w || !g.acc || g.batch <= 0 || g.n <= 0 || g.k <= 0) return PD_ERR_INVALID_ARG;
  if (g.fp8 && (!g.scale_x || !g.scale_w)) return PD_ERR_INVALID_ARG;
  if (g.batch > (g.fp8 ? 128 : 64) && g.batch <= 256 && g.n % (2 * SK_BM) == 0 && g.k % (g.fp8 ? 2 * SK_BK : SK_BK) == 0 &&
      g.ldx % (g.fp8 ? 16 : 8) == 0 && skinny_pair_mode()) {
    pd_status st;
    if (g.batch <= 128) st = g.fp8 ? launch_skinny_pair<128, true>(g, stream) : launch_skinny_pair<128, false>(g, stream);
    else st = g.fp8 ? launch_skinny_pair<256, true>(g, stream) : launch_skinny_pair<256, false>(g, stream);
    if (st != PD_ERR_UNSUPPORTED_SHAPE) return st;  // (clusters of two could not be placed: single-CTA kernel)
  }
  if (g.fp8) {
    if (g.k % (2 * SK_BK) != 0 || g.n % 4 != 0 || g.ldx % 16 != 0) return PD_ERR_UNSUPPORTED_SHAPE;
    if (g.batch <= 16) return launch_skinny<16, 1, true>(g, stream);
    if (g.batch <= 32) return launch_skinny<32, 1, true>(g, stream);
    if (g.batch <= 64) return launch_skinny<64, 1, true>(g, stream);
    if (g.batch <= 128) return launch_skinny<128, 1, true>(g, stream);
    return launch_skinny<256, 1, true>(g, stream);
  }
  if (g.k % SK_BK != 0 || g.n % 4 != 0 || g.ldx % 8 != 0) return PD_ERR_UNSUPPORTED_SHAPE;
  if (g.batch <= 16) return launch_skinny<16, 1, false>(g, stream);
  if (g.batch <= 32) return launch_skinny<32, 1, false>(g, stream);
  if (g.batch <= 64) return launch_skinny<64, 1, false>(g, stream);
  // (two weight sub-tiles per block, MT = 2, measured 10-20 % slower at B = 128..256: one block per SM
  // loses the overlap of one block's epilogue with another's main loop)
  if (g.batch <= 128) return launch_skinny<128, 1, false>(g, stream);
  return launch_skinny<256, 1, false>(g, stream);
}

pd_status launch_skinny_rope_kv(const float* acc, bf16* qkv, const RopeEpilogue& rp, int batch, int* err_word,
                                float* zero_ptr, int zero_cols, cudaStream_t s) {
  if (zero_ptr && zero_cols % 4 != 0) return PD_ERR_UNSUPPORTED_SHAPE;
  PD_CUDA_TRY(launch_pdl(skinny_rope_kv_kernel, dim3(batch), dim3(128), 0, s, acc, qkv, rp, err_word, zero_ptr, zero_cols));
  count_launch();
  return PD_OK;
}

pd_status launch_skinny_residual(const float* acc, const bf16* x, bf16* h, const bf16* gain, bf16* n, int batch, int d,
                                 float eps, float* zero_ptr, int zero_cols, cudaStream_t s, uint8_t* q_out, float* s_out) {
  if (d % 8 != 0 || d > RES_THREADS * RES_MAX_CHUNKS * 8 || (q_out && (!s_out || !n))) return PD_ERR_UNSUPPORTED_SHAPE;
  if (zero_ptr && zero_cols % 4 != 0) return PD_ERR_UNSUPPORTED_SHAPE;
  const bf16* no_gain = nullptr;
  bf16* no_out = nullptr;
  if (n)
    PD_CUDA_TRY(launch_pdl(skinny_residual_kernel<true>, dim3(batch), dim3(RES_THREADS), 0, s, acc, x, h, gain, n, d, eps,
                           zero_ptr, zero_cols, q_out, s_out));
  else
    PD_CUDA_TRY(launch_pdl(skinny_residual_kernel<false>, dim3(batch), dim3(RES_THREADS), 0, s, acc, x, h, no_gain, no_out,
                           d, eps, zero_ptr, zero_cols, q_out, s_out));
  count_launch();
  return PD_OK;
}

pd_status launch_skinny_swiglu(const float* acc, bf16* out, int batch, int f, float* zero_ptr, int zero_cols,
                               cudaStream_t s) {
  if (zero_ptr && zero_cols % 4 != 0) return PD_ERR_UNSUPPORTED_SHAPE;
  const size_t total = static_cast<size_t>(batch) * (f / 8);
  size_t blocks = (total + 255) / 256;
  if (blocks > 148 * 4) blocks = 148 * 4;  // all resident beside the projection blocks they wait for
  PD_CUDA_TRY(launch_pdl(skinny_swiglu_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, s, acc, out, batch, f,
                         zero_ptr, zero_cols));
  count_launch();
  return PD_OK;
}

}  // namespace pd
