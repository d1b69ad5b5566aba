// FP8 (E4M3) GEMM with block-wise scales, and the two quantisers that produce its operands.
//
// Reading of "FP8 deployment" for checkpoints that carry one scale per block (weight_block_size [128, 128]):
//   * W[N, K]: one fp32 scale per 128 x 128 block, scale = max|block| / 448, code = E4M3(w / scale);
//   * X[M, K]: one fp32 scale per row and group of 128 consecutive K elements, computed the same way;
//   * C[m, n] = sum over K blocks kb of ( sum_{k in kb} dec(qx[m, k]) dec(qw[n, k]) ) * sx[m, kb] * sw[n / 128, kb].
// The tensor cores sum the codes' products of ONE K block (128 elements = one shared-memory stage = four
// tcgen05.mma kind::f8f6f4 instructions of K = 32) into a tensor-memory accumulator that starts from zero;
// eight warps then read that accumulator, multiply it by the two scales and add it to fp32 sums they keep in registers
// (half an output row per thread: 64 columns, as packed f32x2 FMAs), while the products of the next K block run into
// the second accumulator.  Tile 128 x 128; the grid is persistent (one block per SM walks the tiles row by row of
// tiles, so that the blocks of a wave share their rows of A and the whole of B in L2), and barrier phases and the
// accumulator turn run on one K-block counter that continues across tiles.
//   warp 0: TMA producer (one lane), warp 1: MMA issuer (one lane), warps 2-9: scaled accumulation and the store
//   (warps 2-5 columns 0-63, warps 6-9 columns 64-127 of the tensor-memory lanes their number allows them to read).
// Every wait is wall-clock bounded and leaves through the common teardown.
#include "pd_common.cuh"
#include "pd_ptx.cuh"

namespace pd {
namespace {

constexpr int FB_TILE = 128;       // rows and columns of an output tile, and K elements per block (128 bytes per row)
constexpr int FB_THREADS = 320;
constexpr int FB_STAGES = 6;
constexpr int FB_OPERAND_BYTES = FB_TILE * 128;          // 128 rows of 128 one-byte codes
constexpr int FB_STAGE_BYTES = 2 * FB_OPERAND_BYTES;     // A rows + B rows
constexpr int FB_SMEM_BYTES = FB_STAGES * FB_STAGE_BYTES + 1024 + 256;
constexpr int FB_TMEM_COLS = 256;                        // two accumulators of 128 columns

struct F8BlockDev {
  bf16* c;
  const float* scale_a;  // [m, k_blocks]
  const float* scale_b;  // [ceil(n / 128), k_blocks]
  int m, n, k_blocks, ldc, tiles_n, n_tiles;
  int* err_word;
  unsigned long long wait_limit_ns;
  int test_skip_load;  // test hook: the producer leaves out one A tile load
};

__global__ void __launch_bounds__(FB_THREADS, 1)
gemm_f8_block_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, F8BlockDev p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;  // tiles: 1024-byte aligned (128-byte swizzle)
  uint8_t* smem_al = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + FB_STAGES * FB_STAGE_BYTES);
  // bars[0..S): full, [S..2S): empty, [2S..2S+2): accumulator full, [2S+2..2S+4): accumulator empty
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * FB_STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar0 = ptx::smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (FB_STAGES + s); };
  auto accf_bar = [&](int a) { return bar0 + 8u * (2 * FB_STAGES + a); };
  auto acce_bar = [&](int a) { return bar0 + 8u * (2 * FB_STAGES + 2 + a); };
  const uint64_t limit = p.wait_limit_ns;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < FB_STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(accf_bar(a), 1);
      ptx::mbar_init(acce_bar(a), 8);  // the eight accumulating warps
    }
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmap_a);
    ptx::prefetch_tensormap(&tmap_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_slot), FB_TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int k_blocks = p.k_blocks;

  ptx::grid_launch_dependents();
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      ptx::grid_dependency_wait();
      for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x) {
        const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!ptx::mbar_wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, limit)) { ok = false; break; }
          const uint32_t sa = smem_base + stage * FB_STAGE_BYTES;
          ptx::mbar_arrive_expect_tx(full_bar(stage), FB_STAGE_BYTES);
          if (!(p.test_skip_load && tile == static_cast<int>(blockIdx.x) && kb == 0))
            ptx::tma_load_2d(sa, &tmap_a, kb * FB_TILE, tm * FB_TILE, full_bar(stage));
          ptx::tma_load_2d(sa + FB_OPERAND_BYTES, &tmap_b, kb * FB_TILE, tn * FB_TILE, full_bar(stage));
          if (++stage == FB_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // give loads already in flight time to land before the block's shared memory is released
#pragma unroll 1
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::umma_idesc_e4m3(FB_TILE, FB_TILE);
      int stage = 0;
      uint32_t phase = 0;
      const long long total = static_cast<long long>((p.n_tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) /
                                                     static_cast<int>(gridDim.x)) * k_blocks;  // K blocks of this block's tiles
      for (long long it = 0; it < total; ++it) {
        const int acc = static_cast<int>(it & 1);
        // the accumulator's previous content (two K blocks ago) has been read out
        if (!ptx::mbar_wait_bounded(acce_bar(acc), (static_cast<uint32_t>(it >> 1) & 1u) ^ 1u, abort_flag, limit)) break;
        if (!ptx::mbar_wait_bounded(full_bar(stage), phase, abort_flag, limit)) break;
        ptx::tc_fence_after();
        const uint32_t sa = smem_base + stage * FB_STAGE_BYTES;
        const uint64_t da = ptx::umma_desc_sw128(sa);
        const uint64_t db = ptx::umma_desc_sw128(sa + FB_OPERAND_BYTES);
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * FB_TILE);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)  // 32 bytes = 32 K elements per instruction
          ptx::umma_f8(d_tmem, da + 2u * kk, db + 2u * kk, idesc, kk > 0 ? 1u : 0u);
        ptx::umma_commit(empty_bar(stage));
        ptx::umma_commit(accf_bar(acc));
        if (++stage == FB_STAGES) { stage = 0; phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------ scaled accumulation, half an output row per thread
    const int lane_group = warp & 3;         // the tensor-memory lanes this warp may touch
    const int half = (warp - 2) >> 2;        // columns 64 * half .. + 63 of the tile
    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(lane_group * 32) << 16) + static_cast<uint32_t>(half * 64);
    ptx::grid_dependency_wait();
    bool ok = true;
    long long it = 0;  // K blocks taken so far, over all tiles of this block (accumulator turn and barrier phase)
    for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x) {
      const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
      const int row = tm * FB_TILE + lane_group * 32 + lane;
      const bool row_ok = row < p.m;
      const float* sa_row = p.scale_a + static_cast<size_t>(row_ok ? row : 0) * k_blocks;
      const float* sb_row = p.scale_b + static_cast<size_t>(tn) * k_blocks;
      uint64_t sum[32];  // 64 fp32 sums, two to a register pair
#pragma unroll
      for (int c = 0; c < 32; ++c) sum[c] = 0ull;
      float s_next = sa_row[0] * sb_row[0];
      for (int kb = 0; kb < k_blocks; ++kb, ++it) {
        const int acc = static_cast<int>(it & 1);
        const uint64_t s2 = ptx::pack_f32x2(s_next, s_next);
        if (kb + 1 < k_blocks) s_next = sa_row[kb + 1] * sb_row[kb + 1];
        ok = __all_sync(0xffffffffu, ptx::mbar_wait_bounded(accf_bar(acc), static_cast<uint32_t>(it >> 1) & 1u, abort_flag, limit));
        if (!ok) break;
        ptx::tc_fence_after();
        uint32_t v[2][32];
        ptx::tmem_ld_32x32(t_row + static_cast<uint32_t>(acc * FB_TILE), v[0]);
        ptx::tmem_ld_32x32(t_row + static_cast<uint32_t>(acc * FB_TILE + 32), v[1]);
        ptx::tmem_ld_wait();
        // the accumulator is in registers: the products two K blocks on may overwrite it
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(acce_bar(acc));
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const uint64_t x2 = ptx::pack_f32x2(__uint_as_float(v[ch][e]), __uint_as_float(v[ch][e + 1]));
            sum[ch * 16 + (e >> 1)] = ptx::fma_f32x2(x2, s2, sum[ch * 16 + (e >> 1)]);
          }
        }
      }
      if (ok && row_ok) {
        bf16* dst = p.c + static_cast<size_t>(row) * p.ldc + tn * FB_TILE + half * 64;
        const int cols = min(FB_TILE, p.n - tn * FB_TILE) - half * 64;  // a multiple of 16, may be <= 0
#pragma unroll
        for (int c = 0; c < 64; c += 8) {
          if (c < cols) {
            float f[8];
#pragma unroll
            for (int q = 0; q < 4; ++q) ptx::unpack_f32x2(sum[(c >> 1) + q], f[2 * q], f[2 * q + 1]);
            uint4 o;
            o.x = ptx::pack_bf16(f[0], f[1]);
            o.y = ptx::pack_bf16(f[2], f[3]);
            o.z = ptx::pack_bf16(f[4], f[5]);
            o.w = ptx::pack_bf16(f[6], f[7]);
            *reinterpret_cast<uint4*>(dst + c) = o;
          }
        }
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag && p.err_word) atomicExch(p.err_word, 1);
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, FB_TMEM_COLS);
  }
}

// ------------------------------------------------------------------ quantisers
// Both take the maximum and the quotients on the bf16 values as stored, in fp32 with IEEE division, and round to
// nearest even with saturation, so that the codes are decided in one fixed precision.  An all-zero group or block gets
// scale 1.

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  f[0] = ptx::bf16_lo(v.x); f[1] = ptx::bf16_hi(v.x);
  f[2] = ptx::bf16_lo(v.y); f[3] = ptx::bf16_hi(v.y);
  f[4] = ptx::bf16_lo(v.z); f[5] = ptx::bf16_hi(v.z);
  f[6] = ptx::bf16_lo(v.w); f[7] = ptx::bf16_hi(v.w);
}

// X[rows, k]: half a warp per (row, group of 128 elements), eight elements (16 bytes) per lane.
constexpr int QG_THREADS = 256;
__global__ void __launch_bounds__(QG_THREADS) quantize_groups_fp8_kernel(const bf16* __restrict__ x, int ldx, int rows,
                                                                         int groups, uint8_t* __restrict__ codes, int ldq,
                                                                         float* __restrict__ scale_out) {
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  const int sub = threadIdx.x & 15;  // lane inside the half warp
  const long long n_units = static_cast<long long>(rows) * groups;
  const long long stride = static_cast<long long>(gridDim.x) * (QG_THREADS / 16);
  // whole warps stay in the loop together (the shuffles below name all 32 lanes): the bound is rounded up to a pair
  for (long long unit = static_cast<long long>(blockIdx.x) * (QG_THREADS / 16) + (threadIdx.x >> 4); unit < ((n_units + 1) & ~1ll);
       unit += stride) {
    const bool live = unit < n_units;
    const int row = live ? static_cast<int>(unit / groups) : 0, g = live ? static_cast<int>(unit % groups) : 0;
    const uint4 v = *reinterpret_cast<const uint4*>(x + static_cast<size_t>(row) * ldx + g * 128 + sub * 8);
    float f[8];
    unpack8(v, f);
    float amax = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(f[e]));
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const float scale = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
    if (live) {
      if (sub == 0) scale_out[static_cast<size_t>(row) * groups + g] = scale;
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] = __fdiv_rn(f[e], scale);
      uint2 o;
      o.x = ptx::cvt_e4m3x2(f[0], f[1]) | (ptx::cvt_e4m3x2(f[2], f[3]) << 16);
      o.y = ptx::cvt_e4m3x2(f[4], f[5]) | (ptx::cvt_e4m3x2(f[6], f[7]) << 16);
      *reinterpret_cast<uint2*>(codes + static_cast<size_t>(row) * ldq + g * 128 + sub * 8) = o;
    }
  }
}

// W[n, k]: one thread block per 128 x 128 block (fewer rows in the last row of blocks); a thread holds half a row.
constexpr int QB_THREADS = 256;
__global__ void __launch_bounds__(QB_THREADS) quantize_blocks_fp8_kernel(const bf16* __restrict__ w, int ldw, int n,
                                                                         int k_blocks, uint8_t* __restrict__ codes,
                                                                         int ldq, float* __restrict__ scale_out) {
  const int bn = blockIdx.x / k_blocks, bk = blockIdx.x % k_blocks;
  const int row = bn * 128 + (threadIdx.x >> 1);
  const int col = bk * 128 + (threadIdx.x & 1) * 64;
  const bool live = row < n;
  uint4 v[8];
  float amax = 0.f;
  if (live) {
    const uint4* src = reinterpret_cast<const uint4*>(w + static_cast<size_t>(row) * ldw + col);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      v[i] = src[i];
      float f[8];
      unpack8(v[i], f);
#pragma unroll
      for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(f[e]));
    }
  }
  __shared__ float red[QB_THREADS / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < QB_THREADS / 32; ++i) tot = fmaxf(tot, red[i]);
  const float scale = tot > 0.f ? __fdiv_rn(tot, 448.f) : 1.f;
  if (threadIdx.x == 0) scale_out[static_cast<size_t>(bn) * k_blocks + bk] = scale;
  if (live) {
    uint2* dst = reinterpret_cast<uint2*>(codes + static_cast<size_t>(row) * ldq + col);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float f[8];
      unpack8(v[i], f);
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] = __fdiv_rn(f[e], scale);
      uint2 o;
      o.x = ptx::cvt_e4m3x2(f[0], f[1]) | (ptx::cvt_e4m3x2(f[2], f[3]) << 16);
      o.y = ptx::cvt_e4m3x2(f[4], f[5]) | (ptx::cvt_e4m3x2(f[6], f[7]) << 16);
      dst[i] = o;
    }
  }
}

}  // namespace

pd_status launch_gemm_f8_block(const uint8_t* a, const float* sa, const uint8_t* b, const float* sb, bf16* c, int m, int n,
                               int k, int* err_word, cudaStream_t st) {
  if (m == 0 || n == 0) return PD_OK;
  if (!a || !sa || !b || !sb || !c || m < 0 || n < 0 || k <= 0) return PD_ERR_INVALID_ARG;
  if (k % FB_TILE != 0 || n % 16 != 0) return PD_ERR_UNSUPPORTED_SHAPE;
  const long long tiles_m = (m + FB_TILE - 1) / FB_TILE, tiles_n = (n + FB_TILE - 1) / FB_TILE;
  if (tiles_m * tiles_n > 0x3fffffffll) return PD_ERR_UNSUPPORTED_SHAPE;
  static PerDeviceInt smem_opt_in;
  PD_TRY(opt_in_smem(smem_opt_in, gemm_f8_block_kernel, FB_SMEM_BYTES));
  CUtensorMap ta, tb;
  PD_TRY(make_tmap_u8(&ta, a, m, k, k, FB_TILE));
  PD_TRY(make_tmap_u8(&tb, b, n, k, k, FB_TILE));
  F8BlockDev p{};
  p.c = c; p.scale_a = sa; p.scale_b = sb;
  p.m = m; p.n = n; p.k_blocks = k / FB_TILE; p.ldc = n; p.tiles_n = static_cast<int>(tiles_n);
  p.n_tiles = static_cast<int>(tiles_m * tiles_n);
  p.err_word = err_word;
  p.wait_limit_ns = 4000000000ull;
  if (take_wait_injection(PD_INJECT_GEMM_FP8_BLOCKWISE, &p.wait_limit_ns)) p.test_skip_load = 1;
  int dev = 0, sms = 0;
  PD_CUDA_TRY(cudaGetDevice(&dev));
  PD_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int grid = p.n_tiles < sms ? p.n_tiles : sms;
  PD_CUDA_TRY(launch_pdl(gemm_f8_block_kernel, dim3(static_cast<unsigned>(grid)), dim3(FB_THREADS), FB_SMEM_BYTES, st, ta, tb, p));
  count_launch();
  return PD_OK;
}

}  // namespace pd

extern "C" pd_status pd_quantize_fp8_groups(const void* x, int32_t ldx, int32_t rows, int32_t k, void* codes, float* scales,
                                            void* stream) {
  if (rows == 0) return PD_OK;
  if (!x || !codes || !scales || rows < 0 || k <= 0) return PD_ERR_INVALID_ARG;
  if (k % 128 != 0 || ldx % 8 != 0 || ldx < k) return PD_ERR_UNSUPPORTED_SHAPE;
  const int groups = k / 128;
  const long long units = static_cast<long long>(rows) * groups;
  long long blocks = (units + pd::QG_THREADS / 16 - 1) / (pd::QG_THREADS / 16);
  if (blocks > 148 * 16) blocks = 148 * 16;  // resident blocks take further units grid-stride
  PD_CUDA_TRY(pd::launch_pdl(pd::quantize_groups_fp8_kernel, dim3(static_cast<unsigned>(blocks)), dim3(pd::QG_THREADS), 0,
                             static_cast<cudaStream_t>(stream), static_cast<const pd::bf16*>(x), ldx, rows, groups,
                             static_cast<uint8_t*>(codes), k, scales));
  pd::count_launch();
  return PD_OK;
}

extern "C" pd_status pd_quantize_fp8_blocks(const void* w, int32_t ldw, int32_t n, int32_t k, void* codes, float* scales,
                                            void* stream) {
  if (n == 0) return PD_OK;
  if (!w || !codes || !scales || n < 0 || k <= 0) return PD_ERR_INVALID_ARG;
  if (k % 128 != 0 || ldw % 8 != 0 || ldw < k) return PD_ERR_UNSUPPORTED_SHAPE;
  const long long blocks = static_cast<long long>((n + 127) / 128) * (k / 128);
  if (blocks > 0x7fffffffll) return PD_ERR_UNSUPPORTED_SHAPE;
  pd::quantize_blocks_fp8_kernel<<<static_cast<unsigned>(blocks), pd::QB_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const pd::bf16*>(w), ldw, n, k / 128, static_cast<uint8_t*>(codes), k, scales);
  PD_CUDA_TRY(cudaGetLastError());
  pd::count_launch();
  return PD_OK;
}

extern "C" pd_status pd_gemm_fp8_blockwise(const void* a_codes, const float* a_scales, const void* b_codes,
                                           const float* b_scales, void* c, int32_t m, int32_t n, int32_t k, int32_t* err_word,
                                           void* stream) {
  return pd::launch_gemm_f8_block(static_cast<const uint8_t*>(a_codes), a_scales, static_cast<const uint8_t*>(b_codes), b_scales,
                                  static_cast<pd::bf16*>(c), m, n, k, err_word, static_cast<cudaStream_t>(stream));
}
