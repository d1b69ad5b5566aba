// C[M,N] = A[M,K] * B[N,K]^T (+ residual), bf16 or FP8 (E4M3) operands, fp32 accumulation.
// With FP8 operands a shared-memory row of 128 bytes holds 128 K elements instead of 64, the
// instruction is tcgen05.mma.kind::f8f6f4 (32 K elements each) and the accumulator is multiplied by
// the row scale of A and the row scale of B before the epilogue proper.
//
// A persistent, warp-specialised kernel.  One thread issues TMA tile
// loads of A (128 x 64) and B (BN x 64) into a ring of shared-memory stages; one thread
// issues tcgen05.mma (128 x BN x 16 per instruction) accumulating in tensor memory; four
// warps drain the accumulator (tcgen05.ld) and run the epilogue.  Two accumulator buffers
// in tensor memory let the epilogue of tile i overlap the main loop of tile i+1.
// Epilogues: plain store, residual add, SwiGLU (gate and up columns interleaved in blocks
// of 64 so one tile holds both halves), and RoPE with the scatter of q, k, v to the q buffer
// and the KV cache (a tile holds whole heads).
// Every barrier wait is wall-clock bounded; on a timeout the block raises a shared abort
// flag, records an error word in global memory and leaves through the normal teardown.
#include <cstdlib>
#include <mutex>

#include "pd_common.cuh"
#include "pd_ptx.cuh"

namespace pd {

// ------------------------------------------------------------------ tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

pd_status make_tmap_bf16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t ld,
                         uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return PD_ERR_CUDA;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) || (ld * 2) % 16 != 0 || box_rows == 0 || box_rows > 256)
    return PD_ERR_INVALID_ARG;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? PD_OK : PD_ERR_INVALID_ARG;
}

pd_status make_tmap_u8(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t ld,
                       uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return PD_ERR_CUDA;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) || ld % 16 != 0 || box_rows == 0 || box_rows > 256)
    return PD_ERR_INVALID_ARG;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld};
  cuuint32_t box[2] = {128, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? PD_OK : PD_ERR_INVALID_ARG;
}

// ---------------------------------------------------------------- tcgen05 GEMM
namespace {

constexpr int BM = 128;
constexpr int BK = 64;        // K elements of a bf16 stage (128 bytes per row)
constexpr int BK_F8 = 128;    // K elements of an FP8 stage (the same 128 bytes per row)
constexpr int GEMM_THREADS = 192;  // warp 0: TMA, warp 1: MMA, warps 2-5: epilogue
constexpr int TMEM_COLS = 512;

template <int BN>
struct GemmCfg {
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (BN >= 256) ? 4 : (BN >= 128 ? 6 : 8);
  static constexpr int ACC_COLS = BN;  // columns per accumulator buffer
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

struct GemmDev {
  bf16* c;
  const bf16* r;
  int m, n, k;
  int ldc, ldr;
  int tiles_m, tiles_n;
  int raster_group;  // row tiles that share the column-tile sweep (their A slab stays in L2)
  // Tail split: the tiles of the last, partly filled wave are each cut in two along K and given to two
  // blocks; the first writes its fp32 partial tile to `split_scratch` and raises a flag per 32-row group,
  // the second adds it before the epilogue and lowers the flag again (so the flags are zero between
  // launches and a captured launch can be replayed).  n_units = main_tiles + 2 * (tiles - main_tiles).
  int n_units, main_tiles;
  int tail_halves;       // 1: instead, tail tiles are cut in two along N (two 128-column halves, no hand-over)
  float* split_scratch;  // [tail tile][128][BN] fp32
  int* split_flags;      // [tail tile][4], 1 while a partial waits to be consumed
  int split_enable;
  int split_all;         // CTA-pair kernel: EVERY tile is cut in two along K (unit 2 i = first half, 2 i + 1 = second half)
  int* err_word;
  unsigned long long wait_limit_ns;  // bound of every wait inside the kernel
  int test_skip_load;                // test hook: the producer leaves out the A tile of its second K block
  const float* scale_a;  // FP8 operands: per-row scale of A [M] and of B [N]
  const float* scale_b;
  RopeEpilogue rope;  // EPI_ROPE_KV only
};

__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  uint4 o;
  o.x = ptx::pack_bf16(f[0], f[1]);
  o.y = ptx::pack_bf16(f[2], f[3]);
  o.z = ptx::pack_bf16(f[4], f[5]);
  o.w = ptx::pack_bf16(f[6], f[7]);
  return o;
}

__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int GROUP, int& tm, int& tn) {
  // Groups of row-tiles sweep the column-tiles together, so concurrently running blocks hit the
  // same A and B tiles in L2 and B is streamed from HBM once per group.
  const int per_group = GROUP * tiles_n;
  const int g = tile / per_group;
  const int first_m = g * GROUP;
  const int rows_in_group = min(GROUP, tiles_m - first_m);
  const int t = tile - g * per_group;
  tm = first_m + t % rows_in_group;
  tn = t / rows_in_group;
}

// Work unit -> tile, K-block range and role (0 whole tile, 1 first K half: writes a partial, 2 second K half:
// adds the partner's partial and runs the epilogue).
// role 3: the unit is the 128-column half `n_half` of its tile (whole K, independent of the other half).
struct UnitInfo {
  int tile, kb_lo, kb_hi, role, n_half;
};
__device__ __forceinline__ UnitInfo unit_info(int unit, int main_tiles, int k_blocks, int tail_halves) {
  UnitInfo u;
  u.n_half = 0;
  if (unit < main_tiles) {
    u.tile = unit; u.kb_lo = 0; u.kb_hi = k_blocks; u.role = 0;
  } else {
    const int v = unit - main_tiles;
    u.tile = main_tiles + (v >> 1);
    if (tail_halves) {
      u.kb_lo = 0; u.kb_hi = k_blocks; u.role = 3; u.n_half = v & 1;
    } else {
      const int kh = k_blocks >> 1;
      if (v & 1) { u.kb_lo = kh; u.kb_hi = k_blocks; u.role = 2; }
      else { u.kb_lo = 0; u.kb_hi = kh; u.role = 1; }
    }
  }
  return u;
}

// Epilogue of one accumulator tile for the thread that owns row `row` (tensor-memory lane of t_row): reads the
// accumulator in chunks of 32 columns and applies the epilogue EPI.  role / n_half as in UnitInfo; part_row is the
// thread's row of the partner's fp32 partial (roles 1 and 2); ok = false skips the work (an aborted wait).
template <int BN, int EPI, bool F8>
__device__ __forceinline__ void epilogue_tile(const GemmDev& p, int role, int n_half, int tm, int tn, int row,
                                              uint32_t t_row, const float* part_row, bool ok) {
  (void)tm;
  // a half-width unit holds columns [128 n_half, 128 n_half + 128) of its tile in accumulator columns 0..127
  const int acc_cols = (role == 3) ? 128 : BN;
  const int col_base = tn * BN + n_half * 128;
  float row_scale = 1.f;
  if constexpr (F8) row_scale = row < p.m ? p.scale_a[row] : 0.f;
  // accumulator chunk -> registers (+ the partner's partial for a K-split tile; x the operand scales for FP8)
  auto load_acc = [&](int col_off, uint32_t (&v)[32]) {
    ptx::tmem_ld_32x32(t_row + col_off, v);
    ptx::tmem_ld_wait();
    if (role == 2) {
#pragma unroll
      for (int j = 0; j < 32; j += 4) {
        const float4 q = __ldcg(reinterpret_cast<const float4*>(part_row + ((col_off + j) >> 2) * (BM * 4)));
        v[j] = __float_as_uint(__uint_as_float(v[j]) + q.x);
        v[j + 1] = __float_as_uint(__uint_as_float(v[j + 1]) + q.y);
        v[j + 2] = __float_as_uint(__uint_as_float(v[j + 2]) + q.z);
        v[j + 3] = __float_as_uint(__uint_as_float(v[j + 3]) + q.w);
      }
    }
    if constexpr (F8) {
      const int col = col_base + col_off;  // row of B = column of the product (a multiple of 32)
#pragma unroll
      for (int j = 0; j < 32; j += 4) {
        float4 sb = make_float4(0.f, 0.f, 0.f, 0.f);
        if (col + j < p.n) sb = __ldg(reinterpret_cast<const float4*>(p.scale_b + col + j));
        v[j] = __float_as_uint(__uint_as_float(v[j]) * (row_scale * sb.x));
        v[j + 1] = __float_as_uint(__uint_as_float(v[j + 1]) * (row_scale * sb.y));
        v[j + 2] = __float_as_uint(__uint_as_float(v[j + 2]) * (row_scale * sb.z));
        v[j + 3] = __float_as_uint(__uint_as_float(v[j + 3]) * (row_scale * sb.w));
      }
    }
  };
  if (role == 1 || !ok) {
    // nothing more to do for this unit
  } else if constexpr (EPI == EPI_STORE || EPI == EPI_RESIDUAL) {
    // The residual of the NEXT chunk is requested before the current one is processed: a thread reads its own row
    // (16 bytes per load, a different line for every lane), and without the lookahead that latency would be
    // exposed once per chunk, which is what bounded the short-K projections.
    uint4 r_next[4];
    auto load_res = [&](int c0, uint4 (&dst)[4]) {
      const bf16* rrow = p.r + static_cast<size_t>(row) * p.ldr + col_base + c0;
#pragma unroll
      for (int q = 0; q < 4; ++q)
        dst[q] = (row < p.m && col_base + c0 + q * 8 < p.n) ? __ldcg(reinterpret_cast<const uint4*>(rrow + q * 8))
                                                            : make_uint4(0u, 0u, 0u, 0u);
    };
    if constexpr (EPI == EPI_RESIDUAL) load_res(0, r_next);
#pragma unroll 1
    for (int c0 = 0; c0 < acc_cols; c0 += 32) {
      uint4 r_cur[4];
      if constexpr (EPI == EPI_RESIDUAL) {
#pragma unroll
        for (int q = 0; q < 4; ++q) r_cur[q] = r_next[q];
        if (c0 + 32 < acc_cols) load_res(c0 + 32, r_next);
      }
      uint32_t v[32];
      load_acc(c0, v);
      const int col = col_base + c0;
      if (row < p.m) {
        bf16* crow = p.c + static_cast<size_t>(row) * p.ldc + col;
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          if (col + j < p.n) {
            float f[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[j + e]);
            if constexpr (EPI == EPI_RESIDUAL) {
              const uint4 rr = r_cur[j >> 3];
              f[0] += ptx::bf16_lo(rr.x); f[1] += ptx::bf16_hi(rr.x);
              f[2] += ptx::bf16_lo(rr.y); f[3] += ptx::bf16_hi(rr.y);
              f[4] += ptx::bf16_lo(rr.z); f[5] += ptx::bf16_hi(rr.z);
              f[6] += ptx::bf16_lo(rr.w); f[7] += ptx::bf16_hi(rr.w);
            }
            *reinterpret_cast<uint4*>(crow + j) = pack8(f);
          }
        }
      }
    }
  } else if constexpr (EPI == EPI_SWIGLU) {
    // columns [128 q, 128 q + 64) of the product are gate features 64 q .., the next 64 the matching up features
    const int f_total = p.n / 2;
#pragma unroll 1
    for (int c0 = 0; c0 < acc_cols / 2; c0 += 32) {
      const int pair = c0 >> 6, within = c0 & 63;
      uint32_t g[32], u[32];
      load_acc(pair * 128 + within, g);
      load_acc(pair * 128 + 64 + within, u);
      const int fcol = (tn * (BN / 128) + n_half + pair) * 64 + within;
      if (row < p.m && fcol < f_total) {
        bf16* crow = p.c + static_cast<size_t>(row) * p.ldc + fcol;
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          float f[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float gv = __uint_as_float(g[j + e]);
            f[e] = gv / (1.f + __expf(-gv)) * __uint_as_float(u[j + e]);
          }
          *reinterpret_cast<uint4*>(crow + j) = pack8(f);
        }
      }
    }
  } else {  // EPI_ROPE_KV
    const RopeEpilogue& rp = p.rope;
    const int hd = rp.head_dim, half = hd >> 1;
    int pos = 0, slot = 0;
    bool row_ok = row < p.m;
    if (row_ok) {
      if (rp.cu_seqlens) {
        int lo = 0, hi = rp.n_req;  // request r with cu[r] <= row < cu[r+1]
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (rp.cu_seqlens[mid] <= row) lo = mid; else hi = mid;
        }
        pos = row - rp.cu_seqlens[lo] + (rp.prefix ? rp.prefix[lo] : 0);
        slot = rp.slots ? rp.slots[lo] : lo;
      } else {
        pos = rp.kv_len[row];
        slot = row;
      }
      if (pos < 0 || pos >= rp.len_cap || pos >= rp.max_pos || slot < 0 || slot >= rp.batch_cap) {
        if (p.err_word) atomicExch(p.err_word, 2);  // would fall outside the cache or the table: skip the row
        row_ok = false;
      }
    }
    const int n_heads = rp.n_q_heads + 2 * rp.n_kv_heads;
    const int heads_per_tile = acc_cols / hd;
    // (cos, sin) of this row's position for 32 rotation pairs at a time: loaded once for all heads of the tile, and
    // the next 32 pairs are requested before the current ones are used (the loads are private to the thread's row).
    const bool any_rotate = col_base / hd < rp.n_q_heads + rp.n_kv_heads;  // warp-uniform
    float4 t_next[16];
    auto load_tab = [&](int i0, float4 (&dst)[16]) {
      const float4* tab = reinterpret_cast<const float4*>(rp.rope_tab + static_cast<size_t>(pos) * half + i0);
#pragma unroll
      for (int q = 0; q < 16; ++q) dst[q] = row_ok ? __ldg(tab + q) : make_float4(1.f, 0.f, 1.f, 0.f);
    };
    if (any_rotate) load_tab(0, t_next);
#pragma unroll 1
    for (int i0 = 0; i0 < half; i0 += 32) {
      float4 t_cur[16];
#pragma unroll
      for (int q = 0; q < 16; ++q) t_cur[q] = t_next[q];
      if (any_rotate && i0 + 32 < half) load_tab(i0 + 32, t_next);
#pragma unroll 1
      for (int hh = 0; hh < heads_per_tile; ++hh) {
        const int head = col_base / hd + hh;
        if (head >= n_heads) break;  // warp-uniform
        uint32_t lo[32], hi[32];
        load_acc(hh * hd + i0, lo);
        load_acc(hh * hd + half + i0, hi);
        if (!row_ok) continue;
        bf16* dst;
        if (head < rp.n_q_heads) {
          dst = p.c + static_cast<size_t>(row) * p.ldc + head * hd;
        } else if (head < rp.n_q_heads + rp.n_kv_heads) {
          dst = rp.k_cache +
                ((static_cast<size_t>(slot) * rp.n_kv_heads + (head - rp.n_q_heads)) * rp.len_cap + pos) * hd;
        } else {
          dst = rp.v_cache + ((static_cast<size_t>(slot) * rp.n_kv_heads + (head - rp.n_q_heads - rp.n_kv_heads)) *
                                  rp.len_cap + pos) * hd;
        }
        const bool rotate = head < rp.n_q_heads + rp.n_kv_heads;
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          float a[8], b[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) { a[e] = __uint_as_float(lo[j + e]); b[e] = __uint_as_float(hi[j + e]); }
          if (rotate) {
#pragma unroll
            for (int e = 0; e < 8; e += 2) {
              const float4 cs = t_cur[(j + e) >> 1];  // (cos, sin) of two consecutive pairs
              const float a0 = a[e], b0 = b[e], a1 = a[e + 1], b1 = b[e + 1];
              a[e] = a0 * cs.x - b0 * cs.y;      b[e] = b0 * cs.x + a0 * cs.y;
              a[e + 1] = a1 * cs.z - b1 * cs.w;  b[e + 1] = b1 * cs.z + a1 * cs.w;
            }
          }
          *reinterpret_cast<uint4*>(dst + i0 + j) = pack8(a);
          *reinterpret_cast<uint4*>(dst + half + i0 + j) = pack8(b);
        }
      }
    }
  }
}

// Hand-over of a K-split tile between its two units (one warp = one 32-row group of the tile).  The fp32 scratch
// tile is laid out [column group of 4][row][4] so that the 32 rows of a warp access 512 contiguous bytes per
// instruction (a thread's own row, 1 KB apart from its neighbours', would cost 32 lines per instruction); part_row
// points at the thread's row inside column group 0.  role 1: park the accumulator rows and raise the group's flag.  role 2: wait (bounded) for the partner's
// flag; the caller's epilogue then adds the parked rows.  Returns false when the wait gave up.
template <int BN>
__device__ __forceinline__ bool split_hand_over(const GemmDev& p, int role, int slot, int lane_group, int lane,
                                                uint32_t t_row, float* part_row, volatile int* abort_flag) {
  int* flag = p.split_flags + slot * 4 + lane_group;
  if (role == 1) {
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += 32) {
      uint32_t v[32];
      ptx::tmem_ld_32x32(t_row + c0, v);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; j += 4)
        __stcg(reinterpret_cast<uint4*>(part_row + ((c0 + j) >> 2) * (BM * 4)), make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]));
    }
    __threadfence();
    __syncwarp();
    if (lane == 0) *reinterpret_cast<volatile int*>(flag) = 1;
    return true;
  }
  bool seen = true;
  if (lane == 0) {
    const uint64_t t0 = ptx::globaltimer_ns();
    uint32_t spins = 0;
    while (*reinterpret_cast<volatile int*>(flag) != 1) {
      if ((++spins & 1023u) == 0u && (*abort_flag || ptx::globaltimer_ns() - t0 > p.wait_limit_ns)) {
        *abort_flag = 1;
        seen = false;
        break;
      }
    }
  }
  const bool ok = __all_sync(0xffffffffu, seen);
  __threadfence();
  return ok;
}

template <int BN, int EPI, bool F8>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, GemmDev p) {
  using Cfg = GemmCfg<BN>;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  // tiles need 1024-byte alignment for the 128-byte swizzle pattern
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * Cfg::STAGE_BYTES);
  // bars[0..S): full, [S..2S): empty, [2S..2S+2): acc full, [2S+2..2S+4): acc empty
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t bar0 = ptx::smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto accf_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
  auto acce_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + 2 + a); };

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(accf_bar(a), 1);
      ptx::mbar_init(acce_bar(a), 4);
    }
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmap_a);
    ptx::prefetch_tensormap(&tmap_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_slot), TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  constexpr int KE = F8 ? BK_F8 : BK;  // K elements per stage
  const int n_units = p.n_units;
  const int k_blocks = p.k / KE;

  // Programmatic dependent launch: the next kernel of the stream may start its own set-up now; this one touches
  // global memory (operand loads, epilogue reads and writes) only after the kernels before it have completed.
  ptx::grid_launch_dependents();
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      ptx::grid_dependency_wait();
      for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x) {
        const UnitInfo ui = unit_info(unit, p.main_tiles, k_blocks, p.tail_halves);
        int tm, tn;
        tile_coords(ui.tile, p.tiles_m, p.tiles_n, p.raster_group, tm, tn);
        for (int kb = ui.kb_lo; kb < ui.kb_hi; ++kb) {
          if (!ptx::mbar_wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
          const uint32_t sa = smem_base + stage * Cfg::STAGE_BYTES;
          const uint32_t sb = sa + Cfg::A_BYTES;
          ptx::mbar_arrive_expect_tx(full_bar(stage), Cfg::STAGE_BYTES);
          if (!(p.test_skip_load && unit == static_cast<int>(blockIdx.x) && kb == ui.kb_lo + 1))
            ptx::tma_load_2d(sa, &tmap_a, kb * KE, tm * BM, full_bar(stage));
          ptx::tma_load_2d(sb, &tmap_b, kb * KE, tn * BN, full_bar(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // give loads already in flight time to land before the block's shared memory is released
#pragma unroll 1
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = F8 ? ptx::umma_idesc_e4m3(BM, BN) : ptx::umma_idesc_bf16(BM, BN);
      constexpr uint32_t idesc_half = F8 ? ptx::umma_idesc_e4m3(BM, 128) : ptx::umma_idesc_bf16(BM, 128);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x) {
        const UnitInfo ui = unit_info(unit, p.main_tiles, k_blocks, p.tail_halves);
        if (!ptx::mbar_wait_bounded(acce_bar(acc), acc_phase ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * Cfg::ACC_COLS);
        for (int kb = ui.kb_lo; kb < ui.kb_hi; ++kb) {
          if (!ptx::mbar_wait_bounded(full_bar(stage), phase, abort_flag, p.wait_limit_ns)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t sa = smem_base + stage * Cfg::STAGE_BYTES;
          const uint32_t sb = sa + Cfg::A_BYTES;
          const uint64_t da = ptx::umma_desc_sw128(sa);
          // a half-width unit multiplies by rows 128 n_half .. of the B tile only (128 rows = 16 KB further on)
          const uint64_t db = ptx::umma_desc_sw128(sb + ui.n_half * (128 * 128));
          const uint32_t idesc_u = (ui.role == 3) ? idesc_half : idesc;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            // one instruction covers 32 bytes along K (16 bf16 or 32 FP8) of the 128-byte swizzled row:
            // +2 in 16-byte units
            const uint32_t accum = (kb > ui.kb_lo || kk > 0) ? 1u : 0u;
            if constexpr (F8) ptx::umma_f8(d_tmem, da + 2u * kk, db + 2u * kk, idesc_u, accum);
            else ptx::umma_bf16(d_tmem, da + 2u * kk, db + 2u * kk, idesc_u, accum);
          }
          ptx::umma_commit(empty_bar(stage));  // stage is free once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::umma_commit(accf_bar(acc));  // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int lane_group = warp & 3;  // tensor-memory lanes 32*lane_group .. +31 belong to this warp
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    ptx::grid_dependency_wait();
    for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x) {
      const UnitInfo ui = unit_info(unit, p.main_tiles, k_blocks, p.tail_halves);
      int tm, tn;
      tile_coords(ui.tile, p.tiles_m, p.tiles_n, p.raster_group, tm, tn);
      // warp-uniform outcome: tcgen05.ld below needs the whole warp
      ok = __all_sync(0xffffffffu, ptx::mbar_wait_bounded(accf_bar(acc), acc_phase, abort_flag, p.wait_limit_ns));
      if (!ok) break;
      ptx::tc_fence_after();
      const int row = tm * BM + lane_group * 32 + lane;
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(lane_group * 32) << 16) +
                             static_cast<uint32_t>(acc * Cfg::ACC_COLS);
      // partner data of a K-split tile: this thread's row of the fp32 partial tile
      float* part_row = nullptr;
      if (ui.role == 1 || ui.role == 2) {
        const int slot = ui.tile - p.main_tiles;
        part_row = p.split_scratch + static_cast<size_t>(slot) * BM * BN + (lane_group * 32 + lane) * 4;
        ok = split_hand_over<BN>(p, ui.role, slot, lane_group, lane, t_row, part_row, abort_flag);
      }
      epilogue_tile<BN, EPI, F8>(p, ui.role, ui.n_half, tm, tn, row, t_row, part_row, ok);
      // all of this warp's reads of the accumulator are complete: hand the buffer back
      ptx::tc_fence_before();
      __syncwarp();
      if (ui.role == 2 && lane == 0) {
        // the partner's partial has been consumed: lower the flag for the next launch
        __threadfence();
        *reinterpret_cast<volatile int*>(p.split_flags + (ui.tile - p.main_tiles) * 4 + lane_group) = 0;
      }
      if (lane == 0) ptx::mbar_arrive(acce_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0 && p.err_word) atomicExch(p.err_word, 1);
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ------------------------------------------------------------- CTA-pair variant
// The same GEMM on pairs of CTAs (cluster of two on one TPC): a pair owns a 256 x 256 tile.  Each CTA loads its
// 128 rows of A and 128 of the tile's 256 rows of B (so a stage is 32 KB per CTA instead of 48 KB and every byte of
// B is read from shared memory once for both SMs), the even CTA's MMA thread issues tcgen05.mma.cta_group::2 for
// both, and each CTA drains its own 128 accumulator rows through the common epilogue.
// Barriers: `full` lives in the even CTA and counts the bytes of both CTAs' loads; `empty` and `accumulator full`
// exist in both CTAs and are signalled together by a multicast commit; `accumulator empty` lives in the even CTA
// and collects the epilogue warps of both.  A CTA only ever WAITS on its own barriers, always bounded.
constexpr int P2_STAGE_BYTES = 2 * BM * 128;  // A rows + B rows of this CTA, 16 KB each
constexpr int P2_STAGES = 7;
constexpr int P2_SMEM_BYTES = P2_STAGES * P2_STAGE_BYTES + 1024 + 256;

// Work unit of the CTA-pair kernel: whole tiles and half-width tail tiles as in unit_info, or, when the problem
// has so few tiles that half of the pairs would idle (split_all), every tile as two K halves on two pairs.
__device__ __forceinline__ UnitInfo pair_unit_info(const GemmDev& p, int unit, int k_blocks) {
  if (!p.split_all) return unit_info(unit, p.main_tiles, k_blocks, 1);
  UnitInfo u;
  u.n_half = 0;
  u.tile = unit >> 1;
  const int kh = k_blocks >> 1;
  if (unit & 1) { u.kb_lo = kh; u.kb_hi = k_blocks; u.role = 2; }
  else { u.kb_lo = 0; u.kb_hi = kh; u.role = 1; }
  return u;
}

template <int EPI, bool F8>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                    const __grid_constant__ CUtensorMap tmap_b_half, GemmDev p) {
  constexpr int BN = 256;
  constexpr int STAGES = P2_STAGES;
  constexpr int KE = F8 ? BK_F8 : BK;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * P2_STAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();
  const uint32_t bar0 = ptx::smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto accf_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
  auto acce_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + 2 + a); };

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(accf_bar(a), 1);
      ptx::mbar_init(acce_bar(a), 8);  // four epilogue warps of each CTA
    }
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmap_a);
    ptx::prefetch_tensormap(&tmap_b);
    ptx::prefetch_tensormap(&tmap_b_half);
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(ptx::smem_u32(tmem_slot), TMEM_COLS);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();  // both CTAs' barriers are initialised before either CTA signals the other
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int k_blocks = p.k / KE;
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int tiles_m2 = (p.tiles_m + 1) >> 1;  // 256-row tiles
  const int n_units = p.n_units;  // whole tiles [0, main_tiles), then the tiles of the last partial wave as two
                                  // independent 128-column halves each (tail_halves), see unit_info
  const int group2 = max(1, p.raster_group >> 1);

  ptx::grid_launch_dependents();  // (see gemm_tc_kernel)
  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      ptx::grid_dependency_wait();
      for (int unit = pair_id; unit < n_units && ok; unit += n_pairs) {
        const UnitInfo ui = pair_unit_info(p, unit, k_blocks);
        int tm2, tn;
        tile_coords(ui.tile, tiles_m2, p.tiles_n, group2, tm2, tn);
        const bool half = ui.role == 3;  // this CTA then supplies 64 of the half tile's 128 rows of B
        for (int kb = ui.kb_lo; kb < ui.kb_hi; ++kb) {
          if (!ptx::mbar_wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
          const uint32_t sa = smem_base + stage * P2_STAGE_BYTES;
          const uint32_t sb = sa + BM * 128;
          const uint32_t lead_full = ptx::map_to_cta(full_bar(stage), 0);
          if (rank == 0) ptx::mbar_arrive_expect_tx(full_bar(stage), half ? 2 * (BM + 64) * 128 : 2 * P2_STAGE_BYTES);
          if (!(p.test_skip_load && rank == 0 && unit == pair_id && kb == ui.kb_lo + 1))
            ptx::tma_load_2d_pair(sa, &tmap_a, kb * KE, (2 * tm2 + static_cast<int>(rank)) * BM, lead_full);
          if (half)
            ptx::tma_load_2d_pair(sb, &tmap_b_half, kb * KE, tn * BN + ui.n_half * 128 + static_cast<int>(rank) * 64, lead_full);
          else
            ptx::tma_load_2d_pair(sb, &tmap_b, kb * KE, tn * BN + static_cast<int>(rank) * 128, lead_full);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
#pragma unroll 1
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc_full = F8 ? ptx::umma_idesc_e4m3(2 * BM, BN) : ptx::umma_idesc_bf16(2 * BM, BN);
      constexpr uint32_t idesc_half = F8 ? ptx::umma_idesc_e4m3(2 * BM, 128) : ptx::umma_idesc_bf16(2 * BM, 128);
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int unit = pair_id; unit < n_units && ok; unit += n_pairs) {
        const UnitInfo ui = pair_unit_info(p, unit, k_blocks);
        const uint32_t idesc = ui.role == 3 ? idesc_half : idesc_full;
        if (!ptx::mbar_wait_bounded(acce_bar(acc), acc_phase ^ 1u, abort_flag, p.wait_limit_ns)) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
        for (int kb = ui.kb_lo; kb < ui.kb_hi; ++kb) {
          if (!ptx::mbar_wait_bounded(full_bar(stage), phase, abort_flag, p.wait_limit_ns)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t sa = smem_base + stage * P2_STAGE_BYTES;
          const uint64_t da = ptx::umma_desc_sw128(sa);
          const uint64_t db = ptx::umma_desc_sw128(sa + BM * 128);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const uint32_t accum = (kb > ui.kb_lo || kk > 0) ? 1u : 0u;
            if constexpr (F8) ptx::umma_f8_pair(d_tmem, da + 2u * kk, db + 2u * kk, idesc, accum);
            else ptx::umma_bf16_pair(d_tmem, da + 2u * kk, db + 2u * kk, idesc, accum);
          }
          ptx::umma_commit_pair(empty_bar(stage), 3);  // the stage is free in both CTAs
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::umma_commit_pair(accf_bar(acc), 3);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    const int lane_group = warp & 3;
    int acc = 0;
    uint32_t acc_phase = 0;
    ptx::grid_dependency_wait();
    for (int unit = pair_id; unit < n_units; unit += n_pairs) {
      const UnitInfo ui = pair_unit_info(p, unit, k_blocks);
      int tm2, tn;
      tile_coords(ui.tile, tiles_m2, p.tiles_n, group2, tm2, tn);
      const int tm = 2 * tm2 + static_cast<int>(rank);
      if (!__all_sync(0xffffffffu, ptx::mbar_wait_bounded(accf_bar(acc), acc_phase, abort_flag, p.wait_limit_ns))) break;
      ptx::tc_fence_after();
      const int row = tm * BM + lane_group * 32 + lane;
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(lane_group * 32) << 16) + static_cast<uint32_t>(acc * BN);
      // K-split tile: this CTA's 128 rows of the fp32 partial live in scratch slot 2 * tile + rank
      float* part_row = nullptr;
      bool ok = true;
      if (ui.role == 1 || ui.role == 2) {
        const int slot = 2 * ui.tile + static_cast<int>(rank);
        part_row = p.split_scratch + static_cast<size_t>(slot) * BM * BN + (lane_group * 32 + lane) * 4;
        ok = split_hand_over<BN>(p, ui.role, slot, lane_group, lane, t_row, part_row, abort_flag);
      }
      epilogue_tile<BN, EPI, F8>(p, ui.role, ui.n_half, tm, tn, row, t_row, part_row, ok);
      ptx::tc_fence_before();
      __syncwarp();
      if (ui.role == 2 && lane == 0) {
        // the partner's partial has been consumed: lower the flag for the next launch
        __threadfence();
        *reinterpret_cast<volatile int*>(p.split_flags + (2 * ui.tile + static_cast<int>(rank)) * 4 + lane_group) = 0;
      }
      if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(acce_bar(acc), 0));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();  // neither CTA leaves (or frees tensor memory) while its peer may still signal it
  if (*abort_flag && threadIdx.x == 0 && p.err_word) atomicExch(p.err_word, 1);
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

// Bytes of L2 a raster group's A slab may occupy while the B tiles stream past it.  The slab stays resident because
// every one of its tiles is re-read for each column tile; PD_RASTER_MB in the environment overrides the size (for
// sweeps).
long long raster_slab_bytes() {
  static const long long bytes = [] {
    const char* v = std::getenv("PD_RASTER_MB");
    const long long mb = v ? std::atoll(v) : 0;
    return (mb > 0 ? mb : 64) << 20;  // half of the 126 MB L2: with K = 14336 the weight matrix is then streamed twice, not three to four times
  }();
  return bytes;
}

// SM count of the current device (remembered per device ordinal).
int sm_count() {
  static PerDeviceInt memo;
  int n = memo.get();
  if (n > 0) return n;
  int dev = 0;
  n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
    n = 148;
  memo.set(n);
  return n;
}

template <int BN, int EPI, bool F8>
pd_status launch_tc(const GemmArgs& g, cudaStream_t stream) {
  using Cfg = GemmCfg<BN>;
  static PerDeviceInt smem_opt_in;
  auto kern = gemm_tc_kernel<BN, EPI, F8>;
  PD_TRY(opt_in_smem(smem_opt_in, kern, Cfg::SMEM_BYTES));
  CUtensorMap ta, tb;
  if (F8) {
    PD_TRY(make_tmap_u8(&ta, g.a, g.m, g.k, g.lda, BM));
    PD_TRY(make_tmap_u8(&tb, g.b, g.n, g.k, g.ldb, BN));
  } else {
    PD_TRY(make_tmap_bf16(&ta, g.a, g.m, g.k, g.lda, BM));
    PD_TRY(make_tmap_bf16(&tb, g.b, g.n, g.k, g.ldb, BN));
  }
  GemmDev p{};
  p.scale_a = g.scale_a; p.scale_b = g.scale_b;
  p.c = g.c; p.r = g.r; p.m = g.m; p.n = g.n; p.k = g.k; p.ldc = g.ldc; p.ldr = g.ldr;
  p.tiles_m = (g.m + BM - 1) / BM;
  p.tiles_n = (g.n + BN - 1) / BN;
  p.err_word = g.err_word;
  p.wait_limit_ns = 4000000000ull;
  if (take_wait_injection(PD_INJECT_GEMM, &p.wait_limit_ns)) p.test_skip_load = 1;
  {
    // keep a group's A slab (group x 128 rows x K) within the L2 share given to it
    long long grp = raster_slab_bytes() / (static_cast<long long>(BM) * g.k * 2);
    p.raster_group = static_cast<int>(grp < 4 ? 4 : (grp > 32 ? 32 : grp));
  }
  if (EPI == EPI_ROPE_KV) p.rope = *g.rope;
  const int tiles = p.tiles_m * p.tiles_n;
  const int sms = sm_count();
  p.n_units = tiles;
  p.main_tiles = tiles;
  p.split_scratch = nullptr; p.split_flags = nullptr; p.split_enable = 0;
  p.tail_halves = 0;
  {
    // last wave holds `tail` tiles: if they occupy at most half of the SMs, cut each in two along K
    const int tail = tiles % sms;
    const size_t need = static_cast<size_t>(tail) * BM * BN * sizeof(float);
    // (pays only for long K: with K = 4096 the parked partial tile and the hand-over cost as much as the
    // half tile they save; measured -6 % on the K = 14336 down projection, +5 % on the K = 4096 ones)
    if (tail > 0 && 2 * tail <= sms && g.k / (F8 ? BK_F8 : BK) >= 128 && g.split_scratch && g.split_flags &&
        need <= g.split_scratch_bytes && tail <= kSplitMaxTiles) {
      p.main_tiles = tiles - tail;
      p.n_units = tiles + tail;
      p.split_scratch = g.split_scratch; p.split_flags = g.split_flags; p.split_enable = 1;
    } else if (BN == 256 && tail > 0 && 2 * tail <= sms && g.n % 256 == 0) {
      // otherwise give the two 128-column halves of every tail tile to different blocks
      p.main_tiles = tiles - tail;
      p.n_units = tiles + tail;
      p.tail_halves = 1;
    }
  }
  const int grid = p.n_units < sms ? p.n_units : sms;
  PD_CUDA_TRY(launch_pdl(kern, dim3(grid), dim3(GEMM_THREADS), Cfg::SMEM_BYTES, stream, ta, tb, p));
  count_launch();
  return PD_OK;
}

// CTA pairs resident at once for the pair kernel (0: clusters of two cannot be placed).
template <int EPI, bool F8>
int pair_capacity() {
  static PerDeviceInt memo;  // per device: the opt-in below and the occupancy answer are the device's
  const int known = memo.get();
  if (known >= 0) return known;
  auto kern = gemm_tc_pair_kernel<EPI, F8>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, P2_SMEM_BYTES) != cudaSuccess) {
    memo.set(0);
    return 0;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(2 * sm_count());
  cfg.blockDim = dim3(GEMM_THREADS);
  cfg.dynamicSmemBytes = P2_SMEM_BYTES;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
  memo.set(n);
  return n;
}

template <int EPI, bool F8>
pd_status launch_tc_pair(const GemmArgs& g, cudaStream_t stream) {
  auto kern = gemm_tc_pair_kernel<EPI, F8>;
  const int cap = pair_capacity<EPI, F8>();
  if (cap <= 0) return PD_ERR_UNSUPPORTED_SHAPE;
  CUtensorMap ta, tb, tbh;
  if (F8) {
    PD_TRY(make_tmap_u8(&ta, g.a, g.m, g.k, g.lda, BM));
    PD_TRY(make_tmap_u8(&tb, g.b, g.n, g.k, g.ldb, 128));
    PD_TRY(make_tmap_u8(&tbh, g.b, g.n, g.k, g.ldb, 64));
  } else {
    PD_TRY(make_tmap_bf16(&ta, g.a, g.m, g.k, g.lda, BM));
    PD_TRY(make_tmap_bf16(&tb, g.b, g.n, g.k, g.ldb, 128));
    PD_TRY(make_tmap_bf16(&tbh, g.b, g.n, g.k, g.ldb, 64));
  }
  GemmDev p{};
  p.scale_a = g.scale_a; p.scale_b = g.scale_b;
  p.c = g.c; p.r = g.r; p.m = g.m; p.n = g.n; p.k = g.k; p.ldc = g.ldc; p.ldr = g.ldr;
  p.tiles_m = (g.m + BM - 1) / BM;
  p.tiles_n = g.n / 256;
  p.err_word = g.err_word;
  p.wait_limit_ns = 4000000000ull;
  if (take_wait_injection(PD_INJECT_GEMM_PAIR, &p.wait_limit_ns)) p.test_skip_load = 1;
  {
    long long grp = raster_slab_bytes() / (static_cast<long long>(BM) * g.k * (F8 ? 1 : 2));
    p.raster_group = static_cast<int>(grp < 4 ? 4 : (grp > 32 ? 32 : grp));
  }
  if (EPI == EPI_ROPE_KV) p.rope = *g.rope;
  const int units = ((p.tiles_m + 1) / 2) * p.tiles_n;
  p.n_units = units; p.main_tiles = units;
  // Few tiles (short batches against N = d_model): when the tiles would fill at most half of the pairs, every tile
  // is cut in two along K and the halves run on two pairs at once; the first parks its fp32 partial in the scratch,
  // the second adds it before its epilogue (the hand-over of the single-CTA kernel's tail split).
  const size_t split_need = static_cast<size_t>(2 * units) * BM * 256 * sizeof(float);
  // (pays only for long K, like the tail split: the hand-over costs about as much as 4096 elements of K)
  if (2 * units <= cap && g.k / (F8 ? BK_F8 : BK) >= 128 && g.split_scratch && g.split_flags &&
      split_need <= g.split_scratch_bytes && 2 * units <= kSplitMaxTiles) {
    p.split_all = 1;
    p.n_units = 2 * units;
    p.split_scratch = g.split_scratch; p.split_flags = g.split_flags;
  } else {
    // the last wave holds `tail` tiles: if they occupy at most half of the pairs, run each as two 128-column halves
    const int tail = units % cap;
    if (tail > 0 && 2 * tail <= cap) {
      p.main_tiles = units - tail;
      p.n_units = units + tail;
      p.tail_halves = 1;
    }
  }
  const int pairs = p.n_units < cap ? p.n_units : cap;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(GEMM_THREADS);
  cfg.dynamicSmemBytes = P2_SMEM_BYTES;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 2 : 1;
  PD_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, ta, tb, tbh, p));
  count_launch();
  return PD_OK;
}

template <bool F8>
pd_status launch_tc_pair_epi(const GemmArgs& g, cudaStream_t stream) {
  switch (g.epilogue) {
    case EPI_RESIDUAL: return launch_tc_pair<EPI_RESIDUAL, F8>(g, stream);
    case EPI_SWIGLU: return launch_tc_pair<EPI_SWIGLU, F8>(g, stream);
    case EPI_ROPE_KV: return launch_tc_pair<EPI_ROPE_KV, F8>(g, stream);
    default: return launch_tc_pair<EPI_STORE, F8>(g, stream);
  }
}

template <int BN, bool F8>
pd_status launch_tc_epi(const GemmArgs& g, cudaStream_t stream) {
  switch (g.epilogue) {
    case EPI_RESIDUAL: return launch_tc<BN, EPI_RESIDUAL, F8>(g, stream);
    case EPI_SWIGLU:
      if constexpr (BN >= 128) return launch_tc<BN, EPI_SWIGLU, F8>(g, stream);
      return PD_ERR_UNSUPPORTED_SHAPE;
    case EPI_ROPE_KV:
      if constexpr (BN >= 128) return launch_tc<BN, EPI_ROPE_KV, F8>(g, stream);
      return PD_ERR_UNSUPPORTED_SHAPE;
    default: return launch_tc<BN, EPI_STORE, F8>(g, stream);
  }
}

}  // namespace

int gemm_block_n(int m, int n, int epilogue) {
  // Pick the tile width by a small cost model: waves over the SMs times a measured relative
  // per-tile time.  Narrow tiles re-read A from shared memory for fewer columns and keep the
  // tensor pipe only about 55 % busy against 85 % for the 256-wide tile, so they pay off only
  // when they remove a mostly idle wave.  The fused epilogues need whole heads / gate-up pairs
  // in a tile, so they do not use the 64-wide tile.
  const int sms = sm_count();
  const int tiles_m = (m + BM - 1) / BM;
  const bool fused = epilogue == EPI_SWIGLU || epilogue == EPI_ROPE_KV;
  int best = 256;
  double best_cost = 1e300;
  const int cands[3] = {256, 128, 64};
  for (int bn : cands) {
    if (bn == 64 && fused) continue;
    if (bn > n && bn != (fused ? 128 : 64)) continue;
    const long long tiles = 1ll * tiles_m * ((n + bn - 1) / bn);
    const long long waves = (tiles + sms - 1) / sms;
    const double cost = static_cast<double>(waves) * (bn == 256 ? 1.0 : (bn == 128 ? 0.77 : 0.47));
    if (cost < best_cost) { best_cost = cost; best = bn; }
  }
  return best;
}

// Eligible problems (256-wide tiles, N a multiple of 256, more than one row tile) run on the CTA-pair kernel;
// PD_GEMM_PAIRS=0 in the environment keeps them on the single-CTA kernel (for A/B timing).
static int pair_mode() {
  static const int mode = [] {
    const char* v = std::getenv("PD_GEMM_PAIRS");
    return (v && v[0] == '0') ? 0 : 1;
  }();
  return mode;
}

static pd_status check_gemm_args(const GemmArgs& g) {
  if (!g.a || !g.b || !g.c || g.m < 0 || g.n <= 0 || g.k <= 0) return PD_ERR_INVALID_ARG;
  if (g.epilogue == EPI_RESIDUAL && !g.r) return PD_ERR_INVALID_ARG;
  if (g.epilogue == EPI_ROPE_KV && !g.rope) return PD_ERR_INVALID_ARG;
  if (g.fp8 && (!g.scale_a || !g.scale_b)) return PD_ERR_INVALID_ARG;
  if (g.k % (g.fp8 ? BK_F8 : BK) != 0 || g.n % 16 != 0) return PD_ERR_UNSUPPORTED_SHAPE;
  const int opa = g.fp8 ? 16 : 8;  // operand row pitches: multiples of 16 bytes
  if (g.lda % opa || g.ldb % opa || g.ldc % 8 || (g.epilogue == EPI_RESIDUAL && g.ldr % 8)) return PD_ERR_UNSUPPORTED_SHAPE;
  if (g.epilogue == EPI_SWIGLU && g.n % 128 != 0) return PD_ERR_UNSUPPORTED_SHAPE;
  return PD_OK;
}

pd_status gemm(const GemmArgs& g, cudaStream_t stream) {
  PD_TRY(check_gemm_args(g));
  if (g.m == 0) return PD_OK;
  const int bn = gemm_block_n(g.m, g.n, g.epilogue);
  // Short batches against a narrow N with a long K (the down projection at a few hundred tokens): the pair kernel
  // with every tile cut in two along K keeps all SMs busy with 256-wide tiles, which beats one wave of narrow
  // single-CTA tiles (measured 73.7 -> 61.5 us at 512 x 4096 x 14336; at K = 4096 the hand-over costs more than the
  // half main loop it saves, 28.7 -> 34.8 us, so short K stays on the narrow tiles).
  bool pair_split = false;
  if (g.n % 256 == 0 && g.m > BM && g.split_scratch && g.split_flags) {
    const int units = ((g.m + 2 * BM - 1) / (2 * BM)) * (g.n / 256);
    pair_split = 2 * units <= sm_count() / 2 && g.k / (g.fp8 ? BK_F8 : BK) >= 128 &&
                 static_cast<size_t>(2 * units) * BM * 256 * sizeof(float) <= g.split_scratch_bytes;
  }
  if ((bn == 256 || pair_split) && g.n % 256 == 0 && g.m > BM && pair_mode() != 0) {
    const pd_status st = g.fp8 ? launch_tc_pair_epi<true>(g, stream) : launch_tc_pair_epi<false>(g, stream);
    if (st != PD_ERR_UNSUPPORTED_SHAPE) return st;  // (clusters of two could not be placed: single-CTA kernel)
  }
  if (g.fp8) {
    switch (bn) {
      case 256: return launch_tc_epi<256, true>(g, stream);
      case 128: return launch_tc_epi<128, true>(g, stream);
      default: return launch_tc_epi<64, true>(g, stream);
    }
  }
  switch (bn) {
    case 256: return launch_tc_epi<256, false>(g, stream);
    case 128: return launch_tc_epi<128, false>(g, stream);
    default: return launch_tc_epi<64, false>(g, stream);
  }
}

}  // namespace pd

extern "C" pd_status pd_gemm_bf16(const void* a, const void* b, void* c, int32_t m, int32_t n, int32_t k,
                                  int32_t* err_word, void* stream) {
  pd::GemmArgs g{};
  g.a = static_cast<const pd::bf16*>(a);
  g.b = static_cast<const pd::bf16*>(b);
  g.c = static_cast<pd::bf16*>(c);
  g.r = nullptr;
  g.m = m; g.n = n; g.k = k;
  g.lda = k; g.ldb = k; g.ldc = n; g.ldr = 0;
  g.epilogue = pd::EPI_STORE;
  g.err_word = err_word;
  return pd::gemm(g, static_cast<cudaStream_t>(stream));
}

// Workspace layout of pd_gemm_bf16_ws: the hand-over flags (cleared by the call), then the fp32 partial tiles.
static constexpr size_t kGemmWsFlagBytes = (pd::kSplitMaxTiles * 4 * sizeof(int) + 255) / 256 * 256;

extern "C" pd_status pd_gemm_workspace_bytes(size_t* out_bytes) {
  if (!out_bytes) return PD_ERR_INVALID_ARG;
  *out_bytes = kGemmWsFlagBytes + pd::kSplitScratchBytes;
  return PD_OK;
}

extern "C" pd_status pd_gemm_bf16_ws(const void* a, const void* b, void* c, int32_t m, int32_t n, int32_t k,
                                     void* workspace, size_t workspace_bytes, int32_t* err_word, void* stream) {
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return PD_ERR_INVALID_ARG;
  if (workspace_bytes < kGemmWsFlagBytes + pd::kSplitScratchBytes) return PD_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  PD_CUDA_TRY(cudaMemsetAsync(workspace, 0, kGemmWsFlagBytes, st));
  pd::GemmArgs g{};
  g.a = static_cast<const pd::bf16*>(a);
  g.b = static_cast<const pd::bf16*>(b);
  g.c = static_cast<pd::bf16*>(c);
  g.m = m; g.n = n; g.k = k;
  g.lda = k; g.ldb = k; g.ldc = n; g.ldr = 0;
  g.epilogue = pd::EPI_STORE;
  g.err_word = err_word;
  g.split_flags = static_cast<int*>(workspace);
  g.split_scratch = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + kGemmWsFlagBytes);
  g.split_scratch_bytes = pd::kSplitScratchBytes;
  return pd::gemm(g, st);
}

extern "C" pd_status pd_gemm_fp8(const void* a_codes, const float* a_scales, const void* b_codes, const float* b_scales,
                                 void* c, int32_t m, int32_t n, int32_t k, int32_t* err_word, void* stream) {
  pd::GemmArgs g{};
  g.a = static_cast<const pd::bf16*>(a_codes);
  g.b = static_cast<const pd::bf16*>(b_codes);
  g.c = static_cast<pd::bf16*>(c);
  g.m = m; g.n = n; g.k = k;
  g.lda = k; g.ldb = k; g.ldc = n; g.ldr = 0;
  g.epilogue = pd::EPI_STORE;
  g.fp8 = 1; g.scale_a = a_scales; g.scale_b = b_scales;
  g.err_word = err_word;
  return pd::gemm(g, static_cast<cudaStream_t>(stream));
}
