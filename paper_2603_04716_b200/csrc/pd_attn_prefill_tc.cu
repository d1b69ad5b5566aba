// Prefill attention on the 5th-generation tensor cores (tcgen05 + tensor memory).
//
// One block owns 256 consecutive query rows of one (request, query head): two row tiles of 128
// that ping-pong, so the softmax of one tile overlaps the MMAs of the other.
//   warp 0      : TMA producer - Q tiles once, then K and V tiles of 128 keys through a 2-stage ring
//   warp 1      : MMA issuer   - S = Q K^T (both operands in shared memory, fp32 S in tensor memory),
//                                O += P V (P read from tensor memory, V as an MN-major operand)
//   warps 2-5   : softmax of row tile 0, one query row per thread (a row lives in one tensor-memory
//   warps 6-9   : softmax of row tile 1  lane, so the row maximum and sum need no shuffles)
// Tensor memory (512 columns): per tile S (128 columns, later overwritten by P as packed bf16 in
// its first 64) and O (head_dim columns).
// The running maximum is updated lazily: O is rescaled only when a row's maximum grew by more
// than 2^8, which bounds p by 256 and makes the rescale rare after the first tiles.
// Keys beyond the request are masked in S; V rows beyond the request are zeroed in shared memory
// before use, because 0 * (uninitialised cache memory) must not produce NaN.
// Every wait is wall-clock bounded and leaves through the common teardown.
#include <math_constants.h>

#include "pd_common.cuh"
#include "pd_ptx.cuh"

namespace pd {
namespace {

constexpr int TQ = 128;                    // rows per tile
constexpr int TK = 128;                    // keys per KV tile
constexpr int ATT_THREADS = 320;
constexpr float LOG2E_F = 1.4426950408889634f;
constexpr float RESCALE_THRESHOLD = 8.0f;  // in log2 units

template <int HD>
struct AttCfg {
  static constexpr int SUB = HD / 64;                       // 64-column sub-tiles per row tile
  static constexpr int TILE_BYTES = TQ * HD * 2;            // one Q, K or V tile
  static constexpr int SUB_BYTES = TQ * 128;                // one 128-row x 64-column sub-tile
  static constexpr int Q_OFF = 0;
  static constexpr int KV_OFF = 2 * TILE_BYTES;             // stage s: K at KV_OFF + s*2*TILE, V after it
  static constexpr int BAR_OFF = KV_OFF + 4 * TILE_BYTES;
  static constexpr int SMEM_BYTES_MIN = BAR_OFF + 256 + 1024;
  // always ask for more than half of the SM's shared memory so that one block owns the SM
  // (two blocks could not both hold 512 tensor-memory columns)
  static constexpr int SMEM_BYTES = SMEM_BYTES_MIN > 120 * 1024 ? SMEM_BYTES_MIN : 120 * 1024;
  static constexpr int S_COL = 0, O_COL = 128, TILE_COLS = 256;  // tensor-memory columns of a row tile
};

struct AttDev {
  bf16* o;
  const int32_t* cu_seqlens;
  const int32_t* slots;
  const int32_t* prefix;
  int n_q_heads, n_kv_heads, len_cap, batch_cap;
  int* err_word;
};

template <int HD>
__global__ void __launch_bounds__(ATT_THREADS, 1)
prefill_attn_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                       const __grid_constant__ CUtensorMap tmap_v, AttDev p) {
  using Cfg = AttCfg<HD>;
  // Launch order = longest blocks first over the whole grid: the block index that varies slowest is the row
  // block, descending, so every head and request runs its last (longest-range) rows before anybody's short ones
  // and no long block is left to start when the rest of the grid is about to drain.
  const int h = blockIdx.x, req = blockIdx.y;
  const int start = p.cu_seqlens[req];
  const int len = p.cu_seqlens[req + 1] - start;
  const int q0 = (gridDim.z - 1 - blockIdx.z) * (2 * TQ);
  if (q0 >= len) return;
  const int slot = p.slots ? p.slots[req] : req;
  if (slot < 0 || slot >= p.batch_cap) return;  // reported by the QKV epilogue
  const int pre = p.prefix ? p.prefix[req] : 0;  // tokens of this request already in the cache (chunked prefill)
  const int kv_total = pre + len;                // keys this request has after the chunk
  const int kvh = h / (p.n_q_heads / p.n_kv_heads);
  const int kv_row0 = (slot * p.n_kv_heads + kvh) * p.len_cap;  // first cache row of this (sequence, KV head)

  // per row tile: number of KV tiles it attends to
  int n_kv[2];
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const int r0 = q0 + t * TQ;
    n_kv[t] = (r0 < len) ? (pre + min(len, r0 + TQ) + TK - 1) / TK : 0;
  }
  const int n_max = max(n_kv[0], n_kv[1]);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + Cfg::BAR_OFF);
  // 0 q_full | 1,2 k_full | 3,4 v_full | 5,6 v_empty | 7,8 s_full | 9,10 p_ready | 11,12 o_done | 13,14 k_empty
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 15);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = ptx::smem_u32(bars);
  auto bar = [&](int i) { return bar0 + 8u * i; };
  constexpr int B_QFULL = 0, B_KFULL = 1, B_VFULL = 3, B_VEMPTY = 5, B_SFULL = 7, B_PREADY = 9, B_ODONE = 11,
                B_KEMPTY = 13;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int i = 0; i < 15; ++i) ptx::mbar_init(bar(i), (i == B_PREADY || i == B_PREADY + 1) ? 4 : 1);
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmap_q);
    ptx::prefetch_tensormap(&tmap_k);
    ptx::prefetch_tensormap(&tmap_v);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_slot), 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Programmatic dependent launch: the set-up above may overlap the tail of the QKV projection; q and the cache
  // are read, and the output written, only after it has completed.
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();

  if (warp == 0) {
    // ---------------------------------------------------------------- producer
    if (lane == 0) {
      const int n_q = (n_kv[1] > 0) ? 2 : 1;
      ptx::mbar_arrive_expect_tx(bar(B_QFULL), n_q * Cfg::TILE_BYTES);
      for (int t = 0; t < n_q; ++t)
        for (int c = 0; c < Cfg::SUB; ++c)
          ptx::tma_load_2d(smem_base + Cfg::Q_OFF + t * Cfg::TILE_BYTES + c * Cfg::SUB_BYTES, &tmap_q, h * HD + c * 64,
                           start + q0 + t * TQ, bar(B_QFULL));
      bool ok = true;
      for (int j = 0; j < n_max && ok; ++j) {
        const int s = j & 1;
        // K and V slots are released separately: K as soon as both tiles' Q K^T have been issued,
        // V only after the P V products, so the next K tile is on its way while the softmax runs
        if (!ptx::mbar_wait_bounded(bar(B_KEMPTY + s), ((j >> 1) & 1) ^ 1u, abort_flag)) { ok = false; break; }
        const uint32_t sk = smem_base + Cfg::KV_OFF + s * 2 * Cfg::TILE_BYTES;
        const uint32_t sv = sk + Cfg::TILE_BYTES;
        ptx::mbar_arrive_expect_tx(bar(B_KFULL + s), Cfg::TILE_BYTES);
        for (int c = 0; c < Cfg::SUB; ++c)
          ptx::tma_load_2d(sk + c * Cfg::SUB_BYTES, &tmap_k, c * 64, kv_row0 + j * TK, bar(B_KFULL + s));
        if (!ptx::mbar_wait_bounded(bar(B_VEMPTY + s), ((j >> 1) & 1) ^ 1u, abort_flag)) { ok = false; break; }
        ptx::mbar_arrive_expect_tx(bar(B_VFULL + s), Cfg::TILE_BYTES);
        for (int c = 0; c < Cfg::SUB; ++c)
          ptx::tma_load_2d(sv + c * Cfg::SUB_BYTES, &tmap_v, c * 64, kv_row0 + j * TK, bar(B_VFULL + s));
      }
      if (!ok) {
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = ptx::umma_idesc_bf16(TQ, TK);
      constexpr uint32_t idesc_pv = ptx::umma_idesc_bf16_bmn(TQ, HD);
      bool ok = true;
      auto issue_s = [&](int t, int j) {  // S_t = Q_t K_j^T; the last tile to use K_j releases its slot
        const int s = j & 1;
        const uint32_t sq = smem_base + Cfg::Q_OFF + t * Cfg::TILE_BYTES;
        const uint32_t sk = smem_base + Cfg::KV_OFF + s * 2 * Cfg::TILE_BYTES;
        const uint32_t d = tmem_base + t * Cfg::TILE_COLS + Cfg::S_COL;
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          const uint32_t off = (kk >> 2) * Cfg::SUB_BYTES + (kk & 3) * 32;
          ptx::umma_bf16(d, ptx::umma_desc_sw128(sq + off), ptx::umma_desc_sw128(sk + off), idesc_qk, kk > 0 ? 1u : 0u);
        }
        ptx::umma_commit(bar(B_SFULL + t));
        if (t == 1 || j >= n_kv[1]) ptx::umma_commit(bar(B_KEMPTY + s));
      };
      auto issue_pv = [&](int t, int j) {  // O_t += P_t V_j
        const int s = j & 1;
        const uint32_t sv = smem_base + Cfg::KV_OFF + s * 2 * Cfg::TILE_BYTES + Cfg::TILE_BYTES;
        const uint32_t d = tmem_base + t * Cfg::TILE_COLS + Cfg::O_COL;
        const uint32_t a = tmem_base + t * Cfg::TILE_COLS + Cfg::S_COL;
#pragma unroll
        for (int kk = 0; kk < TK / 16; ++kk) {
          // 16 keys = 16 rows of 128 bytes further into the V tile; 8 packed columns further into P
          ptx::umma_bf16_ts(d, a + kk * 8, ptx::umma_desc_mn_sw128(sv + kk * 2048, Cfg::SUB_BYTES), idesc_pv,
                            (j > 0 || kk > 0) ? 1u : 0u);
        }
        ptx::umma_commit(bar(B_ODONE + t));
      };
      if (!ptx::mbar_wait_bounded(bar(B_QFULL), 0u, abort_flag)) ok = false;
      if (ok && !ptx::mbar_wait_bounded(bar(B_KFULL + 0), 0u, abort_flag)) ok = false;
      if (ok) {
        ptx::tc_fence_after();
        for (int t = 0; t < 2; ++t)
          if (n_kv[t] > 0) issue_s(t, 0);
      }
      for (int j = 0; j < n_max && ok; ++j) {
        const int s = j & 1;
        bool v_waited = false;
        for (int t = 0; t < 2 && ok; ++t) {
          if (j >= n_kv[t]) continue;
          if (!ptx::mbar_wait_bounded(bar(B_PREADY + t), j & 1, abort_flag)) { ok = false; break; }
          if (!v_waited) {
            if (!ptx::mbar_wait_bounded(bar(B_VFULL + s), (j >> 1) & 1, abort_flag)) { ok = false; break; }
            v_waited = true;
          }
          ptx::tc_fence_after();
          issue_pv(t, j);
          const bool last_user = (t == 1) || (j >= n_kv[1]);
          if (last_user) ptx::umma_commit(bar(B_VEMPTY + s));
          if (j + 1 < n_kv[t]) {
            if (!ptx::mbar_wait_bounded(bar(B_KFULL + (s ^ 1)), ((j + 1) >> 1) & 1, abort_flag)) { ok = false; break; }
            ptx::tc_fence_after();
            issue_s(t, j + 1);
          }
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- softmax
    const int t = (warp - 2) >> 2;       // row tile of this warpgroup
    const int lane_group = warp & 3;     // tensor-memory lanes this warp may touch
    const int row_in_tile = lane_group * 32 + lane;
    const int row = q0 + t * TQ + row_in_tile;  // row inside the request's chunk
    const int row_pos = pre + row;              // its position = last key it may see
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(lane_group * 32) << 16) + t * Cfg::TILE_COLS;
    const float sl2 = rsqrtf(static_cast<float>(HD)) * LOG2E_F;
    const int kv_end = pre + min(len, q0 + t * TQ + TQ);
    float m_used = -CUDART_INF_F, l_sum = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kv[t]; ++j) {
      ok = __all_sync(0xffffffffu, ptx::mbar_wait_bounded(bar(B_SFULL + t), j & 1, abort_flag));
      if (!ok) break;
      ptx::tc_fence_after();
      const int k0 = j * TK;
      uint32_t sv[4][32];
#pragma unroll
      for (int c = 0; c < 4; ++c) ptx::tmem_ld_32x32(t_lane + Cfg::S_COL + c * 32, sv[c]);
      ptx::tmem_ld_wait();
      // raw scores stay in registers; the scale is folded into the exponent (scale > 0, so the
      // maximum can be taken on the raw values)
      const bool need_mask = (k0 + TK - 1 > pre + q0 + t * TQ) || (k0 + TK > kv_end);  // warp-uniform
      if (need_mask) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const int key = k0 + c * 32 + e;
            if (key > row_pos || key >= kv_end) sv[c][e] = 0xff800000u;  // -inf
          }
        }
      }
      // row maximum: four independent chains of three-input maxima (the softmax warps set the pace of the
      // kernel, so their instruction count and dependency depth are what is being minimised here)
      float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
      for (int c = 0; c < 4; ++c) {
#pragma unroll
        for (int e = 0; e < 32; e += 2)
          mx4[(e >> 1) & 3] = ptx::fmax3(mx4[(e >> 1) & 3], __uint_as_float(sv[c][e]), __uint_as_float(sv[c][e + 1]));
      }
      float mx = ptx::fmax3(fmaxf(mx4[0], mx4[1]), mx4[2], mx4[3]);
      mx *= sl2;
      // lazy maximum: keep the old reference unless this tile exceeds it by more than the threshold
      float factor = 1.f;
      bool grow = false;
      if (j == 0) {
        m_used = mx;  // finite: key 0 is visible to every row
      } else if (mx > m_used + RESCALE_THRESHOLD) {
        factor = ptx::ex2_approx(m_used - mx);
        m_used = mx;
        grow = true;
      }
      if (__any_sync(0xffffffffu, grow)) {
        // O must be stable: the P V product of the previous tile has finished
        ok = __all_sync(0xffffffffu, ptx::mbar_wait_bounded(bar(B_ODONE + t), (j - 1) & 1, abort_flag));
        if (!ok) break;
        ptx::tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t ov[32];
          ptx::tmem_ld_32x32(t_lane + Cfg::O_COL + c * 32, ov);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 32; ++e) ov[e] = __float_as_uint(__uint_as_float(ov[e]) * factor);
          ptx::tmem_st_32x32(t_lane + Cfg::O_COL + c * 32, ov);
        }
        ptx::tmem_st_wait();
        l_sum *= factor;
      }
      // p = 2^(s * scale - m) for a pair of keys at a time: one packed FMA, two exponentials, one packed add.
      // (Evaluating a share of the exponentials with a polynomial on the FMA pipe was measured slower, 300 us
      // against 199 us at L_in 4096: the two row tiles alternate, so a scheduler mostly runs one softmax warp at
      // a time and the polynomial's dependent chain is exposed.)
      const uint64_t sl2_2 = ptx::pack_f32x2(sl2, sl2);
      const uint64_t negm_2 = ptx::pack_f32x2(-m_used, -m_used);
      uint64_t ps[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t pk[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          // packed column 32 c + e holds keys 2 (32 c + e) and 2 (32 c + e) + 1
          const int k_lo = (c * 32 + e) * 2;
          const uint64_t x2 = ptx::pack_f32x2(__uint_as_float(sv[k_lo >> 5][k_lo & 31]),
                                              __uint_as_float(sv[k_lo >> 5][(k_lo & 31) + 1]));
          float y0, y1;
          ptx::unpack_f32x2(ptx::fma_f32x2(x2, sl2_2, negm_2), y0, y1);
          const float p0 = ptx::ex2_approx(y0), p1 = ptx::ex2_approx(y1);
          ps[e & 3] = ptx::add_f32x2(ps[e & 3], ptx::pack_f32x2(p0, p1));
          pk[e] = ptx::pack_bf16(p0, p1);
        }
        ptx::tmem_st_32x32(t_lane + Cfg::S_COL + c * 32, pk);
      }
      {
        float a0, a1;
        ptx::unpack_f32x2(ptx::add_f32x2(ptx::add_f32x2(ps[0], ps[1]), ptx::add_f32x2(ps[2], ps[3])), a0, a1);
        l_sum += a0 + a1;
      }
      ptx::tmem_st_wait();
      // the request's last tile may reach past its end: zero those V rows (0 * garbage must stay 0)
      if (k0 + TK > kv_total) {
        // S being ready only proves that K has landed; V has its own barrier
        ok = __all_sync(0xffffffffu, ptx::mbar_wait_bounded(bar(B_VFULL + (j & 1)), (j >> 1) & 1, abort_flag));
        if (!ok) break;
        if (k0 + row_in_tile >= kv_total) {
          const uint32_t svm = smem_base + Cfg::KV_OFF + (j & 1) * 2 * Cfg::TILE_BYTES + Cfg::TILE_BYTES;
#pragma unroll
          for (int c = 0; c < Cfg::SUB; ++c) {
            uint4* dst = reinterpret_cast<uint4*>(smem_al + (svm - smem_base) + c * Cfg::SUB_BYTES + row_in_tile * 128);
#pragma unroll
            for (int q = 0; q < 8; ++q) dst[q] = make_uint4(0u, 0u, 0u, 0u);
          }
        }
        ptx::fence_proxy_async();
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar(B_PREADY + t));
    }
    if (ok && n_kv[t] > 0) {
      ok = __all_sync(0xffffffffu, ptx::mbar_wait_bounded(bar(B_ODONE + t), (n_kv[t] - 1) & 1, abort_flag));
      if (ok) {
        ptx::tc_fence_after();
        const float inv = 1.f / l_sum;
        bf16* dst = p.o + static_cast<size_t>(start + row) * (p.n_q_heads * HD) + h * HD;
#pragma unroll 1
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t ov[32];
          ptx::tmem_ld_32x32(t_lane + Cfg::O_COL + c * 32, ov);
          ptx::tmem_ld_wait();
          if (row < len) {
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
              uint4 o;
              o.x = ptx::pack_bf16(__uint_as_float(ov[e]) * inv, __uint_as_float(ov[e + 1]) * inv);
              o.y = ptx::pack_bf16(__uint_as_float(ov[e + 2]) * inv, __uint_as_float(ov[e + 3]) * inv);
              o.z = ptx::pack_bf16(__uint_as_float(ov[e + 4]) * inv, __uint_as_float(ov[e + 5]) * inv);
              o.w = ptx::pack_bf16(__uint_as_float(ov[e + 6]) * inv, __uint_as_float(ov[e + 7]) * inv);
              *reinterpret_cast<uint4*>(dst + c * 32 + e) = o;
            }
          }
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
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

template <int HD>
pd_status launch_hd(const PrefillAttnArgs& a, int* err_word, cudaStream_t s) {
  using Cfg = AttCfg<HD>;
  static PerDeviceInt smem_opt_in;
  auto kern = prefill_attn_tc_kernel<HD>;
  PD_TRY(opt_in_smem(smem_opt_in, kern, Cfg::SMEM_BYTES));
  CUtensorMap tq, tk, tv;
  const uint64_t cache_rows = static_cast<uint64_t>(a.batch_cap) * a.n_kv_heads * a.len_cap;
  PD_TRY(make_tmap_bf16(&tq, a.q, a.n_tokens, static_cast<uint64_t>(a.n_q_heads) * HD, a.ldq, TQ));
  PD_TRY(make_tmap_bf16(&tk, a.k_cache, cache_rows, HD, HD, TK));
  PD_TRY(make_tmap_bf16(&tv, a.v_cache, cache_rows, HD, HD, TK));
  AttDev p{};
  p.o = a.o; p.cu_seqlens = a.cu_seqlens; p.slots = a.slots; p.prefix = a.prefix;
  p.n_q_heads = a.n_q_heads; p.n_kv_heads = a.n_kv_heads; p.len_cap = a.len_cap; p.batch_cap = a.batch_cap;
  p.err_word = err_word;
  dim3 grid(a.n_q_heads, a.n_req, (a.max_len + 2 * TQ - 1) / (2 * TQ));
  if (grid.y > 65535u || grid.z > 65535u) return PD_ERR_UNSUPPORTED_SHAPE;
  PD_CUDA_TRY(launch_pdl(kern, grid, dim3(ATT_THREADS), Cfg::SMEM_BYTES, s, tq, tk, tv, p));
  count_launch();
  return PD_OK;
}

}  // namespace

pd_status launch_prefill_attention_tc(const PrefillAttnArgs& a, int* err_word, cudaStream_t s) {
  if (a.n_tokens == 0 || a.n_req == 0 || a.max_len == 0) return PD_OK;
  if (a.head_dim == 128) return launch_hd<128>(a, err_word, s);
  if (a.head_dim == 64) return launch_hd<64>(a, err_word, s);
  return PD_ERR_UNSUPPORTED_SHAPE;
}

}  // namespace pd
