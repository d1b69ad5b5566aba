// Decode attention (the prefill kernel lives in pd_attn_prefill_tc.cu).
//
// Memory-bound.  One block per (split of the KV range, KV head, sequence).  The G query heads
// of the group are the (zero-padded) 16 rows of a warp-level MMA, so each K/V row is read from
// HBM once and used by all G heads.  Every warp streams its own 16-key tiles through a private
// 3-stage cp.async ring (16-byte loads, no block-wide barrier in the loop), keeps an online
// softmax per row with warp shuffles, and the warps' and splits' partial (max, sum, output)
// triples are merged at the end.
#include <math_constants.h>

#include "pd_common.cuh"
#include "pd_ptx.cuh"

namespace pd {
namespace {

constexpr float LOG2E = 1.4426950408889634f;

// Byte offset of 16-byte chunk `c` of row `r` in a tile whose rows are HD bf16 long; chunks
// are XOR-swizzled by the row so that ldmatrix reads are free of bank conflicts.
template <int HD>
__device__ __forceinline__ uint32_t tile_off(int r, int c) {
  return static_cast<uint32_t>(r * (HD * 2) + ((c ^ (r & 7)) << 4));
}

// =================================================================== decode
constexpr int DC_WARPS = 4;
constexpr int DC_THREADS = DC_WARPS * 32;
constexpr int DC_KEYS = 16;   // keys per warp tile
constexpr int DC_STAGES = 3;

template <int HD>
struct DecodeSmem {
  static constexpr int TILE_BYTES = DC_KEYS * HD * 2;               // one K (or V) tile of one warp
  static constexpr int WARP_BYTES = DC_STAGES * 2 * TILE_BYTES;     // K and V, all stages
  static constexpr int RING_BYTES = DC_WARPS * WARP_BYTES;
  static constexpr int MERGE_BYTES = DC_WARPS * 16 * (HD + 2) * 4;  // per-warp (o, m, l) of 16 rows
  static constexpr int BYTES = RING_BYTES > MERGE_BYTES ? RING_BYTES : MERGE_BYTES;
};

template <int HD>
__global__ void __launch_bounds__(DC_THREADS) decode_attn_kernel(DecodeAttnArgs a) {
  constexpr int CPR = HD / 8;
  using SM = DecodeSmem<HD>;
  extern __shared__ __align__(128) uint8_t smem[];
  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int group = a.n_q_heads / a.n_kv_heads;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t4 = lane & 3;
  // q and the newest K/V row come from the kernel before this one
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();

  const int total = min(a.kv_len[b] + 1, a.len_cap);
  // split the key range into n_splits runs whose length is a multiple of the block's 64-key step
  const int step = DC_WARPS * DC_KEYS;
  const int per_split = ((total + a.n_splits - 1) / a.n_splits + step - 1) / step * step;
  const int k_begin = min(total, split * per_split);
  const int k_end = min(total, k_begin + per_split);

  const bf16* kbase = a.k_cache + (static_cast<size_t>(b) * a.n_kv_heads + kvh) * a.len_cap * HD;
  const bf16* vbase = a.v_cache + (static_cast<size_t>(b) * a.n_kv_heads + kvh) * a.len_cap * HD;

  // Q fragments of the group's heads (rows >= G are zero); scores are scaled into log2 units
  const float sl2 = rsqrtf(static_cast<float>(HD)) * LOG2E;
  uint32_t qa[HD / 16][4];
  {
    const bf16* qrow = a.q + static_cast<size_t>(b) * a.ldq + (kvh * group) * HD;
#pragma unroll
    for (int kk = 0; kk < HD / 16; ++kk) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int r = g + (e & 1) * 8;
        const int c = kk * 16 + t4 * 2 + (e >> 1) * 8;
        qa[kk][e] = (r < group) ? *reinterpret_cast<const uint32_t*>(qrow + r * HD + c) : 0u;
      }
    }
  }

  const uint32_t s_warp = ptx::smem_u32(smem) + warp * SM::WARP_BYTES;
  // tile i of this warp covers keys k_begin + (i * DC_WARPS + warp) * 16 ...
  const int n_tiles_blk = (k_end - k_begin + DC_KEYS - 1) / DC_KEYS;
  const int my_tiles = (n_tiles_blk > warp) ? (n_tiles_blk - warp + DC_WARPS - 1) / DC_WARPS : 0;
  auto tile_key0 = [&](int i) { return k_begin + (i * DC_WARPS + warp) * DC_KEYS; };
  auto load_tile = [&](int i, int stage) {
    const int key0 = tile_key0(i);
    const uint32_t sk = s_warp + stage * 2 * SM::TILE_BYTES;
    const uint32_t sv = sk + SM::TILE_BYTES;
#pragma unroll
    for (int j = lane; j < DC_KEYS * CPR; j += 32) {
      const int r = j / CPR, c = j - r * CPR;
      const bool ok = (key0 + r) < k_end;
      const size_t off = static_cast<size_t>(ok ? key0 + r : 0) * HD + c * 8;
      ptx::cp_async_16(sk + tile_off<HD>(r, c), kbase + off, ok);
      ptx::cp_async_16(sv + tile_off<HD>(r, c), vbase + off, ok);
    }
  };
#pragma unroll
  for (int s = 0; s < DC_STAGES - 1; ++s) {
    if (s < my_tiles) load_tile(s, s);
    ptx::cp_async_commit();
  }

  float o_acc[HD / 8][4];
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) o_acc[i][0] = o_acc[i][1] = o_acc[i][2] = o_acc[i][3] = 0.f;
  float m_row[2] = {-CUDART_INF_F, -CUDART_INF_F};
  float l_row[2] = {0.f, 0.f};

  for (int i = 0; i < my_tiles; ++i) {
    const int stage = i % DC_STAGES;
    {
      const int nxt = i + DC_STAGES - 1;
      if (nxt < my_tiles) load_tile(nxt, nxt % DC_STAGES);
      ptx::cp_async_commit();
    }
    ptx::cp_async_wait<DC_STAGES - 1>();
    __syncwarp();
    const uint32_t sk = s_warp + stage * 2 * SM::TILE_BYTES;
    const uint32_t sv = sk + SM::TILE_BYTES;
    const int key0 = tile_key0(i);

    float s_acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
    for (int kk = 0; kk < HD / 16; ++kk) {
      uint32_t b0, b1, b2, b3;
      ptx::ldmatrix_x4(sk + tile_off<HD>((lane & 7) + (lane >> 4) * 8, kk * 2 + ((lane >> 3) & 1)), b0, b1, b2, b3);
      ptx::mma_bf16_16816(s_acc[0], qa[kk], b0, b1);
      ptx::mma_bf16_16816(s_acc[1], qa[kk], b2, b3);
    }
    float tmax[2] = {-CUDART_INF_F, -CUDART_INF_F};
    const bool tail = key0 + DC_KEYS > k_end;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        s_acc[nt][e] *= sl2;
        if (tail && key0 + nt * 8 + t4 * 2 + (e & 1) >= k_end) s_acc[nt][e] = -CUDART_INF_F;
        tmax[e >> 1] = fmaxf(tmax[e >> 1], s_acc[nt][e]);
      }
    }
    float corr[2];
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      tmax[rr] = fmaxf(tmax[rr], __shfl_xor_sync(0xffffffffu, tmax[rr], 1));
      tmax[rr] = fmaxf(tmax[rr], __shfl_xor_sync(0xffffffffu, tmax[rr], 2));
      const float m_new = fmaxf(m_row[rr], tmax[rr]);  // finite: every tile holds at least one valid key
      corr[rr] = exp2f(m_row[rr] - m_new);
      m_row[rr] = m_new;
    }
    uint32_t pa[4];
    {
      const float p00 = exp2f(s_acc[0][0] - m_row[0]), p01 = exp2f(s_acc[0][1] - m_row[0]);
      const float p02 = exp2f(s_acc[0][2] - m_row[1]), p03 = exp2f(s_acc[0][3] - m_row[1]);
      const float p10 = exp2f(s_acc[1][0] - m_row[0]), p11 = exp2f(s_acc[1][1] - m_row[0]);
      const float p12 = exp2f(s_acc[1][2] - m_row[1]), p13 = exp2f(s_acc[1][3] - m_row[1]);
      l_row[0] = l_row[0] * corr[0] + (p00 + p01 + p10 + p11);
      l_row[1] = l_row[1] * corr[1] + (p02 + p03 + p12 + p13);
      pa[0] = ptx::pack_bf16(p00, p01);
      pa[1] = ptx::pack_bf16(p02, p03);
      pa[2] = ptx::pack_bf16(p10, p11);
      pa[3] = ptx::pack_bf16(p12, p13);
    }
    // rescale only when some row's running maximum moved (warp-uniform decision)
    if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {
#pragma unroll
      for (int n = 0; n < HD / 8; ++n) {
        o_acc[n][0] *= corr[0]; o_acc[n][1] *= corr[0];
        o_acc[n][2] *= corr[1]; o_acc[n][3] *= corr[1];
      }
    }
#pragma unroll
    for (int np = 0; np < HD / 16; ++np) {
      uint32_t b0, b1, b2, b3;
      ptx::ldmatrix_x4_trans(sv + tile_off<HD>((lane & 7) + ((lane >> 3) & 1) * 8, np * 2 + (lane >> 4)), b0, b1, b2, b3);
      ptx::mma_bf16_16816(o_acc[2 * np], pa, b0, b1);
      ptx::mma_bf16_16816(o_acc[2 * np + 1], pa, b2, b3);
    }
    __syncwarp();  // all lanes are done reading this stage before it is refilled
  }
  ptx::cp_async_wait<0>();
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    l_row[rr] += __shfl_xor_sync(0xffffffffu, l_row[rr], 1);
    l_row[rr] += __shfl_xor_sync(0xffffffffu, l_row[rr], 2);
  }
  __syncthreads();  // every warp has left its ring: the memory is reused for the merge

  // per-warp partials -> shared: [warp][row][HD + 2] floats (o, m, l); only rows < 8 can be heads
  // of the group when G <= 8, rows g + 8 matter only for G > 8.
  float* mrg = reinterpret_cast<float*>(smem);
  constexpr int RS = HD + 2;
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    const int r = g + rr * 8;
    if (r < group) {
      float* dst = mrg + (warp * 16 + r) * RS;
#pragma unroll
      for (int n = 0; n < HD / 8; ++n) {
        dst[n * 8 + t4 * 2] = o_acc[n][rr * 2];
        dst[n * 8 + t4 * 2 + 1] = o_acc[n][rr * 2 + 1];
      }
      if (t4 == 0) {
        dst[HD] = m_row[rr];
        dst[HD + 1] = l_row[rr];
      }
    }
  }
  __syncthreads();
  for (int idx = tid; idx < group * HD; idx += DC_THREADS) {
    const int r = idx / HD, d = idx - r * HD;
    float m = -CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < DC_WARPS; ++w) m = fmaxf(m, mrg[(w * 16 + r) * RS + HD]);
    float l = 0.f, o = 0.f;
    if (m != -CUDART_INF_F) {
#pragma unroll
      for (int w = 0; w < DC_WARPS; ++w) {
        const float* src = mrg + (w * 16 + r) * RS;
        const float sc = exp2f(src[HD] - m);  // 0 for a warp that saw no key
        l += src[HD + 1] * sc;
        o += src[d] * sc;
      }
    }
    if (a.n_splits == 1) {
      // (a sequence with no visible entry at all, kv_len < 0, gives zeros rather than 0 / 0)
      a.o[static_cast<size_t>(b) * (a.n_q_heads * HD) + (kvh * group + r) * HD + d] = __float2bfloat16(l > 0.f ? o / l : 0.f);
    } else {
      float* dst = a.partial +
                   (((static_cast<size_t>(b) * a.n_kv_heads + kvh) * a.n_splits + split) * group + r) * RS;
      dst[d] = o;
      if (d == 0) {
        dst[HD] = m;
        dst[HD + 1] = l;
      }
    }
  }
}

// Merge of the splits' partials: one block per (sequence, query head), one thread per feature.
template <int HD>
__global__ void __launch_bounds__(HD) decode_combine_kernel(DecodeAttnArgs a) {
  constexpr int RS = HD + 2;
  const int b = blockIdx.y, hq = blockIdx.x, d = threadIdx.x;
  const int group = a.n_q_heads / a.n_kv_heads;
  const int kvh = hq / group, r = hq - kvh * group;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  const float* base = a.partial + ((static_cast<size_t>(b) * a.n_kv_heads + kvh) * a.n_splits) * group * RS;
  float m = -CUDART_INF_F;
  for (int s = 0; s < a.n_splits; ++s) m = fmaxf(m, base[(s * group + r) * RS + HD]);
  float l = 0.f, o = 0.f;
  for (int s = 0; s < a.n_splits; ++s) {
    const float* src = base + (s * group + r) * RS;
    const float ms = src[HD];
    if (ms == -CUDART_INF_F) continue;  // empty split
    const float sc = exp2f(ms - m);
    l += src[HD + 1] * sc;
    o += src[d] * sc;
  }
  a.o[static_cast<size_t>(b) * (a.n_q_heads * HD) + hq * HD + d] = __float2bfloat16(l > 0.f ? o / l : 0.f);
}

template <int HD>
pd_status launch_decode_hd(const DecodeAttnArgs& a, cudaStream_t s) {
  using SM = DecodeSmem<HD>;
  static PerDeviceInt smem_opt_in;
  PD_TRY(opt_in_smem(smem_opt_in, decode_attn_kernel<HD>, SM::BYTES));
  dim3 grid(a.n_splits, a.n_kv_heads, a.batch);
  PD_CUDA_TRY(launch_pdl(decode_attn_kernel<HD>, grid, dim3(DC_THREADS), SM::BYTES, s, a));
  count_launch();
  if (a.n_splits > 1) {
    dim3 cgrid(a.n_q_heads, a.batch);
    PD_CUDA_TRY(launch_pdl(decode_combine_kernel<HD>, cgrid, dim3(HD), 0, s, a));
    count_launch();
  }
  return PD_OK;
}

}  // namespace

int decode_attention_splits(int batch, int n_kv_heads, int max_kv_len) {
  // One block per (sequence, KV head) already streams its range through four independent warp rings, so about
  // 110 blocks saturate HBM; below that the KV range is split to get there.  Above it a split only costs
  // (partials, the merge kernel: 5-13 % at uniform lengths), except that the grid is sized from the LONGEST
  // sequence: with ragged lengths an unsplit long sequence is a block that runs on alone after the others
  // have drained (measured 0.48 of the HBM rate at B = 16 with lengths spread 1 : 9).  So a block's key range
  // is capped at about 2048 keys; short sequences leave their later splits empty.  A split shorter than 512
  // keys never paid.
  const long long blocks = 1ll * batch * n_kv_heads;
  if (blocks <= 0) return 1;
  long long want = (112 + blocks - 1) / blocks;
  const long long by_len = (max_kv_len + 1024ll) / 2048;
  if (by_len > want) want = by_len;
  long long cap = max_kv_len / 512;
  if (cap < 1) cap = 1;
  if (want > cap) want = cap;
  if (want < 1) want = 1;
  if (want > 64) want = 64;
  return static_cast<int>(want);
}

pd_status launch_decode_attention(const DecodeAttnArgs& a, cudaStream_t s) {
  if (a.batch == 0) return PD_OK;
  if (a.n_splits > 1 && !a.partial) return PD_ERR_INVALID_ARG;
  if (a.head_dim == 128) return launch_decode_hd<128>(a, s);
  if (a.head_dim == 64) return launch_decode_hd<64>(a, s);
  return PD_ERR_UNSUPPORTED_SHAPE;
}

}  // namespace pd
