// Prefill attention on the 5th-generation tensor cores (tcgen05 + tensor memory), persistent.
//
// A work item is 256 consecutive query rows of one (request, query head): two row tiles of 128 whose
// softmax and MMAs ping-pong.  One block per SM stays resident and takes items, longest first, from a
// counter in global memory until none is left, so that barrier and tensor-memory set-up happen once per
// SM and the loads of the next item run while the current one drains.
//   warp 0      : producer  - fetches and decodes items, publishes them in a shared-memory ring, loads the
//                             K / V tiles of 128 keys (3 K slots, 2 V slots)
//   warp 10     : Q loader  - loads each item's Q tiles (one buffer per row tile) as the buffers fall free
//   warp 1      : MMA issuer - S = Q K^T (both operands in shared memory, fp32 S in tensor memory) and
//                             O += P V (P read from tensor memory, V as an MN-major operand); event driven:
//                             it issues whichever row tile's next product has its inputs ready, so a tile
//                             may run one K/V tile (and one item) ahead of the other
//   warps 2-5   : softmax of row tile 0, one query row per thread (a row lives in one tensor-memory
//   warps 6-9   : softmax of row tile 1  lane, so the row maximum and sum need no shuffles); they also
//                             normalise and store the tile's output rows at the end of an item
// Tensor memory (512 columns): per tile S (128 columns, later overwritten by P as packed bf16 in its
// first 64) and O (head_dim columns).
// The running maximum is updated lazily: O is rescaled only when a row's maximum grew by more than 2^8,
// which bounds p by 256 and makes the rescale rare after the first tiles.
// Keys beyond the request are masked in S; V rows beyond the request are zeroed in shared memory before
// use, because 0 * (uninitialised cache memory) must not produce NaN.
// All barriers run on counters that continue across items (parity = counter bit).  Every wait is
// wall-clock bounded and leaves through the common teardown.
// The three single-thread roles are functions that are never inlined: each gets registers of its own, apart
// from the softmax code, which needs every register the launch bounds allow.  The MMA issuer sets the pace
// of the kernel: the tensor pipe takes a 128 x 128 x 16 product instruction about every 62 cycles, its
// execution time, and queues hardly any, so the pipe is busy exactly while the thread issues and idles while
// the thread polls, commits and keeps its books.  Hence the plain code of that loop: state of it in local
// memory, polls placed between the instructions of a product, or a second issuing thread (the two
// instruction streams interleave in the pipe and every product finishes later) were all measured slower.
#include <math_constants.h>

#include <atomic>

#include "pd_common.cuh"
#include "pd_ptx.cuh"

namespace pd {
namespace {

constexpr int TQ = 128;                    // rows per tile
constexpr int TK = 128;                    // keys per KV tile
constexpr int ATT_THREADS = 352;
constexpr float LOG2E_F = 1.4426950408889634f;
constexpr float RESCALE_THRESHOLD = 8.0f;  // in log2 units
constexpr int K_SLOTS = 3, V_SLOTS = 2, ITEM_SLOTS = 4;

template <int HD>
struct AttCfg {
  static constexpr int SUB = HD / 64;                       // 64-column sub-tiles per row tile
  static constexpr int TILE_BYTES = TQ * HD * 2;            // one Q, K or V tile
  static constexpr int SUB_BYTES = TQ * 128;                // one 128-row x 64-column sub-tile
  static constexpr int Q_OFF = 0;                           // two Q tiles
  static constexpr int K_OFF = 2 * TILE_BYTES;
  static constexpr int V_OFF = K_OFF + K_SLOTS * TILE_BYTES;
  static constexpr int BAR_OFF = V_OFF + V_SLOTS * TILE_BYTES;
  static constexpr int SMEM_BYTES_MIN = BAR_OFF + 512 + 1024;
  // always ask for more than half of the SM's shared memory so that one block owns the SM
  // (two blocks could not both hold 512 tensor-memory columns)
  static constexpr int SMEM_BYTES = SMEM_BYTES_MIN > 120 * 1024 ? SMEM_BYTES_MIN : 120 * 1024;
  static constexpr int S_COL = 0, O_COL = 128, TILE_COLS = 256;  // tensor-memory columns of a row tile
};

// barrier indices
constexpr int B_QFULL = 0, B_QEMPTY = 2, B_KFULL = 4, B_KEMPTY = 7, B_VFULL = 10, B_VEMPTY = 12, B_SFULL = 14,
              B_PREADY = 16, B_ODONE = 18, B_OREAD = 20, B_IFULL = 22, B_IEMPTY = 26, N_BARS = 30;

struct AttDev {
  bf16* o;
  const int32_t* cu_seqlens;
  const int32_t* slots;
  const int32_t* prefix;
  int n_q_heads, n_kv_heads, len_cap, batch_cap;
  int n_req, n_zblocks, n_items;  // items = n_zblocks x n_req x n_q_heads, longest row blocks first
  int* sched;                     // [0] next item, [1] blocks that have finished; both zero between launches
  int* err_word;
  unsigned long long wait_limit_ns;
  int test_skip_load;             // test hook: the producer leaves out one K tile load (see launch_hd)
};

// A decoded work item as the producer publishes it (shared memory).
struct Item {
  int h, start, len, q0, pre, kv_row0, n_kv0, n_kv1;  // n_kv0 = -1: no more items
};

__device__ __forceinline__ bool decode_item(const AttDev& p, int idx, Item& it) {
  // longest first: the row block varies slowest (descending), then the request, the head fastest
  const int h = idx % p.n_q_heads;
  const int rest = idx / p.n_q_heads;
  const int req = rest % p.n_req;
  const int zi = rest / p.n_req;
  const int start = p.cu_seqlens[req];
  const int len = p.cu_seqlens[req + 1] - start;
  const int q0 = (p.n_zblocks - 1 - zi) * (2 * TQ);
  if (q0 >= len) return false;
  const int slot = p.slots ? p.slots[req] : req;
  if (slot < 0 || slot >= p.batch_cap) return false;  // reported by the QKV epilogue
  const int pre = p.prefix ? p.prefix[req] : 0;       // tokens of this request already in the cache (chunked prefill)
  const int kvh = h / (p.n_q_heads / p.n_kv_heads);
  it.h = h; it.start = start; it.len = len; it.q0 = q0; it.pre = pre;
  it.kv_row0 = (slot * p.n_kv_heads + kvh) * p.len_cap;  // first cache row of this (sequence, KV head)
  it.n_kv0 = (pre + min(len, q0 + TQ) + TK - 1) / TK;    // KV tiles row tile 0 attends to
  it.n_kv1 = (q0 + TQ < len) ? (pre + min(len, q0 + 2 * TQ) + TK - 1) / TK : 0;  // >= n_kv0 when the tile exists
  return true;
}

// The MMA issuer's loop, one thread.  A function of its own (never inlined), so that its registers are allocated
// apart from the softmax code, whose pressure would otherwise push this loop's state into local memory.
template <int HD>
__device__ __noinline__ void mma_issuer(const uint32_t smem_base, const uint32_t tmem_base, const uint32_t bar0,
                                        const Item* item_ring, volatile int* abort_flag, const uint64_t limit) {
  using Cfg = AttCfg<HD>;
  auto bar = [&](int i) { return bar0 + 8u * i; };
  constexpr uint32_t idesc_qk = ptx::umma_idesc_bf16(TQ, TK);
  constexpr uint32_t idesc_pv = ptx::umma_idesc_bf16_bmn(TQ, HD);
  // Per row tile: the item it is working on and how far it has got.  The two tiles walk the same item
  // sequence and share the K / V rings, but each advances as soon as its own inputs are ready.
  Item cur[2];
  bool have[2] = {false, false}, done[2] = {false, false};
  int seq[2] = {0, 0};      // items taken from the ring so far
  int base[2] = {0, 0};     // ring position of the current item's first K / V tile
  int n[2] = {0, 0};        // K / V tiles of the current item for this row tile
  int jq[2] = {0, 0};       // next Q K^T to issue
  int jp[2] = {0, 0};       // next P V to issue
  int act[2] = {0, 0};      // items with work for this row tile finished so far
  int pv_cnt[2] = {0, 0};   // P V products issued so far (phase of p_ready)
  uint32_t k_used = 0, v_used = 0;  // users that have consumed the tile in each ring slot, 4 bits per slot
  uint64_t t_idle = 0;
  uint32_t idle_polls = 0;
  bool ok = true;
  while (ok && !(done[0] && done[1])) {
    bool progress = false;
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      if (done[t]) continue;
      if (!have[t]) {
        const int s = seq[t] & (ITEM_SLOTS - 1);
        if (!ptx::mbar_test_wait(bar(B_IFULL + s), (seq[t] / ITEM_SLOTS) & 1)) continue;
        cur[t] = item_ring[s];
        ptx::mbar_arrive(bar(B_IEMPTY + s));
        ++seq[t];
        progress = true;
        if (cur[t].n_kv0 < 0) { done[t] = true; continue; }
        n[t] = t == 0 ? cur[t].n_kv0 : cur[t].n_kv1;
        if (n[t] == 0) {  // this item has rows for the other tile only
          base[t] += max(cur[t].n_kv0, cur[t].n_kv1);
          continue;
        }
        have[t] = true; jq[t] = 0; jp[t] = 0;
      }
      const Item& it = cur[t];
      if (jp[t] < jq[t]) {
        // ---- O_t += P_t V_j
        const int j = jp[t], g = base[t] + j, s = g % V_SLOTS;
        if (!ptx::mbar_test_wait(bar(B_PREADY + t), pv_cnt[t] & 1)) continue;
        if (!ptx::mbar_test_wait(bar(B_VFULL + s), (g / V_SLOTS) & 1)) continue;
        // the first product of an item overwrites O: the previous item's output must have been read out
        if (j == 0 && act[t] > 0 && !ptx::mbar_test_wait(bar(B_OREAD + t), (act[t] - 1) & 1)) continue;
        ptx::tc_fence_after();
        const uint32_t sv = smem_base + Cfg::V_OFF + s * Cfg::TILE_BYTES;
        const uint32_t d = tmem_base + t * Cfg::TILE_COLS + Cfg::O_COL;
        const uint32_t a = tmem_base + t * Cfg::TILE_COLS + Cfg::S_COL;
#pragma unroll
        for (int kk = 0; kk < TK / 16; ++kk) {
          // 16 keys = 16 rows of 128 bytes further into the V tile; 8 packed columns further into P
          ptx::umma_bf16_ts(d, a + kk * 8, ptx::umma_desc_mn_sw128(sv + kk * 2048, Cfg::SUB_BYTES), idesc_pv,
                            (j > 0 || kk > 0) ? 1u : 0u);
        }
        ptx::umma_commit(bar(B_ODONE + t));
        const uint32_t users = (j < it.n_kv0 ? 1u : 0u) + (j < it.n_kv1 ? 1u : 0u);
        v_used += 1u << (4 * s);
        if (((v_used >> (4 * s)) & 15u) == users) { ptx::umma_commit(bar(B_VEMPTY + s)); v_used &= ~(15u << (4 * s)); }
        ++pv_cnt[t]; ++jp[t];
        progress = true;
        if (jp[t] == n[t]) {  // item finished for this tile
          have[t] = false;
          ++act[t];
          base[t] += max(it.n_kv0, it.n_kv1);
          continue;
        }
      }
      if (jq[t] < n[t] && jq[t] == jp[t]) {
        // ---- S_t = Q_t K_j^T (S is free: the P that aliased it has been consumed by the product above)
        const int j = jq[t], g = base[t] + j, s = g % K_SLOTS;
        if (j == 0 && !ptx::mbar_test_wait(bar(B_QFULL + t), act[t] & 1)) continue;
        if (!ptx::mbar_test_wait(bar(B_KFULL + s), (g / K_SLOTS) & 1)) continue;
        ptx::tc_fence_after();
        const uint32_t sq = smem_base + Cfg::Q_OFF + t * Cfg::TILE_BYTES;
        const uint32_t sk = smem_base + Cfg::K_OFF + s * Cfg::TILE_BYTES;
        const uint32_t d = tmem_base + t * Cfg::TILE_COLS + Cfg::S_COL;
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          const uint32_t off = (kk >> 2) * Cfg::SUB_BYTES + (kk & 3) * 32;
          ptx::umma_bf16(d, ptx::umma_desc_sw128(sq + off), ptx::umma_desc_sw128(sk + off), idesc_qk, kk > 0 ? 1u : 0u);
        }
        ptx::umma_commit(bar(B_SFULL + t));
        const uint32_t users = (j < it.n_kv0 ? 1u : 0u) + (j < it.n_kv1 ? 1u : 0u);
        k_used += 1u << (4 * s);
        if (((k_used >> (4 * s)) & 15u) == users) { ptx::umma_commit(bar(B_KEMPTY + s)); k_used &= ~(15u << (4 * s)); }
        ++jq[t];
        if (jq[t] == n[t]) ptx::umma_commit(bar(B_QEMPTY + t));  // the tile's Q buffer may be refilled
        progress = true;
      }
    }
    if (progress) {
      idle_polls = 0;
      t_idle = 0;
    } else if ((++idle_polls & 1023u) == 0u) {
      // nothing could be issued for a while: look at the abort flag and the clock
      if (*abort_flag) { ok = false; break; }
      const uint64_t now = ptx::globaltimer_ns();
      if (t_idle == 0) t_idle = now;
      else if (now - t_idle > limit) { *abort_flag = 1; ok = false; }
    }
  }
}

// The producer's loop (one thread): work items, K and V tiles.  Like the MMA issuer a function of its own.
template <int HD>
__device__ __noinline__ void kv_producer(const CUtensorMap* tmap_k, const CUtensorMap* tmap_v, const AttDev& p,
                                         const uint32_t smem_base, const uint32_t bar0, Item* item_ring,
                                         volatile int* abort_flag, const uint64_t limit) {
  using Cfg = AttCfg<HD>;
  auto bar = [&](int i) { return bar0 + 8u * i; };
  int it_pub = 0;               // items published so far (ring position)
  int g_k = 0, g_v = 0;         // K / V tiles loaded so far (ring positions)
  bool ok = true;
  // the next item is fetched and decoded while the current one's tiles are being loaded
  auto fetch = [&](Item& it) {
    for (;;) {
      const int idx = atomicAdd(p.sched, 1);
      if (idx >= p.n_items) {
        it.h = it.start = it.len = it.q0 = it.pre = it.kv_row0 = it.n_kv1 = 0;
        it.n_kv0 = -1;
        return;
      }
      if (decode_item(p, idx, it)) return;  // (rows beyond a request's length: nothing to do)
    }
  };
  Item nxt;
  fetch(nxt);
  while (ok) {
    const Item it = nxt;
    const bool last = it.n_kv0 < 0;
    {
      const int s = it_pub & (ITEM_SLOTS - 1);
      if (!ptx::mbar_wait_bounded(bar(B_IEMPTY + s), ((it_pub / ITEM_SLOTS) & 1) ^ 1u, abort_flag, limit)) { ok = false; break; }
      item_ring[s] = it;
      ptx::mbar_arrive(bar(B_IFULL + s));  // release: the item is visible to whoever sees the phase flip
      ++it_pub;
    }
    if (last) break;
    const int n_max = max(it.n_kv0, it.n_kv1);
    for (int j = 0; j < n_max && ok; ++j) {
      // K and V slots are released separately: K as soon as the Q K^T products that use it have run, V only
      // after the P V products, so later K tiles are on their way while the softmax runs
      const int sk_i = g_k % K_SLOTS;
      if (!ptx::mbar_wait_bounded(bar(B_KEMPTY + sk_i), ((g_k / K_SLOTS) & 1) ^ 1u, abort_flag, limit)) { ok = false; break; }
      if (!(p.test_skip_load && g_k == 1)) {
        const uint32_t sk = smem_base + Cfg::K_OFF + sk_i * Cfg::TILE_BYTES;
        ptx::mbar_arrive_expect_tx(bar(B_KFULL + sk_i), Cfg::TILE_BYTES);
        for (int c = 0; c < Cfg::SUB; ++c)
          ptx::tma_load_2d(sk + c * Cfg::SUB_BYTES, tmap_k, c * 64, it.kv_row0 + j * TK, bar(B_KFULL + sk_i));
      }
      ++g_k;
      const int sv_i = g_v % V_SLOTS;
      if (!ptx::mbar_wait_bounded(bar(B_VEMPTY + sv_i), ((g_v / V_SLOTS) & 1) ^ 1u, abort_flag, limit)) { ok = false; break; }
      const uint32_t sv = smem_base + Cfg::V_OFF + sv_i * Cfg::TILE_BYTES;
      ptx::mbar_arrive_expect_tx(bar(B_VFULL + sv_i), Cfg::TILE_BYTES);
      for (int c = 0; c < Cfg::SUB; ++c)
        ptx::tma_load_2d(sv + c * Cfg::SUB_BYTES, tmap_v, c * 64, it.kv_row0 + j * TK, bar(B_VFULL + sv_i));
      ++g_v;
      if (j == 0) fetch(nxt);  // (after this item's first loads are on their way)
    }
  }
  if (!ok) {
    // give loads already in flight time to land before the block's shared memory is released
#pragma unroll 1
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
}

// The Q loader's loop (one thread).  Its own thread, so that a wait for one tile's Q buffer never holds up the K / V
// stream of the other tile.
template <int HD>
__device__ __noinline__ void q_loader(const CUtensorMap* tmap_q, const uint32_t smem_base, const uint32_t bar0,
                                      const Item* item_ring, volatile int* abort_flag, const uint64_t limit) {
  using Cfg = AttCfg<HD>;
  auto bar = [&](int i) { return bar0 + 8u * i; };
  int seq = 0;
  int q_cnt[2] = {0, 0};  // Q loads so far per row tile
  bool ok = true;
  while (ok) {
    const int s = seq & (ITEM_SLOTS - 1);
    if (!ptx::mbar_wait_bounded(bar(B_IFULL + s), (seq / ITEM_SLOTS) & 1, abort_flag, limit)) break;
    const Item it = item_ring[s];
    ptx::mbar_arrive(bar(B_IEMPTY + s));
    ++seq;
    if (it.n_kv0 < 0) break;
    for (int t = 0; t < 2; ++t) {
      if (t == 1 && it.n_kv1 == 0) break;
      // the tile's Q buffer is free once the last Q K^T of its previous item has been executed
      if (!ptx::mbar_wait_bounded(bar(B_QEMPTY + t), (q_cnt[t] & 1) ^ 1u, abort_flag, limit)) { ok = false; break; }
      ptx::mbar_arrive_expect_tx(bar(B_QFULL + t), Cfg::TILE_BYTES);
      for (int c = 0; c < Cfg::SUB; ++c)
        ptx::tma_load_2d(smem_base + Cfg::Q_OFF + t * Cfg::TILE_BYTES + c * Cfg::SUB_BYTES, tmap_q, it.h * HD + c * 64,
                         it.start + it.q0 + t * TQ, bar(B_QFULL + t));
      ++q_cnt[t];
    }
  }
  if (!ok) {
#pragma unroll 1
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
}

template <int HD>
__global__ void __launch_bounds__(ATT_THREADS, 1)
prefill_attn_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                       const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ AttDev p) {
  using Cfg = AttCfg<HD>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + Cfg::BAR_OFF);
  Item* item_ring = reinterpret_cast<Item*>(bars + N_BARS);  // ITEM_SLOTS entries of 32 bytes
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(item_ring + ITEM_SLOTS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = ptx::smem_u32(bars);
  auto bar = [&](int i) { return bar0 + 8u * i; };
  const uint64_t limit = p.wait_limit_ns;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int i = 0; i < N_BARS; ++i) {
      int count = 1;
      if (i >= B_PREADY && i < B_PREADY + 2) count = 4;             // the four softmax warps of the tile
      if (i >= B_OREAD && i < B_OREAD + 2) count = 4;
      if (i >= B_IEMPTY && i < B_IEMPTY + ITEM_SLOTS) count = 11;   // eight softmax warps, the MMA thread once per tile, the Q loader
      ptx::mbar_init(bar(i), count);
    }
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
  // are read, the output written and the item counter touched only after it has completed.
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();

  if (warp == 0) {
    // ---------------------------------------------------------------- producer
    if (lane == 0) kv_producer<HD>(&tmap_k, &tmap_v, p, smem_base, bar0, item_ring, abort_flag, limit);
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) mma_issuer<HD>(smem_base, tmem_base, bar0, item_ring, abort_flag, limit);
  } else if (warp == 10) {
    // ---------------------------------------------------------------- Q loader
    if (lane == 0) q_loader<HD>(&tmap_q, smem_base, bar0, item_ring, abort_flag, limit);
  } else {
    // ---------------------------------------------------------------- softmax
    const int t = (warp - 2) >> 2;       // row tile of this warpgroup
    const int lane_group = warp & 3;     // tensor-memory lanes this warp may touch
    const int row_in_tile = lane_group * 32 + lane;
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(lane_group * 32) << 16) + t * Cfg::TILE_COLS;
    const float sl2 = rsqrtf(static_cast<float>(HD)) * LOG2E_F;
    int seq = 0;    // items taken from the ring so far
    int base = 0;   // ring position of the current item's first K / V tile
    int step = 0;   // K/V tiles this row tile has processed so far, over all items (phase of s_full / o_done)
    bool ok = true;
    while (ok) {
      Item it;
      {
        const int s = seq & (ITEM_SLOTS - 1);
        ok = __all_sync(0xffffffffu, ptx::mbar_wait_bounded(bar(B_IFULL + s), (seq / ITEM_SLOTS) & 1, abort_flag, limit));
        if (!ok) break;
        it = item_ring[s];
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar(B_IEMPTY + s));
        ++seq;
      }
      if (it.n_kv0 < 0) break;  // no more items
      const int n_kv = t == 0 ? it.n_kv0 : it.n_kv1;
      const int item_base = base;
      base += max(it.n_kv0, it.n_kv1);
      if (n_kv == 0) continue;  // this item has rows for the other tile only
      const int row = it.q0 + t * TQ + row_in_tile;  // row inside the request's chunk
      const int row_pos = it.pre + row;              // its position = last key it may see
      const int kv_total = it.pre + it.len;          // keys this request has after the chunk
      const int kv_end = it.pre + min(it.len, it.q0 + t * TQ + TQ);
      float m_used = -CUDART_INF_F, l_sum = 0.f;
#pragma unroll 1
      for (int j = 0; j < n_kv; ++j, ++step) {
        ok = __all_sync(0xffffffffu, ptx::mbar_wait_bounded(bar(B_SFULL + t), step & 1, abort_flag, limit));
        if (!ok) break;
        ptx::tc_fence_after();
        const int k0 = j * TK;
        uint32_t sv[4][32];
#pragma unroll
        for (int c = 0; c < 4; ++c) ptx::tmem_ld_32x32(t_lane + Cfg::S_COL + c * 32, sv[c]);
        ptx::tmem_ld_wait();
        // raw scores stay in registers; the scale is folded into the exponent (scale > 0, so the
        // maximum can be taken on the raw values)
        const bool need_mask = (k0 + TK - 1 > it.pre + it.q0 + t * TQ) || (k0 + TK > kv_end);  // warp-uniform
        if (need_mask) {
          // keys with index above `lim` (inside this tile) are invisible to this row: one compare per key
          const int lim = min(row_pos, kv_end - 1) - k0;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
#pragma unroll
            for (int e = 0; e < 32; ++e)
              if (c * 32 + e > lim) sv[c][e] = 0xff800000u;  // -inf
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
          ok = __all_sync(0xffffffffu, ptx::mbar_wait_bounded(bar(B_ODONE + t), (step - 1) & 1, abort_flag, limit));
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
          const int g = item_base + j, sv_i = g % V_SLOTS;
          ok = __all_sync(0xffffffffu, ptx::mbar_wait_bounded(bar(B_VFULL + sv_i), (g / V_SLOTS) & 1, abort_flag, limit));
          if (!ok) break;
          if (k0 + row_in_tile >= kv_total) {
            uint8_t* svm = smem_al + Cfg::V_OFF + sv_i * Cfg::TILE_BYTES;
#pragma unroll
            for (int c = 0; c < Cfg::SUB; ++c) {
              uint4* dst = reinterpret_cast<uint4*>(svm + c * Cfg::SUB_BYTES + row_in_tile * 128);
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
      if (!ok) break;
      // ---- the item's last P V product has finished: normalise and store the tile's rows
      ok = __all_sync(0xffffffffu, ptx::mbar_wait_bounded(bar(B_ODONE + t), (step - 1) & 1, abort_flag, limit));
      if (!ok) break;
      ptx::tc_fence_after();
      const float inv = 1.f / l_sum;
      bf16* dst = p.o + static_cast<size_t>(it.start + row) * (p.n_q_heads * HD) + it.h * HD;
      // the whole row first, so that the next item's first product may overwrite O as early as possible
      uint32_t ov[HD / 32][32];
#pragma unroll
      for (int c = 0; c < HD / 32; ++c) ptx::tmem_ld_32x32(t_lane + Cfg::O_COL + c * 32, ov[c]);
      ptx::tmem_ld_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar(B_OREAD + t));
      if (row < it.len) {
        // a thread owns a row, so every store of a warp touches 32 different lines: 32-byte stores halve their number
#pragma unroll
        for (int c = 0; c < HD / 32; ++c) {
#pragma unroll
          for (int e = 0; e < 32; e += 16) {
            uint32_t w[8];
#pragma unroll
            for (int q = 0; q < 8; ++q)
              w[q] = ptx::pack_bf16(__uint_as_float(ov[c][e + 2 * q]) * inv, __uint_as_float(ov[c][e + 2 * q + 1]) * inv);
            ptx::st_global_v8(dst + c * 32 + e, w);
          }
        }
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    if (*abort_flag && p.err_word) atomicExch(p.err_word, 1);
    // the block that finishes last puts the item counter back to zero for the next launch
    __threadfence();
    if (atomicAdd(p.sched + 1, 1) == static_cast<int>(gridDim.x) - 1) {
      atomicExch(p.sched, 0);
      atomicExch(p.sched + 1, 0);
    }
  }
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

// Item counters for launches that come without a layer object (pd_prefill_attention): a small pool in the
// library image, handed out round robin.  A counter pair is zero whenever no launch that uses it is running,
// so launches that follow each other on a stream may share one; launches that can overlap on the GPU get
// different ones as long as fewer than kSchedPool of them are in flight.
constexpr int kSchedPool = 64;
__device__ int g_sched_pool[2 * kSchedPool];
std::atomic<unsigned> g_sched_next{0};

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
  p.n_req = a.n_req;
  p.n_zblocks = (a.max_len + 2 * TQ - 1) / (2 * TQ);
  const long long items = 1ll * p.n_zblocks * a.n_req * a.n_q_heads;
  if (items > 0x3fffffffll) return PD_ERR_UNSUPPORTED_SHAPE;
  p.n_items = static_cast<int>(items);
  p.wait_limit_ns = a.wait_limit_ns ? a.wait_limit_ns : 4000000000ull;
  p.test_skip_load = a.test_skip_load;
  {
    unsigned long long inj = 0;
    if (take_wait_injection(PD_INJECT_ATTN_PREFILL, &inj)) { p.wait_limit_ns = inj; p.test_skip_load = 1; }
  }
  p.sched = a.sched;
  if (!p.sched) {
    int* pool = nullptr;
    PD_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&pool), g_sched_pool));
    p.sched = pool + 2 * (g_sched_next.fetch_add(1, std::memory_order_relaxed) % kSchedPool);
  }
  int sms = 0, dev = 0;
  PD_CUDA_TRY(cudaGetDevice(&dev));
  PD_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int grid = static_cast<int>(items < sms ? items : sms);
  PD_CUDA_TRY(launch_pdl(kern, dim3(grid), dim3(ATT_THREADS), Cfg::SMEM_BYTES, s, tq, tk, tv, p));
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
