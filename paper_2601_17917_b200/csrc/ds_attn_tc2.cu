// ds_attn_pruned, tensor-core path for bf16 when the stacked query rows of a KV head fill more than one
// 128-row M-tile (GQA groups, wide windows, the unpruned reference, a cache-refresh step): there the
// problem is bound by the tensor cores and the softmax, not by the KV stream, and the shape of the kernel
// follows.
//
// Work item = (batch, KV head, PAIR of 128-row M-tiles).  Both tiles of a pair use every KV tile once
// from shared memory (half the shared-memory and L2 traffic per MMA of the one-tile kernel), and the
// softmax warps alternate with the tensor pipe: while they exponentiate S_a of KV tile j, the pipe runs
// P_b V and Q_b K^T; then the roles swap.
//
// Warp roles (320 threads, one CTA per SM):
//   warps 0-7  softmax + epilogue, M-tile a then M-tile b of every KV tile: half a row (64 columns) per
//              thread, the two halves of a row in the two half-warps (16x32bx2 TMEM accesses)
//   warp  8    TMA producer (prefix tiles by tiled boxes, tail rows gathered through the index list)
//   warp  9    TMEM allocation, MMA issue (one elected lane), in the order
//              P_a V(j-1), Q_a K(j)^T, P_b V(j-1), Q_b K(j)^T
// TMEM: S_a, S_b, O_a, O_b, 128 columns each.  P (bf16) overwrites the first 64 columns of its S; the
// single in-order issuer makes Q K^T of tile j + 1 follow P V of tile j, the only reader of that P, and
// "S of tile j is complete" (a commit after Q K^T) therefore also says that P V of tile j - 1 has
// completed, which is what the lazy rescale of O needs.
//
// Every wait is a bounded mbarrier wait; on expiry DS_DEV_TIMEOUT is raised, the CTA drains and frees
// TMEM.
#include <cuda.h>

#include <cstring>


#include "ds_attn_tiles.cuh"
#include "ds_common.cuh"
#include "ds_sm100.cuh"

namespace ds {
namespace {

using namespace sm100;
using namespace attn;

constexpr int kThreads2 = 320;
constexpr int kProducerWarp = 8, kMmaWarp = 9;
constexpr float kRescaleThreshold = 8.0f;  // log2 units

template <int D>
struct Geo2 {
  static constexpr int kChunks = D / 64;
  static constexpr int kTileBytes = kChunks * kChunkBytes;
  static constexpr int kSlots = (D == 128) ? 4 : 8;
  static constexpr int kOffQ = 0;                       // [2 tiles]
  static constexpr int kOffRing = 2 * kTileBytes;
  static constexpr int kOffBar = kOffRing + kSlots * kTileBytes;
  // barriers: q_full, q_free, s_full[2], p_full[2], o_full, o_free[2], slot_full[kSlots], slot_empty[kSlots]
  static constexpr int kNumBars = 11 + 2 * kSlots;   // + pv_done[2] (single-tile items)
  static constexpr int kOffIdx = kOffBar + 8 * kNumBars;
  static constexpr int kOffIdxQ = kOffIdx + 4 * 128;
  static constexpr int kOffIdxCache = kOffIdxQ + 4 * 128;
  static constexpr int kOffMisc = kOffIdxCache + 4 * kIdxCap;
  static constexpr int kSmemBytes = kOffMisc + 16 + 1024;
  static constexpr int kTmemS = 0, kTmemO = 256;        // + 128 for tile b
};
static_assert(Geo2<128>::kSmemBytes <= 227 * 1024 && Geo2<64>::kSmemBytes <= 227 * 1024, "shared memory budget");

struct Tc2Params : AttnCommon {
  int n_pairs;  // pairs of M-tiles per (batch, KV head)
  int n_items;  // B * Hkv * n_pairs
};

struct Item2 {
  int b, hk, pr, rows_a, rows_b;  // rows of the two tiles (rows_b = 0: the pair has one tile)
};
__device__ __forceinline__ Item2 decode_item2(const Tc2Params &prm, int item) {
  Item2 it;
  it.pr = item % prm.n_pairs;
  const int bh = item / prm.n_pairs;
  it.hk = bh % prm.Hkv;
  it.b = listed_batch(prm, bh / prm.Hkv);
  const int left = prm.G * prm.Lq - it.pr * 2 * kBlockM;
  it.rows_a = min(kBlockM, left);
  it.rows_b = max(0, min(kBlockM, left - kBlockM));
  return it;
}

template <int D>
__global__ void __launch_bounds__(kThreads2, 1) attn_tc2_kernel(const __grid_constant__ Tc2Params prm) {
  using G_ = Geo2<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  const uint32_t bar0 = sbase + G_::kOffBar;
  const uint32_t bar_q_full = bar0;
  const uint32_t bar_q_free = bar0 + 8;
  const uint32_t bar_s_full = bar0 + 16;  // [2] by M-tile
  const uint32_t bar_p_full = bar0 + 32;  // [2] by M-tile
  const uint32_t bar_o_full = bar0 + 48;
  const uint32_t bar_o_free = bar0 + 56;  // [2] by M-tile
  const uint32_t bar_slot_full = bar0 + 72;
  const uint32_t bar_slot_empty = bar_slot_full + 8 * G_::kSlots;
  const uint32_t bar_pv_done = bar_slot_empty + 8 * G_::kSlots;  // [2] by S buffer, items with one M-tile only
  int32_t *idx_s = reinterpret_cast<int32_t *>(smem + G_::kOffIdx);
  int32_t *idxq_s = reinterpret_cast<int32_t *>(smem + G_::kOffIdxQ);
  volatile uint32_t *tmem_base_s = reinterpret_cast<volatile uint32_t *>(smem + G_::kOffMisc);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + G_::kOffMisc + 4);

  const int n_pre = (prm.P + kBlockN - 1) / kBlockN;
  const int n_tail = (prm.Lq + kBlockN - 1) / kBlockN;
  const int n_tiles = n_pre + n_tail;

  if (tid == 0) {
    mbar_init(bar_q_full, 1);
    mbar_init(bar_q_free, 1);
    mbar_init(bar_s_full, 1);
    mbar_init(bar_s_full + 8, 1);
    mbar_init(bar_p_full, 8);
    mbar_init(bar_p_full + 8, 8);
    mbar_init(bar_o_full, 1);
    mbar_init(bar_o_free, 8);
    mbar_init(bar_o_free + 8, 8);
    mbar_init(bar_pv_done, 1);
    mbar_init(bar_pv_done + 8, 1);
    for (int s = 0; s < G_::kSlots; ++s) {
      mbar_init(bar_slot_full + 8 * s, 1);
      mbar_init(bar_slot_empty + 8 * s, 1);
    }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == kMmaWarp) tmem_alloc(sbase + G_::kOffMisc, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_base_s;
  // sequences (hence work items) of this launch: all, or the listed ones with the count read on the device
  const int n_live = live_sequences(prm);
  const int n_items = n_live * prm.Hkv * prm.n_pairs;
  bool timed_out = false;

  if (warp == kProducerWarp) {
    // ============================ TMA producer ============================
    bool bad_index = bad_sequence_numbers(prm, n_live);
    if (lane == 0) {
      auto prefetch_map = [](const CUtensorMap *m) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
      };
      if (prm.P > 0) {
        prefetch_map(&prm.kpre);
        prefetch_map(&prm.vpre);
      }
      prefetch_map(&prm.k32);
      prefetch_map(&prm.k1);
      prefetch_map(&prm.v32);
      prefetch_map(&prm.v1);
      prefetch_map(&prm.q32);
      prefetch_map(&prm.q1);
      prefetch_map(&prm.k128);
      prefetch_map(&prm.v128);
      prefetch_map(&prm.q128);
    }
    const int32_t *idx_cache = nullptr;
    bool list_ok = false;  // the list is known to be in range and strictly ascending
    if (prm.idx_bstride == 0) {
      int32_t *cache = reinterpret_cast<int32_t *>(smem + G_::kOffIdxCache);
      list_ok = cache_shared_index_list(prm, cache, bad_index);
      __syncwarp();
      if (list_ok) idx_cache = cache;  // a malformed list is read entry by entry from global memory
    }
    const int n_my = (n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    int q_next = 0;
    auto issue_q = [&](int kq) {
      const Item2 it = decode_item2(prm, blockIdx.x + kq * gridDim.x);
      uint32_t bytes = gather_rows<D>(prm, &prm.q32, &prm.q1, &prm.q128, sbase + G_::kOffQ, kChunkBytes, bar_q_full,
                                      it.pr * 2 * kBlockM, it.rows_a, it.hk * prm.G, it.b, idxq_s, idx_cache, list_ok, bad_index, false, true);
      if (it.rows_b > 0)
        bytes += gather_rows<D>(prm, &prm.q32, &prm.q1, &prm.q128, sbase + G_::kOffQ + G_::kTileBytes, kChunkBytes, bar_q_full,
                                (it.pr * 2 + 1) * kBlockM, it.rows_b, it.hk * prm.G, it.b, idxq_s, idx_cache, list_ok, bad_index, false, true);
      if (lane == 0) mbar_arrive_expect_tx(bar_q_full, bytes);
    };
    int issued = 0;
    for (int k = 0; k < n_my && !timed_out; ++k) {
      const Item2 it = decode_item2(prm, blockIdx.x + k * gridDim.x);
      for (int j = 0; j < n_tiles && !timed_out; ++j) {
        for (int kv = 0; kv < 2; ++kv) {
          const int slot = issued % G_::kSlots, use = issued / G_::kSlots;
          const uint32_t dst = sbase + G_::kOffRing + slot * G_::kTileBytes;
          const uint32_t full = bar_slot_full + 8 * slot;
          bool got = false;
          for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
            if (q_next <= k) {
              bool ready = (q_next == 0) || mbar_try_wait(bar_q_free, (q_next - 1) & 1);
              ready = __all_sync(0xffffffffu, ready);
              if (ready) {
                issue_q(q_next);
                ++q_next;
                continue;
              }
            }
            bool e = mbar_try_wait(bar_slot_empty + 8 * slot, (use & 1) ^ 1);
            e = __all_sync(0xffffffffu, e);
            if (e) {
              got = true;
              break;
            }
            if (spin > 128) {
              __nanosleep(64);
              if (__any_sync(0xffffffffu, *abort_flag != 0)) break;
            }
          }
          if (!got) {
            *abort_flag = 1;
            timed_out = true;
            break;
          }
          if (j < n_pre) {
            {
              // one lane per 64-column chunk: the copies are issued side by side
              const CUtensorMap *map = kv ? &prm.vpre : &prm.kpre;
              if (lane < G_::kChunks) tma_load_4d(dst + lane * kChunkBytes, map, full, lane * 64, j * kBlockN, it.hk, it.b);
              if (lane == 0) mbar_arrive_expect_tx(full, G_::kTileBytes);
            }
          } else {
            const int t0 = (j - n_pre) * kBlockN;
            const int n = min(kBlockN, prm.Lq - t0);
            if (kv == 1 && n < kBlockN) {
              // rows past the end of a V tile meet P = 0 in the MMA: make them zero, not stale
              uint8_t *tile = smem + G_::kOffRing + slot * G_::kTileBytes + (lane & 7) * 16;
              for (int row = n + (lane >> 3); row < kBlockN; row += 4) {
#pragma unroll
                for (int c = 0; c < G_::kChunks; ++c)
                  *reinterpret_cast<uint4 *>(tile + c * kChunkBytes + row * 128) = make_uint4(0, 0, 0, 0);
              }
              fence_proxy_async();
            }
            const uint32_t bytes = gather_rows<D>(prm, kv ? &prm.v32 : &prm.k32, kv ? &prm.v1 : &prm.k1, kv ? &prm.v128 : &prm.k128, dst, kChunkBytes,
                                                  full, t0, n, it.hk, it.b, idx_s, idx_cache, list_ok, bad_index, kv == 1, true);
            if (lane == 0) mbar_arrive_expect_tx(full, bytes);
          }
          ++issued;
        }
      }
    }
    while (!timed_out && q_next < n_my) {
      bool ok = (q_next == 0) || mbar_wait(bar_q_free, (q_next - 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) {
        timed_out = true;
        break;
      }
      issue_q(q_next);
      ++q_next;
    }
    if (timed_out) {
      for (int f = max(0, issued - G_::kSlots); f < issued; ++f)
        for (uint32_t w = 0; w < 4096 && !mbar_try_wait(bar_slot_full + 8 * (f % G_::kSlots), (f / G_::kSlots) & 1); ++w)
          __nanosleep(256);
    }
    if (bad_index && prm.status) atomicOr(prm.status, DS_DEV_INDEX);
  } else if (warp == kMmaWarp) {
    // ============================ MMA issuer ============================
    constexpr uint32_t idesc_qk = instr_desc(kBlockM, kBlockN, false, false);
    constexpr uint32_t idesc_pv = instr_desc(kBlockM, D, false, true);
    const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
    const uint64_t dq0 = smem_desc(sbase + G_::kOffQ, 16, 1024);
    const uint64_t dk0 = smem_desc(sbase + G_::kOffRing, 16, 1024);           // K tile, K-major
    const uint64_t dv0 = smem_desc(sbase + G_::kOffRing, kChunkBytes, 1024);  // V tile, MN-major
    bool ok = true;
    int g0 = 0, k = 0;
    int ua = 0, ub = 0;  // uses of the S_a / S_b buffers (phases of their barriers) before the current item
    // S[sx] = Q_qx K(g)^T
    auto issue_qk = [&](int sx, int qx, int g, bool commit_k, bool last) {
      const int fill = 2 * g, slot = fill % G_::kSlots;
      if (elect_one()) {
        const uint64_t dk = dk0 + (uint64_t)((slot * G_::kTileBytes) >> 4);
        const uint64_t dq = dq0 + (uint64_t)((qx * G_::kTileBytes) >> 4);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t off = ((ks / 4) * kChunkBytes + (ks % 4) * 32) >> 4;
          umma_ss(tm + G_::kTmemS + 128 * sx, dq + off, dk + off, idesc_qk, ks > 0);
        }
        umma_commit(bar_s_full + 8 * sx);
        if (commit_k) umma_commit(bar_slot_empty + 8 * slot);
        if (last) umma_commit(bar_q_free);
      }
      __syncwarp();
    };
    // O[ox] += P[sx] V(g)
    auto issue_pv = [&](int sx, int ox, int g, bool first, bool commit_v, bool last, bool commit_done) {
      const int fill = 2 * g + 1, slot = fill % G_::kSlots;
      if (elect_one()) {
        const uint64_t dv = dv0 + (uint64_t)((slot * G_::kTileBytes) >> 4);
#pragma unroll
        for (int ks = 0; ks < kBlockN / 16; ++ks)
          umma_ts(tm + G_::kTmemO + 128 * ox, tm + G_::kTmemS + 128 * sx + ks * 8, dv + ((ks * 2048) >> 4), idesc_pv,
                  (!first || ks > 0) ? 1u : 0u);
        if (commit_done) umma_commit(bar_pv_done + 8 * sx);
        if (commit_v) umma_commit(bar_slot_empty + 8 * slot);
        if (last) umma_commit(bar_o_full);
      }
      __syncwarp();
    };
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++k, g0 += n_tiles) {
      const bool has_b = decode_item2(prm, item).rows_b > 0;
      ok = __all_sync(0xffffffffu, mbar_wait(bar_q_full, k & 1, abort_flag));
      if (!has_b) {
        // One M-tile only: its KV tiles alternate between the two S buffers, so that Q K^T of tile j + 1 runs
        // while tile j is in the softmax (the order of the one-tile kernel): Q K^T(0), Q K^T(1), P V(0),
        // Q K^T(2), P V(1), ...  Every P V signals pv_done of its buffer (the lazy rescale of tile j + 1
        // needs P V(j) complete, and here "S(j + 1) complete" does not say so).
        for (int j = -1; j < n_tiles && ok; ++j) {
          if (j + 1 < n_tiles) {
            const int g = g0 + j + 1, fill = 2 * g, slot = fill % G_::kSlots, use = fill / G_::kSlots;
            ok = __all_sync(0xffffffffu, mbar_wait(bar_slot_full + 8 * slot, use & 1, abort_flag));
            if (!ok) break;
            tc_fence_after();
            issue_qk((j + 1) & 1, 0, g, true, j + 1 == n_tiles - 1);
          }
          if (j >= 0) {
            const int g = g0 + j, fill = 2 * g + 1, slot = fill % G_::kSlots, use = fill / G_::kSlots;
            const int sx = j & 1, px = (sx ? ub : ua) + (j >> 1);
            bool w = mbar_wait2(bar_slot_full + 8 * slot, use & 1, bar_p_full + 8 * sx, px & 1, abort_flag);
            if (j == 0 && k > 0) w = w && mbar_wait(bar_o_free, (k - 1) & 1, abort_flag);
            if (!__all_sync(0xffffffffu, w)) {
              ok = false;
              break;
            }
            tc_fence_after();
            issue_pv(sx, 0, g, j == 0, true, j == n_tiles - 1, true);
          }
        }
        ua += (n_tiles + 1) / 2;
        ub += n_tiles / 2;
        continue;
      }
      for (int j = 0; j <= n_tiles && ok; ++j) {
        const int g = g0 + j;  // tile whose Q K^T is issued; P V is issued for tile g - 1
        if (j < n_tiles) {
          const int fill = 2 * g, slot = fill % G_::kSlots, use = fill / G_::kSlots;
          ok = __all_sync(0xffffffffu, mbar_wait(bar_slot_full + 8 * slot, use & 1, abort_flag));
          if (!ok) break;
        }
        for (int x = 0; x < 2 && ok; ++x) {
          if (j > 0) {
            // P_x of the previous tile is in TMEM and its V tile has landed; the epilogue of the previous item
            // has read O_x before the first P V of this one overwrites it
            const int gp = g - 1, fill = 2 * gp + 1, slot = fill % G_::kSlots, use = fill / G_::kSlots;
            const int px = (x ? ub : ua) + j - 1;  // uses of S_x before this P
            bool w = mbar_wait2(bar_slot_full + 8 * slot, use & 1, bar_p_full + 8 * x, px & 1, abort_flag);
            if (j == 1 && k > 0) w = w && mbar_wait(bar_o_free + 8 * x, (k - 1) & 1, abort_flag);
            if (!__all_sync(0xffffffffu, w)) {
              ok = false;
              break;
            }
            tc_fence_after();
            issue_pv(x, x, gp, j == 1, x == 1, x == 1 && j == n_tiles, false);
          }
          if (j < n_tiles) {
            tc_fence_after();
            issue_qk(x, x, g, x == 1, x == 1 && j == n_tiles - 1);
          }
        }
      }
      ua += n_tiles;
      ub += n_tiles;
    }
    timed_out = !ok;
  } else {
    // ============================ softmax + epilogue ============================
    // All eight warps take M-tile a, then M-tile b, of every KV tile: half a row (64 columns) per thread, the
    // two halves of a row in the two half-warps (16x32bx2 accesses).  While they work on one M-tile the
    // issuer runs P V and the next Q K^T of the other.
    const int half = lane >> 4;                            // column half this thread works on
    const int lane0 = (warp & 3) * 32 + (warp >> 2) * 16;   // first TMEM lane of this warp
    const int row = lane0 + (lane & 15);                   // TMEM lane = row of the M-tile
    const uint32_t lane_base = tmem + ((uint32_t)lane0 << 16);
    const float c2 = prm.scale_log2;
    constexpr int kOCols = D / 2;                          // accumulator columns per thread
    bool ok = true;
    int ga0 = 0, gb0 = 0, k = 0;  // uses of the S_a / S_b buffers before the current item (phase counts of their barriers)
    int da0 = 0, db0 = 0;         // the same, counting single-tile items only (phases of pv_done)
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++k) {
      const Item2 it = decode_item2(prm, item);
      const int n_x = it.rows_b > 0 ? 2 : 1;
      const bool lone = n_x == 1;  // one M-tile: its KV tiles alternate between the two S buffers
      float m_used[2] = {-INFINITY, -INFINITY};  // maximum the probabilities are expressed against (log2 units)
      float l_sum[2] = {0.f, 0.f};               // this thread's half of the row sum
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int valid = (j < n_pre) ? min(kBlockN, prm.P - j * kBlockN) : min(kBlockN, prm.Lq - (j - n_pre) * kBlockN);
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          if (x >= n_x) break;
          const bool live = row < (x ? it.rows_b : it.rows_a);
          const int sx = lone ? (j & 1) : x;  // S buffer of this tile
          const int gx = (sx ? gb0 : ga0) + (lone ? (j >> 1) : j);
          ok = __all_sync(0xffffffffu, mbar_wait(bar_s_full + 8 * sx, gx & 1, abort_flag));
          if (!ok) break;
          tc_fence_after();
          const uint32_t s_base = lane_base + G_::kTmemS + 128 * sx, o_base = lane_base + G_::kTmemO + 128 * x;
          uint32_t s[64];
          tmem_ld16x2_32<64>(s_base, &s[0]);        // columns 64 half + 0..31
          tmem_ld16x2_32<64>(s_base + 32, &s[32]);  // columns 64 half + 32..63
          tmem_wait_ld();
          if (valid < kBlockN) {
            // selects, not branches: the two half-warps see different limits
            const int lim = valid - 64 * half;
#pragma unroll
            for (int c = 0; c < 64; ++c) s[c] = (c >= lim) ? 0xff800000u : s[c];  // -inf: columns past the end of a partial tile
          }
          float mx;
          {
            float a[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) a[c] = __uint_as_float(s[c]);
#pragma unroll
            for (int c = 8; c < 56; c += 16) {
#pragma unroll
              for (int u = 0; u < 8; ++u) a[u] = fmax3(a[u], __uint_as_float(s[c + u]), __uint_as_float(s[c + 8 + u]));
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) a[u] = fmaxf(a[u], __uint_as_float(s[56 + u]));
            mx = fmaxf(fmax3(a[0], a[1], a[2]), fmax3(a[3], a[4], a[5]));
            mx = fmax3(mx, a[6], a[7]);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
          }
          const float m_tile = mx * c2;
          float factor = 1.f;
          if (m_tile > m_used[x] + kRescaleThreshold || m_used[x] == -INFINITY) {
            factor = (m_used[x] == -INFINITY) ? 0.f : ex2_approx(m_used[x] - m_tile);
            m_used[x] = m_tile;
          }
          const bool warp_rescales = __any_sync(0xffffffffu, live && factor != 1.f) && (j > 0);
          l_sum[x] *= factor;
          if (warp_rescales) {
            // With two M-tiles, S of this tile being complete means every MMA issued before its Q K^T has
            // completed, the previous P V of this M-tile among them: O_x is quiescent.  With one M-tile the
            // previous P V was issued after this Q K^T and has a barrier of its own.
            if (lone) {
              const int sp = (j - 1) & 1, gp = (sp ? db0 : da0) + ((j - 1) >> 1);
              ok = __all_sync(0xffffffffu, mbar_wait(bar_pv_done + 8 * sp, gp & 1, abort_flag));
              if (!ok) break;
              tc_fence_after();
            }
#pragma unroll
            for (int cb = 0; cb < kOCols; cb += 32) {
              uint32_t o[32];
              tmem_ld16x2_32<kOCols>(o_base + cb, o);
              tmem_wait_ld();
#pragma unroll
              for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * factor);
              tmem_st16x2_32<kOCols>(o_base + cb, o);
            }
          }
          float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
          const float neg_m = -m_used[x];
          uint32_t pk[32];
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const float p0 = ex2_approx(fmaf(__uint_as_float(s[2 * c]), c2, neg_m));
            const float p1 = ex2_approx(fmaf(__uint_as_float(s[2 * c + 1]), c2, neg_m));
            const float p2 = ex2_approx(fmaf(__uint_as_float(s[2 * c + 2]), c2, neg_m));
            const float p3 = ex2_approx(fmaf(__uint_as_float(s[2 * c + 3]), c2, neg_m));
            pk[c] = pack_bf16(p0, p1);
            pk[c + 1] = pack_bf16(p2, p3);
            l0 += p0;
            l1 += p1;
            l2 += p2;
            l3 += p3;
          }
          l_sum[x] += (l0 + l1) + (l2 + l3);
          // P row -> TMEM over the first 64 columns of S_x (two bf16 per column); this thread's 64 keys are
          // columns 32 half .. 32 half + 31
          tmem_st16x2_32<32>(s_base, pk);
          tmem_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_p_full + 8 * sx);
        }
      }
      if (!ok) break;
      // ---- epilogue of the item: the last P V of both M-tiles has completed ----
      ok = __all_sync(0xffffffffu, mbar_wait(bar_o_full, k & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int x = 0; x < 2; ++x) {
        const bool have = x < n_x;
        const bool live = have && row < (x ? it.rows_b : it.rows_a);
        uint32_t o[kOCols];
        if (have) {
#pragma unroll
          for (int cb = 0; cb < kOCols; cb += 32) tmem_ld16x2_32<kOCols>(lane_base + G_::kTmemO + 128 * x + cb, &o[cb]);
          tmem_wait_ld();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_o_free + 8 * x);   // O_x is in registers (or does not exist): it may be overwritten
        const float l_row = l_sum[x] + __shfl_xor_sync(0xffffffffu, l_sum[x], 16);  // the other half of the row
        if (live) {
          const int R = (it.pr * 2 + x) * kBlockM + row;
          const int hq = it.hk * prm.G + R / prm.Lq, i = R % prm.Lq;
          const float inv = 1.f / l_row;
          __nv_bfloat16 *orow = reinterpret_cast<__nv_bfloat16 *>(prm.out) + it.b * prm.out_stride[0] +
                                hq * prm.out_stride[1] + (long long)i * prm.out_stride[2] + kOCols * half;
#pragma unroll
          for (int c = 0; c < kOCols; c += 8) {
            uint4 w;
            w.x = pack_bf16(__uint_as_float(o[c + 0]) * inv, __uint_as_float(o[c + 1]) * inv);
            w.y = pack_bf16(__uint_as_float(o[c + 2]) * inv, __uint_as_float(o[c + 3]) * inv);
            w.z = pack_bf16(__uint_as_float(o[c + 4]) * inv, __uint_as_float(o[c + 5]) * inv);
            w.w = pack_bf16(__uint_as_float(o[c + 6]) * inv, __uint_as_float(o[c + 7]) * inv);
            *reinterpret_cast<uint4 *>(orow + c) = w;
          }
          if (prm.lse && half == 0) prm.lse[((long long)it.b * prm.Hq + hq) * prm.Lq + i] = (m_used[x] + log2f(l_row)) * kLn2;
        }
      }
      ga0 += lone ? (n_tiles + 1) / 2 : n_tiles;
      gb0 += lone ? n_tiles / 2 : n_tiles;
      if (lone) {
        da0 += (n_tiles + 1) / 2;
        db0 += n_tiles / 2;
      }
    }
    timed_out = !ok;
  }

  if (timed_out && prm.status) atomicOr(prm.status, DS_DEV_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

template <int D>
int prepare2_d(const ds_attn_params &p, AttnPrepared &out) {
  static_assert(sizeof(Tc2Params) <= sizeof(out.kernel_params), "parameter struct does not fit the plan");
  Tc2Params &prm = *reinterpret_cast<Tc2Params *>(out.kernel_params);  // plain data, zeroed below
  memset(&prm, 0, sizeof(prm));
  out.path = kAttnPathTc2;
  out.p = p;
  out.grid = 0;
  if (!fill_common(prm, p)) {
    note_cuda_error((int)cudaErrorInvalidValue);  // cuTensorMapEncodeTiled refused the layout
    return DS_ERR_CUDA;
  }
  const long long rows_total = (long long)prm.G * p.Lq;
  prm.n_pairs = (int)((rows_total + 2 * kBlockM - 1) / (2 * kBlockM));
  const long long n_items = (long long)(p.seq_list ? p.n_seq : p.B) * p.Hkv * prm.n_pairs;  // upper bound with a device count
  if (n_items > 0x7fffffffLL) return DS_ERR_UNSUPPORTED;
  prm.n_items = (int)n_items;
  int grid = (int)(n_items < sm_count() ? n_items : sm_count());
  // An odd number of M-tiles leaves a pair with one tile, about half the work of a full pair.  CTA c takes the
  // items c, c + grid, ...; the pair number is the fastest index of an item, so a grid that shares a factor with
  // the number of pairs would hand some CTAs nothing but full pairs: keep the two coprime.
  if ((rows_total + kBlockM - 1) / kBlockM % 2 == 1 && prm.n_pairs > 1 && n_items > grid) {
    auto gcd = [](int a, int b) {
      while (b) {
        const int t = a % b;
        a = b;
        b = t;
      }
      return a;
    };
    while (grid > 1 && gcd(grid, prm.n_pairs) != 1) --grid;
  }
  out.grid = grid;
  return DS_OK;
}

template <int D>
int launch_prepared2_d(const AttnPrepared &a, cudaStream_t stream) {
  if (a.grid == 0) return DS_OK;
  DS_CUDA_OK(cudaFuncSetAttribute(attn_tc2_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo2<D>::kSmemBytes));
  attn_tc2_kernel<D><<<a.grid, kThreads2, Geo2<D>::kSmemBytes, stream>>>(*reinterpret_cast<const Tc2Params *>(a.kernel_params));
  DS_CUDA_OK(cudaGetLastError());
  note_launch(1);
  return DS_OK;
}

}  // namespace

int prepare_attn_tc2(const ds_attn_params &p, AttnPrepared &out) {
  return p.D == 128 ? prepare2_d<128>(p, out) : prepare2_d<64>(p, out);
}
int launch_prepared_tc2(const AttnPrepared &a, cudaStream_t stream) {
  return a.p.D == 128 ? launch_prepared2_d<128>(a, stream) : launch_prepared2_d<64>(a, stream);
}
int launch_attn_tc2(const ds_attn_params &p, cudaStream_t stream) {
  AttnPrepared a;
  const int rc = prepare_attn_tc2(p, a);
  return rc != DS_OK ? rc : launch_prepared_tc2(a, stream);
}

}  // namespace ds
