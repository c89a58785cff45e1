// ds_attn_pruned, tensor-core path for bf16 (Eq. 7-8): TMA-staged KV tiles, tcgen05 MMAs with
// TMEM accumulators, online softmax.
//
// Work item = (batch, KV head, 128-row M-tile).  The query heads of one GQA group are stacked along
// M (row R = head_in_group * Lq + i), so every KV tile is read once per group.  KV is streamed as
// 128-row tiles: first the cached prefix (tiled TMA boxes, out-of-range rows zero-filled), then the
// retained tail rows named by the index list, fetched as one 128-row box when a whole tile (or a
// partial tile that ends with the buffer's last row) is consecutive, as 32-row boxes where the list is
// contiguous and as single-row boxes elsewhere.  CTAs are persistent: CTA c takes items c, c + grid,
// ... and the KV ring keeps streaming across item boundaries.
//
// "Extra" rows.  The retained set is block + window + the trailing position, so the stacked row
// count is often 128 m + 1.  Up to 8 rows beyond the last full M-tile do not get a tile of their own:
// they ride along with that tile as a second, transposed problem  S_x^T = K Q_x^T  (M = 128 keys,
// N = 16) and  O_x^T = V^T P_x^T  (M = D, N = 16), which costs a fraction of a full tile on the
// tensor cores.  There the keys lie along TMEM lanes, so a column maximum would need a cross-lane
// reduction per tile; instead those columns are expressed against a reference exponent that is only
// moved (with an exact rescale) when a score exceeds it by more than 2^24.
//
// Warp roles (512 threads, one CTA per SM):
//   warps 0-7  softmax (and, in launches with extra rows, the items' epilogue).  Warp w works on the 16 TMEM lanes 32 (w % 4) + 16 (w / 4) ..;
//              two threads share a row (lanes l and l + 16 of the warp take the two column halves of
//              every S tile, tcgen05.ld shape 16x32bx2), so a row maximum is one shuffle away and
//              every scheduler has two softmax warps.
//   warp  8    TMA producer of the K/V tiles (lane 0 issues; the warp stages the index list of each gathered tile)
//   warp  9    TMEM allocation; issues Q K^T (one elected lane)
//   warps 10-13 softmax + epilogue of the transposed problem (thread = key of the tile), kept apart so that
//              its cross-warp agreement never sits on the main rows' critical path.  In launches without
//              extra rows they write the items' results instead (thread = row of the M-tile), so that the
//              softmax warps can go straight on to the next item.
//   warp 14    issues P V.  Issuing blocks while the tensor pipe's queue is full, so the two streams
//              have an issuer each; the one dependency the pipe no longer orders by itself (Q K^T of
//              tile g + 2 overwrites the buffer P V of tile g reads) is an explicit barrier wait.
//   warp 15    TMA producer of the query tiles.  Gathering a query tile takes the issuing warp about as long
//              as a KV tile lasts, so it has a warp of its own: the K/V stream starts at once and never
//              pauses for it.  In the kQ2 instantiation (items of few KV tiles) there are two query buffers
//              and four ring slots instead of one and five: the next item's queries are then fetched while
//              the current item runs, which removes the stall at every item boundary.
// Per KV tile:  S[g%2] = Q K^T            (tcgen05.mma, both operands K-major in shared memory)
//               softmax warps: tcgen05.ld S, row maximum, P = 2^(s*c - m) as bf16 written over the
//               first 64 columns of the same S buffer
//               O += P V                   (A = P from TMEM, B = V MN-major straight from its [kv][D]
//                                           layout)
// S/P is double buffered so Q K^T of the next tile runs under the softmax of this one.  O is only
// rescaled when a row maximum grows by more than 2^8 (the stale maximum keeps P within range), which
// removes the TMEM round trip from the steady state.
//
// Barriers are mbarriers waited on by parity.  A parity wait can only tell two consecutive phases
// apart, so every barrier here is arranged such that a waiter is never more than one phase behind
// (barriers that could run ahead are double buffered by tile parity, and per-item barriers are
// waited on by every participant at every item).
//
// Every wait is bounded (no hardware barrier inside the role loops); on expiry the thread raises
// DS_DEV_TIMEOUT in the status word, all roles leave their loops, outstanding TMA copies are waited
// for (bounded), TMEM is freed and the CTA returns.
#include <cuda.h>

#include <cstring>
#include <mutex>


#include "ds_attn_tiles.cuh"
#include "ds_common.cuh"
#include "ds_sm100.cuh"

namespace ds {
namespace {

using namespace sm100;
using namespace attn;

constexpr int kSoftmaxWarps = 8;
constexpr int kXWarps = 4;  // softmax of the transposed problem (one per TMEM lane quadrant)
constexpr int kNumThreads = (kSoftmaxWarps + 4 + kXWarps) * 32;
constexpr int kProducerWarp = kSoftmaxWarps, kMmaWarp = kSoftmaxWarps + 1, kXWarp0 = kSoftmaxWarps + 2;
constexpr int kPvWarp = kXWarp0 + kXWarps;  // second MMA issuer
constexpr int kQWarp = kPvWarp + 1;         // producer of the query tiles
constexpr int kXRows = 16;                  // N of the transposed problem (the smallest N for M = 128)
constexpr int kXMax = 8;                    // extra rows actually served
constexpr int kXChunkBytes = kXRows * 128;
constexpr float kRescaleThreshold = 8.0f;   // log2 units
constexpr int kQ2MaxTiles = 24;             // items of at most this many KV tiles get the two-query-buffer instantiation
constexpr float kXLimit = 24.0f;            // log2 units a transposed score may exceed its reference by

template <int D, bool kQ2>
struct Geo {
  static constexpr int kChunks = D / 64;                    // 64-column chunks per tile
  static constexpr int kTileBytes = kChunks * kChunkBytes;  // Q / K / V tile
  static constexpr int kQBufs = kQ2 ? 2 : 1;                // query buffers (by item parity)
  static constexpr int kSlots = ((D == 128) ? 5 : 10) - (kQ2 ? (D == 128 ? 1 : 2) : 0);  // ring of K/V tiles
  static constexpr int kOffQ = 0;                           // [kQBufs] tiles
  static constexpr int kQxBytes = 2 * kXChunkBytes;         // small query tile: [2 chunks][16 rows][128 B]
  static constexpr int kOffQx = kQBufs * kTileBytes;        // [kQBufs] small tiles
  static constexpr int kOffPx = kOffQx + kQBufs * kQxBytes;  // [2 buffers][2 chunks][16 rows][128 B]
  static constexpr int kOffRing = kOffPx + 4 * kXChunkBytes;
  static constexpr int kOffBar = kOffRing + kSlots * kTileBytes;
  // barriers: q_full, q_free, s_full[2], p_full[2], pv_done[2], o_free, xbar[2], ybar, o_full, px_full[2],
  //           ox_free, sx_full[2], pvx_done[2], slot_full[kSlots], slot_empty[kSlots], q_full / q_free of the
  //           second query buffer
  static constexpr int kNumBars = 22 + 2 * kSlots;
  static constexpr int kOffIdx = kOffBar + 8 * kNumBars;     // int32[128] gathered-row indices of a KV tile
  static constexpr int kOffIdxQ = kOffIdx + 4 * 128;         // int32[128] gathered-row indices of a query tile
  static constexpr int kOffXflag = kOffIdxQ + 4 * 128;       // int[2 parity][4 warps]
  static constexpr int kOffXcol = kOffXflag + 4 * 16;        // float[4 warps][8 columns]
  static constexpr int kOffIdxCache = kOffXcol + 4 * 64;     // int32[kIdxCap] the index list, when all batches share it
  static constexpr int kOffMisc = kOffIdxCache + 4 * kIdxCap;  // tmem base, abort flag
  static constexpr int kSmemBytes = kOffMisc + 16 + 1024;    // + slack to align the base to 1024
  static constexpr int kTmemCols = 512;
  static constexpr int kTmemS0 = 0, kTmemS1 = 128, kTmemO = 256;  // P(g) overwrites columns 0..63 of S(g)
  static constexpr int kTmemSx0 = 384, kTmemSx1 = 400, kTmemOx = 416;
};
static_assert(Geo<128, false>::kSmemBytes <= 227 * 1024 && Geo<128, true>::kSmemBytes <= 227 * 1024, "shared memory budget");
static_assert(Geo<64, false>::kSmemBytes <= 227 * 1024 && Geo<64, true>::kSmemBytes <= 227 * 1024, "shared memory budget");

struct TcParams : attn::AttnCommon {
  int n_mtiles;  // M-tiles per (batch, KV head)
  int x_rows;    // extra rows riding with the last M-tile (0 = none)
  int n_items;   // B * Hkv * n_mtiles * splits
  int q2;        // 1: several items per CTA and few KV tiles per item: the instantiation with two query buffers
  // Few work items (small batches): the KV tiles of an item are split over `splits` CTAs, each writing a
  // normalised partial result and its log-sum-exp to the workspace (out / lse then point there, one copy per
  // split, split_stride elements apart); a second kernel merges them.
  int splits, tiles_per_split, n_tiles;
  long long out_split_stride, lse_split_stride;
};

struct Item {
  int b, hk, mt, m_rows, x_rows;
  int split, t0, nt;  // this CTA's KV tiles: t0 .. t0 + nt - 1 of the item's sequence of tiles
};
// kSplit = false is the launch in which every item takes all its KV tiles: nothing of the split arithmetic
// is left in that instantiation.
template <bool kSplit>
__device__ __forceinline__ Item decode_item(const TcParams &prm, int item) {
  Item it;
  it.split = 0;
  it.t0 = 0;
  it.nt = prm.n_tiles;
  if constexpr (kSplit) {
    it.split = item % prm.splits;
    item /= prm.splits;
    it.t0 = it.split * prm.tiles_per_split;
    it.nt = min(prm.tiles_per_split, prm.n_tiles - it.t0);
  }
  it.mt = item % prm.n_mtiles;
  const int bh = item / prm.n_mtiles;
  it.hk = bh % prm.Hkv;
  it.b = attn::listed_batch(prm, bh / prm.Hkv);
  const int rows_total = prm.G * prm.Lq;
  it.x_rows = (it.mt == prm.n_mtiles - 1) ? prm.x_rows : 0;
  it.m_rows = min(kBlockM, rows_total - it.x_rows - it.mt * kBlockM);
  return it;
}

// ------------------------------------------------------------------------------------------------
// The kernel
// ------------------------------------------------------------------------------------------------
// kX: the launch has rows beyond the last full M-tile (prm.x_rows > 0).  The two cases differ in what warps 10-13
// and the epilogue do, and each instantiation carries only its own code.
template <int D, bool kSplit, bool kQ2, bool kX>
__global__ void __launch_bounds__(kNumThreads, 1) attn_tc_kernel(const __grid_constant__ TcParams prm) {
  static_assert(!kX || D == 128, "extra rows exist for D = 128 only");
  using G_ = Geo<D, kQ2>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  const uint32_t bar0 = sbase + G_::kOffBar;
  const uint32_t bar_q_full = bar0;
  const uint32_t bar_q_free = bar0 + 8;
  const uint32_t bar_s_full = bar0 + 16;     // [2]
  const uint32_t bar_p_full = bar0 + 32;     // [2] a softmax warp may be one tile ahead of another
  const uint32_t bar_pv_done = bar0 + 48;    // [2] by tile parity: a waiter may be two tiles behind the P V stream
  const uint32_t bar_o_free = bar0 + 64;
  const uint32_t bar_x = bar0 + 72;          // [2] transposed problem: "does this tile outgrow the reference" votes
  const uint32_t bar_y = bar0 + 88;          // transposed problem: occasional exchanges (column maxima, sums)
  const uint32_t bar_o_full = bar0 + 96;     // the last P V of an item has completed
  const uint32_t bar_px_full = bar0 + 104;   // [2] P_x^T of a tile is in shared memory
  const uint32_t bar_ox_free = bar0 + 120;   // the epilogue has read O_x^T
  const uint32_t bar_sx_full = bar0 + 128;   // [2] S_x^T of a tile is in TMEM
  const uint32_t bar_pvx_done = bar0 + 144;  // [2] O_x^T += V^T P_x^T of a tile has completed
  const uint32_t bar_slot_full = bar0 + 160;                       // [kSlots]
  const uint32_t bar_slot_empty = bar_slot_full + 8 * G_::kSlots;  // [kSlots]
  const uint32_t bar_q1 = bar_slot_empty + 8 * G_::kSlots;         // q_full, q_free of the second query buffer
  // query buffer of this CTA's k-th item, its two barriers and their phase for that item
  auto q_buf = [](int k) { return kQ2 ? (k & 1) : 0; };
  auto q_phase = [](int k) { return (uint32_t)(kQ2 ? (k >> 1) & 1 : k & 1); };
  auto q_full_bar = [&](int k) { return q_buf(k) ? bar_q1 : bar_q_full; };
  auto q_free_bar = [&](int k) { return q_buf(k) ? bar_q1 + 8 : bar_q_free; };
  int32_t *idx_s = reinterpret_cast<int32_t *>(smem + G_::kOffIdx);
  int32_t *idxq_s = reinterpret_cast<int32_t *>(smem + G_::kOffIdxQ);
  volatile uint32_t *tmem_base_s = reinterpret_cast<volatile uint32_t *>(smem + G_::kOffMisc);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + G_::kOffMisc + 4);

  const int n_pre = (prm.P + kBlockN - 1) / kBlockN;
  const int n_tail = (prm.Lq + kBlockN - 1) / kBlockN;
  const int n_tiles = n_pre + n_tail;

  constexpr bool x_epilogue = !kX;
  if (tid == 0) {
    mbar_init(bar_q_full, 1);
    mbar_init(bar_q_free, 1);
    mbar_init(bar_q1, 1);
    mbar_init(bar_q1 + 8, 1);
    mbar_init(bar_s_full, 1);
    mbar_init(bar_s_full + 8, 1);
    mbar_init(bar_p_full, kSoftmaxWarps);
    mbar_init(bar_p_full + 8, kSoftmaxWarps);
    mbar_init(bar_pv_done, 1);
    mbar_init(bar_pv_done + 8, 1);
    // launches without extra rows: warps 10-13 write the items' results (see their role), so they are the ones
    // that release O, and bar_x is the softmax warps' "row sums handed over"
    mbar_init(bar_o_free, x_epilogue ? kXWarps : kSoftmaxWarps);
    mbar_init(bar_x, x_epilogue ? kSoftmaxWarps : kXWarps);
    mbar_init(bar_x + 8, kXWarps);
    mbar_init(bar_y, kXWarps);
    mbar_init(bar_o_full, 1);
    mbar_init(bar_px_full, kXWarps);
    mbar_init(bar_px_full + 8, kXWarps);
    mbar_init(bar_ox_free, kXWarps);
    mbar_init(bar_sx_full, 1);
    mbar_init(bar_sx_full + 8, 1);
    mbar_init(bar_pvx_done, 1);
    mbar_init(bar_pvx_done + 8, 1);
    for (int s = 0; s < G_::kSlots; ++s) {
      mbar_init(bar_slot_full + 8 * s, 1);
      mbar_init(bar_slot_empty + 8 * s, 1);
    }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == kMmaWarp) tmem_alloc(sbase + G_::kOffMisc, G_::kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_base_s;
  // sequences (hence work items) of this launch: all, or the listed ones with the count read on the device
  const int n_live = attn::live_sequences(prm);
  const int n_items = n_live * prm.Hkv * prm.n_mtiles * (kSplit ? prm.splits : 1);
  bool timed_out = false;

  if (warp == kProducerWarp) {
    // ============================ TMA producer: K/V tiles ============================
    bool bad_index = attn::bad_sequence_numbers(prm, n_live);
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
      prefetch_map(&prm.k128);
      prefetch_map(&prm.v128);
    }
    // One index list for all batches: (the head of) it is kept in shared memory, validated once -- but only
    // when the first tail tile comes up, so that the prefix tiles are requested without waiting for it.
    const int32_t *idx_cache = nullptr;
    bool list_ok = false;  // the list is known to be in range and strictly ascending
    bool list_seen = false;
    const int n_my = (n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;  // items of this CTA
    int issued = 0;  // ring fills issued so far
    for (int k = 0; k < n_my && !timed_out; ++k) {
      const Item it = decode_item<kSplit>(prm, blockIdx.x + k * gridDim.x);
      const int nt_it = kSplit ? it.nt : n_tiles;
      for (int jj = 0; jj < nt_it && !timed_out; ++jj) {
        const int j = (kSplit ? it.t0 : 0) + jj;
        for (int kv = 0; kv < 2; ++kv) {
          const int slot = issued % G_::kSlots, use = issued / G_::kSlots;
          const uint32_t dst = sbase + G_::kOffRing + slot * G_::kTileBytes;
          const uint32_t full = bar_slot_full + 8 * slot;
          if (!__all_sync(0xffffffffu, mbar_wait(bar_slot_empty + 8 * slot, (use & 1) ^ 1, abort_flag))) {
            timed_out = true;
            break;
          }
          if (j < n_pre) {
            // one lane per 64-column chunk: the copies are issued side by side
            const CUtensorMap *map = kv ? &prm.vpre : &prm.kpre;
            if (lane < G_::kChunks) tma_load_4d(dst + lane * kChunkBytes, map, full, lane * 64, j * kBlockN, it.hk, it.b);
            if (lane == 0) mbar_arrive_expect_tx(full, G_::kTileBytes);
          } else {
            if (!list_seen && prm.idx_bstride == 0) {
              int32_t *cache = reinterpret_cast<int32_t *>(smem + G_::kOffIdxCache);
              list_ok = cache_shared_index_list(prm, cache, bad_index);
              __syncwarp();
              if (list_ok) idx_cache = cache;  // a malformed list is read entry by entry from global memory
            }
            list_seen = true;
            const int t0 = (j - n_pre) * kBlockN;
            const int n = min(kBlockN, prm.Lq - t0);
            if (kv == 1 && n < kBlockN) {
              // rows past the end of a V tile meet P = 0 in the MMA: make them zero, not stale
              // (a row of a chunk is 8 x 16 bytes: 4 rows per pass of the warp)
              uint8_t *tile = smem + G_::kOffRing + slot * G_::kTileBytes + (lane & 7) * 16;
              for (int row = n + (lane >> 3); row < kBlockN; row += 4) {
#pragma unroll
                for (int c = 0; c < G_::kChunks; ++c)
                  *reinterpret_cast<uint4 *>(tile + c * kChunkBytes + row * 128) = make_uint4(0, 0, 0, 0);
              }
              fence_proxy_async();
            }
            // the V fill of a tile directly follows its K fill: the staged row list is still valid
            const uint32_t bytes = gather_rows<D>(prm, kv ? &prm.v32 : &prm.k32, kv ? &prm.v1 : &prm.k1, kv ? &prm.v128 : &prm.k128, dst, kChunkBytes,
                                                  full, t0, n, it.hk, it.b, idx_s, idx_cache, list_ok, bad_index, kv == 1, true);
            if (lane == 0) mbar_arrive_expect_tx(full, bytes);
          }
          ++issued;
        }
      }
    }
    if (timed_out) {
      // let copies already in flight land before the CTA's shared memory goes away
      for (int f = max(0, issued - G_::kSlots); f < issued; ++f)
        for (uint32_t w = 0; w < 4096 && !mbar_try_wait(bar_slot_full + 8 * (f % G_::kSlots), (f / G_::kSlots) & 1); ++w)
          __nanosleep(256);
    }
    if (bad_index && prm.status) atomicOr(prm.status, DS_DEV_INDEX);
  } else if (warp == kQWarp) {
    // ============================ TMA producer: query tiles ============================
    // Item k's queries go to buffer q_buf(k) once the item that used it before (k - kQBufs) has issued its
    // last Q K^T.  The row numbers are read from global memory here (every query tile is gathered once; the
    // K/V producer's shared copy of the list may not exist yet).
    bool bad_index = false;
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&prm.q32)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&prm.q1)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&prm.q128)) : "memory");
    }
    const int n_my = (n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;  // items of this CTA
    int k_done = 0;
    for (int k = 0; k < n_my && !timed_out; ++k) {
      if (k >= G_::kQBufs) {
        if (!__all_sync(0xffffffffu, mbar_wait(q_free_bar(k), q_phase(k - G_::kQBufs), abort_flag))) {
          timed_out = true;
          break;
        }
      }
      const Item it = decode_item<kSplit>(prm, blockIdx.x + k * gridDim.x);
      const uint32_t full = q_full_bar(k);
      uint32_t bytes = gather_rows<D>(prm, &prm.q32, &prm.q1, &prm.q128, sbase + G_::kOffQ + q_buf(k) * G_::kTileBytes, kChunkBytes, full,
                                      it.mt * kBlockM, it.m_rows, it.hk * prm.G, it.b, idxq_s, nullptr, false, bad_index, false, true);
      if (kX && it.x_rows > 0) {
        // rows of the small query tile that are not loaded must be finite: clear the tile first
        uint8_t *qx = smem + G_::kOffQx + q_buf(k) * G_::kQxBytes;
        for (int q = lane; q < G_::kQxBytes / 16; q += 32) *reinterpret_cast<uint4 *>(qx + q * 16) = make_uint4(0, 0, 0, 0);
        fence_proxy_async();
        bytes += gather_rows<D>(prm, &prm.q32, &prm.q1, &prm.q128, sbase + G_::kOffQx + q_buf(k) * G_::kQxBytes, kXChunkBytes, full,
                                (it.mt + 1) * kBlockM, it.x_rows, it.hk * prm.G, it.b, idxq_s, nullptr, false, bad_index);
      }
      if (lane == 0) mbar_arrive_expect_tx(full, bytes);
      k_done = k + 1;
    }
    if (timed_out) {
      // let copies already in flight land before the CTA's shared memory goes away
      for (int f = max(0, k_done - G_::kQBufs); f < k_done; ++f)
        for (uint32_t w = 0; w < 4096 && !mbar_try_wait(q_full_bar(f), q_phase(f)); ++w) __nanosleep(256);
    }
    if (bad_index && prm.status) atomicOr(prm.status, DS_DEV_INDEX);
  } else if (warp == kMmaWarp) {
    // ============================ MMA issuer: S = Q K^T ============================
    // The whole warp walks the loop (uniform control flow keeps descriptors in uniform registers);
    // one elected lane issues the MMAs and commits.
    constexpr uint32_t idesc_qk = instr_desc(kBlockM, kBlockN, false, false);
    constexpr uint32_t idesc_qk_x = instr_desc(kBlockM, kXRows, false, false);  // S_x^T = K Q_x^T
    const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
    // descriptors of byte 0 of each operand region; a K-step only adds to the address field
    const uint64_t dq0 = smem_desc(sbase + G_::kOffQ, 16, 1024);
    const uint64_t dqx0 = smem_desc(sbase + G_::kOffQx, 16, 1024);
    const uint64_t dk0 = smem_desc(sbase + G_::kOffRing, 16, 1024);  // K tile, K-major
    bool ok = true;
    int g0 = 0;   // tiles processed by this CTA before the current item
    int k = 0;
    int gx0 = 0;  // tiles of items with extra rows before the current item
    int nt_cur = 0;  // KV tiles of the current item that this CTA processes
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++k, g0 += nt_cur) {
      const int j_lo = kSplit ? decode_item<kSplit>(prm, item).t0 : 0;
      nt_cur = kSplit ? decode_item<kSplit>(prm, item).nt : n_tiles;
      const bool has_x = kX && decode_item<kSplit>(prm, item).x_rows > 0;
      ok = __all_sync(0xffffffffu, mbar_wait(q_full_bar(k), q_phase(k), abort_flag));
      const uint64_t dq = dq0 + (uint64_t)((q_buf(k) * G_::kTileBytes) >> 4);
      const uint64_t dqx = dqx0 + (uint64_t)((q_buf(k) * G_::kQxBytes) >> 4);
      for (int jj = 0; jj < nt_cur && ok; ++jj) {
        const int j = j_lo + jj;
        (void)j;
        const int g = g0 + jj, gx = gx0 + jj;
        const int fill = 2 * g, slot = fill % G_::kSlots, use = fill / G_::kSlots;
        // the K tile has landed, and S[g % 2] is free: P V of tile g - 2, the reader of the P it still
        // holds, has completed
        bool w;
        if (g >= 2)
          w = mbar_wait2(bar_slot_full + 8 * slot, use & 1, bar_pv_done + 8 * (g & 1), ((g - 2) >> 1) & 1, abort_flag);
        else
          w = mbar_wait(bar_slot_full + 8 * slot, use & 1, abort_flag);
        if (!__all_sync(0xffffffffu, w)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const uint64_t dk = dk0 + (uint64_t)((slot * G_::kTileBytes) >> 4);
        if (elect_one()) {
          const uint32_t d = tm + ((g & 1) ? G_::kTmemS1 : G_::kTmemS0);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            const uint32_t off = ((ks / 4) * kChunkBytes + (ks % 4) * 32) >> 4;
            umma_ss(d, dq + off, dk + off, idesc_qk, ks > 0);
          }
          umma_commit(bar_s_full + 8 * (g & 1));
        }
        __syncwarp();
        if (has_x && gx >= 2) {
          // S_x^T and P_x^T buffers of this parity are free once the transposed P V of two such tiles
          // back has completed (which also means its softmax warps have moved on)
          if (!__all_sync(0xffffffffu, mbar_wait(bar_pvx_done + 8 * (gx & 1), ((gx - 2) >> 1) & 1, abort_flag))) {
            ok = false;
            break;
          }
          tc_fence_after();
        }
        if (elect_one()) {
          if (has_x) {
            const uint32_t dx = tm + ((gx & 1) ? G_::kTmemSx1 : G_::kTmemSx0);  // buffers by x-tile parity
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
              const uint32_t off = ((ks / 4) * kChunkBytes + (ks % 4) * 32) >> 4;
              const uint32_t offx = ((ks / 4) * kXChunkBytes + (ks % 4) * 32) >> 4;
              umma_ss(dx, dk + off, dqx + offx, idesc_qk_x, ks > 0);
            }
            umma_commit(bar_sx_full + 8 * (gx & 1));
          }
          umma_commit(bar_slot_empty + 8 * slot);
          if (jj == nt_cur - 1) umma_commit(q_free_bar(k));
        }
        __syncwarp();
      }
      if (has_x) gx0 += nt_cur;
    }
    timed_out = !ok;
  } else if (warp == kPvWarp) {
    // ============================ MMA issuer: O += P V ============================
    constexpr uint32_t idesc_pv = instr_desc(kBlockM, D, false, true);
    constexpr uint32_t idesc_pv_x = instr_desc(kBlockM, kXRows, true, false);  // O_x^T = V^T P_x^T
    const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
    const uint64_t dpx = smem_desc(sbase + G_::kOffPx, 16, 1024);
    const uint64_t dv0 = smem_desc(sbase + G_::kOffRing, kChunkBytes, 1024);  // V tile, MN-major
    bool ok = true;
    int g0 = 0, k = 0;
    int kx = 0;   // items with extra rows before the current one
    int gx0 = 0;  // tiles of such items
    int nt_cur = 0;  // KV tiles of the current item that this CTA processes
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++k, g0 += nt_cur) {
      const int j_lo = kSplit ? decode_item<kSplit>(prm, item).t0 : 0;
      nt_cur = kSplit ? decode_item<kSplit>(prm, item).nt : n_tiles;
      const bool has_x = kX && decode_item<kSplit>(prm, item).x_rows > 0;
      for (int jj = 0; jj < nt_cur && ok; ++jj) {
        const int j = j_lo + jj;
        (void)j;
        const int g = g0 + jj, gx = gx0 + jj;
        const int fill = 2 * g + 1, slot = fill % G_::kSlots, use = fill / G_::kSlots;
        bool w = mbar_wait2(bar_slot_full + 8 * slot, use & 1, bar_p_full + 8 * (g & 1), (g >> 1) & 1, abort_flag);
        // the epilogue of the previous item has read O before this item's first P V overwrites it
        if (jj == 0 && k > 0) w = w && mbar_wait(bar_o_free, (k - 1) & 1, abort_flag);
        if (!__all_sync(0xffffffffu, w)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const uint64_t dv = dv0 + (uint64_t)((slot * G_::kTileBytes) >> 4);
        if (elect_one()) {
#pragma unroll
          for (int ks = 0; ks < kBlockN / 16; ++ks)
            umma_ts(tm + G_::kTmemO, tm + ((g & 1) ? G_::kTmemS1 : G_::kTmemS0) + ks * 8, dv + ((ks * 2048) >> 4),
                    idesc_pv, (jj > 0 || ks > 0) ? 1u : 0u);
          umma_commit(bar_pv_done + 8 * (g & 1));  // frees S[g % 2] for Q K^T of tile g + 2
        }
        __syncwarp();
        if (has_x) {
          // the transposed problem's probabilities come from their own warps
          bool wx = mbar_wait(bar_px_full + 8 * (gx & 1), (gx >> 1) & 1, abort_flag);
          if (jj == 0 && kx > 0) wx = wx && mbar_wait(bar_ox_free, (kx - 1) & 1, abort_flag);
          if (!__all_sync(0xffffffffu, wx)) {
            ok = false;
            break;
          }
          tc_fence_after();
        }
        if (elect_one()) {
          if (has_x) {
            if constexpr (D == 128) {
#pragma unroll
              for (int ks = 0; ks < kBlockN / 16; ++ks) {
                const uint32_t offx = ((gx & 1) * 2 * kXChunkBytes + (ks / 4) * kXChunkBytes + (ks % 4) * 32) >> 4;
                umma_ss(tm + G_::kTmemOx, dv + ((ks * 2048) >> 4), dpx + offx, idesc_pv_x, (jj > 0 || ks > 0) ? 1u : 0u);
              }
              umma_commit(bar_pvx_done + 8 * (gx & 1));
            }
          }
          umma_commit(bar_slot_empty + 8 * slot);
          if (jj == nt_cur - 1) umma_commit(bar_o_full);
        }
        __syncwarp();
      }
      if (has_x) {
        ++kx;
        gx0 += nt_cur;
      }
    }
    timed_out = !ok;
  } else if (x_epilogue && warp >= kXWarp0 && warp < kXWarp0 + kXWarps) {
    // ============================ epilogue of the items (launches without extra rows) ============================
    // The softmax warps leave each row's sum and maximum in shared memory and go straight on to the next item,
    // whose first S tile is already waiting; these four warps, idle otherwise, wait for the item's last P V, read
    // O (thread = row = TMEM lane), release it for the next item, normalise and store.  Measured before: from
    // "last P stored" to the next item's first S tile the softmax warps spent about 5400 cycles against 300
    // between two tiles of one item.
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const float *xl = reinterpret_cast<const float *>(smem + G_::kOffPx);  // [2 item parities][2: sum, maximum][128 rows]
    bool ok = true;
    int k = 0;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++k) {
      const Item it = decode_item<kSplit>(prm, item);
      ok = __all_sync(0xffffffffu, mbar_wait(bar_x, k & 1, abort_flag));
      if (!ok) break;
      const float l_row = xl[((k & 1) * 2 + 0) * 128 + row], m_row = xl[((k & 1) * 2 + 1) * 128 + row];
      ok = __all_sync(0xffffffffu, mbar_wait(bar_o_full, k & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      const bool live = row < it.m_rows;
      const int R = it.mt * kBlockM + row;
      const int hq = it.hk * prm.G + R / prm.Lq, i = R % prm.Lq;
      const float inv = 1.f / l_row;
      __nv_bfloat16 *orow = reinterpret_cast<__nv_bfloat16 *>(prm.out) + (kSplit ? it.split * prm.out_split_stride : 0) + it.b * prm.out_stride[0] +
                            hq * prm.out_stride[1] + (long long)i * prm.out_stride[2];
#pragma unroll
      for (int cb = 0; cb < D; cb += 32) {
        uint32_t o[32];
        tmem_ld32(lane_base + G_::kTmemO + cb, o);
        tmem_wait_ld();
        if (cb + 32 == D) {  // O is in registers: the next item's first P V may overwrite it
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_o_free);
        }
        if (live) {
#pragma unroll
          for (int c = 0; c < 32; c += 8) {
            uint4 w;
            w.x = pack_bf16(__uint_as_float(o[c + 0]) * inv, __uint_as_float(o[c + 1]) * inv);
            w.y = pack_bf16(__uint_as_float(o[c + 2]) * inv, __uint_as_float(o[c + 3]) * inv);
            w.z = pack_bf16(__uint_as_float(o[c + 4]) * inv, __uint_as_float(o[c + 5]) * inv);
            w.w = pack_bf16(__uint_as_float(o[c + 6]) * inv, __uint_as_float(o[c + 7]) * inv);
            *reinterpret_cast<uint4 *>(orow + cb + c) = w;
          }
        }
      }
      if (live && prm.lse)
        prm.lse[(kSplit ? it.split * prm.lse_split_stride : 0) + ((long long)it.b * prm.Hq + hq) * prm.Lq + i] = (m_row + log2f(l_row)) * kLn2;
    }
    timed_out = !ok;
  } else if (kX && warp >= kXWarp0 && warp < kXWarp0 + kXWarps) {
    // ============================ transposed problem: softmax + epilogue ============================
    // Thread = key `row` of the tile (TMEM lane of S_x^T) and, for O_x^T, head-dimension element `row`.
    // The kXMax columns are the extra query rows.
    const int xw = warp - kXWarp0;
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const float c2 = prm.scale_log2;
    volatile int *xflag_s = reinterpret_cast<volatile int *>(smem + G_::kOffXflag);
    volatile float *xcol_s = reinterpret_cast<volatile float *>(smem + G_::kOffXcol);
    bool ok = true;
    int g0 = 0, k = 0, gx0 = 0;
    uint32_t n_y = 0;  // uses of bar_y so far (same in all four warps)
    // exchange through bar_y: every warp has written its part, everyone may read after the wait
    auto sync_y = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_y);
      bool w = mbar_wait(bar_y, n_y & 1, abort_flag);
      ++n_y;
      return __all_sync(0xffffffffu, w);
    };
    int nt_cur = 0;  // KV tiles of the current item that this CTA processes
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++k, g0 += nt_cur) {
      const int j_lo = kSplit ? decode_item<kSplit>(prm, item).t0 : 0;
      nt_cur = kSplit ? decode_item<kSplit>(prm, item).nt : n_tiles;
      const Item it = decode_item<kSplit>(prm, item);
      if (!(kX && it.x_rows > 0)) {
        // nothing to do, but stay in step with the per-item barrier (a parity wait cannot skip phases)
        ok = __all_sync(0xffffffffu, mbar_wait(bar_o_full, k & 1, abort_flag));
        continue;
      }
      float mref[kXMax], lx[kXMax];
#pragma unroll
      for (int i = 0; i < kXMax; ++i) mref[i] = 0.f, lx[i] = 0.f;
      for (int jj = 0; jj < nt_cur; ++jj) {
        const int j = j_lo + jj;
        const int gx = gx0 + jj;
        // S_x^T of this tile is ready (and with it the P_x^T buffer of this parity is free: the issuer
        // waited for the transposed P V of two such tiles back)
        ok = __all_sync(0xffffffffu, mbar_wait(bar_sx_full + 8 * (gx & 1), (gx >> 1) & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        uint32_t sx[kXMax];
        tmem_ld8(lane_base + ((gx & 1) ? G_::kTmemSx1 : G_::kTmemSx0), sx);
        tmem_wait_ld();
        const int valid = (j < n_pre) ? min(kBlockN, prm.P - j * kBlockN) : min(kBlockN, prm.Lq - (j - n_pre) * kBlockN);
        const bool kv_live = row < valid;  // keys past the end of a partial tile do not exist
        // Exponents against the reference.  A tile that outgrows it (and the first tile, which has no
        // reference yet) takes the slow path; the four warps vote.
        float tx[kXMax];
        bool over = (jj == 0);
#pragma unroll
        for (int i = 0; i < kXMax; ++i) {
          tx[i] = kv_live ? fmaf(__uint_as_float(sx[i]), c2, -mref[i]) : -INFINITY;
          over = over || (tx[i] > kXLimit);
        }
        over = __any_sync(0xffffffffu, over);
        if (lane == 0) {
          xflag_s[(gx & 1) * 4 + xw] = over ? 1 : 0;
          mbar_arrive(bar_x + 8 * (gx & 1));
        }
        ok = __all_sync(0xffffffffu, mbar_wait(bar_x + 8 * (gx & 1), (gx >> 1) & 1, abort_flag));
        if (!ok) break;
        const bool x_slow = (xflag_s[(gx & 1) * 4 + 0] | xflag_s[(gx & 1) * 4 + 1] | xflag_s[(gx & 1) * 4 + 2] |
                             xflag_s[(gx & 1) * 4 + 3]) != 0;
        if (x_slow) {
          // exact column maxima over the 128 keys of this tile
          float cm[kXMax], fx[kXMax];
#pragma unroll
          for (int i = 0; i < kXMax; ++i) {
            cm[i] = kv_live ? __uint_as_float(sx[i]) * c2 : -INFINITY;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) cm[i] = fmaxf(cm[i], __shfl_xor_sync(0xffffffffu, cm[i], o));
          }
          if (lane == 0) {
#pragma unroll
            for (int i = 0; i < kXMax; ++i) xcol_s[xw * kXMax + i] = cm[i];
          }
          ok = sync_y();
          if (!ok) break;
#pragma unroll
          for (int i = 0; i < kXMax; ++i) {
            const float c = fmaxf(fmaxf(xcol_s[0 * kXMax + i], xcol_s[1 * kXMax + i]),
                                  fmaxf(xcol_s[2 * kXMax + i], xcol_s[3 * kXMax + i]));
            const float m_new = (jj == 0) ? c : fmaxf(mref[i], c);
            fx[i] = (jj == 0) ? 0.f : ex2_approx(mref[i] - m_new);
            lx[i] *= fx[i];
            mref[i] = m_new;
            tx[i] = kv_live ? fmaf(__uint_as_float(sx[i]), c2, -m_new) : -INFINITY;
          }
          // xcol_s is reused by the next exchange: nobody may still be reading it
          ok = sync_y();
          if (!ok) break;
          if (jj > 0) {
            // O_x^T must be quiescent: the previous transposed P V has completed
            ok = __all_sync(0xffffffffu,
                            mbar_wait(bar_pvx_done + 8 * ((gx - 1) & 1), ((gx - 1) >> 1) & 1, abort_flag));
            if (!ok) break;
            tc_fence_after();
            uint32_t o[kXMax];
            tmem_ld8(lane_base + G_::kTmemOx, o);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < kXMax; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * fx[i]);
            tmem_st8(lane_base + G_::kTmemOx, o);
            tmem_wait_st();
          }
        }
        // P_x^T -> shared memory as a K-major [16 rows][128 keys] operand, 128-byte swizzle
        uint8_t *pxb = smem + G_::kOffPx + (gx & 1) * 2 * kXChunkBytes + (row >> 6) * kXChunkBytes + (row & 7) * 2;
        const int u = (row & 63) >> 3;
#pragma unroll
        for (int i = 0; i < kXMax; ++i) {
          const float px = ex2_approx(tx[i]);
          lx[i] += px;
          *reinterpret_cast<__nv_bfloat16 *>(pxb + i * 128 + ((u ^ (i & 7)) << 4)) = __float2bfloat16_rn(px);
        }
        fence_proxy_async();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_px_full + 8 * (gx & 1));
      }
      if (!ok) break;
      gx0 += nt_cur;
      // ---- epilogue: column sums over all keys, then O_x^T / sum ----
#pragma unroll
      for (int i = 0; i < kXMax; ++i) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) lx[i] += __shfl_xor_sync(0xffffffffu, lx[i], o);
      }
      if (lane == 0) {
#pragma unroll
        for (int i = 0; i < kXMax; ++i) xcol_s[xw * kXMax + i] = lx[i];
      }
      ok = sync_y();
      if (!ok) break;
#pragma unroll
      for (int i = 0; i < kXMax; ++i)
        lx[i] = (xcol_s[0 * kXMax + i] + xcol_s[1 * kXMax + i]) + (xcol_s[2 * kXMax + i] + xcol_s[3 * kXMax + i]);
      ok = __all_sync(0xffffffffu, mbar_wait(bar_o_full, k & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      uint32_t ox[kXMax];
      tmem_ld8(lane_base + G_::kTmemOx, ox);
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_ox_free);
      // xcol_s is free again only when everyone has read it
      ok = sync_y();
      if (!ok) break;
      __nv_bfloat16 *outp = reinterpret_cast<__nv_bfloat16 *>(prm.out) + (kSplit ? it.split * prm.out_split_stride : 0) + it.b * prm.out_stride[0];
#pragma unroll
      for (int i = 0; i < kXMax; ++i) {
        if (i < it.x_rows) {
          const int R = (it.mt + 1) * kBlockM + i;
          const int hq = it.hk * prm.G + R / prm.Lq, ii = R % prm.Lq;
          outp[hq * prm.out_stride[1] + (long long)ii * prm.out_stride[2] + row] =
              __float2bfloat16_rn(__uint_as_float(ox[i]) / lx[i]);
          if (prm.lse && row == 0)
            prm.lse[(kSplit ? it.split * prm.lse_split_stride : 0) + ((long long)it.b * prm.Hq + hq) * prm.Lq + ii] = (mref[i] + log2f(lx[i])) * kLn2;
        }
      }
    }
    timed_out = !ok;
  } else {
    // ============================ softmax + epilogue ============================
    const int half = lane >> 4;                            // column half this thread works on
    const int lane0 = (warp & 3) * 32 + (warp >> 2) * 16;   // first TMEM lane of this warp
    const int row = lane0 + (lane & 15);                   // TMEM lane = row of the M-tile
    const uint32_t lane_base = tmem + ((uint32_t)lane0 << 16);
    const float c2 = prm.scale_log2;
    constexpr int kOCols = D / 2;                          // accumulator columns per thread
    bool ok = true;
    int g0 = 0, k = 0;
    int nt_cur = 0;  // KV tiles of the current item that this CTA processes
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++k, g0 += nt_cur) {
      const int j_lo = kSplit ? decode_item<kSplit>(prm, item).t0 : 0;
      nt_cur = kSplit ? decode_item<kSplit>(prm, item).nt : n_tiles;
      const Item it = decode_item<kSplit>(prm, item);
      const bool live = row < it.m_rows;
      float m_used = -INFINITY;  // maximum the probabilities are expressed against (log2 units)
      float l_sum = 0.f;         // this thread's half of the row sum
      for (int jj = 0; jj < nt_cur; ++jj) {
        const int j = j_lo + jj;
        const int g = g0 + jj;
        ok = mbar_wait(bar_s_full + 8 * (g & 1), (g >> 1) & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t s_base = lane_base + ((g & 1) ? G_::kTmemS1 : G_::kTmemS0);
        uint32_t s[64];
        tmem_ld16x2_32<64>(s_base, &s[0]);        // columns 64 half + 0..31
        tmem_ld16x2_32<64>(s_base + 32, &s[32]);  // columns 64 half + 32..63
        tmem_wait_ld();
        // columns past the end of a partial tile do not exist
        const int valid = (j < n_pre) ? min(kBlockN, prm.P - j * kBlockN) : min(kBlockN, prm.Lq - (j - n_pre) * kBlockN);
        if (valid < kBlockN) {
          // selects, not branches: the two half-warps see different limits
          const int lim = valid - 64 * half;
#pragma unroll
          for (int c = 0; c < 64; ++c) s[c] = (c >= lim) ? 0xff800000u : s[c];  // -inf: columns past the end of a partial tile
        }
        // row maximum: eight independent chains over this half, then the other half by shuffle
        float mx;
        {
          float a[8];
#pragma unroll
          for (int c = 0; c < 8; ++c) a[c] = __uint_as_float(s[c]);
#pragma unroll
          for (int c = 8; c < 56; c += 16) {
#pragma unroll
            for (int u = 0; u < 8; ++u)
              a[u] = fmax3(a[u], __uint_as_float(s[c + u]), __uint_as_float(s[c + 8 + u]));
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) a[u] = fmaxf(a[u], __uint_as_float(s[56 + u]));
          mx = fmaxf(fmax3(a[0], a[1], a[2]), fmax3(a[3], a[4], a[5]));
          mx = fmax3(mx, a[6], a[7]);
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
        }
        const float m_tile = mx * c2;
        float factor = 1.f;
        if (m_tile > m_used + kRescaleThreshold || m_used == -INFINITY) {
          factor = (m_used == -INFINITY) ? 0.f : ex2_approx(m_used - m_tile);
          m_used = m_tile;
        }
        const bool warp_rescales = __any_sync(0xffffffffu, live && factor != 1.f) && (jj > 0);
        l_sum *= factor;
        float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
        const float neg_m = -m_used;
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
        l_sum += (l0 + l1) + (l2 + l3);
        if (warp_rescales) {
          // O must be quiescent: the previous P V has completed
          ok = mbar_wait(bar_pv_done + 8 * ((g - 1) & 1), ((g - 1) >> 1) & 1, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int cb = 0; cb < kOCols; cb += 32) {
            uint32_t o[32];
            tmem_ld16x2_32<kOCols>(lane_base + G_::kTmemO + cb, o);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * factor);
            tmem_st16x2_32<kOCols>(lane_base + G_::kTmemO + cb, o);
          }
        }
        // P row -> TMEM over the first 64 columns of its own S buffer (two bf16 per column); this
        // thread's 64 keys are columns 32 half .. 32 half + 31
        tmem_st16x2_32<32>(s_base, pk);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_p_full + 8 * (g & 1));
      }
      if (!ok) break;
      // ---- epilogue of the item ----
      l_sum += __shfl_xor_sync(0xffffffffu, l_sum, 16);
      if constexpr (x_epilogue) {
        // hand the row's sum and maximum to warps 10-13, which write the item's result, and go on
        float *xl = reinterpret_cast<float *>(smem + G_::kOffPx);
        if (half == 0) {
          xl[((k & 1) * 2 + 0) * 128 + row] = l_sum;
          xl[((k & 1) * 2 + 1) * 128 + row] = m_used;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_x);
        continue;
      }
      // the last P V of the item has completed (its own barrier, waited on once per item by everyone)
      ok = mbar_wait(bar_o_full, k & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t o[kOCols];
#pragma unroll
      for (int cb = 0; cb < kOCols; cb += 32) tmem_ld16x2_32<kOCols>(lane_base + G_::kTmemO + cb, &o[cb]);
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_o_free);
      if (live) {
        const int R = it.mt * kBlockM + row;
        const int hq = it.hk * prm.G + R / prm.Lq, i = R % prm.Lq;
        const float inv = 1.f / l_sum;
        __nv_bfloat16 *orow = reinterpret_cast<__nv_bfloat16 *>(prm.out) + (kSplit ? it.split * prm.out_split_stride : 0) + it.b * prm.out_stride[0] +
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
        if (prm.lse && half == 0)
          prm.lse[(kSplit ? it.split * prm.lse_split_stride : 0) + ((long long)it.b * prm.Hq + hq) * prm.Lq + i] = (m_used + log2f(l_sum)) * kLn2;
      }
    }
    timed_out = !ok;
  }

  if (timed_out && prm.status) atomicOr(prm.status, DS_DEV_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem, G_::kTmemCols);
  }
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
// Stacked query rows of one KV head: full 128-row tiles, and a remainder that either rides along with the
// last full tile (1..kXMax rows, D = 128) or gets a tile of its own.
void tile_counts(const ds_attn_params &p, int &n_mtiles, int &x_rows) {
  const long long rows_total = (long long)(p.Hq / p.Hkv) * p.Lq;
  const int n_full = (int)(rows_total / kBlockM), rem = (int)(rows_total % kBlockM);
  if (p.D == 128 && n_full >= 1 && rem >= 1 && rem <= kXMax) {
    n_mtiles = n_full;
    x_rows = rem;
  } else {
    n_mtiles = n_full + (rem ? 1 : 0);
    x_rows = 0;
  }
}

// Few work items (small batches) leave most SMs idle: split the KV tiles of every item over several CTAs.
struct SplitPlan {
  int splits, tiles_per_split;
  size_t out_bytes, lse_bytes;  // partial results in the workspace
};
SplitPlan choose_splits(const ds_attn_params &p) {
  int n_mtiles, x_rows;
  tile_counts(p, n_mtiles, x_rows);
  const int n_tiles = (p.P + kBlockN - 1) / kBlockN + (p.Lq + kBlockN - 1) / kBlockN;
  const long long base = (long long)(p.seq_list ? p.n_seq : p.B) * p.Hkv * n_mtiles;
  int s = 1;
  if (base > 0 && base * 2 <= sm_count() && n_tiles >= 4) {
    s = (int)(sm_count() / base);
    if (s > n_tiles / 2) s = n_tiles / 2;
    if (s > 8) s = 8;
  }
  SplitPlan sp;
  sp.tiles_per_split = (n_tiles + s - 1) / s;
  // the merge is a second launch and every split fetches the queries again, measured to cost what about
  // six KV tiles take: split only when it takes at least eight tiles off the critical path
  if (n_tiles - sp.tiles_per_split < 8) sp.tiles_per_split = n_tiles;
  sp.splits = (n_tiles + sp.tiles_per_split - 1) / sp.tiles_per_split;
  const size_t rows = (size_t)p.B * p.Hq * p.Lq;
  sp.out_bytes = sp.splits > 1 ? ((size_t)sp.splits * rows * p.D * 2 + 255) / 256 * 256 : 0;
  sp.lse_bytes = sp.splits > 1 ? (size_t)sp.splits * rows * 4 : 0;
  return sp;
}

// Merges the partial results of a split launch: out = sum_s w_s part_s / sum_s w_s with w_s = exp(lse_s - max lse).
// One warp per (sequence, head, row).
template <int D>
__global__ void __launch_bounds__(256) attn_combine_kernel(const __nv_bfloat16 *__restrict__ part, const float *__restrict__ plse,
                                                           int splits, long long out_split_stride, long long lse_split_stride,
                                                           int B, int Hq, int Lq, __nv_bfloat16 *__restrict__ out,
                                                           long long os0, long long os1, long long os2, float *__restrict__ lse,
                                                           const int32_t *__restrict__ seq_list, int n_seq,
                                                           const int32_t *__restrict__ n_seq_dev) {
  int n_live = B;
  if (seq_list != nullptr) {
    n_live = n_seq;
    if (n_seq_dev != nullptr) n_live = max(0, min(n_live, *n_seq_dev));
  }
  const long long r = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= (long long)n_live * Hq * Lq) return;
  const int lane = threadIdx.x & 31;
  const int i = (int)(r % Lq), hq = (int)((r / Lq) % Hq);
  int b = (int)(r / ((long long)Lq * Hq));
  if (seq_list != nullptr) b = min(max(seq_list[b], 0), B - 1);
  const long long prow = ((long long)b * Hq + hq) * Lq + i;
  float m = -INFINITY;
  for (int s = 0; s < splits; ++s) m = fmaxf(m, plse[s * lse_split_stride + prow]);
  constexpr int kPer = D / 32;  // consecutive elements per lane
  float acc[kPer];
#pragma unroll
  for (int c = 0; c < kPer; ++c) acc[c] = 0.f;
  float wsum = 0.f;
  for (int s = 0; s < splits; ++s) {
    const float w = __expf(plse[s * lse_split_stride + prow] - m);
    wsum += w;
    const __nv_bfloat16 *src = part + s * out_split_stride + prow * D + lane * kPer;
#pragma unroll
    for (int c = 0; c < kPer; ++c) acc[c] += w * __bfloat162float(src[c]);
  }
  const float inv = 1.f / wsum;
  __nv_bfloat16 *dst = out + b * os0 + hq * os1 + (long long)i * os2 + lane * kPer;
#pragma unroll
  for (int c = 0; c < kPer; ++c) dst[c] = __float2bfloat16_rn(acc[c] * inv);
  if (lse != nullptr && lane == 0) lse[prow] = m + __logf(wsum);
}

template <int D>
int prepare_d(const ds_attn_params &p, AttnPrepared &out) {
  static_assert(sizeof(TcParams) <= sizeof(out.kernel_params), "parameter struct does not fit the plan");
  TcParams &prm = *reinterpret_cast<TcParams *>(out.kernel_params);  // plain data, zeroed below
  memset(&prm, 0, sizeof(prm));
  out.path = kAttnPathTc;
  out.p = p;
  out.grid = 0;
  if (!fill_common(prm, p)) {
    note_cuda_error((int)cudaErrorInvalidValue);  // cuTensorMapEncodeTiled refused the layout
    return DS_ERR_CUDA;
  }
  tile_counts(p, prm.n_mtiles, prm.x_rows);
  const int n_tiles = (p.P + kBlockN - 1) / kBlockN + (p.Lq + kBlockN - 1) / kBlockN;
  prm.splits = 1;
  prm.tiles_per_split = n_tiles;
  prm.n_tiles = n_tiles;
  const SplitPlan sp = choose_splits(p);
  if (sp.splits > 1 && p.workspace != nullptr && (reinterpret_cast<uintptr_t>(p.workspace) & 255) == 0 &&
      p.workspace_bytes >= sp.out_bytes + sp.lse_bytes) {
    // partial results, one dense [B][Hq][Lq][D] copy (and [B][Hq][Lq] log-sum-exp) per split, in the workspace
    prm.splits = sp.splits;
    prm.tiles_per_split = sp.tiles_per_split;
    prm.out = p.workspace;
    prm.out_stride[0] = (long long)p.Hq * p.Lq * p.D;
    prm.out_stride[1] = (long long)p.Lq * p.D;
    prm.out_stride[2] = p.D;
    prm.out_split_stride = (long long)p.B * p.Hq * p.Lq * p.D;
    prm.lse = reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(p.workspace) + sp.out_bytes);
    prm.lse_split_stride = (long long)p.B * p.Hq * p.Lq;
  }
  const long long n_items = (long long)(p.seq_list ? p.n_seq : p.B) * p.Hkv * prm.n_mtiles * prm.splits;  // upper bound with a device count
  if (n_items > 0x7fffffffLL) return DS_ERR_UNSUPPORTED;
  prm.n_items = (int)n_items;
  out.grid = (int)(n_items < sm_count() ? n_items : sm_count());
  // Two query buffers (and one ring slot fewer) pay when a CTA runs several items and the stall at an item
  // boundary -- about two KV tiles' time with one buffer -- is a visible share of an item.
  prm.q2 = (n_items > out.grid && n_tiles <= kQ2MaxTiles) ? 1 : 0;
  return DS_OK;
}

template <int D, bool kSplit, bool kQ2, bool kX>
int launch_instance(const AttnPrepared &a, const TcParams &prm, cudaStream_t stream) {
  // the attribute is per device: set it at every launch (cheap)
  DS_CUDA_OK(cudaFuncSetAttribute(attn_tc_kernel<D, kSplit, kQ2, kX>, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<D, kQ2>::kSmemBytes));
  attn_tc_kernel<D, kSplit, kQ2, kX><<<a.grid, kNumThreads, Geo<D, kQ2>::kSmemBytes, stream>>>(prm);
  return DS_OK;
}
template <int D, bool kX>
int launch_mode(const AttnPrepared &a, const TcParams &prm, cudaStream_t stream) {
  // split launches: every CTA has one item (a part of one), a second query buffer would have nothing to prefetch
  if (prm.splits > 1) return launch_instance<D, true, false, kX>(a, prm, stream);
  if (prm.q2) return launch_instance<D, false, true, kX>(a, prm, stream);
  return launch_instance<D, false, false, kX>(a, prm, stream);
}

template <int D>
int launch_prepared_d(const AttnPrepared &a, cudaStream_t stream) {
  if (a.grid == 0) return DS_OK;
  const TcParams &prm = *reinterpret_cast<const TcParams *>(a.kernel_params);
  int rc;
  if constexpr (D == 128)
    rc = prm.x_rows > 0 ? launch_mode<D, true>(a, prm, stream) : launch_mode<D, false>(a, prm, stream);
  else
    rc = launch_mode<D, false>(a, prm, stream);
  if (rc != DS_OK) return rc;
  DS_CUDA_OK(cudaGetLastError());
  note_launch(1);
  if (prm.splits > 1) {
    const ds_attn_params &p = a.p;
    const long long rows = (long long)(p.seq_list ? p.n_seq : p.B) * p.Hq * p.Lq;
    attn_combine_kernel<D><<<(unsigned)((rows + 7) / 8), 256, 0, stream>>>(
        reinterpret_cast<const __nv_bfloat16 *>(prm.out), prm.lse, prm.splits, prm.out_split_stride, prm.lse_split_stride, p.B,
        p.Hq, p.Lq, reinterpret_cast<__nv_bfloat16 *>(p.out), p.out_stride[0], p.out_stride[1], p.out_stride[2], p.lse,
        p.seq_list, p.n_seq, p.seq_list ? p.n_seq_dev : nullptr);
    DS_CUDA_OK(cudaGetLastError());
    note_launch(1);
  }
  return DS_OK;
}

}  // namespace

namespace attn {
namespace {
// [B][H][rows][D] bf16 tensor with element strides {batch, head, row}; box = 64 columns x box_rows rows.
bool make_map(CUtensorMap *m, const void *base, int D, long long rows, int H, int B, const int64_t stride[3], int box_rows) {
  EncodeFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)rows, (cuuint64_t)H, (cuuint64_t)B};
  // a dimension of extent 1 may carry any stride; keep them valid multiples of 16 bytes
  const cuuint64_t strides[3] = {(cuuint64_t)stride[2] * 2, (cuuint64_t)(H > 1 ? stride[1] : stride[2] * rows) * 2,
                                 (cuuint64_t)(B > 1 ? stride[0] : (H > 1 ? stride[1] * H : stride[2] * rows)) * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool fill_common(AttnCommon &c, const ds_attn_params &p) {
  const int D = p.D;
  bool ok = true;
  if (p.P > 0) {
    ok = ok && make_map(&c.kpre, p.k_prefix, D, p.P, p.Hkv, p.B, p.kv_prefix_stride, kBlockN);
    ok = ok && make_map(&c.vpre, p.v_prefix, D, p.P, p.Hkv, p.B, p.kv_prefix_stride, kBlockN);
  }
  ok = ok && make_map(&c.k32, p.k_tail, D, p.T, p.Hkv, p.B, p.kv_tail_stride, 32);
  ok = ok && make_map(&c.k1, p.k_tail, D, p.T, p.Hkv, p.B, p.kv_tail_stride, 1);
  ok = ok && make_map(&c.v32, p.v_tail, D, p.T, p.Hkv, p.B, p.kv_tail_stride, 32);
  ok = ok && make_map(&c.v1, p.v_tail, D, p.T, p.Hkv, p.B, p.kv_tail_stride, 1);
  ok = ok && make_map(&c.q32, p.q_tail, D, p.T, p.Hq, p.B, p.q_stride, 32);
  ok = ok && make_map(&c.q1, p.q_tail, D, p.T, p.Hq, p.B, p.q_stride, 1);
  ok = ok && make_map(&c.k128, p.k_tail, D, p.T, p.Hkv, p.B, p.kv_tail_stride, 128);
  ok = ok && make_map(&c.v128, p.v_tail, D, p.T, p.Hkv, p.B, p.kv_tail_stride, 128);
  ok = ok && make_map(&c.q128, p.q_tail, D, p.T, p.Hq, p.B, p.q_stride, 128);
  if (!ok) return false;
  c.idx = p.idx;
  c.idx_bstride = p.idx_batch_stride;
  c.out = p.out;
  for (int k = 0; k < 3; ++k) c.out_stride[k] = p.out_stride[k];
  c.lse = p.lse;
  c.status = p.status;
  c.B = p.B, c.Hq = p.Hq, c.Hkv = p.Hkv, c.G = p.Hq / p.Hkv, c.P = p.P, c.T = p.T, c.Lq = p.Lq;
  c.scale_log2 = p.scale * kLog2e;
  c.seq_list = p.seq_list;
  c.n_seq_dev = p.seq_list ? p.n_seq_dev : nullptr;
  c.n_seq = p.n_seq;
  return true;
}
}  // namespace attn

namespace sm100 {
EncodeFn encode_fn() {
  static EncodeFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeFn>(p);
    else
      (void)cudaGetLastError();
  });
  return fn;
}
}  // namespace sm100

bool attn_tc_supported(const ds_attn_params &p) {
  if (p.dtype != DS_BF16 || (p.D != 64 && p.D != 128)) return false;
  if (!(p.scale > 0.f) || p.scale > 1e30f) return false;  // the running maximum assumes a positive scale
  if ((long long)(p.Hq / p.Hkv) * p.Lq > (1ll << 30)) return false;
  // a tensor map has no broadcast dimension: batch and head strides of extents above 1 must be positive
  const int64_t *st[3] = {p.q_stride, p.kv_tail_stride, p.kv_prefix_stride};
  const int heads[3] = {p.Hq, p.Hkv, p.Hkv};
  for (int k = 0; k < 3; ++k) {
    if (k == 2 && p.P == 0) continue;
    if ((p.B > 1 && st[k][0] <= 0) || (heads[k] > 1 && st[k][1] <= 0)) return false;
  }
  // TMA: 16-byte aligned bases and strides are already guaranteed by validation; extents must fit 32 bits
  return true;
}

size_t attn_tc_workspace_bytes(const ds_attn_params &p) {
  const SplitPlan sp = choose_splits(p);
  return sp.out_bytes + sp.lse_bytes;
}

int prepare_attn_tc(const ds_attn_params &p, AttnPrepared &out) {
  return p.D == 128 ? prepare_d<128>(p, out) : prepare_d<64>(p, out);
}
int launch_prepared_tc(const AttnPrepared &a, cudaStream_t stream) {
  return a.p.D == 128 ? launch_prepared_d<128>(a, stream) : launch_prepared_d<64>(a, stream);
}
int launch_attn_tc(const ds_attn_params &p, cudaStream_t stream) {
  AttnPrepared a;
  const int rc = prepare_attn_tc(p, a);
  return rc != DS_OK ? rc : launch_prepared_tc(a, stream);
}

}  // namespace ds
