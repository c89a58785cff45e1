// Pieces shared by the tensor-core attention kernels: the launch parameters common to both, the gather
// of index-listed rows into swizzled shared-memory tiles, and the tensor-map encoding of the
// [B][H][rows][D] operands.
#pragma once
#include "ds_sm100.cuh"

namespace ds {
namespace attn {

using namespace sm100;

constexpr int kBlockM = 128;
constexpr int kBlockN = 128;
constexpr int kChunkBytes = 128 * 128;  // one [128 rows][64 bf16] swizzled chunk
constexpr int kIdxCap = 2048;           // entries of a shared index list kept in shared memory

struct AttnCommon {
  CUtensorMap kpre, vpre, k32, k1, v32, v1, q32, q1;
  CUtensorMap k128, v128, q128;  // boxes of a whole 128-row tile, for runs of consecutive rows
  const int32_t *idx;
  long long idx_bstride;
  void *out;
  long long out_stride[3];
  float *lse;
  uint32_t *status;
  int B, Hq, Hkv, G, P, T, Lq;
  float scale_log2;  // softmax scale * log2(e)
  // optional restriction to listed sequences (the ones whose block still has masked positions)
  const int32_t *seq_list;   // ascending batch numbers, nullptr = all B
  const int32_t *n_seq_dev;  // device count overriding n_seq (clamped to [0, n_seq]), may be nullptr
  int n_seq;
};

// Number of sequences this launch processes, and the batch number of the s-th of them.
__device__ __forceinline__ int live_sequences(const AttnCommon &c) {
  if (c.seq_list == nullptr) return c.B;
  int n = c.n_seq;
  if (c.n_seq_dev != nullptr) n = max(0, min(n, *c.n_seq_dev));
  return n;
}
__device__ __forceinline__ int listed_batch(const AttnCommon &c, int s) {
  if (c.seq_list == nullptr) return s;
  return min(max(c.seq_list[s], 0), c.B - 1);
}
// Producer warp: flags list entries outside [0, B) (they are clamped by listed_batch).
__device__ __forceinline__ bool bad_sequence_numbers(const AttnCommon &c, int n_live) {
  bool bad = false;
  if (c.seq_list != nullptr)
    for (int s = threadIdx.x & 31; s < n_live; s += 32) {
      const int v = c.seq_list[s];
      bad |= (v < 0 || v >= c.B);
    }
  return bad;
}

// ------------------------------------------------------------------------------------------------
// Producer helper: the index list shared by all batches (idx_bstride == 0) is checked once per CTA --
// every entry in [0, T), strictly ascending -- and its head is kept in shared memory.  Returns true when
// the whole list passed; the caller then passes list_ok = true to gather_rows, which may decide from the
// first and last entry of a run that the rows between them are consecutive.  Entries out of range are
// clamped in the cached copy and flagged.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ bool cache_shared_index_list(const AttnCommon &prm, int32_t *cache, bool &bad_index) {
  const int lane = threadIdx.x & 31;
  bool ok = true;
  for (int i = lane; i < prm.Lq; i += 32) {
    int v = prm.idx[i];
    const int before = (i > 0) ? prm.idx[i - 1] : -1;
    if (v < 0 || v >= prm.T) {
      ok = false;
      v = v < 0 ? 0 : prm.T - 1;
    }
    if (v <= before) ok = false;
    if (i < kIdxCap) cache[i] = v;
  }
  ok = __all_sync(0xffffffffu, ok);
  if (!ok) bad_index = true;
  return ok;
}

// ------------------------------------------------------------------------------------------------
// Producer helper: fetch n gathered rows (logical rows R0 .. R0+n-1 of a stacked sequence whose
// period is Lq) into a swizzled tile whose 64-column chunks are chunk_stride bytes apart.  The whole
// warp calls it; lane 0 issues the copies (a whole-tile fetch: one lane per chunk).  Returns the bytes issued.
// tile_end: the n rows are the last ones of their tile (whatever the copy writes behind them is not used).
//
// Runs of consecutive rows are fetched as one box (128 or 32 rows).  With list_ok (the list is known to be
// strictly ascending and in range) the first and last entry of a run decide; otherwise every entry of the
// run is looked at, and a tile whose entries are not strictly ascending is flagged and fetched row by row.
// ------------------------------------------------------------------------------------------------
template <int D>
__device__ __forceinline__ uint32_t gather_rows(const AttnCommon &prm, const CUtensorMap *map32, const CUtensorMap *map1,
                                                const CUtensorMap *map128, uint32_t dst, uint32_t chunk_stride, uint32_t bar, int R0, int n,
                                                int head0, int b, int32_t *idx_s, const int32_t *idx_cache, bool list_ok,
                                                bool &bad_index, bool staged = false, bool tile_end = false) {
  const int lane = threadIdx.x & 31;
  const int Lq = prm.Lq;
  const int32_t *ix = prm.idx + (long long)b * prm.idx_bstride;
  // position of logical row R0 inside its head; divisions only when the stacking actually wraps
  int head = head0, pos0 = R0;
  if (pos0 >= Lq) {
    head += pos0 / Lq;
    pos0 %= Lq;
  }
  // A full tile of consecutive rows inside one head (the current block and its window, every tile of a
  // cache-refresh step) needs no staging: one box per 64-column chunk fetches it, each chunk issued by a
  // lane of its own.
  // The same box serves a shorter run when it is the last thing in the tile (so that the rows the box brings
  // beyond the run overwrite nothing) and ends with the last row of the buffer: the box then reaches past the
  // end of the tensor, where the copy fills in zeros.  That is every partial tile of compact buffers (T = Lq,
  // idx = 0 .. Lq - 1), the layout ds_rope_gather produces.
  // (Not for a handful of rows: the copy writes all 128 rows of the tile, zeros included.)
  if (pos0 + n <= Lq && (n == 128 || (tile_end && n > 32))) {
    int first, last;
    if (idx_cache != nullptr && pos0 + n - 1 < kIdxCap) {
      first = idx_cache[pos0];
      last = idx_cache[pos0 + n - 1];
    } else {
      first = ix[pos0];
      last = ix[pos0 + n - 1];
    }
    bool whole = (last - first == n - 1 && first >= 0 && last < prm.T) && (n == 128 || last == prm.T - 1);
    if (whole && !list_ok) {
      // the order of the list is not known: all n entries must be the consecutive rows
      bool run = true;
#pragma unroll
      for (int k = 0; k < 4; ++k) run = run && (lane + 32 * k >= n || ix[pos0 + lane + 32 * k] == first + lane + 32 * k);
      whole = __all_sync(0xffffffffu, run);
    }
    if (whole) {
      if (lane < (D / 64)) tma_load_4d(dst + lane * chunk_stride, map128, bar, lane * 64, first, head, b);
      return 128u * 128u * (D / 64);
    }
  }
  __syncwarp();
  if (!staged) {  // otherwise idx_s already holds these rows (the K tile of the same rows came first)
    for (int r = lane; r < n; r += 32) {
      int pos = pos0 + r;
      if (pos >= Lq) pos %= Lq;
      int v;
      if (idx_cache != nullptr && pos < kIdxCap) {
        v = idx_cache[pos];  // validated when it was cached
      } else {
        v = ix[pos];
        if (v < 0 || v >= prm.T) {
          bad_index = true;
          v = v < 0 ? 0 : prm.T - 1;
        }
      }
      idx_s[r] = v;
    }
    __syncwarp();
  }
  // may runs of this tile be fetched as 32-row boxes?  (a box follows the memory order of the rows)
  bool boxes = list_ok;
  if (!list_ok) {
    bool asc = true;
    for (int r = lane + 1; r < n; r += 32) {
      int pos = pos0 + r;
      if (pos >= Lq) pos %= Lq;
      asc = asc && (pos == 0 || idx_s[r] > idx_s[r - 1]);  // the stacking starts the list again at every head
    }
    boxes = __all_sync(0xffffffffu, asc);
    if (!boxes) bad_index = true;
  }
  uint32_t bytes = 0;
  if (lane == 0) {
    // one lane issues: the copies of an SM are taken one after the other whichever lanes issue them
    int r = 0, pos = pos0;
    while (r < n) {
      const int row = idx_s[r];
      const bool box32 = boxes && (r + 32 <= n) && (pos + 32 <= Lq) && (idx_s[r + 31] - row == 31);
      const int step = box32 ? 32 : 1;
#pragma unroll
      for (int c = 0; c < (D / 64); ++c)
        tma_load_4d(dst + c * chunk_stride + r * 128, box32 ? map32 : map1, bar, c * 64, row, head, b);
      bytes += (uint32_t)step * 128u * (D / 64);
      r += step;
      pos += step;
      if (pos >= Lq) {  // a 32-row box never crosses a head, so this is at most one wrap
        pos -= Lq;
        ++head;
      }
    }
  }
  return bytes;
}


// Fills the tensor maps and the fields common to both kernels from the C-ABI parameters.
bool fill_common(AttnCommon &c, const ds_attn_params &p);

}  // namespace attn
}  // namespace ds
