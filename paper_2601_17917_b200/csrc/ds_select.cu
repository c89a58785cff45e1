// ds_unmask_select: Eq. 10 threshold, Eq. 9 selection, Eq. 5 update, block
// termination and the early-exit flag, as warp-level compaction.
//
// One warp owns one sequence.  It walks the block 32 positions at a time:
// a ballot of the mask flags counts n (first pass), the threshold follows in
// fp32 with one rounding per operation, then a second pass takes the ballot of
// "masked and conf >= tau", turns it into ascending output slots with a prefix
// popcount, and tracks the best masked confidence (lowest index among equals)
// for the fallback.  The list of sequences whose block still has masks is an
// ordered compaction over sequences: in the single-CTA launch it follows in
// the same kernel, otherwise in a second one-CTA kernel.
#include <climits>

#include "ds_common.cuh"

namespace ds {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;

__device__ __forceinline__ float eq10_threshold(int n_masked, int K, int extra, float tau0, float alpha) {
  const float r = __fdiv_rn((float)(n_masked + extra), (float)(K + extra));
  const float t1 = __fsub_rn(1.0f, r);
  const float t2 = __fmul_rn(alpha, t1);
  const float t3 = __fsub_rn(1.0f, t2);
  return __fmul_rn(tau0, t3);
}

__device__ void select_sequence(const ds_select_params &p, int b, int lane) {
  const int K = p.K;
  const float *c = p.conf + (long long)b * K;
  const int32_t *t = p.tok + (long long)b * K;
  uint8_t *mk = p.masked + (long long)b * K;
  int32_t *x = p.x_block + (long long)b * K;
  int32_t *si = p.sel_idx + (long long)b * K;

  int nm = 0;
  for (int base = 0; base < K; base += 32) {
    const int i = base + lane;
    const bool m = (i < K) && (mk[i] != 0);
    nm += __popc(__ballot_sync(0xffffffffu, m));
  }
  const float tau = eq10_threshold(nm, K, p.ratio_extra, p.tau0, p.alpha);

  int cnt = 0;
  float best_c = -INFINITY;
  int best_i = INT_MAX;
  bool eos = false;
  for (int base = 0; base < K; base += 32) {
    const int i = base + lane;
    const bool m = (i < K) && (mk[i] != 0);
    const float ci = m ? c[i] : 0.f;
    const bool acc = m && (ci >= tau);
    const unsigned bal = __ballot_sync(0xffffffffu, acc);
    if (acc) {
      const int slot = cnt + __popc(bal & ((1u << lane) - 1u));
      const int ti = t[i];
      si[slot] = i;
      x[i] = ti;
      mk[i] = 0;
      if (p.eos_id >= 0 && ti == p.eos_id && ci >= p.eos_tau) eos = true;
    }
    cnt += __popc(bal);
    if (m && (best_i == INT_MAX || ci > best_c)) {  // ascending i per lane: strict > keeps the lowest index
      best_c = ci;
      best_i = i;
    }
  }
  // fallback candidate: highest confidence, lowest index among equals
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float oc = __shfl_xor_sync(0xffffffffu, best_c, o);
    const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
    const bool take = (oi != INT_MAX) && (best_i == INT_MAX || oc > best_c || (oc == best_c && oi < best_i));
    if (take) {
      best_c = oc;
      best_i = oi;
    }
  }
  if (cnt == 0 && nm > 0) {
    if (lane == 0) {
      const int ti = t[best_i];
      si[0] = best_i;
      x[best_i] = ti;
      mk[best_i] = 0;
      if (p.eos_id >= 0 && ti == p.eos_id && best_c >= p.eos_tau) eos = true;
    }
    cnt = 1;
  }
  for (int i = cnt + lane; i < K; i += 32) si[i] = -1;
  const bool any_eos = __any_sync(0xffffffffu, eos);
  if (lane == 0) {
    p.sel_cnt[b] = cnt;
    p.block_done[b] = (uint8_t)((nm - cnt) == 0);
    if (any_eos) p.eos_exit[b] = 1;
  }
}

__device__ __forceinline__ int listed_count(const ds_select_params &p) {
  int n = p.seq_list ? p.n_seq : p.B;
  if (p.seq_list && p.n_seq_dev) {
    const int d = *p.n_seq_dev;
    n = d < n ? d : n;
    if (n < 0) n = 0;
  }
  return n;
}

// Ordered compaction of the processed sequences whose block is not finished.
// Runs in one CTA of kSelThreads threads.  active_seq may be the array seq_list points to and active_cnt the
// word n_seq_dev points to: every thread has read its entry of a round (and the count) before the barrier
// that precedes the round's writes, and a round only writes positions at or below the ones it read.
__device__ void compact_active(const ds_select_params &p, int n) {
  __shared__ int warp_cnt[kSelWarps];
  __shared__ int running;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  if (tid == 0) running = 0;
  __syncthreads();
  for (int base = 0; base < n; base += kSelThreads) {
    const int s = base + tid;
    int b = -1;
    bool act = false;
    if (s < n) {
      b = p.seq_list ? p.seq_list[s] : s;
      act = (b >= 0 && b < p.B) && p.block_done[b] == 0;
    }
    const unsigned bal = __ballot_sync(0xffffffffu, act);
    if (lane == 0) warp_cnt[wid] = __popc(bal);
    __syncthreads();
    int off = running;
    for (int w = 0; w < wid; ++w) off += warp_cnt[w];
    if (act) p.active_seq[off + __popc(bal & ((1u << lane) - 1u))] = b;
    __syncthreads();
    if (tid == 0) {
      int tot = 0;
      for (int w = 0; w < kSelWarps; ++w) tot += warp_cnt[w];
      running += tot;
    }
    __syncthreads();
  }
  if (tid == 0) *p.active_cnt = running;
}

// Ordered list of the rows b * K + i that are still masked, over the processed sequences in list order.
// Runs in one CTA of kSelThreads threads after the selection: one sequence per warp, kSelWarps per round.
__device__ void compact_masked_rows(const ds_select_params &p, int n) {
  __shared__ int rem_cnt[kSelWarps];
  __shared__ int rows_so_far;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int K = p.K;
  if (tid == 0) rows_so_far = 0;
  __syncthreads();
  for (int s0 = 0; s0 < n; s0 += kSelWarps) {
    const int s = s0 + wid;
    int b = -1;
    if (s < n) {
      b = p.seq_list ? p.seq_list[s] : s;
      if (b < 0 || b >= p.B) b = -1;
    }
    const uint8_t *mk = p.masked + (long long)(b < 0 ? 0 : b) * K;
    int rem = 0;
    if (b >= 0) {
      for (int base = 0; base < K; base += 32) {
        const int i = base + lane;
        rem += __popc(__ballot_sync(0xffffffffu, (i < K) && (mk[i] != 0)));
      }
    }
    if (lane == 0) rem_cnt[wid] = rem;
    __syncthreads();
    int off = rows_so_far;
    for (int w = 0; w < wid; ++w) off += rem_cnt[w];
    if (b >= 0 && rem > 0) {
      for (int base = 0; base < K; base += 32) {
        const int i = base + lane;
        const bool m = (i < K) && (mk[i] != 0);
        const unsigned bal = __ballot_sync(0xffffffffu, m);
        if (m) p.masked_rows[off + __popc(bal & ((1u << lane) - 1u))] = b * K + i;
        off += __popc(bal);
      }
    }
    __syncthreads();
    if (tid == 0) {
      int tot = 0;
      for (int w = 0; w < kSelWarps; ++w) tot += rem_cnt[w];
      rows_so_far += tot;
    }
    __syncthreads();
  }
  if (tid == 0) *p.masked_cnt = rows_so_far;
}

__global__ void __launch_bounds__(kSelThreads) select_fused_kernel(const ds_select_params p) {
  const int n = listed_count(p);
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  for (int s = wid; s < n; s += kSelWarps) {
    const int b = p.seq_list ? p.seq_list[s] : s;
    if (b >= 0 && b < p.B) select_sequence(p, b, lane);
  }
  __syncthreads();  // block_done and the mask flags of every sequence written by this CTA are visible below
  // the row list first: it walks seq_list, which compact_active may overwrite (active_seq may be the same array)
  if (p.masked_rows != nullptr) compact_masked_rows(p, n);
  compact_active(p, n);
}

__global__ void __launch_bounds__(256) select_grid_kernel(const ds_select_params p) {
  const int n = listed_count(p);
  const int lane = threadIdx.x & 31;
  const int s = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (s >= n) return;
  const int b = p.seq_list ? p.seq_list[s] : s;
  if (b >= 0 && b < p.B) select_sequence(p, b, lane);
}

__global__ void __launch_bounds__(kSelThreads) select_compact_kernel(const ds_select_params p) {
  const int n = listed_count(p);
  if (p.masked_rows != nullptr) compact_masked_rows(p, n);
  compact_active(p, n);
}

// Start of a block: mask flags, block tokens and the lists of the sequences that have not exited.
__global__ void __launch_bounds__(kSelThreads) block_begin_kernel(const ds_block_params p) {
  __shared__ int warp_cnt[kSelWarps];
  __shared__ int running;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  if (tid == 0) running = 0;
  __syncthreads();
  for (int base = 0; base < p.B; base += kSelThreads) {  // ordered compaction of the live sequences
    const int b = base + tid;
    const bool live = (b < p.B) && (p.eos_exit[b] == 0);
    const unsigned bal = __ballot_sync(0xffffffffu, live);
    if (lane == 0) warp_cnt[wid] = __popc(bal);
    __syncthreads();
    int off = running;
    for (int w = 0; w < wid; ++w) off += warp_cnt[w];
    if (live) p.active_seq[off + __popc(bal & ((1u << lane) - 1u))] = b;
    __syncthreads();
    if (tid == 0) {
      int tot = 0;
      for (int w = 0; w < kSelWarps; ++w) tot += warp_cnt[w];
      running += tot;
    }
    __syncthreads();
  }
  const int n_live = running;
  if (tid == 0) {
    *p.active_cnt = n_live;
    if (p.masked_cnt) *p.masked_cnt = n_live * p.K;
  }
  // one warp per sequence: its K flags and tokens
  for (int b = wid; b < p.B; b += kSelWarps) {
    const bool live = p.eos_exit[b] == 0;
    for (int i = lane; i < p.K; i += 32) {
      p.masked[(long long)b * p.K + i] = live ? 1 : 0;
      p.x_block[(long long)b * p.K + i] = live ? p.mask_id : p.fill_id;
    }
  }
  if (p.masked_rows) {
    __syncthreads();  // active_seq as written above by this CTA
    for (int a = wid; a < n_live; a += kSelWarps) {
      const int b = p.active_seq[a];
      for (int i = lane; i < p.K; i += 32) p.masked_rows[(long long)a * p.K + i] = b * p.K + i;
    }
  }
}

}  // namespace

int launch_block_begin(const ds_block_params &p, cudaStream_t stream) {
  block_begin_kernel<<<1, kSelThreads, 0, stream>>>(p);
  DS_CUDA_OK(cudaGetLastError());
  note_launch(1);
  return DS_OK;
}

int launch_select(const ds_select_params &p, cudaStream_t stream) {
  const int n = p.seq_list ? p.n_seq : p.B;
  // Up to this many sequence-positions one CTA handles with low latency; beyond it, spread over the GPU.
  const long long work = (long long)n * p.K;
  if (n <= kSelWarps * 8 && work <= 64 * 1024) {
    select_fused_kernel<<<1, kSelThreads, 0, stream>>>(p);
    DS_CUDA_OK(cudaGetLastError());
    note_launch(1);
  } else {
    const int warps_per_cta = 8;
    select_grid_kernel<<<ceil_div(n, warps_per_cta), warps_per_cta * 32, 0, stream>>>(p);
    DS_CUDA_OK(cudaGetLastError());
    select_compact_kernel<<<1, kSelThreads, 0, stream>>>(p);
    DS_CUDA_OK(cudaGetLastError());
    note_launch(2);
  }
  return DS_OK;
}

}  // namespace ds
