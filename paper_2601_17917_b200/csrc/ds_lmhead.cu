// ds_lmhead_confidence: output projection z = W h fused with Eq. 4 (c = max softmax(z), x^ = argmax z).
// The [rows x V] logits are never written to memory: they live as fp32 accumulators in TMEM and are
// reduced to (max, sum of exponentials, arg max) per row and per 256-token tile of the vocabulary;
// a second small kernel merges the per-tile triples of every row.
//
// GEMM shape: C[rows][V] = H[rows][hid] * W[V][hid]^T, both operands K-major bf16, fp32 accumulate.
// CTA tile = 256 rows x 256 tokens, as two tcgen05 MMAs of M = 128, N = 256 that share the W tile in
// shared memory (so a CTA reads 64 B of operands per MMA-clock instead of 96); the two accumulators fill
// the 512 TMEM columns.  K is streamed in 64-element chunks through a 3-stage TMA ring (64 KB per stage:
// two 128-row pieces of H and one 256-row piece of W, 128-byte swizzle).  CTAs are persistent; tiles are
// ordered with the row block fastest, so the CTAs that run at the same time share W tiles through L2
// and W is read from HBM about once.
//
// Warp roles (320 threads, one CTA per SM):
//   warp 0      TMA producer
//   warp 1      TMEM allocation, MMA issue (one elected lane)
//   warps 2-9   epilogue: thread = one row of one accumulator (warps 2-5 rows 0..127, 6-9 rows 128..255),
//               256 columns read 32 at a time; online max / sum of 2^((z - max) log2 e) / lowest arg max
// The accumulators are not double buffered: the epilogue of a tile (a few thousand cycles) is exposed
// once per tile, against 64 K-chunks x 8 MMAs x 128 cycles of MMA time at hid = 4096.
//
// Every wait is a bounded mbarrier wait; on expiry the kernel raises DS_DEV_TIMEOUT in the status word,
// drains and frees TMEM.
#include <cuda.h>

#include <climits>
#include <cstring>

#include "ds_common.cuh"
#include "ds_sm100.cuh"

namespace ds {
namespace {

using namespace sm100;

constexpr int kBM = 256, kBN = 256, kBK = 64;
constexpr int kStages = 3;
constexpr int kEpiWarps = 8;
constexpr int kThreads = (2 + kEpiWarps) * 32;
constexpr int kPieceBytes = 128 * 128;           // 128 rows x 64 bf16
constexpr int kStageBytes = 4 * kPieceBytes;     // H rows 0..127, H rows 128..255, W rows 0..255
constexpr int kOffBar = kStages * kStageBytes;   // full[kStages], empty[kStages], acc_full, acc_free
constexpr int kOffMisc = kOffBar + 8 * (2 * kStages + 2);
constexpr int kSmemBytes = kOffMisc + 16 + 1024;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

struct Triple {
  float m;  // maximum logit of the tile
  float s;  // sum of exp(z - m) over the tile
  int i;    // lowest index attaining m
  int pad;
};

struct LmParams {
  CUtensorMap h_map, w_map;
  Triple *partials;  // [n_ntiles][rows]
  uint32_t *status;
  int rows, V, hid;
  int n_mblk, n_ntiles, n_kchunks;
};

__global__ void __launch_bounds__(kThreads, 1) lmhead_kernel(const __grid_constant__ LmParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t bar_full = sbase + kOffBar;
  const uint32_t bar_empty = bar_full + 8 * kStages;
  const uint32_t bar_acc_full = bar_empty + 8 * kStages;
  const uint32_t bar_acc_free = bar_acc_full + 8;
  volatile uint32_t *tmem_base_s = reinterpret_cast<volatile uint32_t *>(smem + kOffMisc);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kOffMisc + 4);

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    mbar_init(bar_acc_full, 1);
    mbar_init(bar_acc_free, kEpiWarps);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(sbase + kOffMisc, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_base_s;
  const int n_tiles = prm.n_mblk * prm.n_ntiles;
  bool timed_out = false;

  if (warp == 0) {
    // ============================ TMA producer ============================
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&prm.h_map)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&prm.w_map)) : "memory");
    }
    int fill = 0;
    for (int t = blockIdx.x; t < n_tiles && !timed_out; t += gridDim.x) {
      const int mb = t % prm.n_mblk, nt = t / prm.n_mblk;
      const bool two = mb * kBM + 128 < prm.rows;  // does the second 128-row half hold any row?
      for (int kc = 0; kc < prm.n_kchunks; ++kc, ++fill) {
        const int slot = fill % kStages, use = fill / kStages;
        bool ok = mbar_wait(bar_empty + 8 * slot, (use & 1) ^ 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) {
          timed_out = true;
          break;
        }
        if (lane == 0) {
          const uint32_t dst = sbase + slot * kStageBytes, full = bar_full + 8 * slot;
          mbar_arrive_expect_tx(full, two ? kStageBytes : 3 * kPieceBytes);
          tma_load_2d(dst, &prm.h_map, full, kc * kBK, mb * kBM);
          if (two) tma_load_2d(dst + kPieceBytes, &prm.h_map, full, kc * kBK, mb * kBM + 128);
          tma_load_2d(dst + 2 * kPieceBytes, &prm.w_map, full, kc * kBK, nt * kBN);
        }
      }
    }
    if (timed_out) {
      for (int f = max(0, fill - kStages); f < fill; ++f)
        for (uint32_t w = 0; w < 4096 && !mbar_try_wait(bar_full + 8 * (f % kStages), (f / kStages) & 1); ++w)
          __nanosleep(256);
    }
  } else if (warp == 1) {
    // ============================ MMA issuer ============================
    constexpr uint32_t idesc = instr_desc(128, kBN, false, false);
    const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
    const uint64_t d0 = smem_desc(sbase, 16, 1024);
    bool ok = true;
    int fill = 0, it = 0;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++it) {
      const int mb = t % prm.n_mblk;
      const bool two = mb * kBM + 128 < prm.rows;
      // the epilogue has read the accumulators of the previous tile
      if (it > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar_acc_free, (it - 1) & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      for (int kc = 0; kc < prm.n_kchunks && ok; ++kc, ++fill) {
        const int slot = fill % kStages, use = fill / kStages;
        ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * slot, use & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        if (elect_one()) {
          const uint64_t da = d0 + (uint64_t)((slot * kStageBytes) >> 4);
          const uint64_t db = da + (uint64_t)((2 * kPieceBytes) >> 4);
#pragma unroll
          for (int ks = 0; ks < kBK / 16; ++ks) {
            const uint32_t acc = (kc > 0 || ks > 0) ? 1u : 0u;
            umma_ss(tm, da + ((ks * 32) >> 4), db + ((ks * 32) >> 4), idesc, acc);
            if (two) umma_ss(tm + 256, da + ((kPieceBytes + ks * 32) >> 4), db + ((ks * 32) >> 4), idesc, acc);
          }
          umma_commit(bar_empty + 8 * slot);
          if (kc == prm.n_kchunks - 1) umma_commit(bar_acc_full);
        }
        __syncwarp();
      }
    }
    timed_out = !ok;
  } else {
    // ============================ epilogue ============================
    const int e = warp - 2;             // 0..7
    const int half = e >> 2;            // which accumulator
    const int row_in_half = (warp & 3) * 32 + lane;  // TMEM lane (warp w may touch lanes 32 (w % 4) ..)
    const uint32_t acc_base = tmem + ((uint32_t)((warp & 3) * 32) << 16) + half * 256;
    bool ok = true;
    int it = 0;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++it) {
      const int mb = t % prm.n_mblk, nt = t / prm.n_mblk;
      const bool two = mb * kBM + 128 < prm.rows;
      ok = __all_sync(0xffffffffu, mbar_wait(bar_acc_full, it & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      const int row = mb * kBM + half * 128 + row_in_half;
      if (half == 0 || two) {
        float m = -INFINITY, ssum = 0.f, best = -INFINITY;
        int best_i = INT_MAX;
        const int col0 = nt * kBN;
#pragma unroll 1
        for (int cb = 0; cb < kBN; cb += 32) {
          uint32_t z[32];
          tmem_ld32(acc_base + cb, z);
          tmem_wait_ld();
          // tokens past the end of the vocabulary do not exist
          if (col0 + cb + 32 > prm.V) {
#pragma unroll
            for (int c = 0; c < 32; ++c)
              if (col0 + cb + c >= prm.V) z[c] = 0xff800000u;  // -inf
          }
          float cm = __uint_as_float(z[0]);
#pragma unroll
          for (int c = 1; c < 32; ++c) cm = fmaxf(cm, __uint_as_float(z[c]));
          if (cm > m) {
            ssum *= (m == -INFINITY) ? 0.f : ex2_approx((m - cm) * kLog2e);
            m = cm;
          }
          const float nml = -m * kLog2e;
          float s0 = 0.f, s1 = 0.f;
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            s0 += ex2_approx(fmaf(__uint_as_float(z[c]), kLog2e, nml));
            s1 += ex2_approx(fmaf(__uint_as_float(z[c + 1]), kLog2e, nml));
          }
          if (m != -INFINITY) ssum += s0 + s1;
          if (cm > best) {  // strictly greater: an earlier chunk keeps an equal maximum; find the first column
            best = cm;
#pragma unroll
            for (int c = 31; c >= 0; --c)
              if (__uint_as_float(z[c]) == cm) best_i = col0 + cb + c;
          }
        }
        if (row < prm.rows) {
          Triple tr;
          tr.m = m;
          tr.s = ssum;
          tr.i = best_i;
          tr.pad = 0;
          *reinterpret_cast<int4 *>(&prm.partials[(long long)nt * prm.rows + row]) = *reinterpret_cast<int4 *>(&tr);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_acc_free);
    }
    timed_out = !ok;
  }

  if (timed_out && prm.status) atomicOr(prm.status, DS_DEV_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// Merges the per-tile triples of every row: one warp per row, equal maxima resolve to the lowest index.
__global__ void __launch_bounds__(256) lmhead_merge_kernel(const Triple *__restrict__ partials, int rows, int n_ntiles,
                                                           float *__restrict__ conf, int32_t *__restrict__ tok) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  float m = -INFINITY, s = 0.f;
  int idx = INT_MAX;
  auto merge = [&](float om, float os, int oi) {
    const float nm = fmaxf(m, om);
    if (nm == -INFINITY) return;
    const float ea = (m == nm) ? 1.f : ex2_approx((m - nm) * kLog2e);
    const float eb = (om == nm) ? 1.f : ex2_approx((om - nm) * kLog2e);
    if (om > m || (om == m && oi < idx)) idx = oi;
    s = s * ea + os * eb;
    m = nm;
  };
  for (int t = lane; t < n_ntiles; t += 32) {
    const int4 raw = __ldg(reinterpret_cast<const int4 *>(&partials[(long long)t * rows + row]));
    merge(__int_as_float(raw.x), __int_as_float(raw.y), raw.z);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, o);
    const float os = __shfl_xor_sync(0xffffffffu, s, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    merge(om, os, oi);
  }
  if (lane == 0) {
    conf[row] = 1.f / s;
    tok[row] = idx;
  }
}

bool make_map_2d(CUtensorMap *m, const void *base, long long rows, long long cols, long long ld, int box_rows) {
  EncodeFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

size_t lmhead_workspace_bytes(int64_t rows, int64_t V) {
  if (rows <= 0 || V <= 0) return 0;
  return (size_t)((V + kBN - 1) / kBN) * (size_t)rows * sizeof(Triple);
}

int launch_lmhead_confidence(const void *hidden, const void *weight, int64_t rows, int64_t hid, int64_t V, int64_t ld_h,
                             int64_t ld_w, float *conf, int32_t *tok, void *workspace, uint32_t *status,
                             cudaStream_t stream) {
  DS_CUDA_OK(cudaFuncSetAttribute(lmhead_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  LmParams prm;
  memset(&prm, 0, sizeof(prm));
  if (!make_map_2d(&prm.h_map, hidden, rows, hid, ld_h, 128) || !make_map_2d(&prm.w_map, weight, V, hid, ld_w, kBN))
    return DS_ERR_CUDA;
  prm.partials = reinterpret_cast<Triple *>(workspace);
  prm.status = status;
  prm.rows = (int)rows, prm.V = (int)V, prm.hid = (int)hid;
  prm.n_mblk = ceil_div(rows, kBM);
  prm.n_ntiles = ceil_div(V, kBN);
  prm.n_kchunks = ceil_div(hid, kBK);
  const long long n_tiles = (long long)prm.n_mblk * prm.n_ntiles;
  const int grid = (int)(n_tiles < sm_count() ? n_tiles : sm_count());
  lmhead_kernel<<<grid, kThreads, kSmemBytes, stream>>>(prm);
  DS_CUDA_OK(cudaGetLastError());
  lmhead_merge_kernel<<<ceil_div(rows, 8), 256, 0, stream>>>(prm.partials, (int)rows, prm.n_ntiles, conf, tok);
  DS_CUDA_OK(cudaGetLastError());
  note_launch(2);
  return DS_OK;
}

}  // namespace ds
