// ds_attn_pruned, tensor-core path for bf16 (Eq. 7-8): TMA-staged KV tiles, tcgen05 MMAs with
// TMEM accumulators, online softmax.
//
// Work item = (batch, KV head, 128-row M-tile).  The query heads of one GQA group are stacked along
// M (row R = head_in_group * Lq + i), so every KV tile is read once per group.  KV is streamed as
// 128-row tiles: first the cached prefix (tiled TMA boxes, out-of-range rows zero-filled), then the
// retained tail rows named by the index list, fetched as 32-row TMA boxes where the list is
// contiguous and as single-row boxes elsewhere.
//
// Warp roles (192 threads, one CTA per SM):
//   warps 0-3  softmax + epilogue; thread t owns TMEM lane t = S/O row t
//   warp  4    TMA producer (lane 0 issues; the warp pre-loads the index list of each gathered tile)
//   warp  5    TMEM allocation and MMA issue (lane 0)
// Per KV tile j:  S[j%2] = Q K_j^T  (tcgen05.mma, both operands K-major, 128B swizzle)
//                 softmax warps: tcgen05.ld S, running max with lazy rescale, P = 2^(s*c - m) as bf16
//                 into a swizzled shared-memory tile
//                 O += P V_j       (A = P K-major, B = V MN-major straight from its [kv][D] layout)
// S is double buffered so Q K_{j+1}^T runs under the softmax of tile j.  The accumulator O is only
// rescaled when a row maximum grows by more than 2^8 (the stale maximum keeps P within bf16/fp32
// range), which removes the TMEM round trip from the steady state.
//
// Every mbarrier wait is bounded; on expiry the thread raises DS_DEV_TIMEOUT in the status word,
// all roles leave their loops, outstanding TMA copies are waited for (bounded), TMEM is freed and the
// CTA returns.
#include <cuda.h>

#include <cstdio>
#include <mutex>

#include "ds_common.cuh"

namespace ds {
namespace {

constexpr int kBlockM = 128;
constexpr int kBlockN = 128;
constexpr int kNumThreads = 192;
constexpr int kChunkBytes = 128 * 128;  // one [128 rows][64 bf16] swizzled chunk
constexpr int kPBytes = kBlockM * kBlockN * 2;
constexpr uint32_t kSpinLimit = 1u << 20;
constexpr float kRescaleThreshold = 8.0f;  // log2 units

template <int D>
struct Geo {
  static constexpr int kChunks = D / 64;                     // 64-column chunks per tile
  static constexpr int kTileBytes = kChunks * kChunkBytes;   // Q / K / V tile
  static constexpr int kSlots = (D == 128) ? 5 : 10;         // ring of K/V tiles
  static constexpr int kOffQ = 0;
  static constexpr int kOffP = kTileBytes;
  static constexpr int kOffRing = kOffP + kPBytes;
  static constexpr int kOffBar = kOffRing + kSlots * kTileBytes;
  // barriers: q_full, s_full[2], s_free[2], p_full, pv_done, slot_full[kSlots], slot_empty[kSlots]
  static constexpr int kNumBars = 7 + 2 * kSlots;
  static constexpr int kOffIdx = kOffBar + 8 * kNumBars;     // int32[128] gathered-row indices
  static constexpr int kOffMisc = kOffIdx + 4 * 128;         // tmem base, abort flag
  static constexpr int kSmemBytes = kOffMisc + 16 + 1024;    // + slack to align the base to 1024
  static constexpr int kTmemCols = 512;
  static constexpr int kTmemS0 = 0, kTmemS1 = 128, kTmemO = 256;
};

struct TcParams {
  CUtensorMap kpre, vpre, k32, k1, v32, v1, q32, q1;
  const int32_t *idx;
  long long idx_bstride;
  void *out;
  long long out_stride[3];
  float *lse;
  uint32_t *status;
  int B, Hq, Hkv, G, P, T, Lq;
  float scale_log2;  // softmax scale * log2(e)
};

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when it gave up (or another role already did).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 128) {
      __nanosleep(64);
      if (*abort_flag) return false;
    }
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// mbarrier arrives once all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
      ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
        "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
        "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]), "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128.
__host__ __device__ constexpr uint32_t instr_desc(int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(kBlockM >> 4) << 24);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// ------------------------------------------------------------------------------------------------
// Producer helper: fetch up to 128 gathered rows (logical rows R0 .. R0+n-1 of a stacked sequence whose
// period is Lq) into a swizzled tile.  The whole warp calls it; lane 0 issues the copies.
// Returns the bytes issued (valid on lane 0).
// ------------------------------------------------------------------------------------------------
template <int D>
__device__ __forceinline__ uint32_t gather_rows(const TcParams &prm, const CUtensorMap *map32, const CUtensorMap *map1,
                                                uint32_t dst, uint32_t bar, int R0, int n, int head0, int b,
                                                int32_t *idx_s, bool &bad_index) {
  const int lane = threadIdx.x & 31;
  const int32_t *ix = prm.idx + (long long)b * prm.idx_bstride;
  __syncwarp();
  for (int r = lane; r < n; r += 32) {
    int v = ix[(R0 + r) % prm.Lq];
    if (v < 0 || v >= prm.T) {
      bad_index = true;
      v = v < 0 ? 0 : prm.T - 1;
    }
    idx_s[r] = v;
  }
  __syncwarp();
  uint32_t bytes = 0;
  if (lane == 0) {
    int r = 0;
    while (r < n) {
      const int R = R0 + r;
      const int head = head0 + R / prm.Lq;
      const int row = idx_s[r];
      const bool box32 = ((r & 7) == 0) && (r + 32 <= n) && ((R % prm.Lq) + 32 <= prm.Lq) && (idx_s[r + 31] - row == 31);
      if (box32) {
#pragma unroll
        for (int c = 0; c < Geo<D>::kChunks; ++c) tma_load_4d(dst + c * kChunkBytes + r * 128, map32, bar, c * 64, row, head, b);
        bytes += 32u * 128u * Geo<D>::kChunks;
        r += 32;
      } else {
#pragma unroll
        for (int c = 0; c < Geo<D>::kChunks; ++c) tma_load_4d(dst + c * kChunkBytes + r * 128, map1, bar, c * 64, row, head, b);
        bytes += 128u * Geo<D>::kChunks;
        r += 1;
      }
    }
  }
  return bytes;
}

// ------------------------------------------------------------------------------------------------
// The kernel
// ------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(kNumThreads, 1) attn_tc_kernel(const __grid_constant__ TcParams prm) {
  using G_ = Geo<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  const uint32_t bar0 = sbase + G_::kOffBar;
  const uint32_t bar_q_full = bar0;
  const uint32_t bar_s_full = bar0 + 8;    // [2]
  const uint32_t bar_s_free = bar0 + 24;   // [2]
  const uint32_t bar_p_full = bar0 + 40;
  const uint32_t bar_pv_done = bar0 + 48;
  const uint32_t bar_slot_full = bar0 + 56;                       // [kSlots]
  const uint32_t bar_slot_empty = bar_slot_full + 8 * G_::kSlots;  // [kSlots]
  int32_t *idx_s = reinterpret_cast<int32_t *>(smem + G_::kOffIdx);
  volatile uint32_t *tmem_base_s = reinterpret_cast<volatile uint32_t *>(smem + G_::kOffMisc);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + G_::kOffMisc + 4);

  const int mt = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
  const int rows_total = prm.G * prm.Lq;                        // stacked query rows of this KV head
  const int m_rows = min(kBlockM, rows_total - mt * kBlockM);   // valid rows of this M-tile
  const int n_pre = (prm.P + kBlockN - 1) / kBlockN;
  const int n_tail = (prm.Lq + kBlockN - 1) / kBlockN;
  const int n_tiles = n_pre + n_tail;

  if (tid == 0) {
    mbar_init(bar_q_full, 1);
    mbar_init(bar_s_full, 1);
    mbar_init(bar_s_full + 8, 1);
    mbar_init(bar_s_free, 4);
    mbar_init(bar_s_free + 8, 4);
    mbar_init(bar_p_full, 4);
    mbar_init(bar_pv_done, 1);
    for (int s = 0; s < G_::kSlots; ++s) {
      mbar_init(bar_slot_full + 8 * s, 1);
      mbar_init(bar_slot_empty + 8 * s, 1);
    }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 5) tmem_alloc(sbase + G_::kOffMisc, G_::kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_base_s;
  bool timed_out = false;

  if (warp == 4) {
    // ============================ TMA producer ============================
    bool bad_index = false;
    {
      const uint32_t bytes = gather_rows<D>(prm, &prm.q32, &prm.q1, sbase + G_::kOffQ, bar_q_full, mt * kBlockM, m_rows,
                                            hk * prm.G, b, idx_s, bad_index);
      if (lane == 0) mbar_arrive_expect_tx(bar_q_full, bytes);
    }
    int issued = 0;  // ring fills issued so far
    for (int j = 0; j < n_tiles && !timed_out; ++j) {
      for (int kv = 0; kv < 2; ++kv) {
        const int slot = issued % G_::kSlots, use = issued / G_::kSlots;
        const uint32_t dst = sbase + G_::kOffRing + slot * G_::kTileBytes;
        const uint32_t full = bar_slot_full + 8 * slot;
        bool ok = mbar_wait(bar_slot_empty + 8 * slot, (use & 1) ^ 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) {
          timed_out = true;
          break;
        }
        if (j < n_pre) {
          if (lane == 0) {
            const CUtensorMap *map = kv ? &prm.vpre : &prm.kpre;
#pragma unroll
            for (int c = 0; c < G_::kChunks; ++c) tma_load_4d(dst + c * kChunkBytes, map, full, c * 64, j * kBlockN, hk, b);
            mbar_arrive_expect_tx(full, G_::kTileBytes);
          }
        } else {
          const int t0 = (j - n_pre) * kBlockN;
          const int n = min(kBlockN, prm.Lq - t0);
          if (kv == 1 && n < kBlockN) {
            // rows past the end of a V tile meet P = 0 in the MMA: make them zero, not stale
            const int nz_rows = kBlockN - n;
            for (int q = lane; q < nz_rows * 8 * G_::kChunks; q += 32) {
              const int u = q % 8, row = n + (q / 8) % nz_rows, c = q / (8 * nz_rows);
              *reinterpret_cast<uint4 *>(smem + G_::kOffRing + slot * G_::kTileBytes + c * kChunkBytes + row * 128 + u * 16) =
                  make_uint4(0, 0, 0, 0);
            }
            fence_proxy_async();
          }
          const uint32_t bytes = gather_rows<D>(prm, kv ? &prm.v32 : &prm.k32, kv ? &prm.v1 : &prm.k1, dst, full, t0, n, hk, b,
                                                idx_s, bad_index);
          if (lane == 0) mbar_arrive_expect_tx(full, bytes);
        }
        ++issued;
      }
    }
    if (timed_out) {
      // let copies already in flight land before the CTA's shared memory goes away
      for (int k = max(0, issued - G_::kSlots); k < issued; ++k)
        for (uint32_t it = 0; it < 4096 && !mbar_try_wait(bar_slot_full + 8 * (k % G_::kSlots), (k / G_::kSlots) & 1); ++it)
          __nanosleep(256);
    }
    if (bad_index && prm.status) atomicOr(prm.status, DS_DEV_INDEX);
  } else if (warp == 5) {
    // ============================ MMA issuer ============================
    if (lane == 0) {
      constexpr uint32_t idesc_qk = instr_desc(kBlockN, false);
      constexpr uint32_t idesc_pv = instr_desc(D, true);
      const uint32_t q_addr = sbase + G_::kOffQ, p_addr = sbase + G_::kOffP;
      auto issue_qk = [&](int j) -> bool {
        const int fill = 2 * j, slot = fill % G_::kSlots, use = fill / G_::kSlots;
        if (!mbar_wait(bar_slot_full + 8 * slot, use & 1, abort_flag)) return false;
        if (!mbar_wait(bar_s_free + 8 * (j & 1), ((j >> 1) & 1) ^ 1, abort_flag)) return false;
        tc_fence_after();
        const uint32_t k_addr = sbase + G_::kOffRing + slot * G_::kTileBytes;
        const uint32_t d = tmem + ((j & 1) ? G_::kTmemS1 : G_::kTmemS0);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t off = (ks / 4) * kChunkBytes + (ks % 4) * 32;
          umma_bf16(d, smem_desc(q_addr + off, 16, 1024), smem_desc(k_addr + off, 16, 1024), idesc_qk, ks > 0);
        }
        umma_commit(bar_s_full + 8 * (j & 1));
        umma_commit(bar_slot_empty + 8 * slot);
        return true;
      };
      bool ok = mbar_wait(bar_q_full, 0, abort_flag);
      if (ok) ok = issue_qk(0);
      for (int j = 0; j < n_tiles && ok; ++j) {
        if (j + 1 < n_tiles) ok = issue_qk(j + 1);
        if (!ok) break;
        const int fill = 2 * j + 1, slot = fill % G_::kSlots, use = fill / G_::kSlots;
        if (!mbar_wait(bar_slot_full + 8 * slot, use & 1, abort_flag)) { ok = false; break; }
        if (!mbar_wait(bar_p_full, j & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t v_addr = sbase + G_::kOffRing + slot * G_::kTileBytes;
#pragma unroll
        for (int ks = 0; ks < kBlockN / 16; ++ks) {
          const uint64_t a = smem_desc(p_addr + (ks / 4) * kChunkBytes + (ks % 4) * 32, 16, 1024);
          const uint64_t bdesc = smem_desc(v_addr + ks * 2048, kChunkBytes, 1024);
          umma_bf16(tmem + G_::kTmemO, a, bdesc, idesc_pv, (j > 0 || ks > 0) ? 1u : 0u);
        }
        umma_commit(bar_pv_done);
        umma_commit(bar_slot_empty + 8 * slot);
      }
      timed_out = !ok;
    }
  } else {
    // ============================ softmax + epilogue ============================
    const int row = tid;                                  // TMEM lane = row of the M-tile
    const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
    float m_used = -INFINITY;                             // maximum the probabilities are expressed against (log2 units)
    float l_sum = 0.f;
    const float c2 = prm.scale_log2;
    uint8_t *p_row = smem + G_::kOffP + row * 128;
    bool ok = true;
    for (int j = 0; j < n_tiles; ++j) {
      ok = mbar_wait(bar_s_full + 8 * (j & 1), (j >> 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t s[128];
      {
        const uint32_t ta = lane_base + ((j & 1) ? G_::kTmemS1 : G_::kTmemS0);
        tmem_ld32(ta, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
        tmem_ld32(ta + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
        tmem_ld32(ta + 64, *reinterpret_cast<uint32_t(*)[32]>(&s[64]));
        tmem_ld32(ta + 96, *reinterpret_cast<uint32_t(*)[32]>(&s[96]));
        tmem_wait_ld();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_s_free + 8 * (j & 1));
      // columns past the end of a partial tile do not exist
      const int valid = (j < n_pre) ? min(kBlockN, prm.P - j * kBlockN) : min(kBlockN, prm.Lq - (j - n_pre) * kBlockN);
      if (valid < kBlockN) {
#pragma unroll
        for (int k = 0; k < 128; ++k)
          if (k >= valid) s[k] = 0xff800000u;  // -inf
      }
      float mx = __uint_as_float(s[0]);
#pragma unroll
      for (int k = 1; k < 128; ++k) mx = fmaxf(mx, __uint_as_float(s[k]));
      const float m_tile = mx * c2;
      float factor = 1.f;
      if (m_tile > m_used + kRescaleThreshold || m_used == -INFINITY) {
        factor = (m_used == -INFINITY) ? 0.f : ex2_approx(m_used - m_tile);
        m_used = m_tile;
      }
      const bool warp_rescales = __any_sync(0xffffffffu, factor != 1.f) && (j > 0);
      l_sum *= factor;
      float l0 = 0.f, l1 = 0.f;
      const float neg_m = -m_used;
      uint32_t pk[64];
#pragma unroll
      for (int k = 0; k < 64; ++k) {
        const float p0 = ex2_approx(fmaf(__uint_as_float(s[2 * k]), c2, neg_m));
        const float p1 = ex2_approx(fmaf(__uint_as_float(s[2 * k + 1]), c2, neg_m));
        pk[k] = pack_bf16(p0, p1);
        // normalise with the bf16 values the MMA will actually use: sum_j p~_j v_j / sum_j p~_j is then a
        // convex combination of value rows whatever the rounding of p was
        l0 += bf16lo_to_f32(pk[k]);
        l1 += bf16hi_to_f32(pk[k]);
      }
      l_sum += l0 + l1;
      if (j > 0) {
        // P buffer free and O quiescent once the previous P V has completed
        ok = mbar_wait(bar_pv_done, (j - 1) & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        if (warp_rescales) {
#pragma unroll
          for (int cb = 0; cb < D; cb += 32) {
            uint32_t o[32];
            tmem_ld32(lane_base + G_::kTmemO + cb, o);
            tmem_wait_ld();
#pragma unroll
            for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * factor);
            tmem_st32(lane_base + G_::kTmemO + cb, o);
          }
          tmem_wait_st();
        }
      }
      // P row -> shared memory, K-major 128-byte swizzle: 16-byte unit u of a 128-byte row lands at u ^ (row % 8)
#pragma unroll
      for (int g = 0; g < 16; ++g) {
        const int c = g >> 3, u = g & 7;
        *reinterpret_cast<uint4 *>(p_row + c * kChunkBytes + ((u ^ (row & 7)) << 4)) =
            make_uint4(pk[4 * g], pk[4 * g + 1], pk[4 * g + 2], pk[4 * g + 3]);
      }
      fence_proxy_async();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_p_full);
    }
    if (ok) {
      ok = mbar_wait(bar_pv_done, (n_tiles - 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      const int R = mt * kBlockM + row;
      const bool live = row < m_rows;
      const int hq = hk * prm.G + (live ? R / prm.Lq : 0), i = live ? R % prm.Lq : 0;
      const float inv = 1.f / l_sum;
      __nv_bfloat16 *orow = reinterpret_cast<__nv_bfloat16 *>(prm.out) + b * prm.out_stride[0] + hq * prm.out_stride[1] +
                            (long long)i * prm.out_stride[2];
#pragma unroll
      for (int cb = 0; cb < D; cb += 32) {
        uint32_t o[32];
        tmem_ld32(lane_base + G_::kTmemO + cb, o);
        tmem_wait_ld();
        if (live) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint4 w;
            w.x = pack_bf16(__uint_as_float(o[8 * g + 0]) * inv, __uint_as_float(o[8 * g + 1]) * inv);
            w.y = pack_bf16(__uint_as_float(o[8 * g + 2]) * inv, __uint_as_float(o[8 * g + 3]) * inv);
            w.z = pack_bf16(__uint_as_float(o[8 * g + 4]) * inv, __uint_as_float(o[8 * g + 5]) * inv);
            w.w = pack_bf16(__uint_as_float(o[8 * g + 6]) * inv, __uint_as_float(o[8 * g + 7]) * inv);
            *reinterpret_cast<uint4 *>(orow + cb + 8 * g) = w;
          }
        }
      }
      if (live && prm.lse) prm.lse[((long long)b * prm.Hq + hq) * prm.Lq + i] = (m_used + log2f(l_sum)) * kLn2;
      tc_fence_before();
    }
    timed_out = !ok;
  }

  if (timed_out && prm.status) atomicOr(prm.status, DS_DEV_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem, G_::kTmemCols);
  }
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
using EncodeFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                              const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

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

template <int D>
int launch_d(const ds_attn_params &p, cudaStream_t stream) {
  static std::once_flag once;
  static cudaError_t attr_rc = cudaSuccess;
  std::call_once(once, [] {
    attr_rc = cudaFuncSetAttribute(attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<D>::kSmemBytes);
  });
  // the attribute is per device: set it again when the current device changed (cheap)
  DS_CUDA_OK(cudaFuncSetAttribute(attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<D>::kSmemBytes));
  (void)attr_rc;
  TcParams prm;
  memset(&prm, 0, sizeof(prm));
  bool ok = true;
  if (p.P > 0) {
    ok = ok && make_map(&prm.kpre, p.k_prefix, D, p.P, p.Hkv, p.B, p.kv_prefix_stride, kBlockN);
    ok = ok && make_map(&prm.vpre, p.v_prefix, D, p.P, p.Hkv, p.B, p.kv_prefix_stride, kBlockN);
  }
  ok = ok && make_map(&prm.k32, p.k_tail, D, p.T, p.Hkv, p.B, p.kv_tail_stride, 32);
  ok = ok && make_map(&prm.k1, p.k_tail, D, p.T, p.Hkv, p.B, p.kv_tail_stride, 1);
  ok = ok && make_map(&prm.v32, p.v_tail, D, p.T, p.Hkv, p.B, p.kv_tail_stride, 32);
  ok = ok && make_map(&prm.v1, p.v_tail, D, p.T, p.Hkv, p.B, p.kv_tail_stride, 1);
  ok = ok && make_map(&prm.q32, p.q_tail, D, p.T, p.Hq, p.B, p.q_stride, 32);
  ok = ok && make_map(&prm.q1, p.q_tail, D, p.T, p.Hq, p.B, p.q_stride, 1);
  if (!ok) return DS_ERR_CUDA;
  prm.idx = p.idx;
  prm.idx_bstride = p.idx_batch_stride;
  prm.out = p.out;
  for (int k = 0; k < 3; ++k) prm.out_stride[k] = p.out_stride[k];
  prm.lse = p.lse;
  prm.status = p.status;
  prm.B = p.B, prm.Hq = p.Hq, prm.Hkv = p.Hkv, prm.G = p.Hq / p.Hkv, prm.P = p.P, prm.T = p.T, prm.Lq = p.Lq;
  prm.scale_log2 = p.scale * kLog2e;
  const int n_mtiles = ceil_div((long long)prm.G * p.Lq, kBlockM);
  const dim3 grid(n_mtiles, p.Hkv, p.B);
  attn_tc_kernel<D><<<grid, kNumThreads, Geo<D>::kSmemBytes, stream>>>(prm);
  DS_CUDA_OK(cudaGetLastError());
  note_launch(1);
  return DS_OK;
}

}  // namespace

bool attn_tc_supported(const ds_attn_params &p) {
  if (p.dtype != DS_BF16 || (p.D != 64 && p.D != 128)) return false;
  if (!(p.scale > 0.f) || p.scale > 1e30f) return false;  // the running maximum assumes a positive scale
  if (p.Hkv > 65535 || p.B > 65535) return false;
  if ((long long)(p.Hq / p.Hkv) * p.Lq > (1ll << 30)) return false;
  // TMA: 16-byte aligned bases and strides are already guaranteed by validation; extents must fit 32 bits
  return true;
}

size_t attn_tc_workspace_bytes(const ds_attn_params &) { return 0; }

int launch_attn_tc(const ds_attn_params &p, cudaStream_t stream) {
  return p.D == 128 ? launch_d<128>(p, stream) : launch_d<64>(p, stream);
}

}  // namespace ds
