// ds_rope_gather: rotary position encoding of the retained tail rows with their ORIGINAL position ids,
// gathered into compact Q / K / V buffers, and (optionally) the append of a finished block's K / V to
// the prefix cache.  (Eq. 7: the pruned suffix keeps token order through RoPE position ids; Eq. 8: the
// pruned input; prefix KV is cached once per block.)
//
// HBM-bound element-wise work.  One thread owns the 8 elements d0..d0+7 of the low half of one row and
// the 8 matching elements of the high half (the rotate-half pairing couples d with d + D/2), i.e. two
// 16-byte loads and two 16-byte stores per rotated tensor; D/16 consecutive threads cover a row, so a
// warp reads whole 128-byte segments.  The frequencies theta^(-2d/D) come from the host in double,
// split into two floats; the angle position * frequency is formed as an exact product plus correction
// (a position of several thousand times an fp32-rounded frequency would be off by 1e-3 rad), sincosf of
// the leading part is corrected to first order by the rest.  The angle depends on (row, d) only, so a
// thread evaluates it once and applies it to 8 heads.
#include <cmath>

#include "ds_common.cuh"

namespace ds {
namespace {

constexpr int kRopeThreads = 256;
constexpr int kMaxHalf = 128;

struct RopeTable {
  float hi[kMaxHalf], lo[kMaxHalf];  // frequency of pair d = hi[d] + lo[d]
};

struct Bf16x8 {
  uint4 w;
};
__device__ __forceinline__ void unpack8(const uint4 &w, float (&f)[8]) {
  f[0] = bf16lo_to_f32(w.x), f[1] = bf16hi_to_f32(w.x), f[2] = bf16lo_to_f32(w.y), f[3] = bf16hi_to_f32(w.y);
  f[4] = bf16lo_to_f32(w.z), f[5] = bf16hi_to_f32(w.z), f[6] = bf16lo_to_f32(w.w), f[7] = bf16hi_to_f32(w.w);
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t *>(&v);
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  return make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7]));
}

constexpr int kHeadsPerThread = 8;  // heads that share one evaluation of the sines and cosines

__global__ void __launch_bounds__(kRopeThreads) rope_gather_kernel(const ds_rope_params p, const RopeTable tab) {
  const int D = p.D, half = D >> 1, units = half >> 3;  // 16-byte units per half row
  const int Hall = p.Hq + 2 * p.Hkv;                    // query heads, key heads, value heads
  const int chunks = (Hall + kHeadsPerThread - 1) / kHeadsPerThread;
  const long long total = (long long)p.B * p.Lq * chunks * units;
  bool bad_index = false;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (long long)gridDim.x * blockDim.x) {
    const int u = (int)(t % units);
    long long rest = t / units;
    const int ch = (int)(rest % chunks);
    rest /= chunks;
    const int i = (int)(rest % p.Lq);
    const int b = (int)(rest / p.Lq);
    int r = p.idx[(long long)b * p.idx_batch_stride + i];
    if (r < 0 || r >= p.T) {
      bad_index = true;
      r = r < 0 ? 0 : p.T - 1;
    }
    const int d0 = u * 8;
    const int h_begin = ch * kHeadsPerThread, h_end = min(Hall, h_begin + kHeadsPerThread);
    // the angle depends on (row, d) only: one evaluation serves every head of the chunk
    float sn[8], cs[8];
    if (h_begin < p.Hq + p.Hkv) {
      const float pos = (float)(p.pos_offset + r);  // exact below 2^24
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const float f_hi = tab.hi[d0 + k], f_lo = tab.lo[d0 + k];
        const float ang = pos * f_hi;
        const float rest_a = fmaf(pos, f_hi, -ang) + pos * f_lo;  // exact rounding error of the product + low part
        float s0, c0;
        sincosf(ang, &s0, &c0);
        sn[k] = fmaf(rest_a, c0, s0);
        cs[k] = fmaf(-rest_a, s0, c0);
      }
    }
#pragma unroll 4
    for (int hh = h_begin; hh < h_end; ++hh) {
      const __nv_bfloat16 *src;
      __nv_bfloat16 *dst, *cache = nullptr;
      bool rotate = true;
      if (hh < p.Hq) {
        src = reinterpret_cast<const __nv_bfloat16 *>(p.q_raw) + b * p.q_stride[0] + hh * p.q_stride[1] + (long long)r * p.q_stride[2];
        dst = reinterpret_cast<__nv_bfloat16 *>(p.q_out) + b * p.q_out_stride[0] + hh * p.q_out_stride[1] + (long long)i * p.q_out_stride[2];
      } else {
        const bool is_v = hh >= p.Hq + p.Hkv;
        const int h = hh - p.Hq - (is_v ? p.Hkv : 0);
        const void *raw = is_v ? p.v_raw : p.k_raw;
        void *out = is_v ? p.v_out : p.k_out;
        src = reinterpret_cast<const __nv_bfloat16 *>(raw) + b * p.kv_stride[0] + h * p.kv_stride[1] + (long long)r * p.kv_stride[2];
        dst = reinterpret_cast<__nv_bfloat16 *>(out) + b * p.kv_out_stride[0] + h * p.kv_out_stride[1] + (long long)i * p.kv_out_stride[2];
        rotate = !is_v;
        if (i < p.n_append) {
          void *c = is_v ? p.v_cache : p.k_cache;
          cache = reinterpret_cast<__nv_bfloat16 *>(c) + b * p.cache_stride[0] + h * p.cache_stride[1] +
                  (long long)(p.cache_row0 + i) * p.cache_stride[2];
        }
      }
      const uint4 lo = *reinterpret_cast<const uint4 *>(src + d0);
      const uint4 hi = *reinterpret_cast<const uint4 *>(src + half + d0);
      uint4 olo = lo, ohi = hi;
      if (rotate) {
        float a[8], c[8], x[8], y[8];
        unpack8(lo, a);
        unpack8(hi, c);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          x[k] = a[k] * cs[k] - c[k] * sn[k];
          y[k] = c[k] * cs[k] + a[k] * sn[k];
        }
        olo = pack8(x);
        ohi = pack8(y);
      }
      *reinterpret_cast<uint4 *>(dst + d0) = olo;
      *reinterpret_cast<uint4 *>(dst + half + d0) = ohi;
      if (cache) {
        *reinterpret_cast<uint4 *>(cache + d0) = olo;
        *reinterpret_cast<uint4 *>(cache + half + d0) = ohi;
      }
    }
  }
  if (bad_index && p.status) atomicOr(p.status, DS_DEV_INDEX);
}

}  // namespace

int launch_rope_gather(const ds_rope_params &p, cudaStream_t stream) {
  const int chunks = (p.Hq + 2 * p.Hkv + kHeadsPerThread - 1) / kHeadsPerThread;
  const long long total = (long long)p.B * p.Lq * chunks * (p.D / 16);
  if (total == 0) return DS_OK;
  if (p.D / 2 > kMaxHalf) return DS_ERR_UNSUPPORTED;
  long long blocks = (total + kRopeThreads - 1) / kRopeThreads;
  const long long cap = 16LL * sm_count();
  if (blocks > cap) blocks = cap;
  RopeTable tab;
  for (int d = 0; d < p.D / 2; ++d) {
    const double f = std::pow((double)p.rope_theta, -2.0 * d / (double)p.D);
    tab.hi[d] = (float)f;
    tab.lo[d] = (float)(f - (double)tab.hi[d]);
  }
  for (int d = p.D / 2; d < kMaxHalf; ++d) tab.hi[d] = tab.lo[d] = 0.f;
  rope_gather_kernel<<<(unsigned)blocks, kRopeThreads, 0, stream>>>(p, tab);
  DS_CUDA_OK(cudaGetLastError());
  note_launch(1);
  return DS_OK;
}

}  // namespace ds
