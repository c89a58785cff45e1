// ds_attn_pruned, CUDA-core path: fp32 inputs, head dimension 32, 64, 128 or 256.
//
// One warp owns one retained query row (Eq. 8: queries = current block U
// retained suffix).  The lanes split the head dimension; keys are visited
// prefix first, then the retained tail rows named by the index list (Eq. 7),
// four at a time, with an online softmax in fp32 (base-2 exponent, the softmax
// scale folded into the query).
#include "ds_common.cuh"

namespace ds {
namespace {

constexpr int kRowsPerCta = 8;

// A lane's slice of a row.  Rows are only promised 16-byte alignment (bases and strides), so a slice wider
// than that (fp32, D = 256: 32 bytes) is moved as 16-byte pieces.
template <typename T, int N>
struct alignas(sizeof(T) * N < 16 ? sizeof(T) * N : 16) Frag {
  T v[N];
};

template <typename T>
__device__ __forceinline__ float to_f32(T x);
template <>
__device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <typename T>
__device__ __forceinline__ T from_f32(float x);
template <>
__device__ __forceinline__ float from_f32<float>(float x) { return x; }

template <typename T, int DPL>
__device__ __forceinline__ void load_frag(const T *p, float (&out)[DPL]) {
  const Frag<T, DPL> f = *reinterpret_cast<const Frag<T, DPL> *>(p);
#pragma unroll
  for (int k = 0; k < DPL; ++k) out[k] = to_f32<T>(f.v[k]);
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

template <typename T, int DPL>
__global__ void __launch_bounds__(kRowsPerCta * 32) attn_simt_kernel(const ds_attn_params p) {
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.x * kRowsPerCta + (threadIdx.x >> 5);
  if (i >= p.Lq) return;
  const int hq = blockIdx.y;
  int b = blockIdx.z;
  bool bad_index = false;
  if (p.seq_list != nullptr) {  // blockIdx.z counts listed sequences
    int n = p.n_seq;
    if (p.n_seq_dev != nullptr) n = max(0, min(n, *p.n_seq_dev));
    if (b >= n) return;
    b = p.seq_list[b];
    if (b < 0 || b >= p.B) {
      bad_index = true;
      b = b < 0 ? 0 : p.B - 1;
    }
  }
  const int hk = hq / (p.Hq / p.Hkv);
  const int32_t *ix = p.idx + (long long)b * p.idx_batch_stride;
  const int dofs = lane * DPL;

  auto tail_row = [&](int j) {
    int r = ix[j];
    if (r < 0 || r >= p.T) {
      bad_index = true;
      r = r < 0 ? 0 : p.T - 1;
    }
    return r;
  };

  const T *Qt = reinterpret_cast<const T *>(p.q_tail) + b * p.q_stride[0] + hq * p.q_stride[1];
  const T *Kt = reinterpret_cast<const T *>(p.k_tail) + b * p.kv_tail_stride[0] + hk * p.kv_tail_stride[1];
  const T *Vt = reinterpret_cast<const T *>(p.v_tail) + b * p.kv_tail_stride[0] + hk * p.kv_tail_stride[1];
  const T *Kp = reinterpret_cast<const T *>(p.k_prefix) + b * p.kv_prefix_stride[0] + hk * p.kv_prefix_stride[1];
  const T *Vp = reinterpret_cast<const T *>(p.v_prefix) + b * p.kv_prefix_stride[0] + hk * p.kv_prefix_stride[1];

  float q[DPL];
  load_frag<T, DPL>(Qt + (long long)tail_row(i) * p.q_stride[2] + dofs, q);
  if (i > 0 && ix[i] <= ix[i - 1]) bad_index = true;  // the list must be strictly ascending (served as written)
  const float qs = p.scale * kLog2e;
#pragma unroll
  for (int k = 0; k < DPL; ++k) q[k] *= qs;

  float m = -INFINITY, l = 0.f;
  float o[DPL];
#pragma unroll
  for (int k = 0; k < DPL; ++k) o[k] = 0.f;

  const int Lkv = p.P + p.Lq;
  for (int j0 = 0; j0 < Lkv; j0 += 4) {
    float s[4];
    const T *vrow[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int j = j0 + u;
      s[u] = -INFINITY;
      vrow[u] = nullptr;
      if (j < Lkv) {
        const T *krow;
        if (j < p.P) {
          krow = Kp + (long long)j * p.kv_prefix_stride[2];
          vrow[u] = Vp + (long long)j * p.kv_prefix_stride[2];
        } else {
          const long long r = tail_row(j - p.P);
          krow = Kt + r * p.kv_tail_stride[2];
          vrow[u] = Vt + r * p.kv_tail_stride[2];
        }
        float kf[DPL];
        load_frag<T, DPL>(krow + dofs, kf);
        float acc = 0.f;
#pragma unroll
        for (int k = 0; k < DPL; ++k) acc = fmaf(q[k], kf[k], acc);
        s[u] = acc;
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (j0 + u < Lkv) s[u] = warp_sum(s[u]);
    const float m_new = fmaxf(fmaxf(m, fmaxf(s[0], s[1])), fmaxf(s[2], s[3]));
    const float a = ex2_approx(m - m_new);  // m = -inf at the start gives 0
    l *= a;
#pragma unroll
    for (int k = 0; k < DPL; ++k) o[k] *= a;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (j0 + u < Lkv) {
        const float pj = ex2_approx(s[u] - m_new);
        l += pj;
        float vf[DPL];
        load_frag<T, DPL>(vrow[u] + dofs, vf);
#pragma unroll
        for (int k = 0; k < DPL; ++k) o[k] = fmaf(pj, vf[k], o[k]);
      }
    }
    m = m_new;
  }

  const float inv = 1.f / l;
  Frag<T, DPL> f;
#pragma unroll
  for (int k = 0; k < DPL; ++k) f.v[k] = from_f32<T>(o[k] * inv);
  T *orow = reinterpret_cast<T *>(p.out) + b * p.out_stride[0] + hq * p.out_stride[1] +
            (long long)i * p.out_stride[2];
  *reinterpret_cast<Frag<T, DPL> *>(orow + dofs) = f;
  if (p.lse && lane == 0) p.lse[((long long)b * p.Hq + hq) * p.Lq + i] = (m + log2f(l)) * kLn2;
  if (bad_index && p.status && lane == 0) atomicOr(p.status, DS_DEV_INDEX);
}

template <typename T>
int launch_t(const ds_attn_params &p, cudaStream_t stream) {
  const int n_seq = p.seq_list ? p.n_seq : p.B;
  if (n_seq == 0) return DS_OK;
  const dim3 grid(ceil_div(p.Lq, kRowsPerCta), p.Hq, n_seq);
  const dim3 block(kRowsPerCta * 32);
  switch (p.D / 32) {
    case 1: attn_simt_kernel<T, 1><<<grid, block, 0, stream>>>(p); break;
    case 2: attn_simt_kernel<T, 2><<<grid, block, 0, stream>>>(p); break;
    case 4: attn_simt_kernel<T, 4><<<grid, block, 0, stream>>>(p); break;
    case 8: attn_simt_kernel<T, 8><<<grid, block, 0, stream>>>(p); break;
    default: return DS_ERR_UNSUPPORTED;
  }
  DS_CUDA_OK(cudaGetLastError());
  note_launch(1);
  return DS_OK;
}

}  // namespace

int launch_attn_simt(const ds_attn_params &p, cudaStream_t stream) {
  if (p.dtype != DS_F32) return DS_ERR_UNSUPPORTED;
  if (p.Hq > 65535 || p.B > 65535) return DS_ERR_UNSUPPORTED;
  return launch_t<float>(p, stream);
}

}  // namespace ds
