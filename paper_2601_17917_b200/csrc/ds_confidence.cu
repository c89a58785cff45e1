// ds_confidence: Eq. 4, c = max softmax(z) and x^ = argmax, one read of the logits.
//
// HBM-bound streaming reduction.  Every thread streams 16-byte vectors of its
// row (coalesced across the warp), keeping a running maximum m, the sum of
// exp(z - m) and the vector in which the maximum first appeared.  The sum is
// rescaled only when a vector raises the thread's maximum, which happens
// O(log n) times, so the steady state costs one FMA, one MUFU ex2 and one add
// per element.  The position of the maximum is recovered afterwards by
// re-reading that single vector.  (m, sum, index) triples are merged with
// warp shuffles, then across the block's warps through shared memory; equal
// maxima always resolve to the lowest index.  When there are too few rows to
// fill the GPU a row is split over several CTAs, each writing a partial triple
// to the workspace; the CTA that arrives last (atomic ticket) merges them.
#include <cfloat>
#include <climits>
#include <mutex>

#include "ds_common.cuh"

namespace ds {
namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;
constexpr int kMaxSplits = 64;

struct Triple {
  float m;  // maximum
  float s;  // sum of exp(z - m)
  int i;    // lowest index attaining m
  int pad;
};

__device__ __forceinline__ Triple merge(const Triple &a, const Triple &b) {
  Triple r;
  const bool a_wins = (a.m > b.m) || (a.m == b.m && a.i <= b.i);
  r.m = fmaxf(a.m, b.m);
  r.i = a_wins ? a.i : b.i;
  // exp(-inf - finite) = 0; both -inf: keep 0 (avoid inf - inf)
  const float ea = (a.m == r.m) ? 1.f : ex2_approx((a.m - r.m) * kLog2e);
  const float eb = (b.m == r.m) ? 1.f : ex2_approx((b.m - r.m) * kLog2e);
  r.s = a.s * ea + b.s * eb;
  r.pad = 0;
  return r;
}

__device__ __forceinline__ Triple shfl_xor(const Triple &t, int lane_mask) {
  Triple r;
  r.m = __shfl_xor_sync(0xffffffffu, t.m, lane_mask);
  r.s = __shfl_xor_sync(0xffffffffu, t.s, lane_mask);
  r.i = __shfl_xor_sync(0xffffffffu, t.i, lane_mask);
  r.pad = 0;
  return r;
}

template <typename T>
struct Vec;
template <>
struct Vec<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ float at(const uint4 &w, int j) {
    return __uint_as_float(j == 0 ? w.x : j == 1 ? w.y : j == 2 ? w.z : w.w);
  }
  static __device__ __forceinline__ float vmax(const uint4 &w) {
    return fmaxf(fmaxf(__uint_as_float(w.x), __uint_as_float(w.y)),
                 fmaxf(__uint_as_float(w.z), __uint_as_float(w.w)));
  }
  static __device__ __forceinline__ void expsum(const uint4 &w, float nml, float &s0, float &s1) {
    s0 += ex2_approx(fmaf(__uint_as_float(w.x), kLog2e, nml));
    s1 += ex2_approx(fmaf(__uint_as_float(w.y), kLog2e, nml));
    s0 += ex2_approx(fmaf(__uint_as_float(w.z), kLog2e, nml));
    s1 += ex2_approx(fmaf(__uint_as_float(w.w), kLog2e, nml));
  }
  static __device__ __forceinline__ float scalar(const float *p) { return *p; }
};
template <>
struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  static __device__ __forceinline__ float at(const uint4 &w, int j) {
    const uint32_t u = (j >> 1) == 0 ? w.x : (j >> 1) == 1 ? w.y : (j >> 1) == 2 ? w.z : w.w;
    return (j & 1) ? bf16hi_to_f32(u) : bf16lo_to_f32(u);
  }
  static __device__ __forceinline__ float vmax(const uint4 &w) {
    const __nv_bfloat162 a = __hmax2(*reinterpret_cast<const __nv_bfloat162 *>(&w.x),
                                     *reinterpret_cast<const __nv_bfloat162 *>(&w.y));
    const __nv_bfloat162 b = __hmax2(*reinterpret_cast<const __nv_bfloat162 *>(&w.z),
                                     *reinterpret_cast<const __nv_bfloat162 *>(&w.w));
    const __nv_bfloat162 c = __hmax2(a, b);
    const uint32_t u = *reinterpret_cast<const uint32_t *>(&c);
    return fmaxf(bf16lo_to_f32(u), bf16hi_to_f32(u));
  }
  static __device__ __forceinline__ void expsum(const uint4 &w, float nml, float &s0, float &s1) {
    s0 += ex2_approx(fmaf(bf16lo_to_f32(w.x), kLog2e, nml));
    s1 += ex2_approx(fmaf(bf16hi_to_f32(w.x), kLog2e, nml));
    s0 += ex2_approx(fmaf(bf16lo_to_f32(w.y), kLog2e, nml));
    s1 += ex2_approx(fmaf(bf16hi_to_f32(w.y), kLog2e, nml));
    s0 += ex2_approx(fmaf(bf16lo_to_f32(w.z), kLog2e, nml));
    s1 += ex2_approx(fmaf(bf16hi_to_f32(w.z), kLog2e, nml));
    s0 += ex2_approx(fmaf(bf16lo_to_f32(w.w), kLog2e, nml));
    s1 += ex2_approx(fmaf(bf16hi_to_f32(w.w), kLog2e, nml));
  }
  static __device__ __forceinline__ float scalar(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
};

// Running state of one thread.
struct Run {
  float m = -INFINITY;  // running maximum
  float nml = 0.f;      // -m * log2(e), 0 while m = -inf
  float s0 = 0.f, s1 = 0.f;
  long long bvec = -1;  // vector (row-body numbering) where m first appeared
};

template <typename T>
__device__ __forceinline__ void consume(const uint4 &w, long long v, Run &r) {
  const float vm = Vec<T>::vmax(w);
  if (vm > r.m) {  // rare after the first few vectors
    // Terms are 2^(z*log2e + nml); moving the offset multiplies the sum by 2^(nml_new - nml_old) exactly.
    const float nml_new = -vm * kLog2e;
    const float f = (r.m == -INFINITY) ? 0.f : ex2_approx(nml_new - r.nml);
    r.s0 *= f;
    r.s1 *= f;
    r.m = vm;
    r.nml = nml_new;
    r.bvec = v;
  }
  Vec<T>::expsum(w, r.nml, r.s0, r.s1);
}

__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
  uint4 w;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w)
               : "l"(p));
  return w;
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
confidence_kernel(const T *__restrict__ logits, long long V, long long ld,
                  const int32_t *__restrict__ row_list, int splits, float *__restrict__ conf,
                  int32_t *__restrict__ tok, Triple *__restrict__ partials,
                  unsigned *__restrict__ tickets, const int32_t *__restrict__ n_listed_dev, long long rows) {
  constexpr int N = Vec<T>::N;
  const int li = blockIdx.x / splits;  // position in the list of processed rows
  const int sp = blockIdx.x - li * splits;
  if (n_listed_dev != nullptr && li >= *n_listed_dev) return;  // the list is shorter than the launch was sized for
  const long long row = row_list ? (long long)row_list[li] : (long long)li;
  if (row < 0 || row >= rows) return;  // every CTA of the row leaves: no ticket of it is ever awaited
  const T *z = logits + row * ld;
  const int tid = threadIdx.x;

  // Row = [head scalars][16-byte aligned body of vectors][tail scalars].
  const uintptr_t addr = reinterpret_cast<uintptr_t>(z);
  long long head = (long long)(((16 - (addr & 15)) & 15) / sizeof(T));
  if (head > V) head = V;
  const long long nvec = (V - head) / N;
  const long long tail0 = head + nvec * N;  // first tail scalar
  const uint4 *body = reinterpret_cast<const uint4 *>(z + head);

  // this CTA's share of the body
  const long long per = (nvec + splits - 1) / splits;
  const long long vs = per * sp;
  const long long ve = (vs + per < nvec) ? vs + per : nvec;

  Run r;
  long long v = vs + tid;
  for (; v + (long long)(kUnroll - 1) * kThreads < ve; v += (long long)kUnroll * kThreads) {
    uint4 w[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) w[u] = ld_stream(body + v + (long long)u * kThreads);
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) consume<T>(w[u], v + (long long)u * kThreads, r);
  }
  for (; v < ve; v += kThreads) {
    const uint4 w = ld_stream(body + v);
    consume<T>(w, v, r);
  }

  // Resolve the position of this thread's maximum: re-read its vector.
  Triple t;
  t.m = r.m;
  // nml is -m*log2e rounded to fp32; the FMA in the loop is exact up to its own rounding, so the
  // whole sum is off by the single factor 2^(nml + m*log2e), removed here (matters for large |m|).
  t.s = (r.m == -INFINITY) ? 0.f : (r.s0 + r.s1) * ex2_approx(fmaf(-r.m, kLog2e, -r.nml));
  t.i = INT_MAX;
  t.pad = 0;
  if (r.bvec >= 0) {
    const uint4 w = body[r.bvec];
    int j = 0;
#pragma unroll
    for (int k = N - 1; k >= 0; --k)
      if (Vec<T>::at(w, k) == r.m) j = k;
    t.i = (int)(head + r.bvec * N + j);
  }
  // Head scalars belong to split 0, tail scalars to the last split.
  if (sp == 0 && tid < head) {
    Triple e = {Vec<T>::scalar(z + tid), 1.f, tid, 0};
    t = merge(t, e);
  }
  if (sp == splits - 1 && tail0 + tid < V) {
    Triple e = {Vec<T>::scalar(z + tail0 + tid), 1.f, (int)(tail0 + tid), 0};
    t = merge(t, e);
  }

#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t = merge(t, shfl_xor(t, o));
  __shared__ Triple warp_t[kThreads / 32];
  __shared__ bool is_last;
  if ((tid & 31) == 0) warp_t[tid >> 5] = t;
  __syncthreads();
  if (tid < 32) {
    Triple u = (tid < kThreads / 32) ? warp_t[tid] : Triple{-INFINITY, 0.f, INT_MAX, 0};
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) u = merge(u, shfl_xor(u, o));
    if (tid == 0) {
      if (splits == 1) {
        conf[row] = 1.f / u.s;
        tok[row] = u.i;
      } else {
        partials[(long long)li * splits + sp] = u;
        __threadfence();
        const unsigned old = atomicAdd(&tickets[li], 1u);
        is_last = (old == (unsigned)(splits - 1));
      }
    }
  }
  if (splits == 1) return;
  __syncthreads();
  if (!is_last) return;
  if (tid < 32) {
    __threadfence();
    Triple u{-INFINITY, 0.f, INT_MAX, 0};
    for (int k = tid; k < splits; k += 32) {
      const int4 raw = __ldcg(reinterpret_cast<const int4 *>(&partials[(long long)li * splits + k]));
      const Triple p = {__int_as_float(raw.x), __int_as_float(raw.y), raw.z, 0};
      u = merge(u, p);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) u = merge(u, shfl_xor(u, o));
    if (tid == 0) {
      conf[row] = 1.f / u.s;
      tok[row] = u.i;
      tickets[li] = 0u;
    }
  }
}

inline int pick_splits(int64_t n_rows, int64_t V, int dtype) {
  const int n = (dtype == DS_BF16) ? 8 : 4;
  const int64_t nvec = V / n;
  // enough CTAs for ~4 per SM, but at least 2 vectors per thread per CTA
  int64_t want = (4LL * sm_count() + n_rows - 1) / (n_rows > 0 ? n_rows : 1);
  int64_t cap = nvec / (2 * kThreads);
  if (want > cap) want = cap;
  if (want > kMaxSplits) want = kMaxSplits;
  if (want < 1) want = 1;
  return (int)want;
}

// Fixed scratch of ds_confidence_static: one ticket per processed row, then the partial triples.
// It lives in every device that loads the library, for the life of the process.
constexpr int kStaticRows = DS_CONFIDENCE_STATIC_MAX_ROWS;
constexpr int kStaticPartials = 2 * kStaticRows;
constexpr size_t kStaticTicketBytes = (size_t)kStaticRows * sizeof(unsigned);
constexpr size_t kStaticBytes = kStaticTicketBytes + (size_t)kStaticPartials * sizeof(Triple);
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void *g_static_ptr[kMaxDevices];  // device address of g_static_scratch, per device; null until set up

// Device address of the scratch array on the current device.  In host code the array's name is only
// a handle, so the address a kernel can use has to be asked for, once per device, with that
// device current.
int static_scratch(void **out) {
  int dev = -1;
  DS_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return DS_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (!g_static_ptr[dev]) {
    void *ptr = nullptr;
    DS_CUDA_OK(cudaGetSymbolAddress(&ptr, g_static_scratch));
    if (!ptr) return DS_ERR_CUDA;
    g_static_ptr[dev] = ptr;
  }
  *out = g_static_ptr[dev];
  return DS_OK;
}

}  // namespace

int launch_confidence_static(const void *logits, int dtype, int64_t rows, int64_t V, int64_t ld,
                             const int32_t *row_list, int64_t n_listed, float *conf, int32_t *tok,
                             cudaStream_t stream) {
  const int32_t *n_listed_dev = nullptr;
  const int64_t n = row_list ? n_listed : rows;
  if (n == 0) return DS_OK;
  if (n > kStaticRows) return DS_ERR_STATIC_LIMIT;
  const int splits = pick_splits(n, V, dtype);
  // pick_splits keeps n * splits below 4 * SMs + n, far under the 2 * MAX_ROWS partial results the array holds
  // for any n it accepts; the check only guards that arithmetic
  if (n * splits > kStaticPartials) return DS_ERR_STATIC_LIMIT;
  void *base = nullptr;
  const int rc = static_scratch(&base);
  if (rc != DS_OK) return rc;
  unsigned *tickets = reinterpret_cast<unsigned *>(base);
  Triple *partials = reinterpret_cast<Triple *>(reinterpret_cast<unsigned char *>(base) + kStaticTicketBytes);
  // the array keeps whatever the previous call left: the tickets must start at zero
  if (splits > 1) DS_CUDA_OK(cudaMemsetAsync(tickets, 0, (size_t)n * sizeof(unsigned), stream));
  const dim3 grid((unsigned)(n * splits));
  if (dtype == DS_BF16) {
    confidence_kernel<__nv_bfloat16><<<grid, kThreads, 0, stream>>>(
        reinterpret_cast<const __nv_bfloat16 *>(logits), V, ld, row_list, splits, conf, tok, partials, tickets, n_listed_dev, rows);
  } else {
    confidence_kernel<float><<<grid, kThreads, 0, stream>>>(reinterpret_cast<const float *>(logits), V, ld,
                                                           row_list, splits, conf, tok, partials, tickets, n_listed_dev, rows);
  }
  DS_CUDA_OK(cudaGetLastError());
  note_launch(1);
  return DS_OK;
}

size_t confidence_workspace_bytes(int64_t rows, int64_t V, int dtype) {
  if (rows <= 0 || V <= 0) return 0;
  // sized for the largest split count any row subset could need
  const size_t tickets = ((size_t)rows * sizeof(unsigned) + 255) / 256 * 256;
  return tickets + (size_t)rows * kMaxSplits * sizeof(Triple);
}

int launch_confidence(const void *logits, int dtype, int64_t rows, int64_t V, int64_t ld,
                      const int32_t *row_list, int64_t n_listed, const int32_t *n_listed_dev, float *conf,
                      int32_t *tok, void *workspace, size_t workspace_bytes, cudaStream_t stream) {
  const int64_t n = row_list ? n_listed : rows;
  if (n == 0) return DS_OK;
  const int splits = pick_splits(n, V, dtype);
  unsigned *tickets = nullptr;
  Triple *partials = nullptr;
  if (splits > 1) {
    const size_t tk = ((size_t)rows * sizeof(unsigned) + 255) / 256 * 256;
    const size_t need = tk + (size_t)n * splits * sizeof(Triple);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < need)
      return DS_ERR_WORKSPACE;
    tickets = reinterpret_cast<unsigned *>(workspace);
    partials = reinterpret_cast<Triple *>(reinterpret_cast<char *>(workspace) + tk);
    DS_CUDA_OK(cudaMemsetAsync(tickets, 0, (size_t)n * sizeof(unsigned), stream));
  }
  if (n * splits > 0x7fffffffLL) return DS_ERR_UNSUPPORTED;
  const dim3 grid((unsigned)(n * splits));
  if (dtype == DS_BF16) {
    confidence_kernel<__nv_bfloat16><<<grid, kThreads, 0, stream>>>(
        reinterpret_cast<const __nv_bfloat16 *>(logits), V, ld, row_list, splits, conf, tok, partials, tickets, n_listed_dev, rows);
  } else {
    confidence_kernel<float><<<grid, kThreads, 0, stream>>>(reinterpret_cast<const float *>(logits), V, ld,
                                                           row_list, splits, conf, tok, partials, tickets, n_listed_dev, rows);
  }
  DS_CUDA_OK(cudaGetLastError());
  note_launch(1);
  return DS_OK;
}

}  // namespace ds
