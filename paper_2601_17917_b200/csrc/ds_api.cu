// C ABI of the denoising-step library: argument validation and dispatch.
// Every step of the path runs in the CUDA kernels of the sibling files.
#include <atomic>
#include <new>

#include "ds_common.cuh"

namespace ds {

static std::atomic<long long> g_launches{0};
void note_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
thread_local int g_last_cuda_error = 0;
void note_cuda_error(int code) { g_last_cuda_error = code; }

int sm_count() {
  static int cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

namespace {

bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int validate_attn(const ds_attn_params *p) {
  if (!p) return DS_ERR_INVALID_ARG;
  if (p->dtype != DS_F32 && p->dtype != DS_BF16) return DS_ERR_INVALID_ARG;
  if (p->B < 0 || p->Hq <= 0 || p->Hkv <= 0 || p->D <= 0 || p->P < 0 || p->T <= 0) return DS_ERR_INVALID_ARG;
  if (p->Hq % p->Hkv != 0) return DS_ERR_INVALID_ARG;
  if (p->Lq < 1 || p->Lq > p->T) return DS_ERR_INVALID_ARG;
  if (!p->q_tail || !p->k_tail || !p->v_tail || !p->idx || !p->out) return DS_ERR_INVALID_ARG;
  if (p->P > 0 && (!p->k_prefix || !p->v_prefix)) return DS_ERR_INVALID_ARG;
  if (p->idx_batch_stride != 0 && p->idx_batch_stride < p->Lq) return DS_ERR_INVALID_ARG;
  if (!(p->scale == p->scale)) return DS_ERR_INVALID_ARG;
  if (p->seq_list && (p->n_seq < 0 || p->n_seq > p->B || !aligned(p->seq_list, 4) ||
                      (p->n_seq_dev && !aligned(p->n_seq_dev, 4))))
    return DS_ERR_INVALID_ARG;
  const int64_t unit = (p->dtype == DS_BF16) ? 8 : 4;  // 16 bytes
  const void *ptrs[] = {p->q_tail, p->k_tail, p->v_tail, p->out, p->P > 0 ? p->k_prefix : nullptr,
                        p->P > 0 ? p->v_prefix : nullptr};
  for (const void *q : ptrs)
    if (q && !aligned(q, 16)) return DS_ERR_INVALID_ARG;
  if (!aligned(p->idx, 4) || (p->lse && !aligned(p->lse, 4)) || (p->status && !aligned(p->status, 4)))
    return DS_ERR_INVALID_ARG;
  const int64_t *strides[] = {p->q_stride, p->kv_tail_stride, p->out_stride, p->kv_prefix_stride};
  for (int k = 0; k < 4; ++k) {
    if (k == 3 && p->P == 0) continue;
    for (int d = 0; d < 3; ++d) {
      const int64_t s = strides[k][d];
      if (s < 0 || s % unit != 0) return DS_ERR_INVALID_ARG;
    }
    if (strides[k][2] < p->D) return DS_ERR_INVALID_ARG;  // rows must not overlap
  }
  if (p->kernel != DS_ATTN_KERNEL_AUTO && p->kernel != DS_ATTN_KERNEL_ONE_TILE && p->kernel != DS_ATTN_KERNEL_TWO_TILE)
    return DS_ERR_INVALID_ARG;
  // The envelope: bf16 on the tensor cores, fp32 on the CUDA cores; nothing is rerouted.
  if (p->B > 65535 || p->Hq > 65535) return DS_ERR_UNSUPPORTED;
  if (p->dtype == DS_BF16) return attn_tc_supported(*p) ? DS_OK : DS_ERR_UNSUPPORTED;
  if (p->D != 32 && p->D != 64 && p->D != 128 && p->D != 256) return DS_ERR_UNSUPPORTED;
  if (!(p->scale > -1e30f && p->scale < 1e30f)) return DS_ERR_UNSUPPORTED;
  return DS_OK;
}

}  // namespace
}  // namespace ds

extern "C" {

size_t ds_attn_pruned_workspace(const ds_attn_params *p) {
  if (ds::validate_attn(p) != DS_OK) return 0;
  // only the one-tile kernel splits the keys of an item over CTAs
  if (p->dtype == DS_BF16 && p->kernel != DS_ATTN_KERNEL_TWO_TILE) return ds::attn_tc_workspace_bytes(*p);
  return 0;
}

namespace ds {
namespace {
// Several M-tiles per KV head (wide windows, the unpruned reference, a cache-refresh step): the two-tile
// kernel fetches every KV tile once for a pair of M-tiles and keeps the softmax warps busy on one tile while
// the tensor pipe works for the other.  Measured per work item it costs about 1.88 single tiles for a full pair
// and 1.10 for a pair with one tile (which alternates between the two S buffers like the one-tile kernel), so it
// pays when the number of rounds over the SMs does not grow.
bool two_tile_kernel_pays(const ds_attn_params &p) {
  const long long rows = (long long)(p.Hq / p.Hkv) * p.Lq;
  const long long n_full = rows / 128, rem = rows % 128;
  // the one-tile kernel serves a remainder of up to 8 rows together with the last full tile
  const long long n_mt1 = (p.D == 128 && n_full >= 1 && rem >= 1 && rem <= 8) ? n_full : n_full + (rem ? 1 : 0);
  const long long n_mt = n_full + (rem ? 1 : 0), n_pr = (n_mt + 1) / 2;
  if (n_mt < 2) return false;
  const long long heads = (long long)(p.seq_list ? p.n_seq : p.B) * p.Hkv, sms = sm_count();
  const double rounds1 = (double)((heads * n_mt1 + sms - 1) / sms);
  const double rounds2 = (double)((heads * n_pr + sms - 1) / sms);
  const double pair_cost = (1.88 * (double)(n_mt / 2) + 1.10 * (double)(n_mt % 2)) / (double)n_pr;
  return rounds2 * pair_cost < 0.97 * rounds1;
}

// Validation, choice of the kernel and its parameters for one set of arguments.
int resolve_attn(const ds_attn_params *p, AttnPrepared &a) {
  const int rc = validate_attn(p);
  if (rc != DS_OK) return rc;
  a.p = *p;
  a.grid = 0;
  a.path = kAttnPathSimt;
  if (p->B == 0) return DS_OK;
  if (p->dtype == DS_BF16) {
    if (p->kernel == DS_ATTN_KERNEL_TWO_TILE) return prepare_attn_tc2(*p, a);
    if (p->kernel == DS_ATTN_KERNEL_AUTO && two_tile_kernel_pays(*p)) return prepare_attn_tc2(*p, a);
    // a missing or short workspace is not an error: the call then runs without splitting the keys
    return prepare_attn_tc(*p, a);
  }
  a.grid = 1;  // the fp32 launcher sizes its own grid from a.p
  return DS_OK;
}

int launch_resolved(const AttnPrepared &a, cudaStream_t st) {
  if (a.p.B == 0) return DS_OK;
  switch (a.path) {
    case kAttnPathTc: return launch_prepared_tc(a, st);
    case kAttnPathTc2: return launch_prepared_tc2(a, st);
    default: return launch_attn_simt(a.p, st);
  }
}
}  // namespace
}  // namespace ds

struct ds_attn_plan {
  ds::AttnPrepared a;
};

int ds_attn_pruned(const ds_attn_params *p, void *stream) {
  ds::AttnPrepared a;
  const int rc = ds::resolve_attn(p, a);
  if (rc != DS_OK) return rc;
  return ds::launch_resolved(a, reinterpret_cast<cudaStream_t>(stream));
}

int ds_attn_plan_create(const ds_attn_params *p, ds_attn_plan **plan) {
  if (!plan) return DS_ERR_INVALID_ARG;
  *plan = nullptr;
  ds_attn_plan *pl = new (std::nothrow) ds_attn_plan;
  if (!pl) return DS_ERR_CUDA;
  const int rc = ds::resolve_attn(p, pl->a);
  if (rc != DS_OK) {
    delete pl;
    return rc;
  }
  *plan = pl;
  return DS_OK;
}

int ds_attn_plan_launch(const ds_attn_plan *plan, void *stream) {
  if (!plan) return DS_ERR_INVALID_ARG;
  return ds::launch_resolved(plan->a, reinterpret_cast<cudaStream_t>(stream));
}

void ds_attn_plan_destroy(ds_attn_plan *plan) { delete plan; }

size_t ds_confidence_workspace(int64_t rows, int64_t V, int32_t dtype) {
  if (dtype != DS_F32 && dtype != DS_BF16) return 0;
  return ds::confidence_workspace_bytes(rows, V, dtype);
}

int ds_confidence(const void *logits, int32_t dtype, int64_t rows, int64_t V, int64_t ld,
                  const int32_t *row_list, int64_t n_listed, float *conf, int32_t *tok, void *workspace,
                  size_t workspace_bytes, void *stream) {
  if (dtype != DS_F32 && dtype != DS_BF16) return DS_ERR_INVALID_ARG;
  if (rows < 0 || V <= 0 || ld < V || V > 0x7fffffffLL) return DS_ERR_INVALID_ARG;
  if (rows == 0) return DS_OK;
  if (!logits || !conf || !tok) return DS_ERR_INVALID_ARG;
  const size_t esz = dtype == DS_BF16 ? 2 : 4;
  if (!ds::aligned(logits, esz) || !ds::aligned(conf, 4) || !ds::aligned(tok, 4)) return DS_ERR_INVALID_ARG;
  if (row_list && (n_listed < 0 || n_listed > rows)) return DS_ERR_INVALID_ARG;
  return ds::launch_confidence(logits, dtype, rows, V, ld, row_list, n_listed, nullptr, conf, tok, workspace,
                               workspace_bytes, reinterpret_cast<cudaStream_t>(stream));
}

int ds_confidence_listed(const void *logits, int32_t dtype, int64_t rows, int64_t V, int64_t ld,
                         const int32_t *row_list, int64_t n_listed_max, const int32_t *n_listed_dev, float *conf,
                         int32_t *tok, void *workspace, size_t workspace_bytes, void *stream) {
  if (dtype != DS_F32 && dtype != DS_BF16) return DS_ERR_INVALID_ARG;
  if (rows < 0 || V <= 0 || ld < V || V > 0x7fffffffLL) return DS_ERR_INVALID_ARG;
  if (!row_list || !n_listed_dev || n_listed_max < 0 || n_listed_max > rows) return DS_ERR_INVALID_ARG;
  if (rows == 0 || n_listed_max == 0) return DS_OK;
  if (!logits || !conf || !tok) return DS_ERR_INVALID_ARG;
  const size_t esz = dtype == DS_BF16 ? 2 : 4;
  if (!ds::aligned(logits, esz) || !ds::aligned(conf, 4) || !ds::aligned(tok, 4) || !ds::aligned(n_listed_dev, 4))
    return DS_ERR_INVALID_ARG;
  return ds::launch_confidence(logits, dtype, rows, V, ld, row_list, n_listed_max, n_listed_dev, conf, tok, workspace,
                               workspace_bytes, reinterpret_cast<cudaStream_t>(stream));
}

int ds_rope_gather(const ds_rope_params *p, void *stream) {
  if (!p) return DS_ERR_INVALID_ARG;
  if (p->B < 0 || p->Hq <= 0 || p->Hkv <= 0 || p->D <= 0 || p->T <= 0 || p->Lq < 0 || p->Lq > p->T) return DS_ERR_INVALID_ARG;
  if (p->pos_offset < 0 || !(p->rope_theta > 1.0f) || p->n_append < 0 || p->n_append > p->Lq || p->cache_row0 < 0)
    return DS_ERR_INVALID_ARG;
  if (p->D % 16 != 0) return DS_ERR_UNSUPPORTED;
  if (p->B == 0 || p->Lq == 0) return DS_OK;
  if (!p->q_raw || !p->k_raw || !p->v_raw || !p->idx || !p->q_out || !p->k_out || !p->v_out) return DS_ERR_INVALID_ARG;
  if (p->n_append > 0 && (!p->k_cache || !p->v_cache)) return DS_ERR_INVALID_ARG;
  if (p->idx_batch_stride != 0 && p->idx_batch_stride < p->Lq) return DS_ERR_INVALID_ARG;
  const void *ptrs[] = {p->q_raw, p->k_raw, p->v_raw, p->q_out, p->k_out, p->v_out, p->n_append ? p->k_cache : nullptr,
                        p->n_append ? p->v_cache : nullptr};
  for (const void *q : ptrs)
    if (q && !ds::aligned(q, 16)) return DS_ERR_INVALID_ARG;
  const int64_t *strides[] = {p->q_stride, p->kv_stride, p->q_out_stride, p->kv_out_stride, p->cache_stride};
  for (int k = 0; k < 5; ++k) {
    if (k == 4 && p->n_append == 0) continue;
    for (int d = 0; d < 3; ++d)
      if (strides[k][d] < 0 || strides[k][d] % 8 != 0) return DS_ERR_INVALID_ARG;
    if (strides[k][2] < p->D) return DS_ERR_INVALID_ARG;
  }
  return ds::launch_rope_gather(*p, reinterpret_cast<cudaStream_t>(stream));
}

size_t ds_lmhead_confidence_workspace(int64_t rows, int64_t V) { return ds::lmhead_workspace_bytes(rows, V); }

int ds_lmhead_confidence(const void *hidden, const void *weight, int64_t rows, int64_t hid, int64_t V, int64_t ld_h,
                         int64_t ld_w, float *conf, int32_t *tok, void *workspace, size_t workspace_bytes,
                         uint32_t *status, void *stream) {
  if (rows < 0 || hid <= 0 || V <= 0 || ld_h < hid || ld_w < hid) return DS_ERR_INVALID_ARG;
  if (rows > 0x7fffffffLL || V > 0x7fffffffLL || hid > 0x7fffffffLL) return DS_ERR_INVALID_ARG;
  if (rows == 0) return DS_OK;
  if (!hidden || !weight || !conf || !tok) return DS_ERR_INVALID_ARG;
  if (!ds::aligned(hidden, 16) || !ds::aligned(weight, 16) || !ds::aligned(conf, 4) || !ds::aligned(tok, 4) ||
      (status && !ds::aligned(status, 4)))
    return DS_ERR_INVALID_ARG;
  if (hid % 8 != 0 || ld_h % 8 != 0 || ld_w % 8 != 0) return DS_ERR_INVALID_ARG;
  const size_t need = ds::lmhead_workspace_bytes(rows, V);
  if (!workspace || !ds::aligned(workspace, 256) || workspace_bytes < need) return DS_ERR_WORKSPACE;
  return ds::launch_lmhead_confidence(hidden, weight, rows, hid, V, ld_h, ld_w, conf, tok, workspace, status,
                                      reinterpret_cast<cudaStream_t>(stream));
}

int ds_confidence_static(const void *logits, int32_t dtype, int64_t rows, int64_t V, int64_t ld,
                         const int32_t *row_list, int64_t n_listed, float *conf, int32_t *tok, void *stream) {
  if (dtype != DS_F32 && dtype != DS_BF16) return DS_ERR_INVALID_ARG;
  if (rows < 0 || V <= 0 || ld < V || V > 0x7fffffffLL) return DS_ERR_INVALID_ARG;
  if (rows == 0) return DS_OK;
  if (!logits || !conf || !tok) return DS_ERR_INVALID_ARG;
  const size_t esz = dtype == DS_BF16 ? 2 : 4;
  if (!ds::aligned(logits, esz) || !ds::aligned(conf, 4) || !ds::aligned(tok, 4)) return DS_ERR_INVALID_ARG;
  if (row_list && (n_listed < 0 || n_listed > rows)) return DS_ERR_INVALID_ARG;
  return ds::launch_confidence_static(logits, dtype, rows, V, ld, row_list, n_listed, conf, tok,
                                      reinterpret_cast<cudaStream_t>(stream));
}

int ds_unmask_select(const ds_select_params *p, void *stream) {
  if (!p) return DS_ERR_INVALID_ARG;
  if (p->B < 0 || p->K < 1 || p->K > 4096 || p->ratio_extra < 0) return DS_ERR_INVALID_ARG;
  if (!(p->tau0 == p->tau0) || !(p->alpha == p->alpha) || !(p->eos_tau == p->eos_tau)) return DS_ERR_INVALID_ARG;
  if (!p->active_cnt) return DS_ERR_INVALID_ARG;
  if (p->B > 0 && (!p->conf || !p->tok || !p->masked || !p->x_block || !p->sel_idx || !p->sel_cnt ||
                   !p->block_done || !p->eos_exit || !p->active_seq))
    return DS_ERR_INVALID_ARG;
  if (p->seq_list && (p->n_seq < 0 || p->n_seq > p->B)) return DS_ERR_INVALID_ARG;
  if (!p->seq_list && p->n_seq_dev) return DS_ERR_INVALID_ARG;
  if (p->masked_rows && !p->masked_cnt) return DS_ERR_INVALID_ARG;
  if ((long long)p->B * p->K > 0x7fffffffLL) return DS_ERR_UNSUPPORTED;
  return ds::launch_select(*p, reinterpret_cast<cudaStream_t>(stream));
}

int ds_block_begin(const ds_block_params *p, void *stream) {
  if (!p) return DS_ERR_INVALID_ARG;
  if (p->B < 0 || p->K < 1 || p->K > 4096) return DS_ERR_INVALID_ARG;
  if (!p->active_cnt || (p->masked_rows == nullptr) != (p->masked_cnt == nullptr)) return DS_ERR_INVALID_ARG;
  if ((long long)p->B * p->K > 0x7fffffffLL) return DS_ERR_UNSUPPORTED;
  if (p->B > 0 && (!p->eos_exit || !p->masked || !p->x_block || !p->active_seq)) return DS_ERR_INVALID_ARG;
  return ds::launch_block_begin(*p, reinterpret_cast<cudaStream_t>(stream));
}

int ds_selftest_bounded_wait(uint32_t poll_limit, uint32_t *status, int32_t *report, void *stream) {
  if (poll_limit == 0 || poll_limit > (1u << 16)) return DS_ERR_INVALID_ARG;
  if ((status && !ds::aligned(status, 4)) || (report && !ds::aligned(report, 4))) return DS_ERR_INVALID_ARG;
  return ds::launch_bounded_wait_selftest(poll_limit, status, report, reinterpret_cast<cudaStream_t>(stream));
}

int ds_last_cuda_error(void) { return ds::g_last_cuda_error; }
const char *ds_last_cuda_error_name(void) {
  return cudaGetErrorName(static_cast<cudaError_t>(ds::g_last_cuda_error));
}

int ds_read_status(const uint32_t *device_status, void *stream, uint32_t *host_out) {
  if (!device_status || !host_out) return DS_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  DS_CUDA_OK(cudaMemcpyAsync(host_out, device_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
  DS_CUDA_OK(cudaStreamSynchronize(st));
  return DS_OK;
}

const char *ds_strerror(int code) {
  switch (code) {
    case DS_OK: return "ok";
    case DS_ERR_INVALID_ARG: return "invalid argument";
    case DS_ERR_UNSUPPORTED: return "shape or type outside the kernels' envelope";
    case DS_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case DS_ERR_CUDA: return "CUDA call failed";
    case DS_ERR_STATIC_LIMIT:
      return "request exceeds the fixed scratch of the allocation-free entry point (too many rows)";
    default: return "unknown status";
  }
}

int ds_version(void) { return 1000; }

int64_t ds_launch_count(void) { return ds::g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
