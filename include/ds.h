/*
 * ds.h -- C ABI of the B200 (sm_100a) suffix-pruned denoising step.
 *
 * One step of block-diffusion decoding with attenuation-guided suffix pruning
 * and dynamic confidence-aware unmasking has three device stages:
 *
 *   ds_attn_pruned    bidirectional attention of {current block U retained
 *                     suffix rows} over {cached prefix KV ; the same retained
 *                     rows}  (Method, Eq. 7 and Eq. 8, and the query/key
 *                     construction of "Dynamic Confidence Aware Parallel
 *                     Decoding")
 *   ds_confidence     c = max softmax(z), x^ = argmax softmax(z) per logit row
 *                     (Preliminary, Eq. 4)
 *   ds_unmask_select  adaptive threshold (Eq. 10), selection rule (Eq. 9),
 *                     state update (Eq. 5), block-finished test and the
 *                     early-exit flag ("Early Exit For Block Diffusion")
 *
 * Conventions
 *   - Every function returns a ds_status.  Nothing throws, traps or aborts.
 *   - Unless a parameter is marked HOST, pointers are DEVICE pointers on the
 *     current CUDA device.  The caller owns every buffer; the library never
 *     allocates or frees device memory and never synchronises a stream (except
 *     ds_read_status, which says so).  Work is enqueued on `stream`
 *     (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *   - Shapes outside a kernel's envelope return DS_ERR_UNSUPPORTED; there is
 *     no CPU fallback.
 *   - Conditions only the device can see (a retained-row index out of range, a
 *     bounded on-chip wait that ran out) are OR-ed into the optional device
 *     word `status` as DS_DEV_* bits; the kernel still terminates normally.
 *   - Calls on distinct streams may run concurrently provided they do not
 *     share a workspace.
 */
#ifndef DS_H_
#define DS_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define DS_API __attribute__((visibility("default")))
#else
#define DS_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DS_OK = 0,
  DS_ERR_INVALID_ARG = 1, /* null pointer, negative size, inconsistent shape, misaligned pointer/stride */
  DS_ERR_UNSUPPORTED = 2, /* well-formed request outside the kernels' envelope */
  DS_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or smaller than the *_workspace() query */
  DS_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed (launch, tensor-map encode, ...) */
  DS_ERR_STATIC_LIMIT = 5 /* ds_confidence_static only: more rows than its fixed scratch can serve */
} ds_status;

/* bits OR-ed into the optional device status word */
#define DS_DEV_INDEX 1u   /* an entry of idx (or of a sequence list) was out of range and was clamped, or idx was not
                             strictly ascending (its rows are then fetched one by one, in the order given) */
#define DS_DEV_TIMEOUT 2u /* a bounded mbarrier wait expired; outputs of that CTA are invalid */

typedef enum { DS_F32 = 0, DS_BF16 = 1 } ds_dtype;

/* bf16 attention kernels: one 128-row query tile per work item (KV-stream bound shapes), or a pair of query
 * tiles sharing every KV tile (several tiles per KV head: wide windows, GQA groups, a cache-refresh step). */
typedef enum { DS_ATTN_KERNEL_AUTO = 0, DS_ATTN_KERNEL_ONE_TILE = 1, DS_ATTN_KERNEL_TWO_TILE = 2 } ds_attn_kernel;

/* ------------------------------------------------------------------------
 * ds_attn_pruned  (Eq. 7, Eq. 8; "Dynamic Confidence Aware Parallel Decoding")
 *
 * The sequence at a denoising step is [prefix ; current block ; suffix]
 * (Method, region split).  The "tail" is block + suffix, T rows.  The retained
 * set of Eq. 7 arrives as `idx`: Lq tail-relative row numbers, strictly
 * ascending (block rows first, then the window, then the trailing position).
 * The kernels rely on the order to fetch runs of consecutive rows as one
 * box: they check it, and a list that is not strictly ascending raises
 * DS_DEV_INDEX and is served row by row exactly as written.
 * For every batch b and query head h, with KV head g = h / (Hq / Hkv):
 *
 *     Q~ = q_tail[b, h, idx[:], :]                          (Lq x D)
 *     K~ = [ k_prefix[b, g, 0:P, :] ; k_tail[b, g, idx[:], :] ]   ((P + Lq) x D)
 *     V~ likewise
 *     out[b, h, i, :] = sum_j softmax_j(scale * <Q~_i, K~_j>) V~_j
 *
 * There is no mask: the model is bidirectional.  Rotary position encoding is
 * applied by the caller (pruned rows keep their original position ids).
 * Accumulation is fp32; `out` has the input element type.  `lse`, when not
 * NULL, receives log(sum_j exp(scale * <Q~_i, K~_j>)) (natural log, fp32).
 *
 * Layout: element strides (not bytes) for the batch, head and row dimensions;
 * the D dimension is contiguous.  Every base pointer must be 16-byte aligned
 * and every stride a multiple of 16 bytes (8 bf16 / 4 fp32 elements).  P may be 0 (the
 * prefix pointers are then ignored).  idx is either one list shared by all
 * batches (idx_batch_stride = 0) or one per batch.
 *
 * Envelope: DS_BF16 runs on the tensor cores and takes D in {64, 128} and
 * scale > 0; DS_F32 runs on the CUDA cores and takes D in {32, 64, 128, 256}
 * and any finite scale.  Hq % Hkv == 0.  1 <= Lq <= T.  B, Hq <= 65535.
 * Anything else that is well formed returns DS_ERR_UNSUPPORTED: no request is
 * rerouted to another kernel behind the caller's back.
 *
 * Workspace: ds_attn_pruned_workspace(p) bytes, 256-byte aligned; contents need
 * not be preserved between calls.  It is used when the call has few work
 * items (small batches with a long prefix): the keys of every item are then
 * split over several CTAs, which leave normalised partial results and their
 * log-sum-exp in the workspace, and a second kernel merges them.  A call
 * without a (large enough) workspace is not an error; it runs unsplit.
 * Errors: DS_ERR_INVALID_ARG / DS_ERR_UNSUPPORTED before anything is
 * launched; DS_ERR_CUDA if a tensor-map encoding or a launch fails
 * (ds_last_cuda_error tells which runtime error; for a refused encoding it
 * reports cudaErrorInvalidValue).
 * ------------------------------------------------------------------------ */
typedef struct {
  int32_t B, Hq, Hkv, D;
  int32_t P;  /* cached prefix length (prompt + decoded blocks), >= 0 */
  int32_t T;  /* rows in the tail buffers */
  int32_t Lq; /* retained rows: K + R */
  int32_t dtype; /* ds_dtype of q/k/v/out */
  const void *q_tail;                /* [B][Hq ][T][D] */
  const void *k_tail, *v_tail;       /* [B][Hkv][T][D] */
  const void *k_prefix, *v_prefix;   /* [B][Hkv][P][D] */
  int64_t q_stride[3];               /* batch, head, row (elements) */
  int64_t kv_tail_stride[3];
  int64_t kv_prefix_stride[3];
  int64_t out_stride[3];
  const int32_t *idx;                /* [Lq] or [B][Lq] */
  int64_t idx_batch_stride;          /* 0 or >= Lq */
  float scale;                       /* softmax scale, 1/sqrt(D) for the standard definition */
  void *out;                         /* [B][Hq][Lq][D] */
  float *lse;                        /* optional [B][Hq][Lq], dense */
  void *workspace;
  size_t workspace_bytes;
  uint32_t *status;                  /* optional device word, DS_DEV_* bits are OR-ed in */
  /* Optional restriction to some sequences (e.g. ds_unmask_select's active_seq: the sequences whose block
   * still has masked positions).  seq_list = n_seq ascending batch numbers in [0, B); NULL = all B (n_seq and
   * n_seq_dev are then ignored).  n_seq_dev, when not NULL, is a device scalar read by the kernel that
   * overrides n_seq as the count (clamped to [0, n_seq]; n_seq then only sizes the launch), so that a loop
   * over steps needs no host synchronisation.  Outputs of sequences not listed are left untouched; a listed
   * number outside [0, B) sets DS_DEV_INDEX and is clamped. */
  const int32_t *seq_list;
  int32_t n_seq;
  const int32_t *n_seq_dev;
  /* Which bf16 kernel serves the call (ds_attn_kernel).  DS_ATTN_KERNEL_AUTO lets the library choose by
   * shape; the other two values pin the choice (a caller that has timed both on its shapes, a test that
   * wants each kernel on the same inputs).  Ignored for DS_F32.  Any other value: DS_ERR_INVALID_ARG. */
  int32_t kernel;
} ds_attn_params;

/* HOST, pure: bytes of workspace ds_attn_pruned needs for *p (0 when none). */
DS_API size_t ds_attn_pruned_workspace(const ds_attn_params *p);
/* `p` is a HOST pointer; the pointers inside it are device pointers. */
DS_API int ds_attn_pruned(const ds_attn_params *p, void *stream);

/* The same call split in two for loops that repeat it: within a block every iteration runs the attention of
 * a layer on the same buffers, with the same retained rows (Eq. 7 depends on the block, not on the
 * iteration), and only the device-resident sequence list changes.  ds_attn_plan_create validates *p, chooses
 * the kernel and works out its parameters (tensor-map encodings included) once; ds_attn_plan_launch enqueues
 * that kernel on `stream` and does nothing else, so its host cost is that of one kernel launch.  The plan
 * (HOST memory, owned by the caller until ds_attn_plan_destroy) keeps the pointers of *p, not the memory
 * behind them: every buffer must stay valid and in place while the plan is used; what the buffers, the
 * index list, the sequence list and *n_seq_dev contain is read at each launch.  Launches of one plan may be
 * captured into a CUDA graph.  A plan belongs to the device that was current when it was created.
 * Errors of create: those of ds_attn_pruned; *plan is NULL on failure.  Destroying NULL is allowed. */
typedef struct ds_attn_plan ds_attn_plan;
DS_API int ds_attn_plan_create(const ds_attn_params *p, ds_attn_plan **plan);
DS_API int ds_attn_plan_launch(const ds_attn_plan *plan, void *stream);
DS_API void ds_attn_plan_destroy(ds_attn_plan *plan);

/* ------------------------------------------------------------------------
 * ds_confidence  (Eq. 4)
 *
 * For every selected row r of logits[rows][V] (row stride ld >= V elements):
 *     m       = max_j z_rj
 *     tok[r]  = lowest j with z_rj == m
 *     conf[r] = 1 / sum_j exp(z_rj - m)          (= max_j softmax(z_r)_j)
 * computed in fp32 from one read of the row.  `row_list` (n_listed ascending
 * row numbers) restricts the pass to those rows, e.g. the still-masked
 * positions; NULL means all rows.  conf/tok are indexed by row number; rows
 * not listed are left untouched.
 *
 * Workspace: ds_confidence_workspace(rows, V, dtype) bytes, 256-byte aligned;
 * used when a row is split over several CTAs (few rows, large V).  The
 * library clears the part it needs on `stream` before the kernel runs.
 * ------------------------------------------------------------------------ */
DS_API size_t ds_confidence_workspace(int64_t rows, int64_t V, int32_t dtype);
DS_API int ds_confidence(const void *logits, int32_t dtype, int64_t rows, int64_t V, int64_t ld,
                  const int32_t *row_list, int64_t n_listed, float *conf, int32_t *tok,
                  void *workspace, size_t workspace_bytes, void *stream);
/* The same with the length of row_list held on the device: `n_listed_dev` (device scalar, not NULL) is read
 * by the kernel and clamped to [0, n_listed_max]; n_listed_max sizes the launch; the workspace is that of
 * ds_confidence (ds_confidence_workspace(rows, V, dtype)).  A listed row outside [0, rows) is skipped.  Meant for ds_unmask_select's masked_rows /
 * masked_cnt: Eq. 4 is only needed at the positions that are still masked, and the count changes every step. */
DS_API int ds_confidence_listed(const void *logits, int32_t dtype, int64_t rows, int64_t V, int64_t ld,
                         const int32_t *row_list, int64_t n_listed_max, const int32_t *n_listed_dev,
                         float *conf, int32_t *tok, void *workspace, size_t workspace_bytes, void *stream);

/* ------------------------------------------------------------------------
 * ds_rope_gather  (Eq. 7 position ids, Eq. 8 pruned input, prefix-cache append)
 *
 * Pruned tokens keep their place in the sequence through their rotary
 * position ids (Eq. 7 and the text around it): a retained row is rotated with
 * the position it has in the full sequence, not with its rank in the list.  This
 * entry point takes the un-rotated projections of the whole tail and produces
 * what ds_attn_pruned consumes, compact and rotated.  For every batch b and
 * retained row i (tail row r = idx[i], absolute position pos = pos_offset + r):
 *     q_out[b][h][i] = rope(q_raw[b][h][r], pos)      (all Hq heads)
 *     k_out[b][g][i] = rope(k_raw[b][g][r], pos)      (all Hkv heads)
 *     v_out[b][g][i] = v_raw[b][g][r]
 * rope pairs dimension d with d + D/2 ("rotate half"):
 *     out[d]       = x[d] cos(a_d) - x[d + D/2] sin(a_d)
 *     out[d + D/2] = x[d + D/2] cos(a_d) + x[d] sin(a_d),   a_d = pos * rope_theta^(-2d/D)
 * ds_attn_pruned is then called on the compact buffers with T = Lq and
 * idx = 0 .. Lq-1.  When n_append > 0 the first n_append retained rows (the
 * current block, once it is finished) are also written to the prefix cache at
 * rows cache_row0 .. cache_row0 + n_append - 1 (rotated K, plain V).
 *
 * All tensors bf16, D contiguous, D a multiple of 16, element strides for
 * batch / head / row, bases and strides 16-byte aligned.  Out-of-range idx
 * entries are clamped and flagged (DS_DEV_INDEX) like in ds_attn_pruned.
 * ------------------------------------------------------------------------ */
typedef struct {
  int32_t B, Hq, Hkv, D;
  int32_t T;                          /* rows of the raw tail buffers */
  int32_t Lq;                         /* retained rows */
  const void *q_raw;                  /* [B][Hq ][T][D] */
  const void *k_raw, *v_raw;          /* [B][Hkv][T][D] */
  int64_t q_stride[3], kv_stride[3];
  const int32_t *idx;                 /* [Lq] or [B][Lq] */
  int64_t idx_batch_stride;
  int32_t pos_offset;                 /* absolute position of tail row 0 (= prefix length) */
  float rope_theta;                   /* frequency base, > 1 */
  void *q_out;                        /* [B][Hq ][Lq][D] */
  void *k_out, *v_out;                /* [B][Hkv][Lq][D] */
  int64_t q_out_stride[3], kv_out_stride[3];
  void *k_cache, *v_cache;            /* optional [B][Hkv][rows][D]; needed when n_append > 0 */
  int64_t cache_stride[3];
  int32_t cache_row0, n_append;
  uint32_t *status;                   /* optional device word */
} ds_rope_params;

/* `p` is a HOST pointer; the pointers inside it are device pointers. */
DS_API int ds_rope_gather(const ds_rope_params *p, void *stream);

/* ------------------------------------------------------------------------
 * ds_lmhead_confidence  (output projection + Eq. 4, fused)
 *
 * After the attention, the rest of the model turns the hidden states into the
 * prediction logits (Method, "Dynamic Confidence Aware Parallel Decoding"); the
 * last of those components is the output projection z_r = W h_r.  This entry
 * point computes, for every row r,
 *     z_rj    = sum_k hidden[r][k] * weight[j][k]          (j < V, fp32 accumulation)
 *     tok[r]  = lowest j with z_rj == max_j z_rj
 *     conf[r] = 1 / sum_j exp(z_rj - max_j z_rj)            (Eq. 4)
 * without ever writing the [rows x V] logits: they stay on chip as fp32
 * accumulators (so, unlike ds_confidence on stored bf16 logits, they are not
 * rounded to bf16 either).
 *
 * hidden [rows][ld_h] and weight [V][ld_w] are bf16, row-major, hid elements
 * used per row; bases 16-byte aligned, ld_h, ld_w and hid multiples of 8.
 * Workspace: ds_lmhead_confidence_workspace(rows, V) bytes, 256-byte aligned
 * (one 16-byte partial result per row and per 256-token tile of the vocabulary).
 * `status` (optional device word) receives DS_DEV_TIMEOUT if a bounded on-chip
 * wait expires.  Errors: DS_ERR_INVALID_ARG, DS_ERR_WORKSPACE, DS_ERR_CUDA.
 * ------------------------------------------------------------------------ */
DS_API size_t ds_lmhead_confidence_workspace(int64_t rows, int64_t V);
DS_API int ds_lmhead_confidence(const void *hidden, const void *weight, int64_t rows, int64_t hid, int64_t V,
                         int64_t ld_h, int64_t ld_w, float *conf, int32_t *tok, void *workspace,
                         size_t workspace_bytes, uint32_t *status, void *stream);

/* ------------------------------------------------------------------------
 * ds_confidence_static  (no counterpart in the paper: a packaging variant)
 *
 * The same computation and the same kernel as ds_confidence, for callers that
 * have no way to hand over a workspace because they may not allocate device
 * memory at the point of the call: code running inside another framework's
 * memory plan, a plugin whose host forbids cudaMalloc after start-up, a
 * real-time loop that must not touch the allocator.  The scratch the split-row
 * reduction needs (one ticket per processed row plus the partial results)
 * lives instead in a fixed array inside the library's device image:
 * 4 * MAX_ROWS + 32 * MAX_ROWS bytes = 144 KiB, held by every GPU that loads
 * the library until the process exits.
 *
 * Arguments as for ds_confidence, minus the workspace.  This function and
 * everything it calls allocate and free nothing, on the host or the device.
 *
 * Limits and errors: at most DS_CONFIDENCE_STATIC_MAX_ROWS processed rows
 * (`rows`, or `n_listed` with a row list); more returns DS_ERR_STATIC_LIMIT
 * and launches nothing.  The other argument errors are those of
 * ds_confidence.
 *
 * First call on a device: it looks up the device address of the scratch array
 * (a CUDA runtime query, remembered per device; the device that is current at
 * the call is the one set up).  Make that first call outside any stream
 * capture.  The remembered address belongs to the device's current context:
 * after cudaDeviceReset it is stale, and the process must not call this entry
 * point on that device again.
 *
 * Sharing: every call on a device uses the same array, and the array keeps
 * the previous call's contents; the function clears the tickets it is about
 * to use on `stream` before the kernel.  Two calls that can overlap on the GPU
 * (different streams without an ordering between them) race on the array and
 * give wrong results: order them, or use ds_confidence with separate
 * workspaces.
 * ------------------------------------------------------------------------ */
#define DS_CONFIDENCE_STATIC_MAX_ROWS 4096
DS_API int ds_confidence_static(const void *logits, int32_t dtype, int64_t rows, int64_t V, int64_t ld,
                         const int32_t *row_list, int64_t n_listed, float *conf, int32_t *tok,
                         void *stream);

/* ------------------------------------------------------------------------
 * ds_unmask_select  (Eq. 9, Eq. 10, Eq. 5, block termination, early exit)
 *
 * Per processed sequence b, with n = number of masked positions of its block
 * BEFORE this step:
 *     r_mask = (n + ratio_extra) / (K + ratio_extra)
 *     tau    = tau0 * (1 - alpha * (1 - r_mask))           (fp32, one rounding per op)
 *     accept = { i : masked[b][i] and conf[b][i] >= tau }
 *     if accept is empty and n > 0: accept = { lowest i among masked with maximal conf }
 *     for i in accept: x_block[b][i] = tok[b][i]; masked[b][i] = 0
 *     sel_idx[b][0:sel_cnt[b]] = accept ascending, remaining entries -1
 *     block_done[b] = 1 when no masked position is left, else 0
 *     eos_exit[b]  |= 1 when an accepted token equals eos_id with conf >= eos_tau
 *     active_seq    = ascending list of processed sequences with block_done == 0,
 *                     *active_cnt its length
 *     masked_rows   = (optional) ascending list of b * K + i over the processed sequences b and the positions i
 *                     that are still masked after the step, *masked_cnt its length: the rows of a
 *                     [B * K][V] logit matrix the next step needs Eq. 4 for
 * ratio_extra = 0 counts the block only; ratio_extra = R also counts the
 * retained suffix rows of the query (all still masked).  alpha = 0 gives the
 * fixed-threshold rule.  eos_id < 0 disables the early-exit flag.
 * seq_list (n_seq ascending sequence numbers, e.g. the previous step's
 * active_seq) restricts processing; NULL = all B.  With seq_list, n_seq may be
 * given as a device scalar instead (n_seq_dev != NULL overrides n_seq as the
 * count, n_seq then being only the upper bound used to size the launch).
 * Unprocessed sequences' outputs are left untouched.  active_seq may be the same array as seq_list and
 * active_cnt the same word as n_seq_dev (the list is then updated in place, which keeps the pointers of a
 * loop's calls fixed); no other two arguments may overlap.
 * ------------------------------------------------------------------------ */
typedef struct {
  int32_t B, K;                 /* 1 <= K <= 4096 */
  const float *conf;            /* [B][K] */
  const int32_t *tok;           /* [B][K] */
  uint8_t *masked;              /* [B][K] in/out, non-zero = still MASK */
  int32_t *x_block;             /* [B][K] in/out */
  float tau0, alpha;
  int32_t ratio_extra;          /* >= 0 */
  int32_t eos_id;
  float eos_tau;
  const int32_t *seq_list;      /* optional [n_seq] */
  int32_t n_seq;
  const int32_t *n_seq_dev;     /* optional device scalar */
  int32_t *sel_idx;             /* [B][K] */
  int32_t *sel_cnt;             /* [B] */
  uint8_t *block_done;          /* [B] */
  uint8_t *eos_exit;            /* [B] in/out */
  int32_t *active_seq;          /* [B] */
  int32_t *active_cnt;          /* [1] */
  int32_t *masked_rows;         /* optional [B*K] */
  int32_t *masked_cnt;          /* [1], needed with masked_rows */
} ds_select_params;

/* `p` is a HOST pointer; the pointers inside it are device pointers. */
DS_API int ds_unmask_select(const ds_select_params *p, void *stream);

/* ------------------------------------------------------------------------
 * ds_block_begin  (Eq. 1, Eq. 2, block termination rule, early exit)
 *
 * Decoding proceeds block by block: a block whose positions are all unmasked
 * is followed by the next one (end of Preliminary), and a sequence that has
 * predicted EOS with high confidence decodes no further block ("Early Exit For
 * Block Diffusion").  This entry
 * point prepares the device state of the next block from the per-sequence
 * early-exit flags, without the host looking at them:
 *     for b with eos_exit[b] == 0:  masked[b][:] = 1, x_block[b][:] = mask_id   (Eq. 1: K fresh [MASK])
 *     for b with eos_exit[b] != 0:  masked[b][:] = 0, x_block[b][:] = fill_id   (block skipped)
 *     active_seq  = ascending list of the b with eos_exit[b] == 0, *active_cnt its length
 *     masked_rows = b * K + i for those b (list order) and i = 0..K-1, *masked_cnt = *active_cnt * K
 * in the layout ds_unmask_select, ds_confidence_listed and ds_attn_pruned's
 * seq_list read.  masked_rows/masked_cnt are optional (both NULL or both set).
 * Errors: DS_ERR_INVALID_ARG (NULL pointer, B < 0, K outside 1..4096), DS_ERR_UNSUPPORTED (B * K > 2^31 - 1).
 * ------------------------------------------------------------------------ */
typedef struct {
  int32_t B, K;
  int32_t mask_id;              /* token id of [MASK] */
  int32_t fill_id;              /* token written to the block of a sequence that has exited (normally EOS) */
  const uint8_t *eos_exit;      /* [B] */
  uint8_t *masked;              /* [B][K] out */
  int32_t *x_block;             /* [B][K] out */
  int32_t *active_seq;          /* [B] out */
  int32_t *active_cnt;          /* [1] out */
  int32_t *masked_rows;         /* optional [B*K] out */
  int32_t *masked_cnt;          /* optional [1] out */
} ds_block_params;

/* `p` is a HOST pointer; the pointers inside it are device pointers. */
DS_API int ds_block_begin(const ds_block_params *p, void *stream);

/* ------------------------------------------------------------------------
 * Utilities
 * ------------------------------------------------------------------------ */
/* Self-test of the bounded wait (no counterpart in the paper; the tensor-core kernels' failure handling).
 * Every on-chip wait of the attention and projection kernels is a poll loop with a limit, after which the
 * kernel raises DS_DEV_TIMEOUT and leaves in order.  This call runs that same wait, in a one-warp kernel, on
 * a barrier nobody arrives on, with `poll_limit` polls (1 .. 65536; a few microseconds to milliseconds), so
 * that a deployment can check the expiry path on its GPU without a real kernel having to fail:
 *     *status   |= DS_DEV_TIMEOUT                      (optional device word)
 *     report[0]  = 1  the wait gave up                  (optional device int32[3])
 *     report[1]  = 1  the CTA-wide give-up flag was set
 *     report[2]  = 1  after one arrival, a second wait on the same barrier succeeded
 * The kernel always terminates and the context stays usable.  Errors: DS_ERR_INVALID_ARG (limit out of
 * range, misaligned pointer), DS_ERR_CUDA. */
DS_API int ds_selftest_bounded_wait(uint32_t poll_limit, uint32_t *status, int32_t *report, void *stream);
/* Copies the device status word to *host_out (HOST) after synchronising `stream`. */
DS_API int ds_read_status(const uint32_t *device_status, void *stream, uint32_t *host_out);
/* HOST: static string for a ds_status value. */
DS_API const char *ds_strerror(int code);
/* The CUDA runtime's error code (cudaError_t as int) and its name for the most recent call on this host
 * thread that returned DS_ERR_CUDA; 0 / "cudaSuccess" if there was none. */
DS_API int ds_last_cuda_error(void);
DS_API const char *ds_last_cuda_error_name(void);
/* HOST: library version, major * 1000 + minor. */
DS_API int ds_version(void);
/* HOST: number of kernels this library has launched in this process (all entry points). */
DS_API int64_t ds_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* DS_H_ */
