/*
 * omni_mla.h -- C ABI of the sparse MLA decode library (B200 / sm_100a).
 *
 * The operation is the left-hand side of Eq. 1 of the paper's "OmniAttn: Problem
 * Formulation": softmax(Q K_M^T * scale) V_M, attention restricted to a selected index
 * set M, evaluated for one decode query per (request, head).  Eq. 2 (attention sink +
 * recent tokens) is one producer of M; the library accepts any index list.  As the
 * "Layer-wise Compression" paragraph requires, every head of a request shares one M,
 * which is also what multi-latent attention needs: one latent row per token, K = all
 * d_qk = 576 columns (512 latent + 64 rope), V = the first d_v = 512 columns.
 *
 * Conventions shared by every entry point
 *   - Unless a parameter says "host", pointers are DEVICE pointers owned by the caller.
 *     The library allocates no device memory and keeps no per-call state.  What it does keep,
 *     per process: per-device facts looked up once (SM count, kernel attributes, how many
 *     merging clusters fit), a table of tensor-map encodings keyed by (base address, sizes)
 *     so that repeated calls on the same buffers skip the encoding, up to four side streams per
 *     device for omni_sparse_mla_decode_host (chosen by the caller's stream), the address of the static scratch array of
 *     omni_sparse_mla_decode_static, and the two event handles of
 *     omni_sparse_mla_set_profile_events.  All of it is guarded for use from several host
 *     threads except the profile events.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*).  Errors the host
 *     can see (null pointer, bad shape, misalignment, short workspace) are returned at once
 *     and nothing is launched.
 *   - Conditions only the device can see (a token position or page id out of range) never
 *     trap: the offending entry is skipped (it contributes nothing), and if `device_status`
 *     is non-NULL the word it points to is OR-ed with OMNI_DEV_BAD_INDEX.  A bounded wait
 *     that runs out inside a kernel ORs OMNI_DEV_TIMEOUT and the affected outputs are
 *     unspecified.  The caller zeroes the word and reads it back after synchronising.
 *   - Inputs are never modified.  Distinct streams need distinct workspaces.
 */
#ifndef OMNI_MLA_H_
#define OMNI_MLA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
#define OMNI_ALIGNAS(n) alignas(n)
extern "C" {
#else
#define OMNI_ALIGNAS(n) _Alignas(n)
#endif

typedef enum {
    OMNI_OK = 0,
    OMNI_ERR_NULL = 1,      /* a required pointer is NULL                                  */
    OMNI_ERR_SHAPE = 2,     /* unsupported or inconsistent sizes in the descriptor         */
    OMNI_ERR_ALIGN = 3,     /* a pointer misses its required alignment                     */
    OMNI_ERR_WORKSPACE = 4, /* workspace smaller than omni_sparse_mla_workspace_bytes()    */
    OMNI_ERR_INDEX = 5,     /* reserved for host-side index checks                         */
    OMNI_ERR_TIMEOUT = 6,   /* reserved                                                    */
    OMNI_ERR_CUDA = 7,      /* a CUDA runtime / driver call failed (launch, tensor map)    */
    OMNI_ERR_ARCH = 8       /* the current device is not compute capability 10.x           */
} omni_status_t;

/* bits OR-ed into *device_status by kernels */
#define OMNI_DEV_BAD_INDEX 1
#define OMNI_DEV_TIMEOUT 2
/* set together with OMNI_DEV_TIMEOUT by the paired-CTA kernel: whose wait ran out (diagnosis) */
#define OMNI_DEV_ROLE_PRODUCER_K 0x100
#define OMNI_DEV_ROLE_PRODUCER_V 0x200
#define OMNI_DEV_ROLE_MMA 0x400
#define OMNI_DEV_ROLE_SOFTMAX 0x800

/* descriptor flags */
#define OMNI_FLAG_VALIDATE 1  /* run the index validation kernel before the decode kernel  */
#define OMNI_FLAG_SIMT 2      /* use the plain-FMA bring-up kernel instead of tensor cores */
#define OMNI_FLAG_FUSED_MERGE 4 /* paired-CTA kernel merges the split-KV partials itself (one launch) */
#define OMNI_FLAG_NO_CLUSTER_MERGE 8 /* never merge two splits inside a cluster of two CTA pairs */

/* Plain-data problem descriptor; copied at call time. */
typedef struct {
    int64_t num_pages;         /* pages in the pool, >= 1                                  */
    int32_t batch;             /* B >= 1 requests                                          */
    int32_t num_heads;         /* H in [1,128]                                             */
    int32_t d_qk;              /* must be 576                                              */
    int32_t d_v;               /* must be 512                                              */
    int32_t page_size;         /* must be 64                                               */
    int32_t max_pages_per_req; /* row stride of page_table, >= 1                           */
    int32_t max_sel;           /* row stride of sel_idx, >= 1                              */
    int32_t num_splits;        /* 0: library chooses; k >= 1: k split-KV partitions/request*/
    float softmax_scale;       /* multiplies q.k before the softmax, e.g. 1/sqrt(192)      */
    int32_t flags;             /* OMNI_FLAG_* bits                                         */
} omni_mla_desc_t;

/* Library version, major*1000 + minor. */
int omni_version(void);

/* Static, human-readable name of a status code. */
const char *omni_status_string(omni_status_t status);

/*
 * Number of split-KV partitions per request the library will use for this descriptor on
 * the current device (desc->num_splits if that is >= 1).  Returns 0 on a bad descriptor.
 */
int32_t omni_sparse_mla_num_splits(const omni_mla_desc_t *desc);

/*
 * Kernels one omni_sparse_mla_decode call launches for this descriptor on the current device:
 * the decode kernel, plus the split-KV merge kernel unless the splits are merged inside the
 * decode kernel (two splits per request whose CTA clusters are all resident at once, or
 * OMNI_FLAG_FUSED_MERGE), plus the validation kernel if OMNI_FLAG_VALIDATE is set.  Returns 0
 * on a bad descriptor.
 */
int32_t omni_sparse_mla_num_launches(const omni_mla_desc_t *desc);

/*
 * The split-KV plan as a pure function of its inputs (no device needed; what
 * omni_sparse_mla_num_splits / num_launches compute after asking the current device):
 * partitions per request for this descriptor on a device with `sm_count` SMs on which
 * `resident_merge_clusters` clusters of two CTA pairs of the paired-CTA kernel can be resident
 * at once (33 on a 148-SM B200), and, through num_launches if non-NULL, the kernels one decode
 * call launches.  Returns 0 on a bad descriptor or non-positive sm_count.
 */
int32_t omni_sparse_mla_plan_query(const omni_mla_desc_t *desc, int32_t sm_count,
                                   int32_t resident_merge_clusters, int32_t *num_launches);

/*
 * Bytes of device workspace omni_sparse_mla_decode needs for this descriptor: room for the
 * fp32 partial outputs and partial log-sum-exps of every (request, split) and for the
 * arrival counters of the in-kernel merge.  Returns 0 on a bad descriptor.  The workspace
 * must be 256-byte aligned; its contents need no initialisation (the call clears what it
 * needs cleared, on `stream`) and are overwritten.
 */
size_t omni_sparse_mla_workspace_bytes(const omni_mla_desc_t *desc);

/*
 * Decode-phase sparse MLA attention (Eq. 1 left-hand side over the index set of each
 * request; split-KV partition and merge included).
 *
 * For request b, head h, with N = sel_len[b] and t_j = sel_idx[b][j] for j < N:
 *     row_j = page_table[b][t_j / 64] * 64 + t_j % 64
 *     x_j   = softmax_scale * sum_c q[b,h,c] * kv_cache[row_j][c]          c < 576
 *     lse[b,h]   = ln sum_j exp(x_j)                                       (natural log)
 *     out[b,h,d] = sum_j exp(x_j - lse[b,h]) * kv_cache[row_j][d]          d < 512
 * N = 0 gives out = 0 and lse = -inf.  The order of sel_idx does not matter beyond
 * rounding; repeated positions count once per occurrence.
 *
 *   q          bf16 [B, H, 576], contiguous, 16-byte aligned
 *   kv_cache   bf16 [num_pages, 64, 576], contiguous, 128-byte aligned
 *   page_table int32 [B, max_pages_per_req]: physical page id of each logical page
 *   sel_idx    int32 [B, max_sel]: logical token positions; entries at j >= sel_len[b] are
 *              never read as positions
 *   sel_len    int32 [B], each in [0, max_sel]
 *   out        bf16 [B, H, 512]            (written)
 *   lse        fp32 [B, H]                 (written)
 *   workspace  >= omni_sparse_mla_workspace_bytes(desc) bytes, 256-byte aligned
 *   device_status  optional int32 word, see the conventions above; may be NULL
 *
 * Products are bf16 x bf16 accumulated in fp32; the softmax runs in fp32; the tensor-core
 * path rounds the unnormalised weights to bf16 before the weighted sum.
 */
omni_status_t omni_sparse_mla_decode(const omni_mla_desc_t *desc, const void *q,
                                     const void *kv_cache, const int32_t *page_table,
                                     const int32_t *sel_idx, const int32_t *sel_len, void *out,
                                     float *lse, void *workspace, size_t workspace_bytes,
                                     int32_t *device_status, void *stream);

/*
 * The same decode call in two halves, for callers that issue it every step on the same
 * buffers (no counterpart in the paper: host-side packaging of omni_sparse_mla_decode).
 * omni_sparse_mla_plan_init does, once, everything that depends only on the descriptor, the
 * q buffer and the KV pool: the argument checks on those, the split-KV plan, the choice of
 * kernel and merge path, the tensor-map encodings.  It writes the result into `plan`, memory
 * the caller owns (64-byte aligned; plain data: it may be copied, and needs no clean-up).
 * omni_sparse_mla_decode_planned then takes the per-step pointers, checks them, and launches:
 * no table look-up, no lock, no device query beyond "is the plan's device current".
 * Results are those of omni_sparse_mla_decode with the same arguments, bit for bit.
 *
 * A plan stays valid while q and kv_cache keep their addresses and sizes and the descriptor
 * is unchanged; it belongs to the device that was current in plan_init (OMNI_ERR_CUDA from the
 * planned call if another device is current).  A plan that plan_init did not complete is
 * rejected with OMNI_ERR_SHAPE.  workspace / workspace_bytes, device_status and stream are as
 * in omni_sparse_mla_decode; the workspace size is omni_sparse_mla_workspace_bytes(desc).
 */
typedef struct {
    OMNI_ALIGNAS(64) unsigned char opaque[1024];
} omni_mla_plan_t;
omni_status_t omni_sparse_mla_plan_init(const omni_mla_desc_t *desc, const void *q,
                                        const void *kv_cache, omni_mla_plan_t *plan);
omni_status_t omni_sparse_mla_decode_planned(const omni_mla_plan_t *plan, const int32_t *page_table,
                                             const int32_t *sel_idx, const int32_t *sel_len,
                                             void *out, float *lse, void *workspace,
                                             size_t workspace_bytes, int32_t *device_status,
                                             void *stream);

/*
 * The same operation with the index set of Eq. 2 of the paper (attention sink + recent
 * tokens) given as its two parameters instead of an index list, so that no sel_idx array
 * has to be built or read.  Counting positions from 0, request b with context length
 * M = ctx_len[b] attends to [0, min(N_sink, M)) united with [max(M - N_recent, 0), M); where
 * the two ranges overlap the union is taken without repeats, so the selection is the whole
 * context once N_sink + N_recent >= M.  The result is that of omni_sparse_mla_decode on the
 * increasing list of those positions (within rounding: the kernels walk the recent range in
 * page-aligned tiles, which regroups the sums unless the range already starts on a page
 * boundary right behind the sink; then the two results are bit-identical).
 *
 *   ctx_len    int32 [B], each in [0, max_pages_per_req * 64]; a value outside is treated like a
 *              bad sel_len (out = 0, lse = -inf, OMNI_DEV_BAD_INDEX)
 *   n_sink, n_recent   N_sink and N_recent of Eq. 2, >= 0
 *   desc->max_sel      upper bound of the selection size the split-KV plan is made for; must be
 *              at least min(n_sink + n_recent, max_pages_per_req * 64), else OMNI_ERR_SHAPE.
 *              Workspace and split queries apply to this descriptor unchanged.
 * OMNI_FLAG_VALIDATE is ignored (there is no index list to check; page ids are still checked
 * where they are used).  All other arguments are those of omni_sparse_mla_decode.
 */
omni_status_t omni_sparse_mla_decode_sink_recent(const omni_mla_desc_t *desc, const void *q,
                                                 const void *kv_cache, const int32_t *page_table,
                                                 const int32_t *ctx_len, int32_t n_sink,
                                                 int32_t n_recent, void *out, float *lse,
                                                 void *workspace, size_t workspace_bytes,
                                                 int32_t *device_status, void *stream);

/*
 * Rolling cache of a compressed layer (the paper's layer-wise KV-cache compression: a layer
 * whose pattern bit is 1 only ever attends to the index set of Eq. 2, so it needs to store
 * nothing but the attention sink and the recent window).  Per request such a layer owns
 * omni_rolling_pages_per_request(n_sink, n_recent) = ceil(N_sink/64) + ceil(N_recent/64) + 1
 * pages, listed in its page_table row: the first ceil(N_sink/64) hold positions
 * [0, 64*ceil(N_sink/64)) for good, the others are reused round-robin by all later 64-token
 * blocks of the context.  The token at absolute position t is therefore found at position
 *     t                                                     if t / 64 < sink_pages
 *     (sink_pages + (t/64 - sink_pages) % ring_pages)*64 + t%64   otherwise
 * of that short page table, whatever the context length.
 *
 * omni_kv_append_rolling writes one new latent row per request: new_rows[b] (bf16 [B, 576],
 * 16-byte aligned) becomes the token at position ctx_len[b] (the length BEFORE the append; the
 * caller advances its own counter afterwards) and overwrites the oldest block's slot once the
 * ring has gone round.  A negative length or a bad page id sets OMNI_DEV_BAD_INDEX and skips
 * the request.  desc supplies batch, num_pages and max_pages_per_req (>= the pages per request
 * above, else OMNI_ERR_SHAPE).
 *
 * omni_sparse_mla_decode_rolling is omni_sparse_mla_decode_sink_recent over that layout: the
 * same index set, the same result bit for bit as on an uncompressed cache holding the same
 * rows, for any ctx_len[b] >= 0.  desc->max_sel must be at least n_sink + n_recent.
 */
int32_t omni_rolling_pages_per_request(int32_t n_sink, int32_t n_recent);
omni_status_t omni_kv_append_rolling(const omni_mla_desc_t *desc, void *kv_cache,
                                     const int32_t *page_table, const int32_t *ctx_len,
                                     const void *new_rows, int32_t n_sink, int32_t n_recent,
                                     int32_t *device_status, void *stream);
omni_status_t omni_sparse_mla_decode_rolling(const omni_mla_desc_t *desc, const void *q,
                                             const void *kv_cache, const int32_t *page_table,
                                             const int32_t *ctx_len, int32_t n_sink, int32_t n_recent,
                                             void *out, float *lse, void *workspace,
                                             size_t workspace_bytes, int32_t *device_status, void *stream);

/*
 * 8-bit latent cache (the paper serves an INT8-quantised model, Evaluation, "Experimental
 * Setup", and gives no cache format; this one is the library's own).  A token's row is
 * OMNI_Q8_ROW_BYTES = 640 bytes: its 512 latent columns as FP8 E4M3 codes (1-4-3 bits, bias 7,
 * largest magnitude 448, no infinities), then its 64 rope columns unchanged as bf16.  One fp32
 * scale per row lives in a second array; a latent value is code * scale.
 *
 * omni_kv_quantize_q8 writes that form for `num_rows` bf16 rows (kv_rows bf16 [num_rows, 576],
 * 16-byte aligned; kv_q8 uint8 [num_rows, 640], 128-byte aligned; kv_scale fp32 [num_rows]):
 *     scale = max(amax, 2^-60) / 448,  amax = largest |value| of the row's 512 latent columns
 *     code  = E4M3(value / scale)      fp32 division, round to nearest even, saturating at 448
 * Rows map one to one, so a paged pool keeps its page table.
 *
 * omni_sparse_mla_decode_q8 is omni_sparse_mla_decode over such a pool (kv_q8 uint8
 * [num_pages, 64, 640], kv_scale fp32 [num_pages, 64]): the result is DEFINED as Eq. 1's
 * restricted attention over the de-quantised rows (code * scale for the latent columns, the
 * stored bf16 for the rope columns), K = all 576 columns, V = the first 512.  The codes go
 * through the 8-bit tensor-core path unchanged; q and the softmax weights enter it as two
 * E4M3 terms each (value ~ hi + lo), which keeps about the eight significant bits they have in
 * the bf16 path, so the same tolerances apply against that definition.  Needs more than 64
 * heads (OMNI_ERR_SHAPE otherwise, and for OMNI_FLAG_SIMT); descriptor, index arrays,
 * workspace (omni_sparse_mla_workspace_bytes), status word, stream and the remaining flags are
 * those of omni_sparse_mla_decode.  Rows that are not selected are never read, scales included.
 */
#define OMNI_Q8_ROW_BYTES 640
omni_status_t omni_kv_quantize_q8(const void *kv_rows, int64_t num_rows, void *kv_q8, float *kv_scale,
                                  void *stream);
omni_status_t omni_sparse_mla_decode_q8(const omni_mla_desc_t *desc, const void *q, const void *kv_q8,
                                        const float *kv_scale, const int32_t *page_table,
                                        const int32_t *sel_idx, const int32_t *sel_len, void *out,
                                        float *lse, void *workspace, size_t workspace_bytes,
                                        int32_t *device_status, void *stream);

/*
 * Selection producer for token-level sparsity (the step before the decode call when the index
 * set is "the k highest-scoring tokens", as in a top-k sparse attention variant; the paper
 * itself only uses the sink + recent rule of Eq. 2).  For every request b with M = ctx_len[b]
 * (clamped to [0, stride]) it writes into sel_idx[b] the positions of the min(k, M) largest of
 * scores[b][0..M), in increasing order of position, and min(k, M) into sel_len[b]: exactly what
 * omni_sparse_mla_decode reads (descriptor max_sel = k).  Scores compare as IEEE floats with
 * -0 below +0 and NaN below everything; among equal scores at the threshold the lowest
 * positions win, so the result is a deterministic function of the input.
 *
 *   scores   fp32 [batch, stride], stride <= 131072 (else OMNI_ERR_SHAPE)
 *   ctx_len  int32 [batch]
 *   k        1 <= k <= stride
 *   sel_idx  int32 [batch, k] (written; entries at and beyond sel_len[b] are left untouched)
 *   sel_len  int32 [batch]    (written)
 * All pointers are device pointers owned by the caller; nothing is allocated.  One kernel is
 * enqueued on `stream` (NULL: the default stream) and the call returns without waiting for it.
 * Errors: OMNI_ERR_NULL (a null pointer), OMNI_ERR_SHAPE (batch < 1, k outside [1, stride],
 * stride outside [1, 131072]), OMNI_ERR_ALIGN (a pointer not 4-byte aligned), OMNI_ERR_ARCH
 * (not an sm_100 device), OMNI_ERR_CUDA (the launch failed).
 */
omni_status_t omni_topk_select(const float *scores, const int32_t *ctx_len, int32_t batch, int32_t stride,
                               int32_t k, int32_t *sel_idx, int32_t *sel_len, void *stream);

/*
 * Merge of split-KV partial results (the step that follows a partition of M into disjoint
 * ranges; Eq. 1 is recovered exactly because softmax normalisers add):
 *     lse[b,h]   = ln sum_s exp(part_lse[b,s,h])
 *     out[b,h,d] = sum_s exp(part_lse[b,s,h] - lse[b,h]) * part_out[b,s,h,d]
 *
 *   max_splits  row stride S of the partial arrays, >= 1
 *   part_out    fp32 [B, S, H, 512], each partial normalised by its own sum; 16-byte aligned
 *   part_lse    fp32 [B, S, H]; -inf marks an empty partial (weight 0)
 *   num_splits  int32 [B], each in [0, S], or NULL meaning S for every request
 *   out         bf16 [B, H, 512]  (written);  lse fp32 [B, H] (written)
 * If every partial of a (b,h) is empty the result is out = 0, lse = -inf.  Only batch,
 * num_heads and d_v of the descriptor are used.
 */
omni_status_t omni_sparse_mla_combine(const omni_mla_desc_t *desc, int32_t max_splits,
                                      const float *part_out, const float *part_lse,
                                      const int32_t *num_splits, void *out, float *lse,
                                      void *stream);

/*
 * Self-test of the bounded device waits (no counterpart in the paper).  Every wait inside the
 * kernels of this library (on a copy, on the tensor core, on another warp or CTA) gives up
 * after a limit, ORs OMNI_DEV_TIMEOUT plus a role bit into *device_status and lets the kernel
 * return; nothing spins without bound and nothing traps.  This entry point exercises exactly
 * that helper where it can be made to run out on purpose without involving a copy or tensor
 * memory: one warp waits for `limit_cycles` SM clocks (1 .. 2^31) on a barrier nobody arrives
 * on.  Afterwards *device_status carries OMNI_DEV_TIMEOUT and, if waited_cycles is non-NULL
 * (device pointer, 8-byte aligned), *waited_cycles the clocks the wait took.  The context
 * stays usable.  Asynchronous on `stream`.
 */
omni_status_t omni_selftest_bounded_wait(int64_t limit_cycles, int32_t *device_status,
                                         int64_t *waited_cycles, void *stream);

/*
 * Index contract check on the device: ORs OMNI_DEV_BAD_INDEX into *device_status if any
 * sel_len[b] lies outside [0, max_sel], any read position is negative or beyond the page
 * table row, or any page id it reaches lies outside [0, num_pages).  Launches one small
 * kernel; reads nothing but the three index arrays.
 */
omni_status_t omni_sparse_mla_validate(const omni_mla_desc_t *desc, const int32_t *page_table,
                                       const int32_t *sel_idx, const int32_t *sel_len,
                                       int32_t *device_status, void *stream);

/*
 * Physical rows the decode kernel will read, for checking index handling bit for bit:
 * rows[b][j] = row_j (int64) for j < sel_len[b], -1 elsewhere and for entries that violate
 * the index contract.  rows is int64 [B, max_sel].
 */
omni_status_t omni_sparse_mla_resolve_rows(const omni_mla_desc_t *desc,
                                           const int32_t *page_table, const int32_t *sel_idx,
                                           const int32_t *sel_len, int64_t *rows, void *stream);

/*
 * Same operation as omni_sparse_mla_decode for callers whose per-step tensors live in HOST
 * memory: q, page_table, sel_idx, sel_len are host pointers (pinned memory makes the copies
 * asynchronous) and out / lse are host buffers that receive the result.  kv_cache stays a
 * device pointer: the cache is state that persists across decode steps.
 *
 *   staging, staging_bytes   device scratch for the per-step tensors, at least
 *                            omni_sparse_mla_host_staging_bytes(desc), 256-byte aligned
 *                            (the size includes split-KV scratch for the two-part schedule below)
 * Everything is ordered on `stream`: the host buffers may be read after the stream is
 * synchronised.  From a batch of a few megabytes of q and out on (at least 4 requests), the
 * call runs the batch as two parts: the second part's q copy and, later, its kernel and copies
 * out go to a stream the library creates once per device, which waits for `stream` at the
 * start and which `stream` waits for at the end, so that copies in, kernels and copies out of
 * the two parts overlap (PCIe carries both directions at once).  `workspace` is used only when
 * the batch runs as one part.
 */
size_t omni_sparse_mla_host_staging_bytes(const omni_mla_desc_t *desc);
omni_status_t omni_sparse_mla_decode_host(const omni_mla_desc_t *desc, const void *q_host,
                                          const void *kv_cache,
                                          const int32_t *page_table_host,
                                          const int32_t *sel_idx_host,
                                          const int32_t *sel_len_host, void *out_host,
                                          float *lse_host, void *staging, size_t staging_bytes,
                                          void *workspace, size_t workspace_bytes,
                                          int32_t *device_status, void *stream);

/*
 * Decode without a caller-supplied workspace (the paper has no counterpart: this is a
 * packaging variant of omni_sparse_mla_decode, same arithmetic, same results).
 *
 * Who it is for: code that runs the decode step but may not allocate device memory, e.g. an
 * attention plug-in inside a serving engine that has already handed every free byte of the
 * GPU to its KV-cache pool, or a latency-critical decode loop where cudaMalloc / cudaFree are
 * ruled out because they synchronise the device.  Such callers cannot provide the split-KV
 * workspace, so here the library brings its own: a fixed array of OMNI_STATIC_SCRATCH_BYTES
 * that is part of the library image.  The call itself performs no cudaMalloc, cudaFree or any
 * other allocating call.
 *
 * Costs and rules that follow from that:
 *   - every GPU on which the library is used keeps OMNI_STATIC_SCRATCH_BYTES (32 MiB) of
 *     device memory occupied until the process exits;
 *   - a problem whose omni_sparse_mla_workspace_bytes(desc) exceeds OMNI_STATIC_SCRATCH_BYTES
 *     is rejected with OMNI_ERR_WORKSPACE and nothing is launched (lower desc->num_splits or
 *     the batch, or use omni_sparse_mla_decode with a workspace of your own);
 *   - the first call on each device looks up the array's device address (one runtime query,
 *     with that device current) and caches it; make that first call during start-up, before
 *     any stream capture begins AND before the process hands the rest of the device memory to
 *     its own pools: the CUDA runtime may load the library's device image, array included,
 *     only at that first query, and a device with no free memory left then fails it
 *     (OMNI_ERR_CUDA);
 *   - all calls on one device share the one array, which keeps whatever the previous call left
 *     in it.  The caller clears nothing (each call overwrites every partial result it reads
 *     back and clears the few counters it needs at zero itself), but two calls that overlap on the GPU, e.g. on different streams, race on
 *     it: serialise them, or give the concurrent ones omni_sparse_mla_decode with separate
 *     workspaces.
 * All other arguments, results, alignment rules and status codes are those of
 * omni_sparse_mla_decode.
 */
#define OMNI_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
omni_status_t omni_sparse_mla_decode_static(const omni_mla_desc_t *desc, const void *q,
                                            const void *kv_cache, const int32_t *page_table,
                                            const int32_t *sel_idx, const int32_t *sel_len,
                                            void *out, float *lse, int32_t *device_status,
                                            void *stream);

/*
 * Profiling aid (no counterpart in the paper): when both events are non-NULL, every later
 * omni_sparse_mla_decode call on this thread's process records `before` and `after`
 * (cudaEvent_t passed as void*) on its stream immediately around the main decode kernel,
 * excluding the validation and merge kernels, so a caller can time that kernel alone.
 * Pass NULLs to switch it off.  Process-wide and not thread-safe: meant for benchmarks.
 */
void omni_sparse_mla_set_profile_events(void *before, void *after);

#ifdef __cplusplus
}
#endif
#endif /* OMNI_MLA_H_ */
