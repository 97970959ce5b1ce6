// Host side of the C ABI declared in omni_mla.h: argument checks, the split-KV plan,
// workspace carving and kernel launches.  Nothing here allocates device memory.
#include <cuda_runtime.h>

#include <mutex>

#include "combine.cuh"
#include "common.cuh"
#include "simt_decode.cuh"
#include "tc_decode.cuh"
#include "tc2_decode.cuh"
#include "tc2q8_decode.cuh"
#include "topk_select.cuh"

namespace omni {
namespace {

constexpr int kMaxSplits = 32;

cudaEvent_t g_profile_before = nullptr, g_profile_after = nullptr;

struct DeviceInfo {
    int sm_count = 0;
    int cc_major = 0;
    int index = -1;
    bool ok = false;
};

// Per-device facts, looked up once per device and process.
const DeviceInfo &device_info()
{
    static DeviceInfo info[64];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        static DeviceInfo none;
        return none;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (!info[dev].ok) {
        int sms = 0, major = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess) {
            info[dev].sm_count = sms;
            info[dev].cc_major = major;
            info[dev].index = dev;
            info[dev].ok = true;
        }
    }
    return info[dev];
}

bool desc_ok(const omni_mla_desc_t *d)
{
    return d && d->batch >= 1 && d->num_heads >= 1 && d->num_heads <= 128 && d->d_qk == kDqk &&
           d->d_v == kDv && d->page_size == kPage && d->num_pages >= 1 &&
           d->num_pages <= (int64_t)0x7fffffff / kPage && d->max_pages_per_req >= 1 &&
           d->max_sel >= 1 && d->num_splits >= 0 && d->num_splits <= kMaxSplits;
}

// Pages of a compressed layer's rolling cache: the sink pages are kept for good, the ring holds
// the recent window (which can straddle one more page than it fills).
int64_t rolling_sink_pages(int32_t n_sink) { return ((int64_t)n_sink + kPage - 1) / kPage; }
int64_t rolling_ring_pages(int32_t n_recent) { return ((int64_t)n_recent + kPage - 1) / kPage + 1; }

bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// More than 64 heads run on the paired-CTA kernel (one cluster of two CTAs per work unit).
bool use_pair_kernel(const omni_mla_desc_t *d) { return !(d->flags & OMNI_FLAG_SIMT) && d->num_heads > kTcHeads; }

// Work units one split of one request occupies in the kernel that will run.
int units_per_request(const omni_mla_desc_t *d)
{
    if (d->flags & OMNI_FLAG_SIMT)
        return (d->num_heads + kSimtWarps * kSimtHeadsPerWarp - 1) / (kSimtWarps * kSimtHeadsPerWarp);
    if (use_pair_kernel(d)) return 1;
    return (d->num_heads + kTcHeads - 1) / kTcHeads;
}

// Two splits of a request can be merged inside a cluster of two CTA pairs as long as all those
// clusters are resident at once.
bool merge_in_cluster(const omni_mla_desc_t *d, int splits, int resident_merge_clusters = -1)
{
    if (!(splits == 2 && use_pair_kernel(d) && !(d->flags & (OMNI_FLAG_FUSED_MERGE | OMNI_FLAG_NO_CLUSTER_MERGE))))
        return false;
    if (resident_merge_clusters < 0) resident_merge_clusters = tc2_max_merge_clusters();
    return d->batch <= resident_merge_clusters;
}

// Pick the number of split-KV partitions per request.  The kernel's work units run in waves over
// the SMs.  In units of one tile time (64 tokens), as measured: a unit costs a fixed part of about
// 6 (set-up, first-tile latency, epilogue) plus one per granule; a unit that writes fp32 partial
// results to global memory for a later merge costs about 6 more when the grid runs in several
// waves (256 KiB written and read back against 72 KiB per tile; about 2 within one wave, where
// they stay in L2), and so does the merge kernel at the end.  Two splits merged inside a
// cluster of two CTA pairs avoid the partial results and pay about 5 for the exchange.
// Minimise waves * (granules per unit + fixed parts) + merge.
int choose_splits(const omni_mla_desc_t *d, int sm_count, int resident_merge_clusters = -1)
{
    if (d->num_splits >= 1) return d->num_splits;
    if (sm_count <= 0) sm_count = 148;
    const int granule = use_pair_kernel(d) ? kC2Tile : kTile;
    const int granules = (d->max_sel + granule - 1) / granule;
    const long units = (long)d->batch * units_per_request(d);
    if (use_pair_kernel(d)) sm_count /= 2;               // a work unit occupies two SMs
    long best_cost = -1;
    int best = 1;
    for (int s = 1; s <= kMaxSplits && s <= granules; ++s) {
        const long waves = (units * s + sm_count - 1) / sm_count;
        const long per = (granules + s - 1) / s;
        long cost;
        if (s == 1)
            cost = waves * (per + 6);
        else if (merge_in_cluster(d, s, resident_merge_clusters))
            cost = waves * (per + 6) + 5;
        else
            cost = waves * (per + 6 + (waves > 1 ? 6 : 2)) + 6;     // partial results stay in L2 within one wave
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            best = s;
        }
    }
    return best;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

size_t part_out_bytes(const omni_mla_desc_t *d, int splits)
{
    return align_up((size_t)d->batch * splits * d->num_heads * kDv * sizeof(float), 256);
}

size_t part_lse_bytes(const omni_mla_desc_t *d, int splits)
{
    return align_up((size_t)d->batch * splits * d->num_heads * sizeof(float), 256);
}

// Arrival counters of the in-kernel merge: one per (request, head group of 64).
size_t counter_bytes(const omni_mla_desc_t *d)
{
    return align_up((size_t)d->batch * ((d->num_heads + kTcHeads - 1) / kTcHeads) * sizeof(int32_t), 256);
}

size_t workspace_need(const omni_mla_desc_t *d, int splits)
{
    return part_out_bytes(d, splits) + part_lse_bytes(d, splits) + counter_bytes(d);
}

// On request the paired-CTA kernel merges the splits itself (the last CTA to finish a request's
// head half does it); by default a second, programmatically dependent kernel spreads the merge
// over all SMs, which is faster when every split of a batch finishes at about the same time.
bool merge_in_kernel(const omni_mla_desc_t *d)
{
    return use_pair_kernel(d) && (d->flags & OMNI_FLAG_FUSED_MERGE);
}

omni_status_t launch_combine(int batch, int heads, int max_splits, const float *part_out,
                             const float *part_lse, const int32_t *num_splits, void *out,
                             float *lse, cudaStream_t stream)
{
    // Keep the shared-memory / L1 split the decode kernel needs: alternating between two splits
    // makes every launch wait for the SMs to be reconfigured.
    static bool carveout_set = false;
    if (!carveout_set) {
        cudaFuncSetAttribute(combine_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
        carveout_set = true;
    }
    // Programmatic dependent launch: the merge blocks may become resident while the decode kernel
    // is still running and wait (griddepcontrol.wait) until it has completed and its writes are
    // visible, which removes most of the launch gap between the two kernels.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(batch * heads));
    cfg.blockDim = dim3(128);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, combine_kernel, part_out, part_lse, num_splits, max_splits, heads,
                              static_cast<__nv_bfloat16 *>(out), lse) == cudaSuccess
               ? OMNI_OK
               : OMNI_ERR_CUDA;
}

omni_status_t launch_resolve(const omni_mla_desc_t *d, const int32_t *page_table,
                             const int32_t *sel_idx, const int32_t *sel_len, int64_t *rows,
                             int32_t *status, cudaStream_t stream)
{
    dim3 grid((unsigned)min(64, (d->max_sel + 255) / 256), (unsigned)d->batch);
    resolve_rows_kernel<<<grid, 256, 0, stream>>>(page_table, sel_idx, sel_len,
                                                  d->max_pages_per_req, d->max_sel, d->num_pages,
                                                  rows, status);
    return cudaPeekAtLastError() == cudaSuccess ? OMNI_OK : OMNI_ERR_CUDA;
}

// Self-test of the bounded wait every kernel here relies on: one warp waits, with the given
// limit, on a barrier that nobody ever arrives on.  No copy and no tensor memory is involved;
// the warp reports what the product kernels report when a wait runs out and returns.
__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(long long limit_cycles, int32_t *status,
                                                                   long long *waited_cycles)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const long long t0 = clock64();
    bool ok = mbar_wait(&bar, 0, limit_cycles);
    ok = __all_sync(0xffffffffu, ok);
    const long long t1 = clock64();
    if (threadIdx.x == 0) {
        if (!ok) flag_status(status, OMNI_DEV_TIMEOUT | OMNI_DEV_ROLE_SOFTMAX);
        if (waited_cycles) *waited_cycles = t1 - t0;
    }
}

}  // namespace
}  // namespace omni

using namespace omni;

extern "C" {

int omni_version(void) { return 1000; }

void omni_sparse_mla_set_profile_events(void *before, void *after)
{
    g_profile_before = static_cast<cudaEvent_t>(before);
    g_profile_after = static_cast<cudaEvent_t>(after);
}

const char *omni_status_string(omni_status_t status)
{
    switch (status) {
        case OMNI_OK: return "ok";
        case OMNI_ERR_NULL: return "null pointer";
        case OMNI_ERR_SHAPE: return "unsupported or inconsistent shape";
        case OMNI_ERR_ALIGN: return "misaligned pointer";
        case OMNI_ERR_WORKSPACE: return "workspace too small";
        case OMNI_ERR_INDEX: return "index out of range";
        case OMNI_ERR_TIMEOUT: return "device wait timed out";
        case OMNI_ERR_CUDA: return "CUDA call failed";
        case OMNI_ERR_ARCH: return "device is not compute capability 10.x";
    }
    return "unknown status";
}

int32_t omni_sparse_mla_num_splits(const omni_mla_desc_t *desc)
{
    if (!desc_ok(desc)) return 0;
    return choose_splits(desc, device_info().sm_count);
}

int32_t omni_sparse_mla_num_launches(const omni_mla_desc_t *desc)
{
    if (!desc_ok(desc)) return 0;
    const int s = choose_splits(desc, device_info().sm_count);
    int n = 1 + ((desc->flags & OMNI_FLAG_VALIDATE) ? 1 : 0);
    if (s > 1 && !merge_in_cluster(desc, s) && !(use_pair_kernel(desc) && (desc->flags & OMNI_FLAG_FUSED_MERGE))) ++n;
    return n;
}

int32_t omni_sparse_mla_plan_query(const omni_mla_desc_t *desc, int32_t sm_count, int32_t resident_merge_clusters,
                                   int32_t *num_launches)
{
    if (!desc_ok(desc) || sm_count < 1 || resident_merge_clusters < 0) return 0;
    const int s = choose_splits(desc, sm_count, resident_merge_clusters);
    if (num_launches) {
        int n = 1 + ((desc->flags & OMNI_FLAG_VALIDATE) ? 1 : 0);
        if (s > 1 && !merge_in_cluster(desc, s, resident_merge_clusters) &&
            !(use_pair_kernel(desc) && (desc->flags & OMNI_FLAG_FUSED_MERGE)))
            ++n;
        *num_launches = n;
    }
    return s;
}

size_t omni_sparse_mla_workspace_bytes(const omni_mla_desc_t *desc)
{
    if (!desc_ok(desc)) return 0;
    return workspace_need(desc, choose_splits(desc, device_info().sm_count));
}

// Everything about a decode call that depends only on the descriptor, q and the pool: which
// kernel, the split plan, workspace carving, tensor maps.  The ordinary entry points build
// one per call (maps come from the cache); omni_sparse_mla_plan_init stores one in caller
// memory so that omni_sparse_mla_decode_planned only fills in pointers and launches.
constexpr uint32_t kPlanMagic = 0x4c504d4fu;
struct LaunchPlan {
    uint32_t magic;
    int32_t kernel;            // 0 plain-FMA, 1 single-CTA tensor-core, 2 paired-CTA tensor-core, 3 the same over the 8-bit cache
    int32_t splits;
    int32_t cluster_merge, longest_first, fused_merge;
    int32_t device;
    size_t need, part_out, part_lse, counters;
    omni_mla_desc_t desc;
    const void *q, *kv;
    const float *kv_scale;     // 8-bit cache only
    alignas(64) CUtensorMap maps[5];
};
static_assert(sizeof(LaunchPlan) <= sizeof(omni_mla_plan_t), "plan does not fit its public container");
static_assert(alignof(LaunchPlan) <= 64, "plan alignment");

static omni_status_t build_plan(const omni_mla_desc_t *desc, const void *q, const void *kv_cache, bool cached_maps,
                                LaunchPlan *plan, const float *kv_scale = nullptr, bool q8 = false)
{
    if (!desc || !q || !kv_cache || (q8 && !kv_scale)) return OMNI_ERR_NULL;
    if (!desc_ok(desc)) return OMNI_ERR_SHAPE;
    // the 8-bit path exists for the paired-CTA kernel only (more than 64 heads, tensor cores)
    if (q8 && !use_pair_kernel(desc)) return OMNI_ERR_SHAPE;
    if (!aligned(q, 16) || !aligned(kv_cache, 128) || !aligned(kv_scale, 4)) return OMNI_ERR_ALIGN;
    const DeviceInfo &dev = device_info();
    if (!dev.ok) return OMNI_ERR_CUDA;
    if (dev.cc_major != 10) return OMNI_ERR_ARCH;
    plan->desc = *desc;
    plan->q = q;
    plan->kv = kv_cache;
    plan->kv_scale = kv_scale;
    plan->device = dev.index;
    plan->kernel = q8 ? 3 : (desc->flags & OMNI_FLAG_SIMT) ? 0 : use_pair_kernel(desc) ? 2 : 1;
    const int splits = choose_splits(desc, dev.sm_count);
    plan->splits = splits;
    plan->part_out = part_out_bytes(desc, splits);
    plan->part_lse = part_lse_bytes(desc, splits);
    plan->counters = counter_bytes(desc);
    plan->need = workspace_need(desc, splits);
    // Two splits of a request can be merged inside a cluster of two CTA pairs, without partial
    // results in global memory, as long as all those clusters are resident at once.
    plan->cluster_merge = merge_in_cluster(desc, splits) ? 1 : 0;
    plan->fused_merge = (splits > 1 && merge_in_kernel(desc)) ? 1 : 0;
    // several waves of work units: start the longest requests first (the kernel ranks them itself)
    plan->longest_first = (plan->kernel >= 2 && !plan->cluster_merge && desc->batch <= 256 &&
                           (long)desc->batch * splits > dev.sm_count / 2)
                              ? 1
                              : 0;
    DecodeParams shape = {};
    shape.q = static_cast<const __nv_bfloat16 *>(q);
    shape.kv = static_cast<const __nv_bfloat16 *>(kv_cache);
    shape.num_pages = desc->num_pages;
    shape.batch = desc->batch;
    shape.heads = desc->num_heads;
    if (plan->kernel == 3) {
        if (!tc2q8_prepare_device() || !tc2q8_make_maps(shape, plan->maps, cached_maps)) return OMNI_ERR_CUDA;
    } else if (plan->kernel == 2) {
        if (!tc2_prepare_device() || !tc2_make_maps(shape, plan->maps, cached_maps)) return OMNI_ERR_CUDA;
    } else if (plan->kernel == 1) {
        if (!tc_prepare_device() || !tc_make_maps(shape, plan->maps, cached_maps)) return OMNI_ERR_CUDA;
    }
    plan->magic = kPlanMagic;
    return OMNI_OK;
}

// Checks of the per-step arguments that need no device.
static omni_status_t check_step_args(const omni_mla_desc_t *desc, const int32_t *page_table, const int32_t *sel_idx,
                                     const int32_t *sel_len, const int32_t *ctx_len, int32_t n_sink, int32_t n_recent,
                                     bool rolling, const void *out, const float *lse)
{
    const bool ranges = sel_idx == nullptr;
    if (!page_table || !out || !lse) return OMNI_ERR_NULL;
    if (ranges ? !ctx_len : !sel_len) return OMNI_ERR_NULL;
    if (ranges) {
        // max_sel bounds the selection size the split plan is made for
        if (n_sink < 0 || n_recent < 0) return OMNI_ERR_SHAPE;
        const int64_t longest = (int64_t)desc->max_pages_per_req * kPage;
        // a rolling cache holds contexts of any length, so only N_sink + N_recent bounds the selection
        const int64_t bound = (rolling || (int64_t)n_sink + n_recent < longest) ? (int64_t)n_sink + n_recent : longest;
        if ((int64_t)desc->max_sel < bound) return OMNI_ERR_SHAPE;
        if (rolling && (int64_t)desc->max_pages_per_req < rolling_sink_pages(n_sink) + rolling_ring_pages(n_recent))
            return OMNI_ERR_SHAPE;
    }
    if (!aligned(out, 16) || !aligned(lse, 4) || !aligned(page_table, 4) || !aligned(sel_idx, 4) || !aligned(sel_len, 4) ||
        !aligned(ctx_len, 4))
        return OMNI_ERR_ALIGN;
    return OMNI_OK;
}

// The per-call half: pointer checks, workspace carving, launches.  The selection is an index
// list (sel_idx, sel_len) or, with sel_idx == nullptr, Eq. 2's ranges (ctx_len, n_sink, n_recent).
static omni_status_t run_plan(const LaunchPlan &plan, const int32_t *page_table, const int32_t *sel_idx,
                              const int32_t *sel_len, const int32_t *ctx_len, int32_t n_sink, int32_t n_recent,
                              bool rolling, void *out, float *lse, void *workspace, size_t workspace_bytes,
                              int32_t *device_status, void *stream_)
{
    const omni_mla_desc_t *desc = &plan.desc;
    const bool ranges = sel_idx == nullptr;
    omni_status_t args = check_step_args(desc, page_table, sel_idx, sel_len, ctx_len, n_sink, n_recent, rolling, out, lse);
    if (args != OMNI_OK) return args;
    const int splits = plan.splits;
    if (splits > 1) {
        if (!workspace) return OMNI_ERR_NULL;
        if (!aligned(workspace, 256)) return OMNI_ERR_ALIGN;
        if (workspace_bytes < plan.need) return OMNI_ERR_WORKSPACE;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    if ((desc->flags & OMNI_FLAG_VALIDATE) && !ranges) {
        omni_status_t st = launch_resolve(desc, page_table, sel_idx, sel_len, nullptr, device_status, stream);
        if (st != OMNI_OK) return st;
    }

    DecodeParams p;
    p.q = static_cast<const __nv_bfloat16 *>(plan.q);
    p.kv = static_cast<const __nv_bfloat16 *>(plan.kv);
    p.kv_scale = plan.kv_scale;
    p.page_table = page_table;
    p.sel_idx = sel_idx;
    p.sel_len = sel_len;
    p.ctx_len = ctx_len;
    p.n_sink = n_sink;
    p.n_recent = n_recent;
    p.sink_pages = rolling ? (int32_t)rolling_sink_pages(n_sink) : 0;
    p.ring_pages = rolling ? (int32_t)rolling_ring_pages(n_recent) : 0;
    p.out = static_cast<__nv_bfloat16 *>(out);
    p.lse = lse;
    p.part_out = static_cast<float *>(workspace);
    p.part_lse = splits > 1 ? reinterpret_cast<float *>(static_cast<char *>(workspace) + plan.part_out) : nullptr;
    p.status = device_status;
    p.counters = nullptr;
    p.cluster_merge = plan.cluster_merge;
    p.longest_first = plan.longest_first;
    if (plan.fused_merge) {
        p.counters = reinterpret_cast<int32_t *>(static_cast<char *>(workspace) + plan.part_out + plan.part_lse);
        if (cudaMemsetAsync(p.counters, 0, plan.counters, stream) != cudaSuccess) return OMNI_ERR_CUDA;
    }
    p.num_pages = desc->num_pages;
    p.batch = desc->batch;
    p.heads = desc->num_heads;
    p.max_pages = desc->max_pages_per_req;
    p.max_sel = desc->max_sel;
    p.splits = splits;
    p.scale_log2 = desc->softmax_scale * kLog2e;

    const bool profile = g_profile_before && g_profile_after;
    if (profile) cudaEventRecord(g_profile_before, stream);
    omni_status_t st = OMNI_OK;
    if (plan.kernel == 0) {
        const int grid = desc->batch * splits * units_per_request(desc);
        simt_decode_kernel<<<grid, kSimtWarps * 32, 0, stream>>>(p);
        if (cudaPeekAtLastError() != cudaSuccess) st = OMNI_ERR_CUDA;
    } else {
        st = plan.kernel == 3   ? tc2q8_launch(plan.maps, p, stream)
             : plan.kernel == 2 ? tc2_launch(plan.maps, p, stream)
                                : tc_launch(plan.maps, p, stream);
    }
    if (st != OMNI_OK) return st;
    if (profile) cudaEventRecord(g_profile_after, stream);
    if (splits > 1 && p.counters == nullptr && !p.cluster_merge)
        return launch_combine(desc->batch, desc->num_heads, splits, p.part_out, p.part_lse, nullptr,
                              out, lse, stream);
    return OMNI_OK;
}

static omni_status_t decode_impl(const omni_mla_desc_t *desc, const void *q, const void *kv_cache,
                                 const int32_t *page_table, const int32_t *sel_idx,
                                 const int32_t *sel_len, const int32_t *ctx_len, int32_t n_sink,
                                 int32_t n_recent, bool rolling, void *out, float *lse, void *workspace,
                                 size_t workspace_bytes, int32_t *device_status, void *stream)
{
    // everything the host can check is checked before the device is asked anything
    if (!desc || !q || !kv_cache || !page_table || !out || !lse) return OMNI_ERR_NULL;
    if (sel_idx == nullptr ? !ctx_len : !sel_len) return OMNI_ERR_NULL;
    if (!desc_ok(desc)) return OMNI_ERR_SHAPE;
    omni_status_t st = check_step_args(desc, page_table, sel_idx, sel_len, ctx_len, n_sink, n_recent, rolling, out, lse);
    if (st == OMNI_OK && (!aligned(q, 16) || !aligned(kv_cache, 128))) st = OMNI_ERR_ALIGN;
    if (st != OMNI_OK) return st;
    LaunchPlan plan;
    st = build_plan(desc, q, kv_cache, true, &plan);
    if (st != OMNI_OK) return st;
    return run_plan(plan, page_table, sel_idx, sel_len, ctx_len, n_sink, n_recent, rolling, out, lse, workspace,
                    workspace_bytes, device_status, stream);
}

omni_status_t omni_sparse_mla_decode_q8(const omni_mla_desc_t *desc, const void *q, const void *kv_q8,
                                        const float *kv_scale, const int32_t *page_table, const int32_t *sel_idx,
                                        const int32_t *sel_len, void *out, float *lse, void *workspace,
                                        size_t workspace_bytes, int32_t *device_status, void *stream)
{
    if (!desc || !q || !kv_q8 || !kv_scale || !page_table || !sel_idx || !sel_len || !out || !lse) return OMNI_ERR_NULL;
    if (!desc_ok(desc) || !use_pair_kernel(desc)) return OMNI_ERR_SHAPE;
    omni_status_t st = check_step_args(desc, page_table, sel_idx, sel_len, nullptr, 0, 0, false, out, lse);
    if (st == OMNI_OK && (!aligned(q, 16) || !aligned(kv_q8, 128) || !aligned(kv_scale, 4))) st = OMNI_ERR_ALIGN;
    if (st != OMNI_OK) return st;
    LaunchPlan plan;
    st = build_plan(desc, q, kv_q8, true, &plan, kv_scale, true);
    if (st != OMNI_OK) return st;
    return run_plan(plan, page_table, sel_idx, sel_len, nullptr, 0, 0, false, out, lse, workspace, workspace_bytes,
                    device_status, stream);
}

omni_status_t omni_kv_quantize_q8(const void *kv_rows, int64_t num_rows, void *kv_q8, float *kv_scale, void *stream)
{
    if (!kv_rows || !kv_q8 || !kv_scale) return OMNI_ERR_NULL;
    if (num_rows < 1 || num_rows > (int64_t)0x7fffffff * 8) return OMNI_ERR_SHAPE;
    if (!aligned(kv_rows, 16) || !aligned(kv_q8, 128) || !aligned(kv_scale, 4)) return OMNI_ERR_ALIGN;
    const unsigned blocks = (unsigned)((num_rows + 7) / 8);
    quantize_q8_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const __nv_bfloat16 *>(kv_rows), num_rows, static_cast<uint8_t *>(kv_q8), kv_scale);
    return cudaPeekAtLastError() == cudaSuccess ? OMNI_OK : OMNI_ERR_CUDA;
}

omni_status_t omni_sparse_mla_plan_init(const omni_mla_desc_t *desc, const void *q, const void *kv_cache,
                                        omni_mla_plan_t *plan)
{
    if (!plan) return OMNI_ERR_NULL;
    if (!aligned(plan, 64)) return OMNI_ERR_ALIGN;
    LaunchPlan *lp = reinterpret_cast<LaunchPlan *>(plan);
    lp->magic = 0;
    return build_plan(desc, q, kv_cache, false, lp);
}

omni_status_t omni_sparse_mla_decode_planned(const omni_mla_plan_t *plan, const int32_t *page_table,
                                             const int32_t *sel_idx, const int32_t *sel_len, void *out,
                                             float *lse, void *workspace, size_t workspace_bytes,
                                             int32_t *device_status, void *stream)
{
    if (!plan || !sel_idx) return OMNI_ERR_NULL;
    if (!aligned(plan, 64)) return OMNI_ERR_ALIGN;
    const LaunchPlan *lp = reinterpret_cast<const LaunchPlan *>(plan);
    if (lp->magic != kPlanMagic) return OMNI_ERR_SHAPE;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != lp->device) return OMNI_ERR_CUDA;
    return run_plan(*lp, page_table, sel_idx, sel_len, nullptr, 0, 0, false, out, lse, workspace, workspace_bytes,
                    device_status, stream);
}

omni_status_t omni_sparse_mla_decode(const omni_mla_desc_t *desc, const void *q,
                                     const void *kv_cache, const int32_t *page_table,
                                     const int32_t *sel_idx, const int32_t *sel_len, void *out,
                                     float *lse, void *workspace, size_t workspace_bytes,
                                     int32_t *device_status, void *stream)
{
    if (!sel_idx) return OMNI_ERR_NULL;
    return decode_impl(desc, q, kv_cache, page_table, sel_idx, sel_len, nullptr, 0, 0, false, out, lse, workspace,
                       workspace_bytes, device_status, stream);
}

omni_status_t omni_sparse_mla_decode_sink_recent(const omni_mla_desc_t *desc, const void *q,
                                                 const void *kv_cache, const int32_t *page_table,
                                                 const int32_t *ctx_len, int32_t n_sink,
                                                 int32_t n_recent, void *out, float *lse,
                                                 void *workspace, size_t workspace_bytes,
                                                 int32_t *device_status, void *stream)
{
    return decode_impl(desc, q, kv_cache, page_table, nullptr, nullptr, ctx_len, n_sink, n_recent, false, out, lse,
                       workspace, workspace_bytes, device_status, stream);
}

omni_status_t omni_sparse_mla_decode_rolling(const omni_mla_desc_t *desc, const void *q,
                                             const void *kv_cache, const int32_t *page_table,
                                             const int32_t *ctx_len, int32_t n_sink, int32_t n_recent,
                                             void *out, float *lse, void *workspace,
                                             size_t workspace_bytes, int32_t *device_status, void *stream)
{
    return decode_impl(desc, q, kv_cache, page_table, nullptr, nullptr, ctx_len, n_sink, n_recent, true, out, lse,
                       workspace, workspace_bytes, device_status, stream);
}

omni_status_t omni_topk_select(const float *scores, const int32_t *ctx_len, int32_t batch, int32_t stride,
                               int32_t k, int32_t *sel_idx, int32_t *sel_len, void *stream)
{
    if (!scores || !ctx_len || !sel_idx || !sel_len) return OMNI_ERR_NULL;
    if (batch < 1 || stride < 1 || stride > kTopkMaxContext || k < 1 || k > stride) return OMNI_ERR_SHAPE;
    if (!aligned(scores, 4) || !aligned(ctx_len, 4) || !aligned(sel_idx, 4) || !aligned(sel_len, 4)) return OMNI_ERR_ALIGN;
    const DeviceInfo &dev = device_info();
    if (!dev.ok) return OMNI_ERR_CUDA;
    if (dev.cc_major != 10) return OMNI_ERR_ARCH;
    return launch_topk_select(scores, ctx_len, batch, stride, k, sel_idx, sel_len, static_cast<cudaStream_t>(stream));
}

int32_t omni_rolling_pages_per_request(int32_t n_sink, int32_t n_recent)
{
    if (n_sink < 0 || n_recent < 0) return 0;
    const int64_t pages = rolling_sink_pages(n_sink) + rolling_ring_pages(n_recent);
    return pages > 0x7fffffff ? 0 : (int32_t)pages;
}

omni_status_t omni_kv_append_rolling(const omni_mla_desc_t *desc, void *kv_cache,
                                     const int32_t *page_table, const int32_t *ctx_len,
                                     const void *new_rows, int32_t n_sink, int32_t n_recent,
                                     int32_t *device_status, void *stream)
{
    if (!desc || !kv_cache || !page_table || !ctx_len || !new_rows) return OMNI_ERR_NULL;
    if (!desc_ok(desc) || n_sink < 0 || n_recent < 0) return OMNI_ERR_SHAPE;
    if ((int64_t)desc->max_pages_per_req < rolling_sink_pages(n_sink) + rolling_ring_pages(n_recent)) return OMNI_ERR_SHAPE;
    if (!aligned(kv_cache, 128) || !aligned(new_rows, 16) || !aligned(page_table, 4) || !aligned(ctx_len, 4))
        return OMNI_ERR_ALIGN;
    append_rolling_kernel<<<(unsigned)desc->batch, 72, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<__nv_bfloat16 *>(kv_cache), page_table, ctx_len, static_cast<const __nv_bfloat16 *>(new_rows),
        desc->max_pages_per_req, desc->num_pages, (int)rolling_sink_pages(n_sink), (int)rolling_ring_pages(n_recent),
        device_status);
    return cudaPeekAtLastError() == cudaSuccess ? OMNI_OK : OMNI_ERR_CUDA;
}

omni_status_t omni_sparse_mla_combine(const omni_mla_desc_t *desc, int32_t max_splits,
                                      const float *part_out, const float *part_lse,
                                      const int32_t *num_splits, void *out, float *lse,
                                      void *stream)
{
    if (!desc || !part_out || !part_lse || !out || !lse) return OMNI_ERR_NULL;
    if (desc->batch < 1 || desc->num_heads < 1 || desc->d_v != kDv || max_splits < 1)
        return OMNI_ERR_SHAPE;
    if (!aligned(part_out, 16) || !aligned(out, 8) || !aligned(part_lse, 4) || !aligned(lse, 4))
        return OMNI_ERR_ALIGN;
    return launch_combine(desc->batch, desc->num_heads, max_splits, part_out, part_lse, num_splits,
                          out, lse, static_cast<cudaStream_t>(stream));
}

omni_status_t omni_selftest_bounded_wait(int64_t limit_cycles, int32_t *device_status, int64_t *waited_cycles,
                                         void *stream)
{
    if (!device_status) return OMNI_ERR_NULL;
    if (limit_cycles < 1 || limit_cycles > ((int64_t)1 << 31)) return OMNI_ERR_SHAPE;
    if (!aligned(device_status, 4) || !aligned(waited_cycles, 8)) return OMNI_ERR_ALIGN;
    bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
        (long long)limit_cycles, device_status, reinterpret_cast<long long *>(waited_cycles));
    return cudaPeekAtLastError() == cudaSuccess ? OMNI_OK : OMNI_ERR_CUDA;
}

omni_status_t omni_sparse_mla_validate(const omni_mla_desc_t *desc, const int32_t *page_table,
                                       const int32_t *sel_idx, const int32_t *sel_len,
                                       int32_t *device_status, void *stream)
{
    if (!desc || !page_table || !sel_idx || !sel_len || !device_status) return OMNI_ERR_NULL;
    if (!desc_ok(desc)) return OMNI_ERR_SHAPE;
    return launch_resolve(desc, page_table, sel_idx, sel_len, nullptr, device_status,
                          static_cast<cudaStream_t>(stream));
}

omni_status_t omni_sparse_mla_resolve_rows(const omni_mla_desc_t *desc,
                                           const int32_t *page_table, const int32_t *sel_idx,
                                           const int32_t *sel_len, int64_t *rows, void *stream)
{
    if (!desc || !page_table || !sel_idx || !sel_len || !rows) return OMNI_ERR_NULL;
    if (!desc_ok(desc)) return OMNI_ERR_SHAPE;
    return launch_resolve(desc, page_table, sel_idx, sel_len, rows, nullptr,
                          static_cast<cudaStream_t>(stream));
}


// The host-buffer entry point splits a large batch into two parts so that the second part's
// host-to-device copies run under the first half's kernel, and the first half's device-to-host
// copies under the second half's kernel (PCIe carries both directions at once).  The second half
// runs on a stream of the library's own, which forks from and joins back into the caller's.
static size_t host_copy_bytes(const omni_mla_desc_t *desc)
{
    const size_t B = desc->batch, H = desc->num_heads;
    return align_up(B * H * kDqk * 2, 256) + align_up(B * desc->max_pages_per_req * 4, 256) +
           align_up(B * desc->max_sel * 4, 256) + align_up(B * 4, 256) +
           align_up(B * H * kDv * 2, 256) + align_up(B * H * 4, 256);
}

static bool host_pipelined(const omni_mla_desc_t *desc)
{
    const size_t B = desc->batch, H = desc->num_heads;
    return desc->batch >= 4 && B * H * (kDqk + kDv) * 2 >= (size_t)(2u << 20);
}

static omni_mla_desc_t host_half_desc(const omni_mla_desc_t *desc, int half)
{
    omni_mla_desc_t d = *desc;
    const int first = (desc->batch + 1) / 2;       // even halves measured better than 5/8 : 3/8
    d.batch = half == 0 ? first : desc->batch - first;
    return d;
}

static size_t host_half_workspace(const omni_mla_desc_t *desc, int half)
{
    const omni_mla_desc_t d = host_half_desc(desc, half);
    return align_up(workspace_need(&d, choose_splits(&d, device_info().sm_count)), 256);
}

// Side streams of the host-buffer entry point: a few per device, chosen by the caller's stream, so
// that calls in flight on different streams do not queue their second halves behind one another.
constexpr int kHostSideStreams = 4;
static cudaStream_t host_side_stream(cudaStream_t caller)
{
    static std::mutex lock;
    static cudaStream_t streams[64][kHostSideStreams] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    const uintptr_t h = reinterpret_cast<uintptr_t>(caller);
    const int slot = (int)(((h >> 4) ^ (h >> 12) ^ (h >> 20)) % kHostSideStreams);
    std::lock_guard<std::mutex> guard(lock);
    if (!streams[dev][slot] && cudaStreamCreateWithFlags(&streams[dev][slot], cudaStreamNonBlocking) != cudaSuccess)
        streams[dev][slot] = nullptr;
    return streams[dev][slot];
}

size_t omni_sparse_mla_host_staging_bytes(const omni_mla_desc_t *desc)
{
    if (!desc_ok(desc)) return 0;
    size_t n = host_copy_bytes(desc);
    if (host_pipelined(desc)) n += host_half_workspace(desc, 0) + host_half_workspace(desc, 1);
    return n;
}

omni_status_t omni_sparse_mla_decode_host(const omni_mla_desc_t *desc, const void *q_host,
                                          const void *kv_cache,
                                          const int32_t *page_table_host,
                                          const int32_t *sel_idx_host,
                                          const int32_t *sel_len_host, void *out_host,
                                          float *lse_host, void *staging, size_t staging_bytes,
                                          void *workspace, size_t workspace_bytes,
                                          int32_t *device_status, void *stream_)
{
    if (!desc || !q_host || !kv_cache || !page_table_host || !sel_idx_host || !sel_len_host ||
        !out_host || !lse_host || !staging)
        return OMNI_ERR_NULL;
    if (!desc_ok(desc)) return OMNI_ERR_SHAPE;
    if (!aligned(staging, 256)) return OMNI_ERR_ALIGN;
    if (staging_bytes < omni_sparse_mla_host_staging_bytes(desc)) return OMNI_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const size_t B = desc->batch, H = desc->num_heads;
    const size_t rq = H * kDqk * 2, rpt = (size_t)desc->max_pages_per_req * 4, rsi = (size_t)desc->max_sel * 4,
                 rsl = 4, rout = H * kDv * 2, rlse = H * 4;                      // bytes per request
    char *base = static_cast<char *>(staging);
    char *dq = base;
    char *dpt = dq + align_up(B * rq, 256);
    char *dsi = dpt + align_up(B * rpt, 256);
    char *dsl = dsi + align_up(B * rsi, 256);
    char *dout = dsl + align_up(B * rsl, 256);
    char *dlse = dout + align_up(B * rout, 256);
    char *half_ws = dlse + align_up(B * rlse, 256);

    auto h2d = [](void *dst, const void *src, size_t n, cudaStream_t s) {
        return cudaMemcpyAsync(dst, src, n, cudaMemcpyHostToDevice, s) == cudaSuccess;
    };
    // the three index arrays of all requests (small: one copy each)
    auto copy_indices = [&](cudaStream_t s) {
        return h2d(dpt, page_table_host, B * rpt, s) && h2d(dsi, sel_idx_host, B * rsi, s) && h2d(dsl, sel_len_host, B * rsl, s);
    };
    auto copy_q = [&](size_t b0, size_t n, cudaStream_t s) {
        return h2d(dq + b0 * rq, static_cast<const char *>(q_host) + b0 * rq, n * rq, s);
    };
    // requests [b0, b0 + d.batch) on stream s: decode and copies out
    auto decode_and_copy_out = [&](const omni_mla_desc_t &d, size_t b0, void *ws, size_t ws_bytes, cudaStream_t s) -> omni_status_t {
        const size_t n = d.batch;
        omni_status_t st = omni_sparse_mla_decode(
            &d, dq + b0 * rq, kv_cache, reinterpret_cast<int32_t *>(dpt + b0 * rpt), reinterpret_cast<int32_t *>(dsi + b0 * rsi),
            reinterpret_cast<int32_t *>(dsl + b0 * rsl), dout + b0 * rout, reinterpret_cast<float *>(dlse + b0 * rlse), ws,
            ws_bytes, device_status, s);
        if (st != OMNI_OK) return st;
        if (cudaMemcpyAsync(static_cast<char *>(out_host) + b0 * rout, dout + b0 * rout, n * rout, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaMemcpyAsync(reinterpret_cast<char *>(lse_host) + b0 * rlse, dlse + b0 * rlse, n * rlse, cudaMemcpyDeviceToHost, s) != cudaSuccess)
            return OMNI_ERR_CUDA;
        return OMNI_OK;
    };

    cudaStream_t side = host_pipelined(desc) ? host_side_stream(stream) : nullptr;
    if (!side) {
        if (!copy_q(0, B, stream) || !copy_indices(stream)) return OMNI_ERR_CUDA;
        return decode_and_copy_out(*desc, 0, workspace, workspace_bytes, stream);
    }
    const omni_mla_desc_t first = host_half_desc(desc, 0), second = host_half_desc(desc, 1);
    const size_t ws0 = host_half_workspace(desc, 0), ws1 = host_half_workspace(desc, 1);
    cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};     // first q in | indices in | second half done
    for (int e = 0; e < 3; ++e)
        if (cudaEventCreateWithFlags(&ev[e], cudaEventDisableTiming) != cudaSuccess) {
            for (int f = 0; f < e; ++f) cudaEventDestroy(ev[f]);
            return OMNI_ERR_CUDA;
        }
    // caller's stream: q of the first half | indices | kernel | copies out           | join
    // side stream:                         | q of the second half     | kernel | copies out
    bool ok = copy_q(0, (size_t)first.batch, stream) && cudaEventRecord(ev[0], stream) == cudaSuccess &&
              cudaStreamWaitEvent(side, ev[0], 0) == cudaSuccess;
    const bool forked = ok;
    ok = ok && copy_q((size_t)first.batch, (size_t)second.batch, side);
    ok = ok && copy_indices(stream) && cudaEventRecord(ev[1], stream) == cudaSuccess &&
         cudaStreamWaitEvent(side, ev[1], 0) == cudaSuccess;
    omni_status_t st = ok ? OMNI_OK : OMNI_ERR_CUDA;
    if (st == OMNI_OK) st = decode_and_copy_out(first, 0, half_ws, ws0, stream);
    if (st == OMNI_OK) st = decode_and_copy_out(second, (size_t)first.batch, half_ws + ws0, ws1, side);
    if (forked && (cudaEventRecord(ev[2], side) != cudaSuccess || cudaStreamWaitEvent(stream, ev[2], 0) != cudaSuccess))
        st = st != OMNI_OK ? st : OMNI_ERR_CUDA;
    for (int e = 0; e < 3; ++e) cudaEventDestroy(ev[e]);  // released by the runtime once the work that uses them is done
    return st;
}

}  // extern "C"
