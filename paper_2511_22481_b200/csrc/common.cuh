// Shared device-side definitions of the sparse MLA decode kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "omni_mla.h"

namespace omni {

constexpr int kDqk = 576;        // latent row: 512 "nope" + 64 rope columns, all used as K
constexpr int kDv = 512;         // the first 512 columns of the same row are V
constexpr int kPage = 64;        // tokens per page
constexpr int kTile = 64;        // tokens per split-KV granule (split boundaries fall on these)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Everything a kernel needs to find its data; passed by value.
struct DecodeParams {
    const __nv_bfloat16 *q;        // [B, H, 576]
    const __nv_bfloat16 *kv;       // [num_pages * 64, 576]; the 8-bit kernel: bytes [num_pages * 64, 640]
    const float *kv_scale;         // 8-bit cache only: one scale per pool row
    const int32_t *page_table;     // [B, max_pages]
    const int32_t *sel_idx;        // [B, max_sel]; null: the selection is Eq. 2's two ranges
    const int32_t *sel_len;        // [B]
    const int32_t *ctx_len;        // [B] context length in tokens (range selection only)
    int32_t n_sink, n_recent;      // Eq. 2's N_sink and N_recent (range selection only)
    int32_t sink_pages, ring_pages; // rolling cache of a compressed layer (ring_pages > 0), see rolling_position
    __nv_bfloat16 *out;            // [B, H, 512]
    float *lse;                    // [B, H]
    float *part_out;               // [B, S, H, 512]  (S > 1 only)
    float *part_lse;               // [B, S, H]
    int32_t *status;               // may be null
    int32_t *counters;             // [B, head groups] arrivals per merge unit, zeroed before the
                                   // launch; null: the caller merges with a kernel of its own
    int64_t num_pages;
    int32_t batch, heads, max_pages, max_sel, splits;
    int32_t cluster_merge;         // 1: two splits, merged inside a cluster of two CTA pairs
    int32_t longest_first;         // 1: work units take the requests in order of decreasing selection size
    float scale_log2;              // softmax_scale * log2(e)
};

// Token range [begin, end) of split s of a request with n selected tokens: the n tokens are
// cut into granules (64 tokens unless a kernel works on larger tiles) and the granules are
// dealt out in contiguous, equal runs.
__device__ __forceinline__ void split_range(int n, int splits, int s, int &begin, int &end,
                                            int granule = kTile)
{
    const int granules = (n + granule - 1) / granule;
    const int per = (granules + splits - 1) / splits;
    begin = min(n, s * per * granule);
    end = min(n, (s + 1) * per * granule);
}

// Rolling cache of a compressed layer.  Such a layer only ever attends to the first N_sink and
// the last N_recent tokens (Eq. 2), so it stores nothing else: `sink_pages` pages hold positions
// [0, 64 * sink_pages) for good, and `ring_pages` = ceil(N_recent / 64) + 1 further pages are
// reused round-robin by all later 64-token blocks of the context.  A token at absolute position t
// lives at this position of the request's (short) page table:
__host__ __device__ __forceinline__ int32_t rolling_position(int32_t t, int32_t sink_pages, int32_t ring_pages)
{
    const int32_t block = t / kPage;
    if (block < sink_pages) return t;
    return (sink_pages + (block - sink_pages) % ring_pages) * kPage + t % kPage;
}

// The selection of one request: the caller's index list, or the index set of Eq. 2 of the
// paper (attention sink + recent tokens) kept as two ranges, [0, ns) and [rs, M), so that no
// index list has to exist in memory.  Entry j of the selection is list[j] or, for ranges, j
// itself below ns and a position of the recent range from `vstart` on.  Between the two ranges
// up to 63 padding entries (kSelectionPad: "no token", weight zero, not an error) shift the
// recent range so that position t sits at offset t mod 64 of its 64-entry tile: the tiles of the
// recent window then coincide with pages and are loaded as boxes wherever the window starts,
// instead of every tile straddling two pages.
constexpr int32_t kSelectionPad = -2;
struct Selection {
    const int32_t *list;   // null for ranges
    int n;                 // entries (selected tokens, plus padding for ranges)
    int ns, rs;            // ranges only: end of the sink range, start of the recent range
    int vstart;            // ranges only: entry of position rs
    int sink_pages, ring_pages;   // ranges over a rolling cache (ring_pages > 0)
    bool bad;              // the length breaks the contract (n was set to 0)
    uint64_t keep;         // L2 policy of the index loads (see ldg_index)
};

// Index data (token positions, page ids) is a few bytes per token and is read by several warps of
// both CTAs that serve a request; the cache rows stream through L2 at a thousand times the volume
// and would push it out between two uses.  Its loads therefore ask L2 to evict these lines last.
__device__ __forceinline__ uint64_t index_load_policy()
{
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
__device__ __forceinline__ int32_t ldg_index(const int32_t *ptr, uint64_t policy)
{
    int32_t v;
    asm volatile("ld.global.nc.L2::cache_hint.b32 %0, [%1], %2;" : "=r"(v) : "l"(ptr), "l"(policy));
    return v;
}

__device__ __forceinline__ Selection load_selection(const DecodeParams &p, int b)
{
    Selection s;
    s.bad = false;
    s.ns = s.rs = s.vstart = 0;
    s.sink_pages = p.sink_pages;
    s.ring_pages = p.ring_pages;
    s.keep = index_load_policy();
    if (p.sel_idx != nullptr) {
        s.list = p.sel_idx + (size_t)b * p.max_sel;
        s.n = __ldg(p.sel_len + b);
        if (s.n < 0 || s.n > p.max_sel) {
            s.bad = true;
            s.n = 0;
        }
    } else {
        s.list = nullptr;
        int m = __ldg(p.ctx_len + b);
        // a rolling cache holds contexts of any length in its few pages
        if (m < 0 || (p.ring_pages == 0 && (int64_t)m > (int64_t)p.max_pages * kPage)) {
            s.bad = true;
            m = 0;
        }
        // 0-based Eq. 2: [0, N_sink) united with [M - N_recent, M); where the two overlap, the
        // union without repeats
        s.ns = min(p.n_sink, m);
        s.rs = max(s.ns, m - min(p.n_recent, m));
        s.vstart = s.ns + (m > s.rs ? ((s.rs - s.ns) % kPage) : 0);
        s.n = s.vstart + (m - s.rs);
    }
    return s;
}

// Whether entry value t is range padding ("no token") rather than a position the caller wrote:
// only the range form pads, so in an index list -2 is a negative position like any other and
// breaks the index contract.
__device__ __forceinline__ bool is_padding(const Selection &s, int32_t t)
{
    return s.list == nullptr && t == kSelectionPad;
}

__device__ __forceinline__ int32_t selection_at(const Selection &s, int j)
{
    if (s.list != nullptr) return ldg_index(s.list + j, s.keep);
    if (j >= s.ns && j < s.vstart) return kSelectionPad;
    const int32_t t = j < s.ns ? j : s.rs + (j - s.vstart);
    return s.ring_pages > 0 ? rolling_position(t, s.sink_pages, s.ring_pages) : t;
}

// Logical token position -> physical pool row, or -1 if the entry breaks the index contract.
__device__ __forceinline__ int64_t resolve_row(const int32_t *page_table_row, int32_t t,
                                               int32_t max_pages, int64_t num_pages)
{
    if (t < 0) return -1;
    const int32_t lp = t / kPage;
    if (lp >= max_pages) return -1;
    const int32_t page = __ldg(page_table_row + lp);
    if (page < 0 || (int64_t)page >= num_pages) return -1;
    return (int64_t)page * kPage + (t % kPage);
}

// 2^x for the softmax weights: the hardware approximation alone (ex2.approx.ftz, about 2 ulp,
// -inf gives 0, results below 2^-126 are flushed to 0), where exp2f adds a range-scaling sequence
// around it for subnormal results, four more instructions per weight in the hottest loop.  A
// weight that small contributes nothing at the precision the weights are kept in.
__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void flag_status(int32_t *status, int32_t bits)
{
    if (status != nullptr) atomicOr(status, bits);
}

}  // namespace omni
