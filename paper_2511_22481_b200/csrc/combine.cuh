// Split-KV merge and the small index kernels (validation, row export).
#pragma once

#include "common.cuh"

namespace omni {

// One block per (request, head); thread t owns value columns 4t..4t+3.
// lse = ln sum_s exp(lse_s); out = sum_s exp(lse_s - lse) * out_s.
__global__ void __launch_bounds__(128) combine_kernel(const float *__restrict__ part_out,
                                                      const float *__restrict__ part_lse,
                                                      const int32_t *__restrict__ num_splits,
                                                      int max_splits, int heads,
                                                      __nv_bfloat16 *__restrict__ out,
                                                      float *__restrict__ lse)
{
    // no-op unless launched as a programmatic dependent: then wait for the producing kernel;
    // the kernel that follows may be scheduled early in turn (it waits before it reads)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int b = blockIdx.x / heads, h = blockIdx.x % heads;
    int ns = num_splits ? __ldg(num_splits + b) : max_splits;
    ns = max(0, min(ns, max_splits));
    const float *pl = part_lse + (size_t)b * max_splits * heads + h;
    float mx = -INFINITY;
    for (int s = 0; s < ns; ++s) mx = fmaxf(mx, __ldg(pl + (size_t)s * heads));
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float total = -INFINITY;
    if (mx > -INFINITY) {
        float z = 0.f;
        for (int s = 0; s < ns; ++s) z += exp2f((__ldg(pl + (size_t)s * heads) - mx) * kLog2e);
        total = mx + logf(z);
        for (int s = 0; s < ns; ++s) {
            const float ls = __ldg(pl + (size_t)s * heads);
            if (ls == -INFINITY) continue;
            const float w = exp2f((ls - total) * kLog2e);
            const float4 v = __ldg(reinterpret_cast<const float4 *>(
                                       part_out + (((size_t)b * max_splits + s) * heads + h) * kDv) +
                                   threadIdx.x);
            acc.x = fmaf(w, v.x, acc.x);
            acc.y = fmaf(w, v.y, acc.y);
            acc.z = fmaf(w, v.z, acc.z);
            acc.w = fmaf(w, v.w, acc.w);
        }
    }
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t *>(&lo);
    packed.y = *reinterpret_cast<uint32_t *>(&hi);
    reinterpret_cast<uint2 *>(out + ((size_t)b * heads + h) * kDv)[threadIdx.x] = packed;
    if (threadIdx.x == 0) lse[(size_t)b * heads + h] = total;
}

// rows[b][j] = physical row of the j-th selected token (-1 outside sel_len or on a contract
// violation); with rows == nullptr it only checks and flags.
__global__ void __launch_bounds__(256) resolve_rows_kernel(const int32_t *__restrict__ page_table,
                                                           const int32_t *__restrict__ sel_idx,
                                                           const int32_t *__restrict__ sel_len,
                                                           int max_pages, int max_sel,
                                                           int64_t num_pages, int64_t *rows,
                                                           int32_t *status)
{
    const int b = blockIdx.y;
    int n = __ldg(sel_len + b);
    bool bad = false;
    if (n < 0 || n > max_sel) {
        bad = true;
        n = 0;
    }
    for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < max_sel; j += gridDim.x * blockDim.x) {
        int64_t r = -1;
        if (j < n) {
            r = resolve_row(page_table + (size_t)b * max_pages, __ldg(sel_idx + (size_t)b * max_sel + j),
                            max_pages, num_pages);
            bad |= (r < 0);
        }
        if (rows) rows[(size_t)b * max_sel + j] = r;
    }
    if (bad) flag_status(status, OMNI_DEV_BAD_INDEX);
}

// Appends one latent row per request to the rolling cache of a compressed layer: the row of the
// token at absolute position ctx_len[b] goes to rolling_position(ctx_len[b]) of the request's
// page table.  72 threads per request, 16 bytes each.
__global__ void __launch_bounds__(72) append_rolling_kernel(__nv_bfloat16 *__restrict__ kv,
                                                            const int32_t *__restrict__ page_table,
                                                            const int32_t *__restrict__ ctx_len,
                                                            const __nv_bfloat16 *__restrict__ new_rows,
                                                            int max_pages, int64_t num_pages, int sink_pages,
                                                            int ring_pages, int32_t *status)
{
    const int b = blockIdx.x;
    const int32_t t = __ldg(ctx_len + b);
    int64_t row = -1;
    if (t >= 0) {
        const int32_t pos = rolling_position(t, sink_pages, ring_pages);
        row = resolve_row(page_table + (size_t)b * max_pages, pos, max_pages, num_pages);
    }
    if (row < 0) {
        if (threadIdx.x == 0) flag_status(status, OMNI_DEV_BAD_INDEX);
        return;
    }
    const uint4 *src = reinterpret_cast<const uint4 *>(new_rows + (size_t)b * kDqk);
    uint4 *dst = reinterpret_cast<uint4 *>(kv + (size_t)row * kDqk);
    dst[threadIdx.x] = __ldg(src + threadIdx.x);
}

}  // namespace omni
