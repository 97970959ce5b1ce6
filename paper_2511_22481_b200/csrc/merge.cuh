// In-kernel split-KV merge: the decode CTA that finishes a (request, head group) last combines
// the partial results of all splits, so the merge needs no second launch.
//
//     lse = ln sum_s exp(lse_s),   out = sum_s exp(lse_s - lse) * out_s
//
// Every CTA that produced a partial result calls merge_if_last with all of its threads after
// its own partial stores (each storing thread fences them).  A counter per (request, head
// group), zeroed by the host before the launch, tells the last arrival apart.
#pragma once

#include "common.cuh"

namespace omni {

constexpr int kMergeMaxSplits = 32;

// unit / units: head group of this CTA and head groups per request; h0, rows: its head range;
// scratch: at least rows * splits floats of shared memory nobody else uses any more;
// flag: a shared-memory word.
__device__ __forceinline__ void merge_if_last(const DecodeParams &p, int b, int unit, int units, int h0, int rows,
                                              float *scratch, uint32_t *flag)
{
    __syncthreads();                                   // every thread's partial stores are issued and fenced
    if (threadIdx.x == 0) {
        __threadfence();
        const int arrived = atomicAdd(p.counters + (size_t)b * units + unit, 1);
        *flag = (arrived == p.splits - 1) ? 1u : 0u;
    }
    __syncthreads();
    if (*flag == 0u) return;
    __threadfence();                                   // the other splits' stores are visible from here on

    const int S = p.splits;
    const int nthreads = (int)blockDim.x;
    // weights per (row, split), final log-sum-exp per row
    for (int r = (int)threadIdx.x; r < rows; r += nthreads) {
        const float *pl = p.part_lse + (size_t)b * S * p.heads + h0 + r;
        float mx = -INFINITY;
        for (int s = 0; s < S; ++s) mx = fmaxf(mx, __ldcg(pl + (size_t)s * p.heads));
        float total = -INFINITY;
        if (mx > -INFINITY) {
            float z = 0.f;
            for (int s = 0; s < S; ++s) z += exp2f((__ldcg(pl + (size_t)s * p.heads) - mx) * kLog2e);
            total = mx + logf(z);
        }
        for (int s = 0; s < S; ++s) {
            const float ls = __ldcg(pl + (size_t)s * p.heads);
            scratch[r * S + s] = (ls == -INFINITY || total == -INFINITY) ? 0.f : exp2f((ls - total) * kLog2e);
        }
        p.lse[(size_t)b * p.heads + h0 + r] = total;
    }
    __syncthreads();

    // items: (row, group of four value columns); four items per thread in flight
    constexpr int kCols4 = kDv / 4;
    const int total_items = rows * kCols4;
    const float4 *part = reinterpret_cast<const float4 *>(p.part_out);
    for (int base = (int)threadIdx.x; base < total_items; base += 4 * nthreads) {
        float4 acc[4];
        size_t src[4];
        int rr[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int item = min(base + k * nthreads, total_items - 1);
            rr[k] = item / kCols4;
            src[k] = ((size_t)b * S * p.heads + h0 + rr[k]) * kCols4 + item % kCols4;
            acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (int s = 0; s < S; ++s) {
            float4 v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) v[k] = __ldcg(part + src[k] + (size_t)s * p.heads * kCols4);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float w = scratch[rr[k] * S + s];
                acc[k].x = fmaf(w, v[k].x, acc[k].x);
                acc[k].y = fmaf(w, v[k].y, acc[k].y);
                acc[k].z = fmaf(w, v[k].z, acc[k].z);
                acc[k].w = fmaf(w, v[k].w, acc[k].w);
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int item = base + k * nthreads;
            if (item >= total_items) break;
            __nv_bfloat162 lo = __floats2bfloat162_rn(acc[k].x, acc[k].y), hi = __floats2bfloat162_rn(acc[k].z, acc[k].w);
            uint2 packed;
            packed.x = *reinterpret_cast<uint32_t *>(&lo);
            packed.y = *reinterpret_cast<uint32_t *>(&hi);
            reinterpret_cast<uint2 *>(p.out + ((size_t)b * p.heads + h0 + rr[k]) * kDv)[item % kCols4] = packed;
        }
    }
}

}  // namespace omni
