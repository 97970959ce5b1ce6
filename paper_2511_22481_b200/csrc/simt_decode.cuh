// Bring-up kernel: the whole decode path with plain FMA arithmetic, no tensor cores.
// One warp owns four heads of one (request, split); it walks the split's selected tokens
// one by one, so its index handling is easy to audit.  It is the second GPU opinion next
// to the tensor-core kernel and is selected with OMNI_FLAG_SIMT.
#pragma once

#include "common.cuh"

namespace omni {

constexpr int kSimtHeadsPerWarp = 4;
constexpr int kSimtWarps = 4;

__device__ __forceinline__ float2 bf16x2_to_float2(uint32_t v)
{
    float2 r;
    r.x = __uint_as_float(v << 16);
    r.y = __uint_as_float(v & 0xffff0000u);
    return r;
}

__global__ void __launch_bounds__(kSimtWarps * 32) simt_decode_kernel(DecodeParams p)
{
    const int head_groups = (p.heads + kSimtWarps * kSimtHeadsPerWarp - 1) /
                            (kSimtWarps * kSimtHeadsPerWarp);
    const int hg = blockIdx.x % head_groups;
    const int s = (blockIdx.x / head_groups) % p.splits;
    const int b = blockIdx.x / (head_groups * p.splits);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h0 = (hg * kSimtWarps + warp) * kSimtHeadsPerWarp;
    if (h0 >= p.heads) return;

    const Selection selection = load_selection(p, b);
    const int n = selection.n;
    if (selection.bad && threadIdx.x == 0) flag_status(p.status, OMNI_DEV_BAD_INDEX);
    int begin, end;
    split_range(n, p.splits, s, begin, end);

    // lane owns column pairs lane + 32*i (i < 9) of the 288 bf16 pairs of a latent row;
    // the first 8 of them (pairs < 256) are value columns.
    float2 qr[kSimtHeadsPerWarp][9];
#pragma unroll
    for (int g = 0; g < kSimtHeadsPerWarp; ++g) {
        const int h = min(h0 + g, p.heads - 1);
        const uint32_t *qp = reinterpret_cast<const uint32_t *>(p.q + ((size_t)b * p.heads + h) * kDqk);
#pragma unroll
        for (int i = 0; i < 9; ++i) qr[g][i] = bf16x2_to_float2(__ldg(qp + lane + 32 * i));
    }
    float2 acc[kSimtHeadsPerWarp][8];
    float m[kSimtHeadsPerWarp], l[kSimtHeadsPerWarp];
#pragma unroll
    for (int g = 0; g < kSimtHeadsPerWarp; ++g) {
        m[g] = -INFINITY;
        l[g] = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[g][i] = make_float2(0.f, 0.f);
    }

    const int32_t *pt = p.page_table + (size_t)b * p.max_pages;
    for (int j = begin; j < end; ++j) {
        const int32_t t = selection_at(selection, j);
        if (is_padding(selection, t)) continue;
        const int64_t row = resolve_row(pt, t, p.max_pages, p.num_pages);
        if (row < 0) {
            if (lane == 0) flag_status(p.status, OMNI_DEV_BAD_INDEX);
            continue;
        }
        const uint32_t *kp = reinterpret_cast<const uint32_t *>(p.kv + (size_t)row * kDqk);
        float2 kr[9];
#pragma unroll
        for (int i = 0; i < 9; ++i) kr[i] = bf16x2_to_float2(__ldg(kp + lane + 32 * i));
#pragma unroll
        for (int g = 0; g < kSimtHeadsPerWarp; ++g) {
            float d = 0.f;
#pragma unroll
            for (int i = 0; i < 9; ++i) d = fmaf(qr[g][i].x, kr[i].x, fmaf(qr[g][i].y, kr[i].y, d));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
            const float x = d * p.scale_log2;
            const float mn = fmaxf(m[g], x);
            const float corr = exp2f(m[g] - mn);       // exp2f(-inf) == 0 on the first token
            const float w = exp2f(x - mn);
            m[g] = mn;
            l[g] = l[g] * corr + w;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                acc[g][i].x = fmaf(w, kr[i].x, acc[g][i].x * corr);
                acc[g][i].y = fmaf(w, kr[i].y, acc[g][i].y * corr);
            }
        }
    }

#pragma unroll
    for (int g = 0; g < kSimtHeadsPerWarp; ++g) {
        const int h = h0 + g;
        if (h >= p.heads) break;
        const float inv = l[g] > 0.f ? 1.f / l[g] : 0.f;
        const float lse = l[g] > 0.f ? (m[g] + log2f(l[g])) * kLn2 : -INFINITY;
        if (p.splits == 1) {
            __nv_bfloat162 *op = reinterpret_cast<__nv_bfloat162 *>(p.out + ((size_t)b * p.heads + h) * kDv);
#pragma unroll
            for (int i = 0; i < 8; ++i)
                op[lane + 32 * i] = __floats2bfloat162_rn(acc[g][i].x * inv, acc[g][i].y * inv);
            if (lane == 0) p.lse[(size_t)b * p.heads + h] = lse;
        } else {
            const size_t u = ((size_t)b * p.splits + s) * p.heads + h;
            float2 *op = reinterpret_cast<float2 *>(p.part_out + u * kDv);
#pragma unroll
            for (int i = 0; i < 8; ++i)
                op[lane + 32 * i] = make_float2(acc[g][i].x * inv, acc[g][i].y * inv);
            if (lane == 0) p.part_lse[u] = lse;
        }
    }
}

}  // namespace omni
