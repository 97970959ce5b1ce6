// Paired-CTA decode kernel over the 8-bit latent cache (sm_100a).
//
// Cache row of a token: 512 FP8 E4M3 codes (the latent columns), then the 64 rope columns as
// bf16 (128 bytes): 640 bytes, five 128-byte panels.  One fp32 scale per row in a separate array:
// latent value = code * scale.  The result is attention over those de-quantised rows.
//
// The kernel keeps the structure of tc2_decode_kernel (a CTA pair = all heads of one (request,
// split), cta_group::2 MMAs with M = 128, K role / V role loads, eight softmax warps) and changes
// what the 8-bit rows change:
//
//  * Scores.  The latent part runs on the 8-bit tensor-core kind (kind::f8f6f4, K = 32 per
//    instruction): S8 = Q8 K8^T.  q arrives as bf16; at the start of a work unit the softmax warps
//    rewrite its 512 latent columns as TWO E4M3 terms per value, hi = E4M3(q / a) and
//    lo = E4M3(q / a - hi), with a a power of two per head row, so that hi + lo carries the eight
//    significant bits of the bf16 value; both terms accumulate into the same S8.  The rope part
//    is an ordinary bf16 MMA (K = 64) into a second accumulator Sr, because S8 still has to be
//    multiplied by a[row] * scale[token]:  x = (a * scale_t * S8 + Sr) * softmax_scale.
//  * Weighted sum.  V = code * scale_t, so the token's scale is folded into its weight: the
//    softmax runs on y = x + log2(scale_t), P' = exp2(y - m) = p * scale_t is what multiplies the
//    codes, and the row sum uses p = P' / scale_t.  Because the reference m follows max y, P' stays
//    below 448 whatever the data, which is what lets it be written as E4M3: again as two
//    terms hi + lo, side by side in one 128-byte row of the P buffer, [hi tokens 0..63 | lo tokens
//    0..63], so that O += [P_hi | P_lo] [V8 ; V8] is four K = 32 steps per accumulator.
//  * Shared memory.  A K-role stage is 20 KiB and a V-role stage 16 KiB (36 and 32 KiB for bf16
//    rows), so the same budget holds four K stages and three V stages: twice the tokens in flight.
//    The bf16 copy of q (latent panels) sits in the V stages and P buffers while it is converted.
//
// Work split, merge paths, index handling, time-outs: as in tc2_decode_kernel.
#pragma once

#include <cuda_fp16.h>

#include "tc2_decode.cuh"

namespace omni {

constexpr int kQ8RowBytes = 640;
constexpr int kQ8Panels = 5;                              // four panels of 128 codes, one of 64 bf16 rope columns
constexpr int kQ8KStages = 4, kQ8VStages = 3;
constexpr int kQ8KPanel = 32 * 128;
constexpr int kQ8KBytes = kQ8Panels * kQ8KPanel;          // K role: 32 tokens x 640 B
constexpr int kQ8VBytes = 2 * kPanelBytes;                // V role: 64 tokens x 256 codes
constexpr int kQ8SmemQHi = 0;                             // 4 panels x [64 heads x 128 codes]
constexpr int kQ8SmemQLo = 4 * kPanelBytes;
constexpr int kQ8SmemQRope = 8 * kPanelBytes;             // [64 heads x 64 bf16]
constexpr int kQ8SmemK = kTileBytes;
constexpr int kQ8SmemV = kQ8SmemK + kQ8KStages * kQ8KBytes;
constexpr int kQ8SmemP = kQ8SmemV + kQ8VStages * kQ8VBytes;     // 2 buffers x [64 heads x (64 hi + 64 lo codes)]
constexpr int kQ8SmemAux = kQ8SmemP + 2 * kPanelBytes;
constexpr int kQ8SmemQTemp = kQ8SmemV;                    // 8 bf16 panels of q during set-up: V stages + P buffers
constexpr int kQ8ScaleRing = 8;                           // as the validity-mask ring
constexpr uint32_t kQ8ColS8 = 256, kQ8ColSr = 352;
// The weights P' = exp2(y - m) are written as E4M3, whose range is [2^-9, 448].  The reference m is
// therefore kept below the running maximum of y: it is set kQ8Headroom under the tile maximum
// whenever that maximum has risen more than kQ8RescaleWindow above it, so the largest weight
// lies in (2^-.., 2^8.75 = 431] and a token is only lost to underflow when its weight is more
// than 2^18 times smaller than the largest one seen.
constexpr float kQ8Headroom = 8.f, kQ8RescaleWindow = 8.75f;

struct Q8Aux {
    float q_scale[64];                        // a[row]
    float tok_scale[kQ8ScaleRing][64];        // scale of each token of a tile
    float tok_log2[kQ8ScaleRing][64];         // its base-2 logarithm
    float tok_rcp[kQ8ScaleRing][64];          // its reciprocal
};
static_assert(kQ8SmemQRope + kPanelBytes == kTileBytes, "q area");
static_assert(kQ8SmemAux + (int)sizeof(Q8Aux) <= kC2SmemCtl, "auxiliary arrays must end below the control block");
static_assert(kQ8SmemQTemp + 8 * kPanelBytes <= kQ8SmemAux, "the temporary copy of q must not reach the auxiliary arrays");

struct Q8Control {
    uint64_t q_full;                     // this CTA's bf16 q has landed (local)
    uint64_t q_ready;                    // leader: both CTAs have rewritten q as E4M3 terms
    uint64_t q_conv;                     // local: the temporary copy of q is dead
    uint64_t k_full[kQ8KStages];
    uint64_t k_empty[kQ8KStages];
    uint64_t v_full[kQ8VStages];
    uint64_t v_empty[kQ8VStages];
    uint64_t s_full[3];
    uint64_t s_empty[3];
    uint64_t p_full[2];
    uint64_t p_free[2];                  // P V of a tile retired: its P buffer may be rewritten, O may be rescaled
    uint64_t x_bar;
    uint64_t exit_bar;
    uint64_t recv_bar;
    uint64_t ready_bar;
    uint64_t valid_mask[kMaskRing];
    float xchg[2][4][64];
    uint32_t tmem_base;
    uint32_t abort;
    uint32_t merge_flag;
    uint32_t xfail;
    int32_t k_progress;
};
static_assert(sizeof(Q8Control) <= kC2SmemCtlBytes, "control block too large");

// Instruction descriptor of kind::f8f6f4 with E4M3 inputs and fp32 accumulation (same fields as
// instr_desc; the two format fields are 0 for E4M3).
__host__ __device__ constexpr uint32_t instr_desc_e4m3(int m, int n, int b_mn_major)
{
    return (1u << 4) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

template <bool kAccumulate>
__device__ __forceinline__ void tc_mma8_pair_elect(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                                   uint32_t b_hi, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "elect.sync _|q, 0xffffffff;\n\t"
        "@q tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "n"(kAccumulate ? 1 : 0)
        : "memory");
}

// Two floats -> two E4M3 codes (round to nearest even, saturating), `lo` in the low byte.
__device__ __forceinline__ uint32_t e4m3x2(float lo, float hi)
{
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
// Two E4M3 codes -> their exact values.
__device__ __forceinline__ float2 e4m3x2_values(uint32_t codes)
{
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)codes));
    return __half22float2(*reinterpret_cast<const __half2 *>(&h2));
}
// Sixteen values as two-term E4M3: hi codes and lo codes (value ~ hi + lo), 16 bytes each.
__device__ __forceinline__ void split_e4m3(const float (&v)[16], uint4 &hi, uint4 &lo)
{
    uint32_t h[4], l[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t h0 = e4m3x2(v[4 * k], v[4 * k + 1]), h1 = e4m3x2(v[4 * k + 2], v[4 * k + 3]);
        const float2 b0 = e4m3x2_values(h0), b1 = e4m3x2_values(h1);
        const uint32_t l0 = e4m3x2(v[4 * k] - b0.x, v[4 * k + 1] - b0.y), l1 = e4m3x2(v[4 * k + 2] - b1.x, v[4 * k + 3] - b1.y);
        h[k] = h0 | (h1 << 16);
        l[k] = l0 | (l1 << 16);
    }
    hi = make_uint4(h[0], h[1], h[2], h[3]);
    lo = make_uint4(l[0], l[1], l[2], l[3]);
}

// Row gathers of the 8-bit layout (see gather_k_rows / gather_v_rows): 640-byte rows, K role
// 32 rows x 5 panels, V role 64 rows x the two panels of this CTA's value columns.
__device__ __noinline__ void gather_k_rows_q8(uint32_t dst, const char *kv_bytes, int own_row, int lane)
{
    const int ch = lane & 7;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        const int r = 4 * g + (lane >> 3);
        const int src_row = __shfl_sync(0xffffffffu, own_row, r);
        const char *src = kv_bytes + (size_t)src_row * kQ8RowBytes + ch * 16;
        const uint32_t d = dst + r * 128 + ((ch ^ (r & 7)) << 4);
#pragma unroll
        for (int c = 0; c < kQ8Panels; ++c) cp_async16(d + c * kQ8KPanel, src + c * 128);
    }
    cp_async_commit();
}

__device__ __noinline__ void gather_v_rows_q8(uint32_t dst, const char *kv_cols, int row_lo, int row_hi, int lane)
{
    const int ch = lane & 7;
#pragma unroll
    for (int g = 0; g < 16; ++g) {
        const int r = 4 * g + (lane >> 3);
        const int a = __shfl_sync(0xffffffffu, row_lo, r & 31), c2 = __shfl_sync(0xffffffffu, row_hi, r & 31);
        const int src_row = r < 32 ? a : c2;
        const char *src = kv_cols + (size_t)src_row * kQ8RowBytes + ch * 16;
        const uint32_t d = dst + r * 128 + ((ch ^ (r & 7)) << 4);
#pragma unroll
        for (int c = 0; c < 2; ++c) cp_async16(d + c * kPanelBytes, src + c * 128);
    }
    cp_async_commit();
}

// Two instances, as for the bf16 kernel: with and without the in-cluster merge of two splits, each
// carrying only its own merge and epilogue code.  The 8-bit entry point takes an index list only.
template <bool kClusterMerge>
__device__ __forceinline__ void tc2q8_decode_body(const CUtensorMap &q_nope_map, const CUtensorMap &q_rope_map,
                                                  const CUtensorMap &kv_k_map, const CUtensorMap &kv_v_map,
                                                  const CUtensorMap &kv_page_map, const DecodeParams &p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw;
    if (smem_u32(smem_raw) & 1023u) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (threadIdx.x == 0) flag_status(p.status, OMNI_DEV_TIMEOUT);
        return;
    }
    Q8Control *ctl = reinterpret_cast<Q8Control *>(smem + kC2SmemCtl);
    Q8Aux *aux = reinterpret_cast<Q8Aux *>(smem + kQ8SmemAux);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t crank = cluster_rank();
    const uint32_t rank = crank & 1u, leader = crank & ~1u, peer = crank ^ 1u;
    const uint16_t pair_mask = (uint16_t)(3u << leader);

    const int pair = blockIdx.x >> 1;
    const int s = kClusterMerge ? (int)(crank >> 1) : pair % p.splits;
    int b = kClusterMerge ? (int)(blockIdx.x >> 2) : pair / p.splits;
    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;  // warp-uniform
    const int h0 = (int)rank * kTcHeads;
    const int head_rows = min(kTcHeads, p.heads - h0);

    // ---- set-up (no global memory access before the dependent-launch wait) -------------------
    if (threadIdx.x == 0) {
        mbar_init(&ctl->q_full, 1);
        mbar_init(&ctl->q_ready, 16);
        mbar_init(&ctl->q_conv, 8);
        for (int i = 0; i < kQ8KStages; ++i) {
            mbar_init(&ctl->k_full[i], 1);
            mbar_init(&ctl->k_empty[i], 1);
        }
        for (int i = 0; i < kQ8VStages; ++i) {
            mbar_init(&ctl->v_full[i], 1);
            mbar_init(&ctl->v_empty[i], 1);
        }
        for (int i = 0; i < 3; ++i) {
            mbar_init(&ctl->s_full[i], 1);
            mbar_init(&ctl->s_empty[i], 16);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&ctl->p_full[i], 16);
            mbar_init(&ctl->p_free[i], 1);
        }
        mbar_init(&ctl->x_bar, 256);
        mbar_init(&ctl->exit_bar, 2);
        mbar_init(&ctl->recv_bar, 1);
        mbar_init(&ctl->ready_bar, 1);
        ctl->abort = 0;
        ctl->xfail = 0;
        ctl->k_progress = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_after_init();
    tc_fence_after();
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (!kClusterMerge && p.longest_first) b = c2_request_by_length_rank(p, reinterpret_cast<int *>(smem), &ctl->merge_flag, b);
    const Selection selection = load_selection(p, b);
    __builtin_assume(selection.list != nullptr);
    const int n = selection.n;
    const bool bad_len = selection.bad;
    int begin, end;
    split_range(n, p.splits, s, begin, end, kC2Tile);
    const int tiles = (end - begin + kC2Tile - 1) / kC2Tile;

    const bool active = tiles > 0;
    if (!active && bad_len && threadIdx.x == 0 && crank == 0) flag_status(p.status, OMNI_DEV_BAD_INDEX);
    if (!kClusterMerge && !active) c2_store_empty(p, b, s, h0, head_rows, warp, lane);

    const uint32_t tmem = ctl->tmem_base;
    volatile uint32_t *abort_flag = &ctl->abort;
    const int32_t *pt = p.page_table + (size_t)b * p.max_pages;
    const char *kv_bytes = reinterpret_cast<const char *>(p.kv);

    // Index pipeline of the producers: as in tc2_decode_kernel (lane l serves tokens l and l+32).
    struct TileIdx {
        int t0, t1;
        int pg0, pg1;
    };
    auto stage_tokens = [&](int tile, TileIdx &x) {
        const int j0 = begin + tile * kC2Tile + lane, j1 = j0 + 32;
        x.t0 = (tile < tiles && j0 < end) ? selection_at(selection, j0) : -1;
        x.t1 = (tile < tiles && j1 < end) ? selection_at(selection, j1) : -1;
    };
    auto stage_pages = [&](TileIdx &x) {
        x.pg0 = (x.t0 >= 0 && x.t0 / kPage < p.max_pages) ? ldg_index(pt + x.t0 / kPage, selection.keep) : -1;
        x.pg1 = (x.t1 >= 0 && x.t1 / kPage < p.max_pages) ? ldg_index(pt + x.t1 / kPage, selection.keep) : -1;
    };
    auto stage_rows = [&](int tile, const TileIdx &x, int &row_lo, int &row_hi, uint64_t &mask, bool &contig,
                          bool &contig_lo, bool &contig_hi, bool &any_bad) {
        const int j0 = begin + tile * kC2Tile + lane, j1 = j0 + 32;
        const bool ok0 = x.pg0 >= 0 && (int64_t)x.pg0 < p.num_pages, ok1 = x.pg1 >= 0 && (int64_t)x.pg1 < p.num_pages;
        any_bad |= (j0 < end && !ok0 && !is_padding(selection, x.t0)) || (j1 < end && !ok1 && !is_padding(selection, x.t1));
        const int r0 = ok0 ? x.pg0 * kPage + x.t0 % kPage : -1, r1 = ok1 ? x.pg1 * kPage + x.t1 % kPage : -1;
        const uint32_t m0 = __ballot_sync(0xffffffffu, r0 >= 0), m1 = __ballot_sync(0xffffffffu, r1 >= 0);
        mask = (uint64_t)m0 | ((uint64_t)m1 << 32);
        int stand_in = 0;
        if (m0)
            stand_in = __shfl_sync(0xffffffffu, r0, __ffs(m0) - 1);
        else if (m1)
            stand_in = __shfl_sync(0xffffffffu, r1, __ffs(m1) - 1);
        row_lo = r0 >= 0 ? r0 : stand_in;
        row_hi = r1 >= 0 ? r1 : stand_in;
        const int base_lo = __shfl_sync(0xffffffffu, row_lo, 0), base_hi = __shfl_sync(0xffffffffu, row_hi, 0);
        contig_lo = __all_sync(0xffffffffu, r0 == base_lo + lane);
        contig_hi = __all_sync(0xffffffffu, r1 == base_hi + lane);
        contig = contig_lo && contig_hi && base_hi == base_lo + 32;
    };

    float cm_lse = -INFINITY, cm_inv = 0.f;
    bool softmax_ok = true;

    if (!active) {
        // an empty split inside a merging cluster: no pipeline, but it takes part in the exchange
    } else if (warp == 0) {
        // =========================== K-role producer =====================================
        if (lane == 0) {
            // q, bf16: the eight latent panels go to a temporary place, the rope panel to its own
            mbar_expect_tx(&ctl->q_full, kTileBytes);
            tma_box3d(smem_base + kQ8SmemQTemp, &q_nope_map, &ctl->q_full, b * p.heads + h0, 0);
            tma_box3d(smem_base + kQ8SmemQRope, &q_rope_map, &ctl->q_full, b * p.heads + h0, 8);
        }
        bool any_bad = bad_len;
        TileIdx x1, x2;
        int row_lo, row_hi;
        uint64_t mask;
        bool contig, contig_lo, contig_hi;
        float sc_lo, sc_hi;                  // scales of the rows of the tile about to be loaded
        {
            TileIdx x0;
            stage_tokens(0, x0);
            stage_tokens(1, x1);
            stage_tokens(2, x2);
            stage_pages(x0);
            stage_pages(x1);
            stage_rows(0, x0, row_lo, row_hi, mask, contig, contig_lo, contig_hi, any_bad);
            sc_lo = __ldg(p.kv_scale + row_lo);
            sc_hi = __ldg(p.kv_scale + row_hi);
        }
        bool ok = true;
        int pending = -1;
        for (int i = 0; ok && i < tiles; ++i) {
            const int st = i % kQ8KStages;
            if (lane == 0) *const_cast<volatile int32_t *>(&ctl->k_progress) = i;
            if (i >= kQ8KStages) ok = mbar_wait(&ctl->k_empty[st], ((i / kQ8KStages) - 1) & 1);
            ok = __all_sync(0xffffffffu, ok) && (*abort_flag == 0);
            if (!ok) break;
            {
                // what the softmax warps need to know about tile i, published before its copy is
                // requested: which tokens count, and every token's scale, its logarithm and reciprocal
                const int ring = i % kQ8ScaleRing;
                aux->tok_scale[ring][lane] = sc_lo;
                aux->tok_scale[ring][lane + 32] = sc_hi;
                aux->tok_log2[ring][lane] = log2f(sc_lo);
                aux->tok_log2[ring][lane + 32] = log2f(sc_hi);
                aux->tok_rcp[ring][lane] = 1.f / sc_lo;
                aux->tok_rcp[ring][lane + 32] = 1.f / sc_hi;
                if (lane == 0) ctl->valid_mask[i % kMaskRing] = mask;
                __threadfence_block();
            }
            const uint32_t bar = map_to_rank(smem_u32(&ctl->k_full[st]), leader);
            if (lane == 0 && rank == 0) mbar_expect_tx(&ctl->k_full[st], 2 * kQ8KBytes);
            __syncwarp();
            const uint32_t dst = smem_base + kQ8SmemK + st * kQ8KBytes;
            const int own_row = rank ? row_hi : row_lo;
            bool gathered = false;
            if (rank ? contig_hi : contig_lo) {
                if (lane == 0) tma_box3d_pair(dst, &kv_k_map, bar, own_row, 0);
            } else {
                gathered = true;
                gather_k_rows_q8(dst, kv_bytes, own_row, lane);
            }
            if (pending >= 0) {
                retire_gathered_stage(map_to_rank(smem_u32(&ctl->k_full[pending]), leader), kQ8KBytes, gathered, lane);
                pending = -1;
            }
            if (gathered) pending = st;
            if (i + 1 < tiles) {
                stage_rows(i + 1, x1, row_lo, row_hi, mask, contig, contig_lo, contig_hi, any_bad);
                sc_lo = __ldg(p.kv_scale + row_lo);
                sc_hi = __ldg(p.kv_scale + row_hi);
            }
            x1 = x2;
            stage_pages(x1);
            stage_tokens(i + 3, x2);
        }
        if (pending >= 0) retire_gathered_stage(map_to_rank(smem_u32(&ctl->k_full[pending]), leader), kQ8KBytes, false, lane);
        if (lane == 0) *const_cast<volatile int32_t *>(&ctl->k_progress) = 0x7fffffff;
        if (!ok && lane == 0) {
            flag_status(p.status, OMNI_DEV_TIMEOUT | OMNI_DEV_ROLE_PRODUCER_K);
            *abort_flag = 1;
        }
        if (__any_sync(0xffffffffu, any_bad) && lane == 0 && rank == 0) flag_status(p.status, OMNI_DEV_BAD_INDEX);
    } else if (warp == 6) {
        // =========================== V-role producer =====================================
        // This CTA's V columns are [256*rank, 256*rank+256): code panels 2*rank and 2*rank+1.
        bool any_bad = false;
        TileIdx x1, x2;
        int row_lo, row_hi;
        uint64_t mask_unused;
        bool contig, contig_lo, contig_hi;
        {
            TileIdx x0;
            stage_tokens(0, x0);
            stage_tokens(1, x1);
            stage_tokens(2, x2);
            stage_pages(x0);
            stage_pages(x1);
            stage_rows(0, x0, row_lo, row_hi, mask_unused, contig, contig_lo, contig_hi, any_bad);
        }
        // the V stages hold the temporary copy of q until the softmax warps have converted it
        bool ok = mbar_wait(&ctl->q_conv, 0);
        ok = __all_sync(0xffffffffu, ok);
        int pending = -1;
        for (int i = 0; ok && i < tiles; ++i) {
            const int st = i % kQ8VStages;
            if (i >= kQ8VStages) ok = mbar_wait(&ctl->v_empty[st], ((i / kQ8VStages) - 1) & 1);
            ok = __all_sync(0xffffffffu, ok) && (*abort_flag == 0);
            if (!ok) break;
            const uint32_t bar = map_to_rank(smem_u32(&ctl->v_full[st]), leader);
            if (lane == 0 && rank == 0) mbar_expect_tx(&ctl->v_full[st], 2 * kQ8VBytes);
            __syncwarp();
            const uint32_t dst = smem_base + kQ8SmemV + st * kQ8VBytes;
            bool gathered = false;
            if (contig) {
                if (lane == 0) tma_box3d_pair(dst, &kv_v_map, bar, row_lo, 2 * (int)rank);
            } else {
                gathered = true;
                gather_v_rows_q8(dst, kv_bytes + (int)rank * 256, row_lo, row_hi, lane);
            }
            if (pending >= 0) {
                retire_gathered_stage(map_to_rank(smem_u32(&ctl->v_full[pending]), leader), kQ8VBytes, gathered, lane);
                pending = -1;
            }
            if (gathered) pending = st;
            if (i + 1 < tiles) stage_rows(i + 1, x1, row_lo, row_hi, mask_unused, contig, contig_lo, contig_hi, any_bad);
            x1 = x2;
            stage_pages(x1);
            stage_tokens(i + 3, x2);
        }
        if (pending >= 0) retire_gathered_stage(map_to_rank(smem_u32(&ctl->v_full[pending]), leader), kQ8VBytes, false, lane);
        if (!ok && lane == 0) {
            flag_status(p.status, OMNI_DEV_TIMEOUT | OMNI_DEV_ROLE_PRODUCER_V);
            *abort_flag = 1;
        }
    } else if (warp == 7) {
        // =========================== L2 prefetcher (CTA 0 only) ==========================
        if (rank == 0) {
            for (int t0 = 0; t0 < tiles; t0 += 32) {
                const int t = t0 + lane;
                const int j0 = begin + t * kC2Tile;
                int row = -1;
                if (t < tiles && j0 + kC2Tile <= end) {
                    const int first = selection_at(selection, j0), last = selection_at(selection, j0 + kC2Tile - 1);
                    if (first >= 0 && first % kPage == 0 && last == first + kC2Tile - 1 && first / kPage < p.max_pages) {
                        const int pg = ldg_index(pt + first / kPage, selection.keep);
                        if (pg >= 0 && (int64_t)pg < p.num_pages) row = pg * kPage;
                    }
                }
                const int count = min(32, tiles - t0);
                bool ok = true;
                if (!__any_sync(0xffffffffu, row >= 0)) continue;
                for (int k = 0; ok && k < count; ++k) {
                    const int i = t0 + k;
                    const volatile int32_t *progress = &ctl->k_progress;
                    for (int naps = 0; *progress < i - kPrefetchAhead && *abort_flag == 0; ++naps) {
                        if (naps > (1 << 22)) {
                            ok = false;
                            break;
                        }
                        __nanosleep(200);
                    }
                    ok = ok && (*abort_flag == 0);
                    if (ok && lane == k && row >= 0)
                        asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(&kv_page_map),
                                     "r"(0), "r"(row), "r"(0)
                                     : "memory");
                }
                if (!ok) break;
            }
        }
    } else if (warp == 1) {
        // =========================== MMA issuer (CTA 0 only) =============================
        if (rank == 0) {
            constexpr uint32_t idesc_qk8 = instr_desc_e4m3(128, kC2Tile, 0);
            constexpr uint32_t idesc_qkr = instr_desc(128, kC2Tile, 0);
            constexpr uint32_t idesc_pv8 = instr_desc_e4m3(128, 256, 1);
            const uint64_t q_desc = smem_desc(smem_base + kQ8SmemQHi, 16, 1024);
            const uint64_t k_desc = smem_desc(smem_base + kQ8SmemK, 16, 1024);
            const uint64_t p_desc = smem_desc(smem_base + kQ8SmemP, 16, 1024);
            const uint64_t v_desc = smem_desc(smem_base + kQ8SmemV, kPanelBytes, 1024);
            const uint32_t q_lo = (uint32_t)q_desc, k_lo = (uint32_t)k_desc, p_lo = (uint32_t)p_desc, v_lo = (uint32_t)v_desc;
            const uint32_t kmaj_hi = (uint32_t)(q_desc >> 32), v_hi = (uint32_t)(v_desc >> 32);
            const int tiles_u = __shfl_sync(0xffffffffu, tiles, 0);
            const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem, 0);
            // S8(t) = [Q_hi | Q_lo] [K8 ; K8]^T: two terms x 16 steps of 32 codes; Sr(t) = Q_rope K_rope^T: 4 steps of 16 bf16
            auto issue_qk = [&](int kst, int sbuf) {
                const uint32_t d8 = tmem_u + kQ8ColS8 + 32 * sbuf, dr = tmem_u + kQ8ColSr + 32 * sbuf;
                const uint32_t kb = k_lo + ((kst * kQ8KBytes) >> 4);
                tc_mma8_pair_elect<false>(d8, q_lo, kmaj_hi, kb, kmaj_hi, idesc_qk8);
#pragma unroll
                for (int kk = 1; kk < 32; ++kk) {
                    const int term = kk >> 4, c = kk & 15;
                    tc_mma8_pair_elect<true>(d8, q_lo + ((term * kQ8SmemQLo + (c >> 2) * kPanelBytes + (c & 3) * 32) >> 4), kmaj_hi,
                                             kb + (((c >> 2) * kQ8KPanel + (c & 3) * 32) >> 4), kmaj_hi, idesc_qk8);
                }
                tc_mma_pair_elect<false>(dr, q_lo + (kQ8SmemQRope >> 4), kmaj_hi, kb + ((4 * kQ8KPanel) >> 4), kmaj_hi, idesc_qkr);
#pragma unroll
                for (int kk = 1; kk < 4; ++kk)
                    tc_mma_pair_elect<true>(dr, q_lo + ((kQ8SmemQRope + kk * 32) >> 4), kmaj_hi,
                                            kb + ((4 * kQ8KPanel + kk * 32) >> 4), kmaj_hi, idesc_qkr);
                tc_commit_pair_elect(&ctl->k_empty[kst], pair_mask);
                tc_commit_pair_elect(&ctl->s_full[sbuf], pair_mask);
            };
            // O += [P_hi | P_lo] [V8 ; V8]: four steps of 32 codes of a P row (hi tokens 0..31, 32..63,
            // then lo), each against the matching 32 tokens of the stage, two N = 256 accumulators
            auto issue_pv = [&](int vst, int pbuf, bool first) {
                const uint32_t a = p_lo + ((pbuf * kPanelBytes) >> 4);
                const uint32_t bd = v_lo + ((vst * kQ8VBytes) >> 4);
                if (first) {
                    tc_mma8_pair_elect<false>(tmem_u + kColO, a, kmaj_hi, bd, v_hi, idesc_pv8);
                    tc_mma8_pair_elect<false>(tmem_u + kColO + 128, a, kmaj_hi, bd + (kPanelBytes >> 4), v_hi, idesc_pv8);
                } else {
                    tc_mma8_pair_elect<true>(tmem_u + kColO, a, kmaj_hi, bd, v_hi, idesc_pv8);
                    tc_mma8_pair_elect<true>(tmem_u + kColO + 128, a, kmaj_hi, bd + (kPanelBytes >> 4), v_hi, idesc_pv8);
                }
#pragma unroll
                for (int k = 1; k < 4; ++k) {
                    const uint32_t ak = a + ((k * 32) >> 4), bk = bd + (((k & 1) * 4096) >> 4);
                    tc_mma8_pair_elect<true>(tmem_u + kColO, ak, kmaj_hi, bk, v_hi, idesc_pv8);
                    tc_mma8_pair_elect<true>(tmem_u + kColO + 128, ak, kmaj_hi, bk + (kPanelBytes >> 4), v_hi, idesc_pv8);
                }
                tc_commit_pair_elect(&ctl->v_empty[vst], pair_mask);
                tc_commit_pair_elect(&ctl->p_free[pbuf], pair_mask);
            };
            auto qk_tile = [&](int t) -> bool {
                const int kst = t % kQ8KStages, sbuf = t % 3;
                bool good = mbar_wait(&ctl->k_full[kst], (t / kQ8KStages) & 1) &&
                            (t < 3 || mbar_wait(&ctl->s_empty[sbuf], ((t / 3) - 1) & 1));
                good = __all_sync(0xffffffffu, good);
                if (!good) return false;
                tc_fence_after();
                issue_qk(kst, sbuf);
                return true;
            };
            auto pv_tile = [&](int i) -> bool {
                const int vst = i % kQ8VStages, pbuf = i & 1;
                bool good = mbar_wait(&ctl->p_full[pbuf], (i >> 1) & 1) && mbar_wait(&ctl->v_full[vst], (i / kQ8VStages) & 1);
                good = __all_sync(0xffffffffu, good);
                if (!good) return false;
                tc_fence_after();
                issue_pv(vst, pbuf, i == 0);
                return true;
            };
            bool ok = mbar_wait(&ctl->q_ready, 0);
            ok = __all_sync(0xffffffffu, ok);
            if (ok) tc_fence_after();
            if (ok) ok = qk_tile(0);
            if (ok && tiles_u > 1) ok = qk_tile(1);
            for (int i = 0; ok && i < tiles_u; ++i) {
                if (i + 2 < tiles_u) ok = qk_tile(i + 2);
                if (ok) ok = pv_tile(i);
            }
            if (!ok && lane == 0) {
                flag_status(p.status, OMNI_DEV_TIMEOUT | OMNI_DEV_ROLE_MMA);
                *abort_flag = 1;
            }
        }
        __syncwarp();
    } else {
        // =========================== softmax + epilogue =================================
        const int quarter = warp & 3;
        const int sub = warp >= 8 ? 1 : 0;
        const int row = (quarter & 1) * 32 + lane;
        const int half = quarter >> 1;
        const int part = half * 2 + sub;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const uint32_t s_empty_leader = map_to_rank(smem_u32(&ctl->s_empty[0]), leader);
        const uint32_t p_full_leader0 = map_to_rank(smem_u32(&ctl->p_full[0]), leader);
        const uint32_t p_full_leader1 = map_to_rank(smem_u32(&ctl->p_full[1]), leader);
        bool ok = true;
        float a_row = 1.f;
        {
            // ---- rewrite q's latent columns as two E4M3 terms per value -------------------
            // This thread: head row `row`, latent columns [128 * part, 128 * part + 128), i.e. bf16
            // panels 2*part and 2*part+1 of the temporary copy and code panel `part` of each term.
            ok = mbar_wait(&ctl->q_full, 0);
            ok = __all_sync(0xffffffffu, ok);
            float amax = 0.f;
            const uint8_t *src = smem + kQ8SmemQTemp + (size_t)(2 * part) * kPanelBytes + row * 128;
            if (ok) {
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const uint4 w = *reinterpret_cast<const uint4 *>(src + (c >> 3) * kPanelBytes + (((c & 7) ^ (row & 7)) << 4));
                    const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        amax = fmaxf(amax, fabsf(__uint_as_float(ws[k] << 16)));
                        amax = fmaxf(amax, fabsf(__uint_as_float(ws[k] & 0xffff0000u)));
                    }
                }
                ctl->xchg[0][part][row] = amax;
            }
            asm volatile("bar.sync 2, 256;" ::: "memory");        // the eight softmax warps
            if (ok) {
                amax = fmaxf(fmaxf(ctl->xchg[0][0][row], ctl->xchg[0][1][row]), fmaxf(ctl->xchg[0][2][row], ctl->xchg[0][3][row]));
                // a power of two with |q| / a < 448: the division is exact
                int e = 0;
                if (amax > 0.f) (void)frexpf(amax * (1.f / 448.f), &e);
                a_row = amax > 0.f ? ldexpf(1.f, e) : 1.f;
                const float inv_a = 1.f / a_row;
                uint8_t *hi_row = smem + kQ8SmemQHi + (size_t)part * kPanelBytes + row * 128;
                uint8_t *lo_row = smem + kQ8SmemQLo + (size_t)part * kPanelBytes + row * 128;
#pragma unroll
                for (int c = 0; c < 8; ++c) {                    // 16 columns = one 16-byte chunk of codes
                    float v[16];
#pragma unroll
                    for (int hc = 0; hc < 2; ++hc) {
                        const int cc = 2 * c + hc;               // bf16 chunk (8 columns) within the thread's 128
                        const uint4 w = *reinterpret_cast<const uint4 *>(src + (cc >> 3) * kPanelBytes + (((cc & 7) ^ (row & 7)) << 4));
                        const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            v[8 * hc + 2 * k] = __uint_as_float(ws[k] << 16) * inv_a;
                            v[8 * hc + 2 * k + 1] = __uint_as_float(ws[k] & 0xffff0000u) * inv_a;
                        }
                    }
                    uint4 hi, lo;
                    split_e4m3(v, hi, lo);
                    *reinterpret_cast<uint4 *>(hi_row + ((c ^ (row & 7)) << 4)) = hi;
                    *reinterpret_cast<uint4 *>(lo_row + ((c ^ (row & 7)) << 4)) = lo;
                }
                if (part == 0) aux->q_scale[row] = a_row;
            }
            fence_async_smem();                                   // the tensor core reads what the threads wrote
            asm volatile("bar.sync 2, 256;" ::: "memory");        // every read of the temporary copy is done
            if (lane == 0) {
                mbar_arrive(&ctl->q_conv);
                mbar_arrive_cluster(map_to_rank(smem_u32(&ctl->q_ready), leader));
            }
            a_row = aux->q_scale[row];
        }
        float m_ref = -INFINITY, l = 0.f;
        for (int i = 0; ok && i < tiles; ++i) {
            const int buf = i & 1, sbuf = i % 3, ring = i % kQ8ScaleRing;
            ok = mbar_wait(&ctl->s_full[sbuf], (i / 3) & 1);
            if (!__all_sync(0xffffffffu, ok)) {
                ok = false;
                break;
            }
            tc_fence_after();
            uint32_t s8[16], sr[16];
            tc_ld16(tmem + lane_base + kQ8ColS8 + 32 * sbuf + 16 * sub, s8);
            tc_ld16(tmem + lane_base + kQ8ColSr + 32 * sbuf + 16 * sub, sr);
            tc_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(s_empty_leader + 8 * sbuf);
            const uint32_t valid = (uint32_t)(ctl->valid_mask[i % kMaskRing] >> (16 * part)) & 0xffffu;
            const float4 *ts = reinterpret_cast<const float4 *>(&aux->tok_scale[ring][16 * part]);
            const float4 *tl = reinterpret_cast<const float4 *>(&aux->tok_log2[ring][16 * part]);
            float y[16];
            float mt = -INFINITY;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                const float4 sc = ts[g], lg = tl[g];
                const float scv[4] = {sc.x, sc.y, sc.z, sc.w}, lgv[4] = {lg.x, lg.y, lg.z, lg.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int j = 4 * g + k;
                    const float xv = (__uint_as_float(s8[j]) * (a_row * scv[k]) + __uint_as_float(sr[j])) * p.scale_log2;
                    const bool on = (valid >> j) & 1u;
                    y[j] = on ? xv + lgv[k] : -INFINITY;
                    mt = fmaxf(mt, y[j]);
                }
            }
            ctl->xchg[i & 1][part][row] = mt;
            mbar_arrive(&ctl->x_bar);
            ok = mbar_wait(&ctl->x_bar, i & 1);
            if (!__all_sync(0xffffffffu, ok)) {
                ok = false;
                break;
            }
            mt = fmaxf(fmaxf(ctl->xchg[i & 1][0][row], ctl->xchg[i & 1][1][row]),
                       fmaxf(ctl->xchg[i & 1][2][row], ctl->xchg[i & 1][3][row]));
            float factor = 1.f;
            bool moved = false;
            if (mt > m_ref + kQ8RescaleWindow || (m_ref == -INFINITY && mt > -INFINITY)) {
                // the new reference sits kQ8Headroom below the tile maximum (see the constants)
                factor = exp2f(m_ref - (mt - kQ8Headroom));
                m_ref = mt - kQ8Headroom;
                moved = true;
            }
            const float mr = (m_ref == -INFINITY) ? 0.f : m_ref;
            const float4 *tr = reinterpret_cast<const float4 *>(&aux->tok_rcp[ring][16 * part]);
            float sum = 0.f;
            float pw[16];
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                const float4 rc = tr[g];
                const float rcv[4] = {rc.x, rc.y, rc.z, rc.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int j = 4 * g + k;
                    pw[j] = fast_exp2(y[j] - mr);                    // p * scale_t, below 448; 0 for a masked token
                    sum += ((valid >> j) & 1u) ? pw[j] * rcv[k] : 0.f;      // p
                }
            }
            l = l * factor + sum;
            uint4 p_hi, p_lo;
            split_e4m3(pw, p_hi, p_lo);
            // the P buffer is free once P V of tile i-2 retired; O may be rescaled once P V of tile i-1 did
            if (i >= 2) {
                ok = mbar_wait(&ctl->p_free[buf], ((i >> 1) - 1) & 1);
                if (!__all_sync(0xffffffffu, ok)) {
                    ok = false;
                    break;
                }
            }
            if (i >= 1 && __any_sync(0xffffffffu, moved)) {
                ok = mbar_wait(&ctl->p_free[buf ^ 1], ((i - 1) >> 1) & 1);
                if (!__all_sync(0xffffffffu, ok)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
#pragma unroll 1
                for (int c = 0; c < 128; c += 32) {
                    uint32_t ov[32];
                    tc_ld32(tmem + lane_base + kColO + 128 * sub + c, ov);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * factor);
                    tc_st32(tmem + lane_base + kColO + 128 * sub + c, ov);
                }
                tc_wait_st();
            }
            // this thread's 16 tokens: hi codes in 16-byte chunk `part`, lo codes in chunk 4 + part of the row
            uint8_t *p_row = smem + kQ8SmemP + buf * kPanelBytes + row * 128;
            *reinterpret_cast<uint4 *>(p_row + ((part ^ (row & 7)) << 4)) = p_hi;
            *reinterpret_cast<uint4 *>(p_row + (((4 + part) ^ (row & 7)) << 4)) = p_lo;
            fence_async_smem();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(buf ? p_full_leader1 : p_full_leader0);
        }
        if (ok) {
            ok = mbar_wait(&ctl->p_free[(tiles - 1) & 1], ((tiles - 1) >> 1) & 1);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            ctl->xchg[tiles & 1][part][row] = l;
            mbar_arrive(&ctl->x_bar);
            ok = mbar_wait(&ctl->x_bar, tiles & 1);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (kClusterMerge && ok) {
            if (warp == 2 && lane == 0) mbar_arrive_cluster(map_to_rank(smem_u32(&ctl->ready_bar), crank ^ 2u));
            const float lt = (ctl->xchg[tiles & 1][0][row] + ctl->xchg[tiles & 1][1][row]) +
                             (ctl->xchg[tiles & 1][2][row] + ctl->xchg[tiles & 1][3][row]);
            cm_inv = lt > 0.f ? 1.f / lt : 0.f;
            cm_lse = lt > 0.f ? (m_ref + log2f(lt)) * kLn2 : -INFINITY;
        } else if (!kClusterMerge && ok) {
            tc_fence_after();
            const float lt = (ctl->xchg[tiles & 1][0][row] + ctl->xchg[tiles & 1][1][row]) +
                             (ctl->xchg[tiles & 1][2][row] + ctl->xchg[tiles & 1][3][row]);
            c2_store_result(p, smem, tmem, warp, lane, b, s, h0, head_rows, lt, m_ref);
            if (p.splits != 1 && p.counters != nullptr) __threadfence();
        }
        if (!ok && lane == 0) {
            flag_status(p.status, OMNI_DEV_TIMEOUT | OMNI_DEV_ROLE_SOFTMAX);
            *abort_flag = 1;
        }
        softmax_ok = ok;
    }

    // ---- tear-down (as in tc2_decode_kernel) ---------------------------------------------------
    if (*abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    if (kClusterMerge) cluster_merge_exchange(p, ctl, smem, tmem, b, s, crank, h0, head_rows, active, softmax_ok, cm_lse, cm_inv);
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) {
        mbar_arrive(&ctl->exit_bar);
        mbar_arrive_cluster(map_to_rank(smem_u32(&ctl->exit_bar), peer));
    }
    if (warp == 1) {
        mbar_wait(&ctl->exit_bar, 0);
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
    if (kClusterMerge) cluster_sync_relaxed();
    if (!kClusterMerge && p.splits > 1 && p.counters != nullptr)
        merge_if_last(p, b, (int)rank, 2, h0, head_rows, reinterpret_cast<float *>(smem), &ctl->merge_flag);
}

__global__ void __launch_bounds__(kC2Threads, 1)
tc2q8_decode_kernel(const __grid_constant__ CUtensorMap q_nope_map, const __grid_constant__ CUtensorMap q_rope_map,
                    const __grid_constant__ CUtensorMap kv_k_map, const __grid_constant__ CUtensorMap kv_v_map,
                    const __grid_constant__ CUtensorMap kv_page_map, DecodeParams p)
{
    tc2q8_decode_body<false>(q_nope_map, q_rope_map, kv_k_map, kv_v_map, kv_page_map, p);
}

__global__ void __launch_bounds__(kC2Threads, 1)
tc2q8_decode_cm_kernel(const __grid_constant__ CUtensorMap q_nope_map, const __grid_constant__ CUtensorMap q_rope_map,
                       const __grid_constant__ CUtensorMap kv_k_map, const __grid_constant__ CUtensorMap kv_v_map,
                       const __grid_constant__ CUtensorMap kv_page_map, DecodeParams p)
{
    tc2q8_decode_body<true>(q_nope_map, q_rope_map, kv_k_map, kv_v_map, kv_page_map, p);
}

// Quantiser of the 8-bit cache: one warp per row.  scale = max(amax, 2^-60) / 448 with amax the
// largest magnitude of the row's 512 latent columns, code = E4M3(value / scale) with the division
// in fp32 and round-to-nearest-even, saturating conversion; the 64 rope columns are copied.
__global__ void __launch_bounds__(256) quantize_q8_kernel(const __nv_bfloat16 *__restrict__ rows, int64_t num_rows,
                                                           uint8_t *__restrict__ out, float *__restrict__ scale)
{
    const int64_t r = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= num_rows) return;
    const uint4 *src = reinterpret_cast<const uint4 *>(rows + r * kDqk);
    const uint4 w0 = __ldg(src + 2 * lane), w1 = __ldg(src + 2 * lane + 1);      // 16 latent columns
    const uint32_t ws[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
    float v[16];
    float amax = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        v[2 * k] = __uint_as_float(ws[k] << 16);
        v[2 * k + 1] = __uint_as_float(ws[k] & 0xffff0000u);
        amax = fmaxf(amax, fmaxf(fabsf(v[2 * k]), fabsf(v[2 * k + 1])));
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
    const float sc = __fdiv_rn(fmaxf(amax, 0x1p-60f), 448.f);
    uint32_t c[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
        c[k] = e4m3x2(__fdiv_rn(v[4 * k], sc), __fdiv_rn(v[4 * k + 1], sc)) |
               (e4m3x2(__fdiv_rn(v[4 * k + 2], sc), __fdiv_rn(v[4 * k + 3], sc)) << 16);
    uint8_t *dst = out + r * kQ8RowBytes;
    *reinterpret_cast<uint4 *>(dst + 16 * lane) = make_uint4(c[0], c[1], c[2], c[3]);
    if (lane < 8) *reinterpret_cast<uint4 *>(dst + 512 + 16 * lane) = __ldg(src + 64 + lane);          // rope columns
    if (lane == 0) scale[r] = sc;
}

// ---------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------
// The 8-bit pool seen as [rows, 5 panels of 128 bytes]: boxes {128 bytes, box_rows, n panels}.
inline bool encode_q8_panel_map(CUtensorMap *map, const void *base, uint64_t rows, uint32_t box_rows, uint32_t box_panels)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {128, (cuuint64_t)rows, (cuuint64_t)kQ8Panels};
    const cuuint64_t strides[2] = {(cuuint64_t)kQ8RowBytes, 128};
    const cuuint32_t box[3] = {128, box_rows, box_panels};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline bool tc2q8_prepare_device()
{
    static bool attr_set[64] = {};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    std::lock_guard<std::mutex> lock(mu);
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(tc2q8_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kC2SmemBytes) !=
                cudaSuccess ||
            cudaFuncSetAttribute(tc2q8_decode_cm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kC2SmemBytes) !=
                cudaSuccess)
            return false;
        attr_set[dev] = true;
    }
    return true;
}

// maps[0] = q latent panels, maps[1] = q rope panel, maps[2] = K role, maps[3] = V role, maps[4] = whole pages
inline bool tc2q8_make_maps(const DecodeParams &p, CUtensorMap *maps, bool cached)
{
    const uint64_t rows = (uint64_t)p.num_pages * kPage, qrows = (uint64_t)p.batch * p.heads;
    if (cached)
        return cached_map(&maps[0], p.q, qrows, kTcHeads, 8, 1, encode_panel_map) &&
               cached_map(&maps[1], p.q, qrows, kTcHeads, 1, 1, encode_panel_map) &&
               cached_map(&maps[2], p.kv, rows, 32, kQ8Panels, 2, encode_q8_panel_map) &&
               cached_map(&maps[3], p.kv, rows, kTile, 2, 2, encode_q8_panel_map) &&
               cached_map(&maps[4], p.kv, rows, kTile, kQ8Panels, 2, encode_q8_panel_map);
    return encode_panel_map(&maps[0], p.q, qrows, kTcHeads, 8) && encode_panel_map(&maps[1], p.q, qrows, kTcHeads, 1) &&
           encode_q8_panel_map(&maps[2], p.kv, rows, 32, kQ8Panels) && encode_q8_panel_map(&maps[3], p.kv, rows, kTile, 2) &&
           encode_q8_panel_map(&maps[4], p.kv, rows, kTile, kQ8Panels);
}

inline omni_status_t tc2q8_launch(const CUtensorMap *maps, const DecodeParams &p, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.batch * p.splits * 2));
    cfg.blockDim = dim3(kC2Threads);
    cfg.dynamicSmemBytes = kC2SmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = p.cluster_merge ? 4 : 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, p.cluster_merge ? tc2q8_decode_cm_kernel : tc2q8_decode_kernel, maps[0], maps[1], maps[2],
                              maps[3], maps[4], p) == cudaSuccess
               ? OMNI_OK
               : OMNI_ERR_CUDA;
}

}  // namespace omni
