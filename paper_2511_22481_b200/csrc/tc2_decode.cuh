// Paired-CTA tensor-core decode kernel for sm_100a (the fast path for more than 64 heads).
//
// A cluster of two CTAs owns all heads of one (request, split): CTA r serves heads
// [64r, 64r+64).  The pair issues cta_group::2 MMAs with M = 128 (64 rows per CTA), which run
// the tensor pipe of each SM at full rate where a lone M = 64 MMA runs it at half rate, and it
// halves the operand bytes each SM must hold:
//   S = Q K^T   M=128, N=128 tokens, K=576: every CTA supplies its 64 Q rows and the K rows of
//               ITS 64 tokens of the 128-token tile ("K role": 64 tokens x 576 columns)
//   O += P V    M=128, N=256 per instruction, K=128 tokens: every CTA supplies its 64 P rows
//               and, for all 128 tokens, ITS 256 value columns ("V role": 128 tokens x 256
//               columns; CTA r holds columns [256r, 256r+256))
// The two roles overlap only in a quarter of the tile, at different addresses in the two CTAs,
// so each role is loaded on its own (1.9x the tile's bytes cross L2 -> shared memory, but each
// byte leaves HBM once when the pair runs together).
//
// Shared memory has room for one tile per role, so the buffers are refilled piecewise while
// they are consumed: the 9 column panels of the K role form three groups with their own
// full/empty barrier pairs (a group is reloaded for the next tile as soon as its twelve MMAs
// retire) and the V role is split in its two 64-token halves.  Every refill is ONE 3-D TMA box
// {64 columns, 64 rows, 3 or 4 panels}: the copy engine sustains only about 4 M instructions/s
// per SM, so 8 KiB boxes cap an SM near 32 GB/s while 24-72 KiB boxes reach 90-150 GB/s.  All MMAs are issued by one thread of CTA 0 in
// "whatever is ready" order; completion is broadcast to both CTAs with multicast commits.
//
// Warps per CTA: 0 K-role producer, 1 MMA issuer (CTA 0 only) + tensor-memory owner,
// 2-5 softmax / epilogue, 6 V-role producer.
//
// Tensor memory per CTA (a 64-row slice of an M=128 pair accumulator keeps columns [0, N/2) in
// lanes 0-63 and columns [N/2, N) in lanes 64-127):
//   columns   0..255  O: two N=256 accumulators; lane L, column x  <->  head row L%64,
//                        value column 256*(L/64) + x
//   columns 256..319  S buffer 0: lane L, column x <-> head row L%64, token 64*(L/64) + x
//   columns 320..383  S buffer 1
#pragma once

#include "tc_decode.cuh"

namespace omni {

constexpr int kC2Tile = 128;                          // tokens per tile of the pair
constexpr int kC2Threads = 224;
constexpr int kC2SmemQ = 0;                           // 9 panels x 8 KiB
constexpr int kC2SmemK = kC2SmemQ + kTileBytes;       // K role: 9 panels x [64 tokens x 128 B]
constexpr int kC2VHalfBytes = 4 * kPanelBytes;        // V role, one 64-token half: 4 panels
constexpr int kC2SmemV = kC2SmemK + kTileBytes;
constexpr int kC2SmemP = kC2SmemV + 2 * kC2VHalfBytes;  // P: 2 panels x [64 heads x 128 B]
constexpr int kC2SmemCtl = kC2SmemP + 2 * kPanelBytes;
constexpr int kC2SmemCtlBytes = 2048;
constexpr int kC2SmemBytes = kC2SmemCtl + kC2SmemCtlBytes + 1024;
constexpr uint32_t kC2ColS = 256;
constexpr int kMaskRing = 4;
constexpr int kKGroups = 3;                           // the K role is refilled in 3 groups of 3 column panels
constexpr int kKGroupBytes = 3 * kPanelBytes;

struct C2Control {
    uint64_t q_full;
    uint64_t k_full[kKGroups];
    uint64_t k_empty[kKGroups];
    uint64_t v_full[2];
    uint64_t v_empty[2];
    uint64_t s_full[2];
    uint64_t s_empty[2];
    uint64_t p_full;
    uint64_t pv_done;
    uint64_t x_bar;                      // softmax threads: row-maximum exchange
    uint64_t valid_mask[kMaskRing][2];   // per tile: validity of tokens 0..63 and 64..127
    float xchg[2][2][64];                // [tile parity][token half][head row]
    uint32_t tmem_base;
    uint32_t abort;
};
static_assert(sizeof(C2Control) <= kC2SmemCtlBytes, "control block too large");
static_assert(kC2SmemBytes <= 232448, "shared memory budget");

__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}

__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    // default (CTA-scope release) semantics: a cluster-scope release costs ~0.6 us per arrive here,
    // and what must be ordered before it is already ordered by the tcgen05 / async-proxy fences
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Box load of one CTA of a pair; the transaction bytes are credited to `bar_cluster_addr`, which
// may be a barrier of the other CTA of the pair.
__device__ __forceinline__ void tma_box2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar_cluster_addr,
                                               int col, int row)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(col), "r"(row), "r"(bar_cluster_addr)
        : "memory");
}

// 3-D box {64 columns, 64 rows, n column panels}: lands panel-major, i.e. as n consecutive
// [64 rows x 128 B] swizzled panels, in one instruction.
__device__ __forceinline__ void tma_box3d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar_cluster_addr,
                                               int row, int panel)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(0), "r"(row), "r"(panel), "r"(bar_cluster_addr)
        : "memory");
}

__device__ __forceinline__ void tma_gather4_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar_cluster_addr,
                                                 int col, int r0, int r1, int r2, int r3)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(col), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(bar_cluster_addr)
        : "memory");
}

template <bool kAccumulate>
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "n"(kAccumulate ? 1 : 0)
        : "memory");
}

// The same, executed by a whole converged warp: one elected lane issues the instruction.  The
// descriptors arrive as 32-bit halves so that stepping through a tile is a 32-bit add.
template <bool kAccumulate>
__device__ __forceinline__ void tc_mma_pair_elect(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                                  uint32_t b_hi, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "elect.sync _|q, 0xffffffff;\n\t"
        "@q tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "n"(kAccumulate ? 1 : 0)
        : "memory");
}

__device__ __forceinline__ void tc_commit_pair_elect(uint64_t *bar)
{
    const uint16_t both = 3;
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "elect.sync _|q, 0xffffffff;\n\t"
        "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n\t}"
        ::"r"(smem_u32(bar)), "h"(both)
        : "memory");
}

// Arrive on the barrier at this shared-memory offset in BOTH CTAs once all MMAs issued so far
// by this thread have retired.
__device__ __forceinline__ void tc_commit_pair(uint64_t *bar)
{
    const uint16_t both = 3;
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(smem_u32(bar)), "h"(both)
        : "memory");
}

__global__ void __launch_bounds__(kC2Threads, 1)
tc2_decode_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap kv_map,
                  const __grid_constant__ CUtensorMap kv_k_map, const __grid_constant__ CUtensorMap kv_v_map,
                  DecodeParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    C2Control *ctl = reinterpret_cast<C2Control *>(smem + kC2SmemCtl);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t rank = cluster_rank();

    const int pair = blockIdx.x >> 1;
    const int s = pair % p.splits;
    const int b = pair / p.splits;
    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;  // warp-uniform
    const int h0 = (int)rank * kTcHeads;

    int n = __ldg(p.sel_len + b);
    bool bad_len = false;
    if (n < 0 || n > p.max_sel) {
        bad_len = true;
        n = 0;
    }
    int begin, end;
    split_range(n, p.splits, s, begin, end, kC2Tile);
    const int tiles = (end - begin + kC2Tile - 1) / kC2Tile;

    if (tiles == 0) {
        // empty split (the same decision in both CTAs of the pair): zeros and -inf, no cluster work
        if (threadIdx.x == 0 && bad_len && rank == 0) flag_status(p.status, OMNI_DEV_BAD_INDEX);
        for (int r = warp; r < kTcHeads; r += kC2Threads / 32) {
            const int h = h0 + r;
            if (h >= p.heads) break;
            if (p.splits == 1) {
                uint4 *o = reinterpret_cast<uint4 *>(p.out + ((size_t)b * p.heads + h) * kDv);
                for (int i = lane; i < kDv * 2 / 16; i += 32) o[i] = make_uint4(0, 0, 0, 0);
                if (lane == 0) p.lse[(size_t)b * p.heads + h] = -INFINITY;
            } else {
                const size_t u = ((size_t)b * p.splits + s) * p.heads + h;
                float4 *o = reinterpret_cast<float4 *>(p.part_out + u * kDv);
                for (int i = lane; i < kDv / 4; i += 32) o[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (lane == 0) p.part_lse[u] = -INFINITY;
            }
        }
        return;
    }

    // ---- set-up ---------------------------------------------------------------------------
    if (threadIdx.x == 0) {
        mbar_init(&ctl->q_full, 1);
        for (int i = 0; i < kKGroups; ++i) {
            mbar_init(&ctl->k_full[i], 1);
            mbar_init(&ctl->k_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&ctl->v_full[i], 1);
            mbar_init(&ctl->v_empty[i], 1);
            mbar_init(&ctl->s_full[i], 1);
            mbar_init(&ctl->s_empty[i], 8);      // one arrival per softmax warp of either CTA
        }
        mbar_init(&ctl->p_full, 8);
        mbar_init(&ctl->pv_done, 1);
        mbar_init(&ctl->x_bar, 128);
        ctl->abort = 0;
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
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;
    volatile uint32_t *abort_flag = &ctl->abort;

    const int32_t *sel = p.sel_idx + (size_t)b * p.max_sel;
    const int32_t *pt = p.page_table + (size_t)b * p.max_pages;

    // Index pipeline of the producers.  Lane l serves tokens l and l+32 of one 64-token half of a
    // tile.  The three dependent steps (token position -> page id -> pool row) run in different
    // loop iterations, one tile apart, so no load is consumed in the iteration that issued it.
    struct HalfIdx {
        int t0, t1;        // token positions (stage 1)
        int pg0, pg1;      // physical page ids, -1 if the position breaks the contract (stage 2)
    };
    auto stage_tokens = [&](int tile, int half, HalfIdx &x) {
        const int j0 = begin + tile * kC2Tile + half * 64 + lane, j1 = j0 + 32;
        x.t0 = (tile < tiles && j0 < end) ? __ldg(sel + j0) : -1;
        x.t1 = (tile < tiles && j1 < end) ? __ldg(sel + j1) : -1;
    };
    auto stage_pages = [&](HalfIdx &x) {
        x.pg0 = (x.t0 >= 0 && x.t0 / kPage < p.max_pages) ? __ldg(pt + x.t0 / kPage) : -1;
        x.pg1 = (x.t1 >= 0 && x.t1 / kPage < p.max_pages) ? __ldg(pt + x.t1 / kPage) : -1;
    };
    auto stage_rows = [&](int tile, int half, const HalfIdx &x, int &row_lo, int &row_hi, uint64_t &mask, bool &contig,
                          bool &any_bad) {
        const int j0 = begin + tile * kC2Tile + half * 64 + lane, j1 = j0 + 32;
        const bool ok0 = x.pg0 >= 0 && (int64_t)x.pg0 < p.num_pages, ok1 = x.pg1 >= 0 && (int64_t)x.pg1 < p.num_pages;
        any_bad |= (j0 < end && !ok0) || (j1 < end && !ok1);
        const int r0 = ok0 ? x.pg0 * kPage + x.t0 % kPage : -1, r1 = ok1 ? x.pg1 * kPage + x.t1 % kPage : -1;
        const uint32_t m0 = __ballot_sync(0xffffffffu, r0 >= 0), m1 = __ballot_sync(0xffffffffu, r1 >= 0);
        mask = (uint64_t)m0 | ((uint64_t)m1 << 32);
        row_lo = r0 >= 0 ? r0 : 0;           // masked tokens still load a real row (row 0)
        row_hi = r1 >= 0 ? r1 : 0;
        const int base = __shfl_sync(0xffffffffu, row_lo, 0);
        contig = __all_sync(0xffffffffu, r0 == base + lane && r1 == base + 32 + lane);
    };
    // Lane g < 16 takes the rows of tokens 4g..4g+3 of a half.
    auto rows_of_four = [&](int row_lo, int row_hi, int (&r)[4]) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int src = (4 * lane + k) & 31;
            const int a = __shfl_sync(0xffffffffu, row_lo, src), c = __shfl_sync(0xffffffffu, row_hi, src);
            r[k] = lane < 8 ? a : c;
        }
    };

    if (warp == 0) {
        // =========================== K-role producer =====================================
        const uint32_t q_bar = map_to_rank(smem_u32(&ctl->q_full), 0);
        if (lane == 0) {
            if (rank == 0) mbar_expect_tx(&ctl->q_full, 2 * kTileBytes);
            tma_box3d_pair(smem_base + kC2SmemQ, &q_map, q_bar, b * p.heads + h0, 0);
        }
        bool any_bad = bad_len;
        // This CTA's K rows are the tokens of half `rank`; the other half is resolved too because
        // the softmax threads need the validity of all 128 tokens of a tile.
        const int own = (int)rank, oth = own ^ 1;
        HalfIdx a1, b1, a2, b2;              // own / other half, one and two tiles ahead
        int own_lo, own_hi, oth_lo, oth_hi;
        uint64_t mask_own, mask_oth;
        bool contig, contig_oth;
        stage_tokens(0, own, a1);
        stage_tokens(0, oth, b1);
        stage_pages(a1);
        stage_pages(b1);
        stage_rows(0, own, a1, own_lo, own_hi, mask_own, contig, any_bad);
        stage_rows(0, oth, b1, oth_lo, oth_hi, mask_oth, contig_oth, any_bad);
        stage_tokens(1, own, a1);
        stage_tokens(1, oth, b1);
        stage_pages(a1);
        stage_pages(b1);
        stage_tokens(2, own, a2);
        stage_tokens(2, oth, b2);
        bool ok = true;
        for (int i = 0; ok && i < tiles; ++i) {
            if (lane == 0) {
                ctl->valid_mask[i % kMaskRing][own] = mask_own;
                ctl->valid_mask[i % kMaskRing][oth] = mask_oth;
                __threadfence_block();
            }
            int r[4];
            rows_of_four(own_lo, own_hi, r);
            for (int g = 0; g < kKGroups; ++g) {
                if (i > 0) ok = mbar_wait(&ctl->k_empty[g], (i - 1) & 1);
                ok = __all_sync(0xffffffffu, ok) && (*abort_flag == 0);
                if (!ok) break;
                const uint32_t bar = map_to_rank(smem_u32(&ctl->k_full[g]), 0);
                if (lane == 0 && rank == 0) mbar_expect_tx(&ctl->k_full[g], 2 * kKGroupBytes);
                __syncwarp();
                const uint32_t dst = smem_base + kC2SmemK + g * kKGroupBytes;
                if (contig) {
                    if (lane == 0) tma_box3d_pair(dst, &kv_k_map, bar, own_lo, 3 * g);
                } else if (lane < 16) {
#pragma unroll
                    for (int c = 0; c < 3; ++c)
                        tma_gather4_pair(dst + c * kPanelBytes + lane * 512, &kv_map, bar, (3 * g + c) * 64, r[0], r[1], r[2],
                                         r[3]);
                }
            }
            if (!ok) break;
            // advance the index pipeline: rows of tile i+1, page ids of tile i+2, positions of tile i+3
            if (i + 1 < tiles) {
                stage_rows(i + 1, own, a1, own_lo, own_hi, mask_own, contig, any_bad);
                stage_rows(i + 1, oth, b1, oth_lo, oth_hi, mask_oth, contig_oth, any_bad);
            }
            a1 = a2;
            b1 = b2;
            stage_pages(a1);
            stage_pages(b1);
            stage_tokens(i + 3, own, a2);
            stage_tokens(i + 3, oth, b2);
        }
        if (!ok && lane == 0) {
            flag_status(p.status, OMNI_DEV_TIMEOUT);
            *abort_flag = 1;
        }
        if (__any_sync(0xffffffffu, any_bad) && lane == 0 && rank == 0) flag_status(p.status, OMNI_DEV_BAD_INDEX);
    } else if (warp == 6) {
        // =========================== V-role producer =====================================
        bool any_bad = false;
        HalfIdx x1[2], x2[2];
        int lo[2], hi[2];
        uint64_t mask_unused;
        bool contig[2];
        for (int h = 0; h < 2; ++h) {
            stage_tokens(0, h, x1[h]);
            stage_pages(x1[h]);
            stage_rows(0, h, x1[h], lo[h], hi[h], mask_unused, contig[h], any_bad);
            stage_tokens(1, h, x1[h]);
            stage_pages(x1[h]);
            stage_tokens(2, h, x2[h]);
        }
        bool ok = true;
        for (int i = 0; ok && i < tiles; ++i) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (i > 0) ok = mbar_wait(&ctl->v_empty[h], (i - 1) & 1);
                ok = __all_sync(0xffffffffu, ok) && (*abort_flag == 0);
                if (!ok) break;
                const uint32_t bar = map_to_rank(smem_u32(&ctl->v_full[h]), 0);
                if (lane == 0 && rank == 0) mbar_expect_tx(&ctl->v_full[h], 2 * kC2VHalfBytes);
                __syncwarp();
                const uint32_t dst = smem_base + kC2SmemV + h * kC2VHalfBytes;
                if (contig[h]) {
                    if (lane == 0) tma_box3d_pair(dst, &kv_v_map, bar, lo[h], 4 * (int)rank);
                } else {
                    int r[4];
                    rows_of_four(lo[h], hi[h], r);
                    if (lane < 16) {
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            tma_gather4_pair(dst + c * kPanelBytes + lane * 512, &kv_map, bar, ((int)rank * 4 + c) * 64, r[0],
                                             r[1], r[2], r[3]);
                    }
                }
            }
            if (!ok) break;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (i + 1 < tiles) stage_rows(i + 1, h, x1[h], lo[h], hi[h], mask_unused, contig[h], any_bad);
                x1[h] = x2[h];
                stage_pages(x1[h]);
                stage_tokens(i + 3, h, x2[h]);
            }
        }
        if (!ok && lane == 0) {
            flag_status(p.status, OMNI_DEV_TIMEOUT);
            *abort_flag = 1;
        }
    } else if (warp == 1) {
        // =========================== MMA issuer (CTA 0 only) =============================
        // The whole warp runs this loop with warp-uniform control flow and one elected lane issues
        // each MMA / commit: descriptor arithmetic then stays cheap enough to issue an MMA every
        // 32 clocks, which a lone diverged thread cannot.
        if (rank == 0) {
            constexpr uint32_t idesc_qk = instr_desc(128, kC2Tile, 0);
            constexpr uint32_t idesc_pv = instr_desc(128, 256, 1);
            const uint64_t q_desc = smem_desc(smem_base + kC2SmemQ, 16, 1024);
            const uint64_t k_desc = smem_desc(smem_base + kC2SmemK, 16, 1024);
            const uint64_t p_desc = smem_desc(smem_base + kC2SmemP, 16, 1024);
            const uint64_t v_desc = smem_desc(smem_base + kC2SmemV, kPanelBytes, 1024);
            const uint32_t q_lo = (uint32_t)q_desc, k_lo = (uint32_t)k_desc, p_lo = (uint32_t)p_desc, v_lo = (uint32_t)v_desc;
            const uint32_t kmaj_hi = (uint32_t)(q_desc >> 32), v_hi = (uint32_t)(v_desc >> 32);
            bool ok = mbar_wait(&ctl->q_full, 0);
            int qk_t = 0, qk_c = 0, pv_t = 0, pv_h = 0;
            long long idle_since = clock64();
            while (ok && pv_t < tiles) {
                bool progress = false;
                // ---- one 64-token half of O += P V ----
                if (pv_t < qk_t && (pv_h == 1 || mbar_test(&ctl->p_full, pv_t & 1)) &&
                    mbar_test(&ctl->v_full[pv_h], pv_t & 1)) {
                    tc_fence_after();
                    const uint32_t a = p_lo + ((pv_h * kPanelBytes) >> 4);
                    const uint32_t bd = v_lo + ((pv_h * kC2VHalfBytes) >> 4);
                    if (pv_t == 0 && pv_h == 0) {
                        tc_mma_pair_elect<false>(tmem + kColO, a, kmaj_hi, bd, v_hi, idesc_pv);
                        tc_mma_pair_elect<false>(tmem + kColO + 128, a, kmaj_hi, bd + ((2 * kPanelBytes) >> 4), v_hi, idesc_pv);
                    } else {
                        tc_mma_pair_elect<true>(tmem + kColO, a, kmaj_hi, bd, v_hi, idesc_pv);
                        tc_mma_pair_elect<true>(tmem + kColO + 128, a, kmaj_hi, bd + ((2 * kPanelBytes) >> 4), v_hi, idesc_pv);
                    }
#pragma unroll
                    for (int k = 1; k < 4; ++k) {
                        const uint32_t ak = a + ((k * 32) >> 4), bk = bd + ((k * 2048) >> 4);
                        tc_mma_pair_elect<true>(tmem + kColO, ak, kmaj_hi, bk, v_hi, idesc_pv);
                        tc_mma_pair_elect<true>(tmem + kColO + 128, ak, kmaj_hi, bk + ((2 * kPanelBytes) >> 4), v_hi, idesc_pv);
                    }
                    tc_commit_pair_elect(&ctl->v_empty[pv_h]);
                    if (pv_h == 1) {
                        tc_commit_pair_elect(&ctl->pv_done);
                        ++pv_t;
                        pv_h = 0;
                    } else {
                        pv_h = 1;
                    }
                    progress = true;
                }
                // ---- one group of three 64-column panels of S = Q K^T ----
                if (qk_t < tiles && mbar_test(&ctl->k_full[qk_c], qk_t & 1) &&
                    (qk_c > 0 || qk_t < 2 || mbar_test(&ctl->s_empty[qk_t & 1], ((qk_t >> 1) - 1) & 1))) {
                    tc_fence_after();
                    const uint32_t d = tmem + kC2ColS + 64 * (qk_t & 1);
                    const uint32_t off = (qk_c * kKGroupBytes) >> 4;
                    if (qk_c == 0)
                        tc_mma_pair_elect<false>(d, q_lo, kmaj_hi, k_lo, kmaj_hi, idesc_qk);
                    else
                        tc_mma_pair_elect<true>(d, q_lo + off, kmaj_hi, k_lo + off, kmaj_hi, idesc_qk);
#pragma unroll
                    for (int k = 1; k < 12; ++k) {
                        const uint32_t o = off + (((k >> 2) * kPanelBytes + (k & 3) * 32) >> 4);
                        tc_mma_pair_elect<true>(d, q_lo + o, kmaj_hi, k_lo + o, kmaj_hi, idesc_qk);
                    }
                    tc_commit_pair_elect(&ctl->k_empty[qk_c]);
                    if (++qk_c == kKGroups) {
                        tc_commit_pair_elect(&ctl->s_full[qk_t & 1]);
                        qk_c = 0;
                        ++qk_t;
                    }
                    progress = true;
                }
                if (progress)
                    idle_since = clock64();
                else if (clock64() - idle_since > kWaitCycles || *abort_flag)
                    ok = false;
                ok = __all_sync(0xffffffffu, ok);
            }
            if (!ok && lane == 0) {
                flag_status(p.status, OMNI_DEV_TIMEOUT);
                *abort_flag = 1;
            }
        }
        __syncwarp();
    } else {
        // =========================== softmax + epilogue =================================
        const int quarter = warp & 3;
        const int row = (quarter & 1) * 32 + lane;          // head row within this CTA
        const int half = quarter >> 1;                      // token half of S / column half of O
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const uint32_t s_empty0 = map_to_rank(smem_u32(&ctl->s_empty[0]), 0);
        const uint32_t s_empty1 = map_to_rank(smem_u32(&ctl->s_empty[1]), 0);
        const uint32_t p_full_leader = map_to_rank(smem_u32(&ctl->p_full), 0);
        uint8_t *p_row = smem + kC2SmemP + half * kPanelBytes + row * 128;
        float m_ref = -INFINITY, l = 0.f;
        bool ok = true;
        for (int i = 0; i < tiles; ++i) {
            const int buf = i & 1;
            ok = mbar_wait(&ctl->s_full[buf], (i >> 1) & 1);
            if (!__all_sync(0xffffffffu, ok)) {
                ok = false;
                break;
            }
            tc_fence_after();
            uint32_t sv[64];
            tc_ld32(tmem + lane_base + kC2ColS + 64 * buf, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
            tc_ld32(tmem + lane_base + kC2ColS + 64 * buf + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
            tc_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(buf ? s_empty1 : s_empty0);
            const uint64_t valid = ctl->valid_mask[i % kMaskRing][half];
            float mt = -INFINITY;
#pragma unroll
            for (int j = 0; j < 64; ++j) {
                const float x = ((valid >> j) & 1ull) ? __uint_as_float(sv[j]) * p.scale_log2 : -INFINITY;
                sv[j] = __float_as_uint(x);
                mt = fmaxf(mt, x);
            }
            // the other token half of this row lives in the warp two quarters away
            ctl->xchg[i & 1][half][row] = mt;
            mbar_arrive(&ctl->x_bar);
            ok = mbar_wait(&ctl->x_bar, i & 1);
            if (!__all_sync(0xffffffffu, ok)) {
                ok = false;
                break;
            }
            mt = fmaxf(mt, ctl->xchg[i & 1][half ^ 1][row]);
            float factor = 1.f;
            bool moved = false;
            if (mt > m_ref + kRescaleThreshold || (m_ref == -INFINITY && mt > -INFINITY)) {
                factor = exp2f(m_ref - mt);
                m_ref = mt;
                moved = true;
            }
            const float mr = (m_ref == -INFINITY) ? 0.f : m_ref;
            float sum = 0.f;
            uint32_t pk[32];
#pragma unroll
            for (int j = 0; j < 64; j += 2) {
                const float e0 = exp2f(__uint_as_float(sv[j]) - mr), e1 = exp2f(__uint_as_float(sv[j + 1]) - mr);
                sum += e0 + e1;
                pk[j >> 1] = pack_bf16(e0, e1);
            }
            l = l * factor + sum;
            if (i > 0) {
                ok = mbar_wait(&ctl->pv_done, (i - 1) & 1);
                if (!__all_sync(0xffffffffu, ok)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                if (__any_sync(0xffffffffu, moved)) {
#pragma unroll 1
                    for (int c = 0; c < 256; c += 32) {
                        uint32_t ov[32];
                        tc_ld32(tmem + lane_base + kColO + c, ov);
                        tc_wait_ld();
#pragma unroll
                        for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * factor);
                        tc_st32(tmem + lane_base + kColO + c, ov);
                    }
                    tc_wait_st();
                }
            }
            // P row half: 64 tokens x bf16 = 128 B = eight 16-byte chunks, chunk c stored at c ^ (row % 8)
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int chunk = c ^ (row & 7);
                *reinterpret_cast<uint4 *>(p_row + chunk * 16) =
                    make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
            }
            fence_async_smem();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(p_full_leader);
        }
        if (ok) {
            ok = mbar_wait(&ctl->pv_done, (tiles - 1) & 1);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            // total row sum: add the other token half's partial sum
            ctl->xchg[tiles & 1][half][row] = l;
            mbar_arrive(&ctl->x_bar);
            ok = mbar_wait(&ctl->x_bar, tiles & 1);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            const float lt = l + ctl->xchg[tiles & 1][half ^ 1][row];
            const float inv = lt > 0.f ? 1.f / lt : 0.f;
            const int h = h0 + row;
            const bool store = h < p.heads;
            const size_t u = p.splits == 1 ? ((size_t)b * p.heads + h) : (((size_t)b * p.splits + s) * p.heads + h);
#pragma unroll 1
            for (int c = 0; c < 256; c += 32) {
                uint32_t ov[32];
                __syncwarp();
                tc_ld32(tmem + lane_base + kColO + c, ov);
                tc_wait_ld();
                const int col = half * 256 + c;
                if (!store) {
                    // padded head row: nothing to write
                } else if (p.splits == 1) {
                    uint4 *o = reinterpret_cast<uint4 *>(p.out + u * kDv + col);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint4 w;
                        w.x = pack_bf16(__uint_as_float(ov[8 * j]) * inv, __uint_as_float(ov[8 * j + 1]) * inv);
                        w.y = pack_bf16(__uint_as_float(ov[8 * j + 2]) * inv, __uint_as_float(ov[8 * j + 3]) * inv);
                        w.z = pack_bf16(__uint_as_float(ov[8 * j + 4]) * inv, __uint_as_float(ov[8 * j + 5]) * inv);
                        w.w = pack_bf16(__uint_as_float(ov[8 * j + 6]) * inv, __uint_as_float(ov[8 * j + 7]) * inv);
                        o[j] = w;
                    }
                } else {
                    float4 *o = reinterpret_cast<float4 *>(p.part_out + u * kDv + col);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        o[j] = make_float4(__uint_as_float(ov[4 * j]) * inv, __uint_as_float(ov[4 * j + 1]) * inv,
                                           __uint_as_float(ov[4 * j + 2]) * inv, __uint_as_float(ov[4 * j + 3]) * inv);
                }
            }
            if (store && half == 0) {
                const float lse = lt > 0.f ? (m_ref + log2f(lt)) * kLn2 : -INFINITY;
                if (p.splits == 1)
                    p.lse[u] = lse;
                else
                    p.part_lse[u] = lse;
            }
        } else if (lane == 0) {
            flag_status(p.status, OMNI_DEV_TIMEOUT);
            *abort_flag = 1;
        }
    }

    // ---- tear-down: nobody leaves while the other CTA may still touch this one's memory --
    if (*abort_flag) {
        // a wait ran out: give copies that are still in flight time to land before anyone exits
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

inline omni_status_t launch_tc2_decode(const DecodeParams &p, cudaStream_t stream)
{
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return OMNI_ERR_CUDA;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(tc2_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kC2SmemBytes) !=
            cudaSuccess)
            return OMNI_ERR_CUDA;
        attr_set[dev] = true;
    }
    CUtensorMap q_map, kv_map, kv_k_map, kv_v_map;
    if (!make_panel_map(&q_map, p.q, (uint64_t)p.batch * p.heads, kPanels)) return OMNI_ERR_CUDA;
    if (!make_row_map(&kv_map, p.kv, (uint64_t)p.num_pages * kPage, 1)) return OMNI_ERR_CUDA;
    if (!make_panel_map(&kv_k_map, p.kv, (uint64_t)p.num_pages * kPage, 3)) return OMNI_ERR_CUDA;
    if (!make_panel_map(&kv_v_map, p.kv, (uint64_t)p.num_pages * kPage, 4)) return OMNI_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.batch * p.splits * 2));
    cfg.blockDim = dim3(kC2Threads);
    cfg.dynamicSmemBytes = kC2SmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, tc2_decode_kernel, q_map, kv_map, kv_k_map, kv_v_map, p) == cudaSuccess ? OMNI_OK
                                                                                                      : OMNI_ERR_CUDA;
}

}  // namespace omni
