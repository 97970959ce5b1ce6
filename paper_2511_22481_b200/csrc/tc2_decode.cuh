// Paired-CTA tensor-core decode kernel for sm_100a (the fast path for more than 64 heads).
//
// A cluster of two CTAs owns all heads of one (request, split): CTA r serves heads
// [64r, 64r+64).  The pair issues cta_group::2 MMAs with M = 128 (64 rows per CTA), which run
// the tensor pipe of each SM at full rate where a lone M = 64 MMA runs it at half rate, and it
// halves the operand bytes each SM must hold.  Per 64-token tile:
//   S = Q K^T   M=128, N=64 tokens, K=576: every CTA supplies its 64 Q rows and the K rows of
//               ITS 32 tokens of the tile ("K role": 32 tokens x 576 columns, 36 KiB)
//   O += P V    M=128, N=256 per instruction (two of them), K=64 tokens: every CTA supplies its
//               64 P rows and, for all 64 tokens, ITS 256 value columns ("V role": 64 tokens x
//               256 columns, 32 KiB; CTA r holds columns [256r, 256r+256))
// The two roles overlap only in a quarter of the tile, at different addresses in the two CTAs,
// so each role is loaded on its own (1.9x the tile's bytes cross L2 -> shared memory, which L2
// sustains; each byte leaves HBM once because the pair runs together).
//
// Both roles, P and S are double buffered, so the loads of tile i+2 are in flight while tile i
// is consumed and Q K^T of tile i+1 overlaps the softmax of tile i.  Every refill is ONE 3-D TMA
// box {64 columns, rows, panels}: the copy engine sustains only about 4 M instructions/s per SM,
// so 8 KiB boxes cap an SM near 32 GB/s while 32-72 KiB boxes reach 90-150 GB/s.  Tiles that are
// not 64 consecutive pool rows are gathered row by row with cp.async (see below).
//
// All MMAs are issued by warp 1 of CTA 0 in "whatever is ready" order: the whole warp runs the
// loop with warp-uniform control flow and one elected lane issues each instruction (a lone
// diverged thread cannot feed the tensor pipe: it needs ~110 clocks per MMA, the elected form
// issues one every 25-64 clocks).  Completion is broadcast to both CTAs with multicast commits.
//
// Warps per CTA: 0 K-role producer, 1 MMA issuer (CTA 0 only) + tensor-memory owner,
// 2-5 and 8-11 softmax / epilogue (two groups of four warps that take the tiles in turn: warps
// 2-5 the even tiles, 8-11 the odd ones, 32 of a tile's 64 tokens per thread; all eight share
// the epilogue), 6 V-role producer, 7 L2 prefetcher (CTA 0 only): shared memory holds
// only two tiles, about one HBM latency of work, so each whole page is pulled into L2 one tile
// before its K-role load and the shared-memory refills start from a line already on its way.
//
// Tensor memory per CTA (a 64-row slice of an M=128 pair accumulator keeps columns [0, N/2) in
// lanes 0-63 and columns [N/2, N) in lanes 64-127):
//   columns   0..255  O: two N=256 accumulators; lane L, column x  <->  head row L%64,
//                        value column 256*(L/64) + x
//   columns 256..287  S buffer 0: lane L, column x <-> head row L%64, token 32*(L/64) + x
//   columns 288..319, 320..351  S buffers 1, 2 (Q K^T runs two tiles ahead of P V)
//
// Splits of a request are merged in one of three ways chosen by the host: inside a cluster of
// two pairs (two splits, see cluster_merge_exchange), by a separate merge kernel over fp32
// partial results, or by the last CTA to finish a request's head half (a counter per (request,
// head half) in the workspace).
#pragma once

#include <type_traits>

#include "merge.cuh"
#include "tc_decode.cuh"

namespace omni {

constexpr int kC2Tile = 64;                              // tokens per tile of the pair
constexpr int kC2Threads = 384;
// Tiles the L2 prefetch runs ahead of the K-role loads.  Measured on B200: the further ahead, the
// slower (1: 30.4 us, 5: 32.3 us, 12: 35.0 us per step on the batch-32 benchmark shape; the same
// order at batch 128): a line prefetched long before its use is often gone again by then.
constexpr int kPrefetchAhead = 1;
constexpr int kC2KBytes = kPanels * 32 * 128;            // K role: 9 panels x [32 tokens x 128 B]
constexpr int kC2KPanel = 32 * 128;
constexpr int kC2VBytes = 4 * kPanelBytes;               // V role: 4 panels x [64 tokens x 128 B]
constexpr int kC2SmemQ = 0;                              // 9 panels x [64 heads x 128 B]
constexpr int kC2SmemK = kC2SmemQ + kTileBytes;          // 2 stages
constexpr int kC2SmemV = kC2SmemK + 2 * kC2KBytes;       // 2 stages
constexpr int kC2SmemP = kC2SmemV + 2 * kC2VBytes;       // 2 buffers x [64 heads x 128 B]
constexpr int kC2SmemCtl = kC2SmemP + 2 * kPanelBytes;
constexpr int kC2SmemCtlBytes = 3072;
constexpr int kC2SmemBytes = kC2SmemCtl + kC2SmemCtlBytes;   // no alignment slack: the base is checked at run time
constexpr uint32_t kC2ColS = 256;
// Validity masks travel from the K producer to the softmax warps through a small ring.  The
// producer writes the mask of tile i+1 once the score MMAs of tile i-2 have retired, and those
// were issued only after every softmax warp had read the scores of tile i-5 (three score
// buffers), i.e. after tile i-6 was finished: seven tiles can be live, so the ring holds eight.
constexpr int kMaskRing = 8;

struct C2Control {
    uint64_t q_full;
    uint64_t k_full[2];
    uint64_t k_empty[2];
    uint64_t v_full[2];
    uint64_t s_full[3];
    uint64_t s_empty[3];
    uint64_t p_full[2];
    uint64_t pv_done[2];                 // P V of a tile retired: frees its V stage and its P buffer
    uint64_t x_bar;                      // all softmax threads: exchange of the final row sums
    uint64_t exit_bar;                   // both CTAs of the pair are done with tensor memory
    uint64_t valid_mask[kMaskRing];      // per tile: validity of its 64 tokens
    float xchg[2][4][64];                // row maxima: [group][2 * parity of the group's tile + token half][head row]; at the end the slots a group no longer uses carry its partial row sums
    uint32_t tmem_base;
    uint32_t abort;
    uint32_t merge_flag;
    uint32_t xfail;                      // cluster merge: some wait of this CTA ran out (decided CTA-wide)
    int32_t k_progress;                  // tiles whose K loads the producer has started (L2 prefetch pacing)
    uint64_t recv_bar;                   // cluster merge: the partner's block has arrived
    uint64_t ready_bar;                  // cluster merge: the partner's main loop is over
    uint64_t xg_bar[2];                  // row-maximum exchange inside either softmax group
    uint64_t ref_bar;                    // the reference maxima after a tile are published (4 warps of its group)
    float ref[2][64];                    // [tile parity][head row]: running reference maximum after that tile
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

// Execution-only rendezvous of the pair (no memory ordering): used before the tensor-memory
// release, where the release-ordered form would first wait for every global store of the
// epilogue to be acknowledged (about 9 us here).
__device__ __forceinline__ void cluster_sync_relaxed()
{
    asm volatile("barrier.cluster.arrive.relaxed.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");
}

// Rendezvous of the cluster after the barriers were initialised.  The initialising thread has
// issued the barrier-init fence, so the arrive needs no release of its own (a release-ordered
// arrive cost half a microsecond of every launch); nothing else that the other CTAs read was
// written before it.
__device__ __forceinline__ void cluster_sync_after_init()
{
    asm volatile("barrier.cluster.arrive.relaxed.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// 3-D box {64 columns, box rows, n column panels} loaded by one CTA of a pair: lands panel-major,
// i.e. as n consecutive [rows x 128 B] swizzled panels.  The transaction bytes are credited to
// `bar_cluster_addr`, which may be a barrier of the other CTA of the pair.
__device__ __forceinline__ void tma_box3d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar_cluster_addr,
                                               int row, int panel)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(0), "r"(row), "r"(panel), "r"(bar_cluster_addr)
        : "memory");
}

// Row gathers without the copy engine.  A 4-row TMA gather moves 512 bytes per instruction and
// the engine takes ~60 clocks for each, which bounds token-level selections; a warp-wide 16-byte
// cp.async moves the same 512 bytes (four rows x 128 B, eight lanes per row) through the load/store
// path at several times that rate.  The lanes place their chunks in the 128-byte-swizzled operand
// layout themselves, and the warp credits the bytes to the stage's barrier with an explicit
// complete_tx once its copies have landed, exactly as a TMA copy would have.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int kPending>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(kPending) : "memory");
}
// All lanes: wait for this lane's copies of the stage (all but the `newer` most recent groups),
// make them visible to the tensor core's proxy, then lane 0 credits `bytes` to the barrier.
__device__ __noinline__ void retire_gathered_stage(uint32_t bar_cluster_addr, uint32_t bytes, bool newer_in_flight,
                                                      int lane)
{
    if (newer_in_flight)
        cp_async_wait<1>();
    else
        cp_async_wait<0>();
    fence_async_smem();
    __syncwarp();
    if (lane == 0) {
        // The rows are in this CTA's shared memory (wait_group returned in every lane, the proxy
        // fence and the warp barrier order them before this point) and it is this CTA's own
        // tensor core that will read them, so a CTA-scope fence is what orders them before the
        // credit.  A cluster-scope fence here would also wait for the next tile's copies and the
        // index loads this lane has in flight: measured at ~0.9 us per tile.
        asm volatile("fence.acq_rel.cta;" ::: "memory");
        asm volatile("mbarrier.complete_tx.relaxed.cluster.shared::cluster.b64 [%0], %1;" ::"r"(bar_cluster_addr), "r"(bytes)
                     : "memory");
    }
}

// The two gathers are kept out of line so that the producers' loops stay as small as they are
// for selections that never need them.
// K role: 32 rows x 9 panels; eight lanes per row, four rows per instruction; chunk c of row r
// lands at chunk c ^ (r % 8) of its 128-byte line.
__device__ __noinline__ void gather_k_rows(uint32_t dst, const char *kv_bytes, int own_row, int lane)
{
    const int ch = lane & 7;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        const int r = 4 * g + (lane >> 3);
        const int src_row = __shfl_sync(0xffffffffu, own_row, r);
        const char *src = kv_bytes + (size_t)src_row * (kDqk * 2) + ch * 16;
        const uint32_t d = dst + r * 128 + ((ch ^ (r & 7)) << 4);
#pragma unroll
        for (int c = 0; c < kPanels; ++c) cp_async16(d + c * (32 * 128), src + c * 128);
    }
    cp_async_commit();
}

// V role: 64 rows x the four panels of this CTA's value columns (`kv_cols` points at the first).
__device__ __noinline__ void gather_v_rows(uint32_t dst, const char *kv_cols, int row_lo, int row_hi, int lane)
{
    const int ch = lane & 7;
#pragma unroll
    for (int g = 0; g < 16; ++g) {
        const int r = 4 * g + (lane >> 3);
        const int a = __shfl_sync(0xffffffffu, row_lo, r & 31), c2 = __shfl_sync(0xffffffffu, row_hi, r & 31);
        const int src_row = r < 32 ? a : c2;
        const char *src = kv_cols + (size_t)src_row * (kDqk * 2) + ch * 16;
        const uint32_t d = dst + r * 128 + ((ch ^ (r & 7)) << 4);
#pragma unroll
        for (int c = 0; c < 4; ++c) cp_async16(d + c * kPanelBytes, src + c * 128);
    }
    cp_async_commit();
}

// Pair MMA executed by a whole converged warp: one elected lane issues the instruction.  The
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

// Arrive on the barrier at this shared-memory offset in BOTH CTAs once all MMAs issued so far by
// the elected lane have retired.
__device__ __forceinline__ void tc_commit_pair_elect(uint64_t *bar, uint16_t both)
{
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "elect.sync _|q, 0xffffffff;\n\t"
        "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n\t}"
        ::"r"(smem_u32(bar)), "h"(both)
        : "memory");
}

// Split-KV merge inside a cluster of two pairs, i.e. the two splits of one request (cluster
// merge).  CTA `crank` and its partner `crank ^ 2` serve the same 64 heads in the two splits.
// Instead of writing fp32 partial results to global memory for a second kernel to read back,
// the two exchange what the other needs through distributed shared memory.  Of every head row
// split 0 finishes value columns [0,128) and [256,384), split 1 the other two quarters: these are
// the columns of softmax warps 2-5 and 8-11 in tensor memory, so in either CTA one warp per
// scheduler is a "sender" (its columns are finished by the partner) and one a "keeper":
//   1. the senders normalise their half by the row sums and write it, followed by the
//      log-sum-exp of the split for every head row, to one block of shared memory, which four
//      bulk shared-memory-to-shared-memory copies take to the partner, each as soon as its
//      quarter of the block is written;
//   2. the keepers wait for the partner's block, weigh their own half (still in tensor memory)
//      and the received one by exp(lse_split - lse_total), add them and store bf16 rows as whole
//      128-byte lines through warp-private staging tiles.
// The copy lands in shared memory that held the partner's operand tiles, so it is not sent
// before the partner has said that its main loop is over (`ready_bar`, a remote arrive that the
// partner fires as soon as its last P V has retired, while this CTA is still staging).
// Called by every thread of the CTA after the main loop.
template <class Control>
__device__ __forceinline__ void cluster_merge_exchange(const DecodeParams &p, Control *ctl, uint8_t *smem,
                                                       uint32_t tmem, int b, int s, uint32_t crank, int h0,
                                                       int head_rows, bool active, bool main_ok, float cm_lse, float cm_inv)
{
    // The block travels as four chunks, so that the copy of one overlaps the staging of the next:
    // chunk q holds, for every head row, the q-th 32 columns of both 128-column runs that are sent.
    constexpr uint32_t kChunkPitch = 2 * 128 + 16;       // row-per-lane 16-byte accesses do not conflict
    constexpr uint32_t kChunkBytes = 64 * kChunkPitch;   // 17,408
    constexpr uint32_t kRowsBytes = 4 * kChunkBytes;
    constexpr uint32_t kBlockBytes = kRowsBytes + 256;   // + 64 log-sum-exps: 69,888
    constexpr uint32_t kStagePitch = 144, kStageBytes = 32 * kStagePitch;
    static_assert(2 * kBlockBytes + 8 * kStageBytes <= 221184, "exchange tiles must end below the control block and the 8-bit kernel's auxiliary arrays");
    uint8_t *send = smem, *stages = smem + kBlockBytes, *recv = smem + kBlockBytes + 8 * kStageBytes;
    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;
    const bool is_softmax = (warp >= 2 && warp <= 5) || warp >= 8;
    if (!is_softmax) return;
    const int quarter = warp & 3, sub = warp >= 8 ? 1 : 0;
    const int row = (quarter & 1) * 32 + lane, half = quarter >> 1;
    const uint32_t partner = crank ^ 2u;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    volatile uint32_t *xfail = &ctl->xfail;
    if (!main_ok && lane == 0) *xfail = 1u;
    // The partner may overwrite this CTA's operand tiles once it has been told that the main loop
    // here is over.  Warp 2 says so at the end of a main loop that went well; after one that did
    // not (or that never ran: an empty split) the same thread says so here, so that the arrive is
    // fired exactly once per launch whatever happened.
    if (warp == 2 && lane == 0 && (!active || !main_ok)) mbar_arrive_cluster(map_to_rank(smem_u32(&ctl->ready_bar), partner));

    // No warp leaves this function early and no barrier below depends on how a wait ended: the
    // four sending warps always meet at their named barrier, every wait is bounded, and a wait
    // that ran out only marks the launch as failed (its results are then unspecified).
    tc_fence_after();
    if (sub != s) {
        // ---- sender: this thread's 128 value columns are finished by the other split ----------
        if (half == 0) reinterpret_cast<float *>(send + kRowsBytes)[row] = cm_lse;
        bool ready = true;                                // (sending warp) the partner's operand tiles are dead
#pragma unroll 1
        for (int q = 0; q < 4; ++q) {
            uint32_t ov[32];
            __syncwarp();
            if (active) {
                tc_ld32(tmem + lane_base + kColO + 128 * sub + q * 32, ov);
                tc_wait_ld();
            }
            uint4 *o = reinterpret_cast<uint4 *>(send + q * kChunkBytes + (size_t)row * kChunkPitch + half * 128);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                // an empty or fully masked split contributes exact zeros
                o[j] = (active && cm_inv != 0.f)
                           ? make_uint4(__float_as_uint(__uint_as_float(ov[4 * j]) * cm_inv),
                                        __float_as_uint(__uint_as_float(ov[4 * j + 1]) * cm_inv),
                                        __float_as_uint(__uint_as_float(ov[4 * j + 2]) * cm_inv),
                                        __float_as_uint(__uint_as_float(ov[4 * j + 3]) * cm_inv))
                           : make_uint4(0u, 0u, 0u, 0u);
            }
            fence_async_smem();                           // the bulk copy reads what the threads wrote
            asm volatile("bar.sync 2, 128;" ::: "memory"); // the four sending warps
            if (quarter == 0) {
                if (q == 0) {
                    ready = mbar_wait(&ctl->ready_bar, 0);
                    ready = __all_sync(0xffffffffu, ready);
                    if (!ready && lane == 0) {
                        *xfail = 1u;
                        flag_status(p.status, OMNI_DEV_TIMEOUT | OMNI_DEV_ROLE_SOFTMAX);
                    }
                }
                if (ready && lane == 0) {
                    const uint32_t bytes = q == 3 ? kChunkBytes + 256 : kChunkBytes;       // the last one takes the log-sum-exps along
                    const uint32_t dst = map_to_rank(smem_u32(recv + q * kChunkBytes), partner);
                    const uint32_t bar = map_to_rank(smem_u32(&ctl->recv_bar), partner);
                    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(dst), "r"(smem_u32(send + q * kChunkBytes)), "r"(bytes), "r"(bar)
                                 : "memory");
                }
            }
        }
    } else if (quarter == 0 && lane == 0) {
        mbar_expect_tx(&ctl->recv_bar, kBlockBytes);
    }

    // ---- finish: the columns kept here (those of the warps with sub == s) never left tensor
    // memory.  Once the partner's block is in, all eight warps take part: a warp can read any
    // column of its tensor-memory lane quarter, so the keeping warp of a quarter finishes the
    // first 64 of its 128 columns and the sending warp of the same quarter, its block gone, the
    // other 64.  A thread mixes its accumulator row with the received one and the warp writes the
    // bf16 rows out as whole 128-byte lines through its private staging tile.
    {
        bool got = mbar_wait(&ctl->recv_bar, 0);
        got = __all_sync(0xffffffffu, got);
        if (!got && lane == 0) {
            *xfail = 1u;
            flag_status(p.status, OMNI_DEV_TIMEOUT | OMNI_DEV_ROLE_SOFTMAX);
        }
    }
    // weights of the two splits for this head row, final log-sum-exp
    const float other = reinterpret_cast<const float *>(recv + kRowsBytes)[row];
    const float mx = fmaxf(cm_lse, other);
    float total = -INFINITY, w_own = 0.f, w_other = 0.f;
    if (mx > -INFINITY) {
        total = mx + logf(exp2f((cm_lse - mx) * kLog2e) + exp2f((other - mx) * kLog2e));
        if (cm_lse > -INFINITY) w_own = exp2f((cm_lse - total) * kLog2e);
        if (other > -INFINITY) w_other = exp2f((other - total) * kLog2e);
    }
    if (s == 0 && sub == 0 && half == 0 && row < head_rows) p.lse[(size_t)b * p.heads + h0 + row] = total;
    // An accumulator that carries no weight is not read at all (that of an empty split was never
    // written, that of a fully masked one may hold anything); the partner sends exact zeros then.
    const bool use_own = active && cm_inv != 0.f && w_own != 0.f;
    const float f_own = use_own ? w_own * cm_inv : 0.f, f_other = w_other;
    const int col = 128 * s + (sub == s ? 0 : 64);                        // first of this thread's 64 columns within its half
    uint8_t *buf = stages + (size_t)(sub * 4 + quarter) * kStageBytes;
    const int row0 = (quarter & 1) * 32;                                  // first head row of this warp
    uint8_t *gq = reinterpret_cast<uint8_t *>(p.out + ((size_t)b * p.heads + h0 + row0) * kDv + half * 256 + col);
    const int rows_here = max(0, min(32, head_rows - row0));
    const uint8_t *theirs = recv + (sub == s ? 0 : 2) * kChunkBytes + (size_t)row * kChunkPitch + half * 128;
    uint4 *mine = reinterpret_cast<uint4 *>(buf + lane * kStagePitch);
    tc_fence_after();
#pragma unroll
    for (int c2 = 0; c2 < 2; ++c2) {
        uint32_t ov[32];
        if (use_own) {
            tc_ld32(tmem + lane_base + kColO + col + c2 * 32, ov);
            tc_wait_ld();
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) ov[j] = 0u;
        }
        const uint4 *r4 = reinterpret_cast<const uint4 *>(theirs + c2 * kChunkBytes);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint4 ra = r4[2 * j], rb = r4[2 * j + 1];
            auto mix = [&](uint32_t own, uint32_t got) { return fmaf(f_own, __uint_as_float(own), f_other * __uint_as_float(got)); };
            uint4 w;
            w.x = pack_bf16(mix(ov[8 * j], ra.x), mix(ov[8 * j + 1], ra.y));
            w.y = pack_bf16(mix(ov[8 * j + 2], ra.z), mix(ov[8 * j + 3], ra.w));
            w.z = pack_bf16(mix(ov[8 * j + 4], rb.x), mix(ov[8 * j + 5], rb.y));
            w.w = pack_bf16(mix(ov[8 * j + 6], rb.z), mix(ov[8 * j + 7], rb.w));
            mine[c2 * 4 + j] = w;
        }
    }
    __syncwarp();
    uint4 v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k)
        v[k] = *reinterpret_cast<const uint4 *>(buf + (4 * k + (lane >> 3)) * kStagePitch + (lane & 7) * 16);
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int r = 4 * k + (lane >> 3);
        if (r < rows_here) *reinterpret_cast<uint4 *>(gq + (size_t)r * (kDv * 2) + (lane & 7) * 16) = v[k];
    }
}

// An empty split (no tokens): zeros and -inf in place of a result.  Called by all threads.
__device__ __forceinline__ void c2_store_empty(const DecodeParams &p, int b, int s, int h0, int head_rows, int warp, int lane)
{
    for (int r = warp; r < head_rows; r += kC2Threads / 32) {
        const int h = h0 + r;
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
    if (p.splits > 1 && p.counters != nullptr) __threadfence();
}

// With more work units than the device runs at once, CTAs start in index order, so the requests
// are taken longest first (ties by index): a long request that started last would otherwise run
// on alone at the end.  Every CTA ranks the (at most 256) selection sizes itself: request j has
// rank #{i : n_i > n_j, or n_i = n_j and i < j}, and the pair whose place in the grid is `slot`
// takes the request of that rank.  lens: shared memory nobody uses yet (batch ints); flag: a
// shared word.  Called by all threads; returns the request.
__device__ __forceinline__ int c2_request_by_length_rank(const DecodeParams &p, int *lens, uint32_t *flag, int slot)
{
    for (int j = threadIdx.x; j < p.batch; j += kC2Threads) lens[j] = load_selection(p, j).n;
    __syncthreads();
    for (int j = threadIdx.x; j < p.batch; j += kC2Threads) {
        const int nj = lens[j];
        int before = 0;
        for (int i = 0; i < p.batch; ++i) before += (lens[i] > nj) || (lens[i] == nj && i < j);
        if (before == slot) *flag = (uint32_t)j;
    }
    __syncthreads();
    const int b = (int)*flag;
    __syncthreads();                                          // the shared memory is handed to the producers next
    return b;
}

// Epilogue of a work unit whose result leaves through global memory (final bf16 rows, or fp32
// partial rows of a split).  Each of the eight softmax warps owns 32 rows x 128 value columns
// of the accumulator: warp quarter q = warp % 4 serves head rows 32 * (q % 2) + lane and value
// columns 256 * (q / 2) + 128 * sub + [0, 128), sub = 1 for warps 8-11.  It moves them out in
// rounds of 128 bytes per row: tensor memory -> registers (scaled by 1 / lt) -> a warp-private
// staging tile in shared memory (all operand buffers are dead by now; 144-byte pitch, so
// neither the row-per-lane writes nor the line-per-8-lanes reads conflict) -> global memory as
// whole 128-byte lines, four rows per instruction.  The staging tile is double buffered and no
// CTA-wide barrier is needed, so the stores of one round overlap the tensor-memory reads of the
// next.  lt: the row's sum of weights; m_ref: its reference maximum (log2 units).
__device__ __forceinline__ void c2_store_result(const DecodeParams &p, uint8_t *smem, uint32_t tmem, int warp, int lane,
                                                int b, int s, int h0, int head_rows, float lt, float m_ref)
{
    const int quarter = warp & 3;
    const int sub = warp >= 8 ? 1 : 0;
    const int row = (quarter & 1) * 32 + lane;
    const int part = (quarter >> 1) * 2 + sub;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const float inv = lt > 0.f ? 1.f / lt : 0.f;
    const int h = h0 + row;
    const bool final_out = p.splits == 1;
    const size_t u = final_out ? ((size_t)b * p.heads + h) : (((size_t)b * p.splits + s) * p.heads + h);
    constexpr uint32_t kStagePitch = 144, kStageBytes = 32 * kStagePitch;
    const int widx = sub * 4 + ((warp - 2) & 3);                         // 0..7
    uint8_t *stage = smem + (size_t)widx * 2 * kStageBytes;
    const uint32_t row_bytes = final_out ? kDv * 2 : kDv * 4;
    const int row0 = (quarter & 1) * 32;                                  // first head row of this warp
    // global address of (row0, this warp's first value column)
    const size_t u0 = final_out ? ((size_t)b * p.heads + h0 + row0) : (((size_t)b * p.splits + s) * p.heads + h0 + row0);
    uint8_t *gbase = (final_out ? reinterpret_cast<uint8_t *>(p.out + u0 * kDv)
                                : reinterpret_cast<uint8_t *>(p.part_out + u0 * kDv)) + part * (row_bytes / 4);
    const int rows_here = max(0, min(32, head_rows - row0));              // rows of this warp that exist
    const int rounds = final_out ? 2 : 4;
#pragma unroll 1
    for (int q = 0; q < rounds; ++q) {
        uint8_t *buf = stage + (q & 1) * kStageBytes;
        uint4 *mine = reinterpret_cast<uint4 *>(buf + lane * kStagePitch);
        __syncwarp();
        if (final_out) {
            // 64 columns -> 128 bytes of bf16
#pragma unroll
            for (int c2 = 0; c2 < 2; ++c2) {
                uint32_t ov[32];
                tc_ld32(tmem + lane_base + kColO + 128 * sub + q * 64 + c2 * 32, ov);
                tc_wait_ld();
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint4 w;
                    w.x = pack_bf16(__uint_as_float(ov[8 * j]) * inv, __uint_as_float(ov[8 * j + 1]) * inv);
                    w.y = pack_bf16(__uint_as_float(ov[8 * j + 2]) * inv, __uint_as_float(ov[8 * j + 3]) * inv);
                    w.z = pack_bf16(__uint_as_float(ov[8 * j + 4]) * inv, __uint_as_float(ov[8 * j + 5]) * inv);
                    w.w = pack_bf16(__uint_as_float(ov[8 * j + 6]) * inv, __uint_as_float(ov[8 * j + 7]) * inv);
                    mine[c2 * 4 + j] = w;
                }
            }
        } else {
            // 32 columns -> 128 bytes of fp32
            uint32_t ov[32];
            tc_ld32(tmem + lane_base + kColO + 128 * sub + q * 32, ov);
            tc_wait_ld();
#pragma unroll
            for (int j = 0; j < 8; ++j)
                mine[j] = make_uint4(__float_as_uint(__uint_as_float(ov[4 * j]) * inv),
                                     __float_as_uint(__uint_as_float(ov[4 * j + 1]) * inv),
                                     __float_as_uint(__uint_as_float(ov[4 * j + 2]) * inv),
                                     __float_as_uint(__uint_as_float(ov[4 * j + 3]) * inv));
        }
        __syncwarp();
        uint8_t *gq = gbase + q * 128;
        uint4 v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k)
            v[k] = *reinterpret_cast<const uint4 *>(buf + (4 * k + (lane >> 3)) * kStagePitch + (lane & 7) * 16);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int r = 4 * k + (lane >> 3);
            if (r < rows_here) *reinterpret_cast<uint4 *>(gq + (size_t)r * row_bytes + (lane & 7) * 16) = v[k];
        }
    }
    if (h < p.heads && part == 0) {
        const float lse = lt > 0.f ? (m_ref + log2f(lt)) * kLn2 : -INFINITY;
        if (final_out)
            p.lse[u] = lse;
        else
            p.part_lse[u] = lse;
    }
}

// The kernel body in two instances: kClusterMerge = true, the two splits of a request merged
// inside a cluster of two pairs; false, every other form (no split, merge kernel, fused merge).
// kRanges = false: the selection is the caller's index list; true: Eq. 2's two ranges (with or
// without a rolling cache).  Each instance carries only its own merge, epilogue and index code.
template <bool kClusterMerge, bool kRanges>
__device__ __forceinline__ void tc2_decode_body(const CUtensorMap &q_map, const CUtensorMap &kv_k_map,
                                                const CUtensorMap &kv_v_map, const CUtensorMap &kv_tile_map,
                                                const DecodeParams &p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw;
    if (smem_u32(smem_raw) & 1023u) {
        // the swizzled operand layouts need a 1024-byte aligned base; never seen otherwise, but say so
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (threadIdx.x == 0) flag_status(p.status, OMNI_DEV_TIMEOUT);
        return;
    }
    C2Control *ctl = reinterpret_cast<C2Control *>(smem + kC2SmemCtl);
    const uint32_t smem_base = smem_u32(smem);
    // A cluster is one pair, or (cluster merge) the two pairs that serve the two splits of a
    // request.  `rank` is the CTA's place within its pair; the pair's barriers live in `leader`.
    const uint32_t crank = cluster_rank();
    const uint32_t rank = crank & 1u, leader = crank & ~1u, peer = crank ^ 1u;
    const uint16_t pair_mask = (uint16_t)(3u << leader);

    const int pair = blockIdx.x >> 1;
    const int s = kClusterMerge ? (int)(crank >> 1) : pair % p.splits;
    int b = kClusterMerge ? (int)(blockIdx.x >> 2) : pair / p.splits;
    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;  // warp-uniform
    const int h0 = (int)rank * kTcHeads;
    const int head_rows = min(kTcHeads, p.heads - h0);

    // ---- set-up: barriers and tensor memory (nothing here touches global memory, so with a
    // programmatic dependent launch it overlaps the tail of the kernel before this one) --------
    if (threadIdx.x == 0) {
        mbar_init(&ctl->q_full, 1);
        // arrivals per tile on the pair's score / weight barriers: one per softmax warp that works on
        // the tile, in either CTA (the four warps of the tile's group)
        constexpr uint32_t kTileWarps = 8;
        for (int i = 0; i < 2; ++i) {
            mbar_init(&ctl->k_full[i], 1);
            mbar_init(&ctl->k_empty[i], 1);
            mbar_init(&ctl->v_full[i], 1);
            mbar_init(&ctl->p_full[i], kTileWarps);
            mbar_init(&ctl->pv_done[i], 1);
            mbar_init(&ctl->xg_bar[i], 128);
        }
        for (int i = 0; i < 3; ++i) {
            mbar_init(&ctl->s_full[i], 1);
            mbar_init(&ctl->s_empty[i], kTileWarps);
        }
        mbar_init(&ctl->ref_bar, 4);
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
    // Programmatic dependent launch, both ways.  This grid may have been scheduled while the
    // kernel before it in the stream was still finishing: nothing in global memory is touched
    // until that kernel has completed and its writes are visible.  And the kernel after this one
    // may be scheduled as soon as resources allow; it waits in the same way before it reads.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (!kClusterMerge && p.longest_first) b = c2_request_by_length_rank(p, reinterpret_cast<int *>(smem), &ctl->merge_flag, b);
    const Selection selection = load_selection(p, b);
    __builtin_assume(kRanges ? selection.list == nullptr : selection.list != nullptr);
    const int n = selection.n;
    const bool bad_len = selection.bad;
    int begin, end;
    split_range(n, p.splits, s, begin, end, kC2Tile);
    const int tiles = (end - begin + kC2Tile - 1) / kC2Tile;

    const bool active = tiles > 0;
    if (!active && bad_len && threadIdx.x == 0 && crank == 0) flag_status(p.status, OMNI_DEV_BAD_INDEX);
    if (!kClusterMerge && !active) {
        // empty split (the same decision in both CTAs of the pair): zeros and -inf, no pipeline
        c2_store_empty(p, b, s, h0, head_rows, warp, lane);
    }

    const uint32_t tmem = ctl->tmem_base;
    volatile uint32_t *abort_flag = &ctl->abort;

    const int32_t *pt = p.page_table + (size_t)b * p.max_pages;

    // Index pipeline of the producers.  Lane l serves tokens l and l+32 of a tile.  The three
    // dependent steps (token position -> page id -> pool row) run in different loop iterations,
    // one tile apart, so no load is consumed in the iteration that issued it.
    struct TileIdx {
        int t0, t1;        // token positions (stage 1)
        int pg0, pg1;      // physical page ids, -1 if the position breaks the contract (stage 2)
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
    // row_lo / row_hi: pool rows of tokens lane and lane+32 (a masked token repeats the row of the
    // tile's first valid token: real cache contents, multiplied by a weight of exactly zero);
    // contig: all 64 tokens valid and in consecutive rows; contig_lo / contig_hi: the same per 32.
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

    // what the cluster merge needs from the softmax warps after the main loop
    float cm_lse = -INFINITY, cm_inv = 0.f;
    bool softmax_ok = true;              // false in a softmax warp whose main loop ran into a bounded wait

    if (!active) {
        // an empty split inside a merging cluster: no pipeline, but it takes part in the exchange
    } else if (warp == 0) {
        // =========================== K-role producer =====================================
        // This CTA's K rows are tokens [32*rank, 32*rank+32) of every tile.
        const uint32_t q_bar = map_to_rank(smem_u32(&ctl->q_full), leader);
        if (lane == 0) {
            if (rank == 0) mbar_expect_tx(&ctl->q_full, 2 * kTileBytes);
            tma_box3d_pair(smem_base + kC2SmemQ, &q_map, q_bar, b * p.heads + h0, 0);
        }
        bool any_bad = bad_len;
        TileIdx x1, x2;                      // one and two tiles ahead
        int row_lo, row_hi;
        uint64_t mask;
        bool contig, contig_lo, contig_hi;
        {
            // the position loads of the first three tiles go out together, then the two page-id
            // loads that depend on them: two cache misses in a row before the first copy, not four
            TileIdx x0;
            stage_tokens(0, x0);
            stage_tokens(1, x1);
            stage_tokens(2, x2);
            stage_pages(x0);
            stage_pages(x1);
            stage_rows(0, x0, row_lo, row_hi, mask, contig, contig_lo, contig_hi, any_bad);
        }
        // The mask of a tile is published (store + fence) right after its rows are resolved and
        // BEFORE the next index loads go out: a fence waits for the loads its thread has in
        // flight, so a fence placed after them put their whole latency in front of every refill.
        auto publish_mask = [&](int tile) {
            if (lane == 0) {
                ctl->valid_mask[tile % kMaskRing] = mask;
                __threadfence_block();
            }
        };
        publish_mask(0);
        bool ok = true;
        int pending = -1;                    // stage of a gathered tile whose bytes are not credited yet
        const char *kv_bytes = reinterpret_cast<const char *>(p.kv);
        for (int i = 0; ok && i < tiles; ++i) {
            const int st = i & 1;
            if (lane == 0) *const_cast<volatile int32_t *>(&ctl->k_progress) = i;
            if (i >= 2) ok = mbar_wait(&ctl->k_empty[st], ((i >> 1) - 1) & 1);
            ok = __all_sync(0xffffffffu, ok) && (*abort_flag == 0);
            if (!ok) break;
            const uint32_t bar = map_to_rank(smem_u32(&ctl->k_full[st]), leader);
            if (lane == 0 && rank == 0) mbar_expect_tx(&ctl->k_full[st], 2 * kC2KBytes);
            __syncwarp();
            const uint32_t dst = smem_base + kC2SmemK + st * kC2KBytes;
            const int own_row = rank ? row_hi : row_lo;
            bool gathered = false;
            if (rank ? contig_hi : contig_lo) {
                if (lane == 0) tma_box3d_pair(dst, &kv_k_map, bar, own_row, 0);
            } else {
                // scattered rows: eight lanes per row, four rows per instruction, chunk c of row r
                // lands at chunk c ^ (r % 8) of its 128-byte line
                gathered = true;
                gather_k_rows(dst, kv_bytes, own_row, lane);
            }
            if (pending >= 0) {
                retire_gathered_stage(map_to_rank(smem_u32(&ctl->k_full[pending]), leader), kC2KBytes, gathered, lane);
                pending = -1;
            }
            if (gathered) pending = st;
            // advance the index pipeline: rows of tile i+1, page ids of tile i+2, positions of tile i+3
            if (i + 1 < tiles) {
                stage_rows(i + 1, x1, row_lo, row_hi, mask, contig, contig_lo, contig_hi, any_bad);
                publish_mask(i + 1);
            }
            x1 = x2;
            stage_pages(x1);
            stage_tokens(i + 3, x2);
        }
        if (pending >= 0) retire_gathered_stage(map_to_rank(smem_u32(&ctl->k_full[pending]), leader), kC2KBytes, false, lane);
        if (lane == 0) *const_cast<volatile int32_t *>(&ctl->k_progress) = 0x7fffffff;
        if (!ok && lane == 0) {
            flag_status(p.status, OMNI_DEV_TIMEOUT | OMNI_DEV_ROLE_PRODUCER_K);
            *abort_flag = 1;
        }
        if (__any_sync(0xffffffffu, any_bad) && lane == 0 && rank == 0) flag_status(p.status, OMNI_DEV_BAD_INDEX);
    } else if (warp == 6) {
        // =========================== V-role producer =====================================
        // This CTA's V columns are [256*rank, 256*rank+256) = panels [4*rank, 4*rank+4) of all 64 tokens.
        bool any_bad = false;
        TileIdx x1, x2;
        int row_lo, row_hi;
        uint64_t mask_unused;
        bool contig, contig_lo, contig_hi;
        {
            // the position loads of the first three tiles go out together, then the two page-id
            // loads that depend on them: two cache misses in a row before the first copy, not four
            TileIdx x0;
            stage_tokens(0, x0);
            stage_tokens(1, x1);
            stage_tokens(2, x2);
            stage_pages(x0);
            stage_pages(x1);
            stage_rows(0, x0, row_lo, row_hi, mask_unused, contig, contig_lo, contig_hi, any_bad);
        }
        bool ok = true;
        int pending = -1;                    // stage of a gathered tile whose bytes are not credited yet
        const char *kv_bytes = reinterpret_cast<const char *>(p.kv);
        for (int i = 0; ok && i < tiles; ++i) {
            const int st = i & 1;
            if (i >= 2) ok = mbar_wait(&ctl->pv_done[st], ((i >> 1) - 1) & 1);
            ok = __all_sync(0xffffffffu, ok) && (*abort_flag == 0);
            if (!ok) break;
            const uint32_t bar = map_to_rank(smem_u32(&ctl->v_full[st]), leader);
            if (lane == 0 && rank == 0) mbar_expect_tx(&ctl->v_full[st], 2 * kC2VBytes);
            __syncwarp();
            const uint32_t dst = smem_base + kC2SmemV + st * kC2VBytes;
            bool gathered = false;
            if (contig) {
                if (lane == 0) tma_box3d_pair(dst, &kv_v_map, bar, row_lo, 4 * (int)rank);
            } else {
                // scattered rows: the four panels of this CTA's value columns, 64 tokens
                gathered = true;
                gather_v_rows(dst, kv_bytes + (int)rank * 512, row_lo, row_hi, lane);
            }
            if (pending >= 0) {
                retire_gathered_stage(map_to_rank(smem_u32(&ctl->v_full[pending]), leader), kC2VBytes, gathered, lane);
                pending = -1;
            }
            if (gathered) pending = st;
            if (i + 1 < tiles) stage_rows(i + 1, x1, row_lo, row_hi, mask_unused, contig, contig_lo, contig_hi, any_bad);
            x1 = x2;
            stage_pages(x1);
            stage_tokens(i + 3, x2);
        }
        if (pending >= 0) retire_gathered_stage(map_to_rank(smem_u32(&ctl->v_full[pending]), leader), kC2VBytes, false, lane);
        if (!ok && lane == 0) {
            flag_status(p.status, OMNI_DEV_TIMEOUT | OMNI_DEV_ROLE_PRODUCER_V);
            *abort_flag = 1;
        }
    } else if (warp == 7) {
        // =========================== L2 prefetcher (CTA 0 only) ==========================
        // A hint only: tiles that look like a whole page in order (first position page-aligned,
        // last position 63 further) get their page prefetched into L2; anything else is left to
        // the demand loads.  Lane l resolves tiles l, l+32, ... of a batch of 32 in parallel.
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
                // nothing to pace out where no tile of the batch is a whole page (token-level selections)
                if (!__any_sync(0xffffffffu, row >= 0)) continue;
                for (int k = 0; ok && k < count; ++k) {
                    // tile i is prefetched once the K loads of tile i - kPrefetchAhead have started (a
                    // monotonic counter, polled with a bounded number of naps)
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
                        asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(&kv_tile_map),
                                     "r"(0), "r"(row), "r"(0)
                                     : "memory");
                }
                if (!ok) break;
            }
        }
    } else if (warp == 1) {
        // =========================== MMA issuer (CTA 0 only) =============================
        if (rank == 0) {
            constexpr uint32_t idesc_qk = instr_desc(128, kC2Tile, 0);
            constexpr uint32_t idesc_pv = instr_desc(128, 256, 1);
            const uint64_t q_desc = smem_desc(smem_base + kC2SmemQ, 16, 1024);
            const uint64_t k_desc = smem_desc(smem_base + kC2SmemK, 16, 1024);
            const uint64_t p_desc = smem_desc(smem_base + kC2SmemP, 16, 1024);
            const uint64_t v_desc = smem_desc(smem_base + kC2SmemV, kPanelBytes, 1024);
            const uint32_t q_lo = (uint32_t)q_desc, k_lo = (uint32_t)k_desc, p_lo = (uint32_t)p_desc, v_lo = (uint32_t)v_desc;
            const uint32_t kmaj_hi = (uint32_t)(q_desc >> 32), v_hi = (uint32_t)(v_desc >> 32);
            // Values that steer the loop are broadcast from lane 0 so that the compiler can see
            // they are warp-uniform and keep the descriptor arithmetic on the uniform datapath;
            // with thread-dependent control flow every MMA costs ~70 clocks to issue instead of ~25.
            const int tiles_u = __shfl_sync(0xffffffffu, tiles, 0);
            const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem, 0);
            // One copy of each issue routine: stage and buffer enter as warp-uniform run-time values
            // (every operand of an MMA is then a uniform base plus a compile-time offset), which
            // keeps the issuing warp's code a few kilobytes instead of several tens (an issue loop
            // unrolled over the buffer parities ran config-2-sized launches 5 % slower, token-level
            // ones 8 %: a launch starts with cold instruction caches and this loop is its critical path).
            auto issue_qk = [&](int kpar, int sbuf) {
                const uint32_t d = tmem_u + kC2ColS + 32 * sbuf;
                const uint32_t kb = k_lo + ((kpar * kC2KBytes) >> 4);
                tc_mma_pair_elect<false>(d, q_lo, kmaj_hi, kb, kmaj_hi, idesc_qk);
#pragma unroll
                for (int kk = 1; kk < kDqk / 16; ++kk)
                    tc_mma_pair_elect<true>(d, q_lo + (((kk >> 2) * kPanelBytes + (kk & 3) * 32) >> 4), kmaj_hi,
                                            kb + (((kk >> 2) * kC2KPanel + (kk & 3) * 32) >> 4), kmaj_hi, idesc_qk);
                tc_commit_pair_elect(&ctl->k_empty[kpar], pair_mask);
                tc_commit_pair_elect(&ctl->s_full[sbuf], pair_mask);
            };
            auto issue_pv = [&](int par, bool first) {
                const uint32_t a = p_lo + ((par * kPanelBytes) >> 4);
                const uint32_t bd = v_lo + ((par * kC2VBytes) >> 4);
                if (first) {
                    tc_mma_pair_elect<false>(tmem_u + kColO, a, kmaj_hi, bd, v_hi, idesc_pv);
                    tc_mma_pair_elect<false>(tmem_u + kColO + 128, a, kmaj_hi, bd + ((2 * kPanelBytes) >> 4), v_hi, idesc_pv);
                } else {
                    tc_mma_pair_elect<true>(tmem_u + kColO, a, kmaj_hi, bd, v_hi, idesc_pv);
                    tc_mma_pair_elect<true>(tmem_u + kColO + 128, a, kmaj_hi, bd + ((2 * kPanelBytes) >> 4), v_hi, idesc_pv);
                }
#pragma unroll
                for (int k = 1; k < 4; ++k) {
                    const uint32_t ak = a + ((k * 32) >> 4), bk = bd + ((k * 2048) >> 4);
                    tc_mma_pair_elect<true>(tmem_u + kColO, ak, kmaj_hi, bk, v_hi, idesc_pv);
                    tc_mma_pair_elect<true>(tmem_u + kColO + 128, ak, kmaj_hi, bk + ((2 * kPanelBytes) >> 4), v_hi, idesc_pv);
                }
                tc_commit_pair_elect(&ctl->pv_done[par], pair_mask);
            };
            // S(t) lives in buffer t % 3, K(t) in stage t & 1; Q K^T runs two tiles ahead of P V
            auto qk_tile = [&](int t) -> bool {
                const int kpar = t & 1, sbuf = t % 3;
                bool good = mbar_wait(&ctl->k_full[kpar], (t >> 1) & 1) &&
                            (t < 3 || mbar_wait(&ctl->s_empty[sbuf], ((t / 3) - 1) & 1));
                good = __all_sync(0xffffffffu, good);
                if (!good) return false;
                tc_fence_after();
                issue_qk(kpar, sbuf);
                return true;
            };
            auto pv_tile = [&](int i) -> bool {
                const int par = i & 1;
                bool good = mbar_wait(&ctl->p_full[par], (i >> 1) & 1) && mbar_wait(&ctl->v_full[par], (i >> 1) & 1);
                good = __all_sync(0xffffffffu, good);
                if (!good) return false;
                tc_fence_after();
                issue_pv(par, i == 0);
                return true;
            };
            bool ok = mbar_wait(&ctl->q_full, 0);
            ok = __all_sync(0xffffffffu, ok);
            if (ok) ok = qk_tile(0);
            if (ok && tiles_u > 1) ok = qk_tile(1);
            for (int i = 0; ok && i < tiles_u; ++i) {
                // if the K rows of tile i+2 have not landed yet while P and V of tile i are ready, P V goes first
                bool qk_todo = i + 2 < tiles_u;
                if (qk_todo) {
                    const int kpar = i & 1;
                    const bool k_ready = __all_sync(0xffffffffu, mbar_test(&ctl->k_full[kpar], ((i + 2) >> 1) & 1));
                    const bool pv_ready = __all_sync(0xffffffffu, mbar_test(&ctl->p_full[kpar], (i >> 1) & 1) &&
                                                                      mbar_test(&ctl->v_full[kpar], (i >> 1) & 1));
                    if (k_ready || !pv_ready) {
                        ok = qk_tile(i + 2);
                        qk_todo = false;
                    }
                }
                if (ok) ok = pv_tile(i);
                if (ok && qk_todo) ok = qk_tile(i + 2);
            }
            if (!ok && lane == 0) {
                flag_status(p.status, OMNI_DEV_TIMEOUT | OMNI_DEV_ROLE_MMA);
                *abort_flag = 1;
            }
        }
        __syncwarp();
    } else {
        // =========================== softmax + epilogue =================================
        // Eight warps (2-5 and 8-11): two per tensor-memory lane quarter, one in each of two groups
        // (sub = 0 for warps 2-5, 1 for warps 8-11).  A thread serves head row L % 64 (L = its
        // tensor-memory lane); in the epilogue it owns value columns 256 * (L / 64) + 128 * sub +
        // [0, 128) of that row.
        const int quarter = warp & 3;
        const int sub = warp >= 8 ? 1 : 0;
        const int row = (quarter & 1) * 32 + lane;          // head row within this CTA
        const int half = quarter >> 1;                      // token half of S / column half of O
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const uint32_t s_empty_leader = map_to_rank(smem_u32(&ctl->s_empty[0]), leader);   // [1], [2] follow at +8, +16
        const uint32_t p_full_leader0 = map_to_rank(smem_u32(&ctl->p_full[0]), leader);
        const uint32_t p_full_leader1 = map_to_rank(smem_u32(&ctl->p_full[1]), leader);
        float m_ref = -INFINITY, l = 0.f;
        bool ok = true;
        // Tiles alternate between two groups of four warps (2-5: even tiles, 8-11: odd tiles), so
        // the chain scores -> weights of one tile overlaps the next tile's instead of all eight warps
        // marching through every tile together.  In its group a thread serves head row `row` and
        // the token half `half` of the tile (32 tokens, all 32 score columns of its lane).  The
        // running reference maximum of a row is shared by the groups through ctl->ref: tile i reads
        // what tile i-1 left and publishes its own decision at once, before its exponentials.
        const int grp = sub;
        for (int i = grp; ok && i < tiles; i += 2) {
            const int sbuf = i % 3, it = i >> 1;
            ok = mbar_wait(&ctl->s_full[sbuf], (i / 3) & 1);
            if (!__all_sync(0xffffffffu, ok)) {
                ok = false;
                break;
            }
            tc_fence_after();
            uint32_t sv[32];
            tc_ld32(tmem + lane_base + kC2ColS + 32 * sbuf, sv);
            tc_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(s_empty_leader + 8 * sbuf);
            const uint32_t valid = (uint32_t)(ctl->valid_mask[i % kMaskRing] >> (32 * half));
            // x[j] * xs is the scaled score of token j.  A full tile under a positive scale keeps the
            // raw scores (xs = the scale): the maximum is taken on them and the scale rides on the
            // fused multiply-add in front of the exponential, one instruction less per token.
            float x[32];
            float mt = -INFINITY;
            float xs = 1.f;
            if (valid == 0xffffffffu && p.scale_log2 > 0.f) {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    x[j] = __uint_as_float(sv[j]);
                    mt = fmaxf(mt, x[j]);
                }
                xs = p.scale_log2;
                mt *= xs;
            } else if (valid == 0xffffffffu) {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    x[j] = __uint_as_float(sv[j]) * p.scale_log2;
                    mt = fmaxf(mt, x[j]);
                }
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    x[j] = ((valid >> j) & 1u) ? __uint_as_float(sv[j]) * p.scale_log2 : -INFINITY;
                    mt = fmaxf(mt, x[j]);
                }
            }
            // the row's other half is served by the thread of the same lane two warps on
            float *xg = &ctl->xchg[0][0][0] + ((grp * 2 + (it & 1)) * 2) * 64;      // [group][parity][half][row]
            xg[half * 64 + row] = mt;
            mbar_arrive(&ctl->xg_bar[grp]);
            ok = mbar_wait(&ctl->xg_bar[grp], it & 1);
            if (i > 0) ok = ok && mbar_wait(&ctl->ref_bar, (i - 1) & 1);
            if (!__all_sync(0xffffffffu, ok)) {
                ok = false;
                break;
            }
            mt = fmaxf(mt, xg[(half ^ 1) * 64 + row]);
            const float ref_in = i > 0 ? ctl->ref[(i - 1) & 1][row] : -INFINITY;
            // move the reference only when the tile maximum leaves the window above it
            float ref_out = ref_in;
            bool moved = false;
            if (mt > ref_in + kRescaleThreshold || (ref_in == -INFINITY && mt > -INFINITY)) {
                ref_out = mt;
                moved = true;
            }
            if (half == 0) ctl->ref[i & 1][row] = ref_out;
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->ref_bar);
            // this thread's own sum was last brought to reference m_ref
            if (ref_out != m_ref) {
                l *= (m_ref == -INFINITY) ? 0.f : exp2f(m_ref - ref_out);
                m_ref = ref_out;
            }
            const float mr = (m_ref == -INFINITY) ? 0.f : m_ref;
            float sum = 0.f;
            uint32_t pk[16];
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
                const float e0 = fast_exp2(fmaf(x[j], xs, -mr)), e1 = fast_exp2(fmaf(x[j + 1], xs, -mr));
                sum += e0 + e1;
                pk[j >> 1] = pack_bf16(e0, e1);
            }
            l += sum;
            // this group's P buffer is free once P V of tile i-2 retired; O may be rescaled once P V of tile i-1 did
            if (i >= 2) {
                ok = mbar_wait(&ctl->pv_done[grp], ((i >> 1) - 1) & 1);
                if (!__all_sync(0xffffffffu, ok)) {
                    ok = false;
                    break;
                }
            }
            if (i >= 1 && __any_sync(0xffffffffu, moved)) {
                ok = mbar_wait(&ctl->pv_done[grp ^ 1], ((i - 1) >> 1) & 1);
                if (!__all_sync(0xffffffffu, ok)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                // the four warps of the group cover all 128 lanes: each thread rescales the 256 value columns of its lane
                const float factor = moved ? ((ref_in == -INFINITY) ? 0.f : exp2f(ref_in - ref_out)) : 1.f;
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
            // half a P row: 32 tokens x bf16 = four 16-byte chunks, chunk c stored at c ^ (row % 8)
            uint8_t *p_row = smem + kC2SmemP + grp * kPanelBytes + row * 128;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int chunk = (half * 4 + c) ^ (row & 7);
                *reinterpret_cast<uint4 *>(p_row + chunk * 16) =
                    make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
            }
            fence_async_smem();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(grp ? p_full_leader1 : p_full_leader0);
        }
        // The row sums are final as soon as the last tile's weights are written, before its P V has
        // run: their exchange and what follows from them overlap that last P V.
        if (ok) {
            // the reference after the last tile is the final one
            ok = mbar_wait(&ctl->ref_bar, (tiles - 1) & 1);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            const float ref_final = ctl->ref[(tiles - 1) & 1][row];
            if (ref_final != m_ref) {
                l *= (m_ref == -INFINITY) ? 0.f : exp2f(m_ref - ref_final);
                m_ref = ref_final;
            }
        }
        // Slot of a group's partial row sums: the group's row-maximum slots of the parity it did NOT
        // use for its last tile.  Every thread of the group has passed the exchange barrier of that
        // last tile, which each thread reached only after reading the slots of the tile before, so
        // nobody reads them any more (a group without tiles never used its slots at all).
        auto sum_slot = [&](int g) -> float * {
            const int last = (tiles - 1) - ((((tiles - 1) & 1) != g) ? 1 : 0);      // the group's last tile, -1 if none
            const int parity = last >= 0 ? (((last >> 1) & 1) ^ 1) : 0;
            return &ctl->xchg[0][0][0] + ((g * 2 + parity) * 2) * 64;                // [half][row]
        };
        float lt = 0.f;
        if (ok) {
            sum_slot(grp)[half * 64 + row] = l;
            mbar_arrive(&ctl->x_bar);
            ok = mbar_wait(&ctl->x_bar, 0);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            const float *s0 = sum_slot(0), *s1 = sum_slot(1);
            lt = (s0[row] + s0[64 + row]) + (s1[row] + s1[64 + row]);
            cm_inv = lt > 0.f ? 1.f / lt : 0.f;
            cm_lse = lt > 0.f ? (m_ref + log2f(lt)) * kLn2 : -INFINITY;
            // now the last tile's P V
            ok = mbar_wait(&ctl->pv_done[(tiles - 1) & 1], ((tiles - 1) >> 1) & 1);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (kClusterMerge && ok) {
            // every MMA of the pair has retired and every copy has landed: the partner in the other
            // split may overwrite this CTA's operand tiles from now on.  The result stays in tensor
            // memory: the exchange after the main loop normalises it and hands half of it to the CTA
            // that serves the same heads in the other split.
            if (warp == 2 && lane == 0) mbar_arrive_cluster(map_to_rank(smem_u32(&ctl->ready_bar), crank ^ 2u));
        } else if (!kClusterMerge && ok) {
            tc_fence_after();
            c2_store_result(p, smem, tmem, warp, lane, b, s, h0, head_rows, lt, m_ref);
            const bool final_out = p.splits == 1;
            // with the in-kernel merge the partial results must be visible before this CTA is counted
            if (!final_out && p.counters != nullptr) __threadfence();
        }
        if (!ok && lane == 0) {
            flag_status(p.status, OMNI_DEV_TIMEOUT | OMNI_DEV_ROLE_SOFTMAX);
            *abort_flag = 1;
        }
        softmax_ok = ok;
    }

    // ---- tear-down: nobody leaves while the other CTA may still touch this one's memory --
    if (*abort_flag) {
        // a wait ran out: give copies that are still in flight time to land before anyone exits
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    if (kClusterMerge) cluster_merge_exchange(p, ctl, smem, tmem, b, s, crank, h0, head_rows, active, softmax_ok, cm_lse, cm_inv);
    tc_fence_before();
    __syncthreads();
    // Tensor memory was allocated for the pair, so it is released only when both CTAs are done
    // with it.  The rendezvous is an mbarrier in each CTA that both CTAs arrive on (the hardware
    // cluster barrier took 6-9 us at this point); warp 1 stays until the peer's arrival has
    // landed, which also keeps this CTA's shared memory alive for it.
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
    // the bulk copy a CTA sent to its partner reads this CTA's shared memory: nobody leaves
    // before every CTA of the cluster has received its block
    if (kClusterMerge) cluster_sync_relaxed();
    // ---- split merge by whichever CTA finishes a (request, head half) last ---------------
    if (!kClusterMerge && p.splits > 1 && p.counters != nullptr)
        merge_if_last(p, b, (int)rank, 2, h0, head_rows, reinterpret_cast<float *>(smem), &ctl->merge_flag);
}

#define OMNI_C2_KERNEL(name, cluster_merge, ranges)                                                                    \
    __global__ void __launch_bounds__(kC2Threads, 1)                                                                   \
    name(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap kv_k_map,                      \
         const __grid_constant__ CUtensorMap kv_v_map, const __grid_constant__ CUtensorMap kv_tile_map, DecodeParams p) \
    {                                                                                                                  \
        tc2_decode_body<cluster_merge, ranges>(q_map, kv_k_map, kv_v_map, kv_tile_map, p);                             \
    }
OMNI_C2_KERNEL(tc2_decode_kernel, false, false)
OMNI_C2_KERNEL(tc2_decode_cm_kernel, true, false)
OMNI_C2_KERNEL(tc2_decode_rng_kernel, false, true)
OMNI_C2_KERNEL(tc2_decode_cm_rng_kernel, true, true)
#undef OMNI_C2_KERNEL

using C2KernelFn = void (*)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, DecodeParams);
inline C2KernelFn tc2_kernel_for(bool cluster_merge, bool ranges)
{
    return cluster_merge ? (ranges ? tc2_decode_cm_rng_kernel : tc2_decode_cm_kernel)
                         : (ranges ? tc2_decode_rng_kernel : tc2_decode_kernel);
}

// Clusters of two pairs (cluster merge) that can be resident at once on the current device, or 0.
inline int tc2_max_merge_clusters()
{
    static int cached[64];
    static bool known[64] = {};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    std::lock_guard<std::mutex> lock(mu);
    if (!known[dev]) {
        int n = 0;
        if (cudaFuncSetAttribute(tc2_decode_cm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kC2SmemBytes) == cudaSuccess) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(4 * 64);
            cfg.blockDim = dim3(kC2Threads);
            cfg.dynamicSmemBytes = kC2SmemBytes;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 4;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            if (cudaOccupancyMaxActiveClusters(&n, tc2_decode_cm_kernel, &cfg) != cudaSuccess) {
                cudaGetLastError();
                n = 0;
            }
        }
        cached[dev] = n;
        known[dev] = true;
    }
    return cached[dev];
}

inline bool tc2_prepare_device()
{
    static bool attr_set[64] = {};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    std::lock_guard<std::mutex> lock(mu);
    if (!attr_set[dev]) {
        for (int k = 0; k < 4; ++k)
            if (cudaFuncSetAttribute(tc2_kernel_for((k & 1) != 0, (k & 2) != 0), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kC2SmemBytes) != cudaSuccess)
                return false;
        attr_set[dev] = true;
    }
    return true;
}

// maps[0] = q, maps[1] = K role boxes, maps[2] = V role boxes, maps[3] = whole pages
inline bool tc2_make_maps(const DecodeParams &p, CUtensorMap *maps, bool cached)
{
    const uint64_t rows = (uint64_t)p.num_pages * kPage, qrows = (uint64_t)p.batch * p.heads;
    if (cached)
        return make_panel_map(&maps[0], p.q, qrows, kTcHeads, kPanels) && make_panel_map(&maps[1], p.kv, rows, 32, kPanels) &&
               make_panel_map(&maps[2], p.kv, rows, kTile, 4) && make_panel_map(&maps[3], p.kv, rows, kTile, kPanels);
    return encode_panel_map(&maps[0], p.q, qrows, kTcHeads, kPanels) && encode_panel_map(&maps[1], p.kv, rows, 32, kPanels) &&
           encode_panel_map(&maps[2], p.kv, rows, kTile, 4) && encode_panel_map(&maps[3], p.kv, rows, kTile, kPanels);
}

inline omni_status_t tc2_launch(const CUtensorMap *maps, const DecodeParams &p, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.batch * p.splits * 2));
    cfg.blockDim = dim3(kC2Threads);
    cfg.dynamicSmemBytes = kC2SmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = p.cluster_merge ? 4 : 2;      // cluster merge: both splits of a request in one cluster
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // the launch may overlap the tail of the previous kernel in the stream (the kernel waits
    // before its first global access), which hides the launch latency between decode steps
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, tc2_kernel_for(p.cluster_merge != 0, p.sel_idx == nullptr), maps[0], maps[1],
                                               maps[2], maps[3], p);
    return err == cudaSuccess ? OMNI_OK : OMNI_ERR_CUDA;
}

}  // namespace omni
