// Tensor-core decode kernel for sm_100a: TMA row gather through the page table, tcgen05 MMAs
// with fp32 accumulators in tensor memory, fp32 online softmax.
//
// One CTA owns 64 heads of one (request, split) and walks the split's selected tokens in
// 64-token tiles:
//   warp 0      producer: resolves token positions to pool rows and brings the rows into a
//               2-stage ring of 128B-swizzled tiles with TMA: one 64x64 box per column panel
//               when the tile is 64 consecutive pool rows (a page in order), otherwise
//               row gathers of 4 rows per instruction
//   warp 1      MMA issuer: S = Q K^T (M=64 heads, N=64 tokens, K=576) and O += P V
//               (M=64, N=512, K=64); owns the tensor-memory allocation
//   warps 2-5   softmax: read S from tensor memory, keep the running reference maximum and
//               row sums, write P (bf16) to shared memory, rescale O when the reference
//               moves, and run the epilogue
//
// Tensor-memory map (an M=64 accumulator occupies lanes 0-15 of each 32-lane quarter, so two
// accumulators share a column range at lane offsets 0 and 16):
//   columns   0..255  O   (lane offset 0: value columns 0..255, lane offset 16: 256..511)
//   columns 256..319  S buffer 0 (one M=64 x N=64 accumulator, lanes 0-15 of each quarter)
//   columns 320..383  S buffer 1
// Every softmax thread owns half a row: lane l of a warp serves head row 16*(warp%4)+l%16 and
// the token half (of S) / value-column half (of O) l/16.
#pragma once

#include <cuda.h>

#include <mutex>
#include <type_traits>

#include "common.cuh"

namespace omni {

constexpr int kTcHeads = 64;                       // heads per CTA (MMA M)
constexpr int kTcThreads = 192;
constexpr int kPanelBytes = kTile * 128;           // 64 rows x 64 bf16 columns, 128B-swizzled
constexpr int kPanels = kDqk / 64;                 // 9 column panels per latent row
constexpr int kTileBytes = kPanels * kPanelBytes;  // 73,728
constexpr int kStages = 2;
constexpr int kPBytes = kTcHeads * kTile * 2;      // 8,192
constexpr int kSmemQ = 0;
constexpr int kSmemKV = kSmemQ + kTileBytes;
constexpr int kSmemP = kSmemKV + kStages * kTileBytes;
constexpr int kSmemCtl = kSmemP + kPBytes;
constexpr int kSmemCtlBytes = 256;
constexpr int kTcSmemBytes = kSmemCtl + kSmemCtlBytes + 1024;  // + slack for 1024B alignment
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColO = 0, kColS = 256;
constexpr uint32_t kLane16 = 16u << 16;
constexpr float kRescaleThreshold = 8.f;           // log2 units the reference max may lag
constexpr long long kWaitCycles = 1ll << 31;         // about a second of SM clocks per wait

struct TcControl {
    uint64_t q_full;
    uint64_t kv_full[kStages];
    uint64_t kv_empty[kStages];
    uint64_t s_full[2];
    uint64_t s_empty[2];
    uint64_t p_full;
    uint64_t pv_done;
    uint64_t valid_mask[kStages];
    uint32_t tmem_base;
    uint32_t abort;
};
static_assert(sizeof(TcControl) <= kSmemCtlBytes, "control block too large");

// ---------------------------------------------------------------------------------------
// thin PTX wrappers
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}

// Bounded wait on a phase parity; false if `limit` SM clocks (about a second by default) passed
// without the phase completing.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, long long limit = kWaitCycles)
{
    const uint32_t addr = smem_u32(bar);
    auto attempt = [&]() {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(addr), "r"(parity)
            : "memory");
        return done != 0;
    };
    // the clock is only read once the first attempt has failed: most waits of the pipeline find
    // their phase complete or completing, and they sit on its critical path
    if (attempt()) return true;
    const long long start = clock64();
    for (uint32_t it = 0;; ++it) {
        if (attempt()) return true;
        if ((it & 63u) == 63u && clock64() - start > limit) return false;
    }
}

__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap *map, uint64_t *bar, int col,
                                            int r0, int r1, int r2, int r3)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cta.global.tile::gather4.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(col), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void tma_box2d(uint32_t dst, const CUtensorMap *map, uint64_t *bar, int col, int row)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(col), "r"(row), "r"(smem_u32(bar))
        : "memory");
}

// 3-D box {64 columns, rows, panels} of the [rows, 9 panels, 64 columns] view: lands panel by panel.
__device__ __forceinline__ void tma_box3d(uint32_t dst, const CUtensorMap *map, uint64_t *bar, int row, int panel)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cta.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(0), "r"(row), "r"(panel), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
          "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
          "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}

__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory operand descriptor, 128-byte swizzle.  Field layout (bits): [0,14) start
// address >> 4, [16,30) leading byte offset >> 4, [32,46) stride byte offset >> 4,
// [46,48) descriptor version (1 on sm_100), [61,64) swizzle mode (2 = 128 B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
           ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor for kind::f16 with bf16 inputs and fp32 accumulation: [4,6) D type
// (1 = f32), [7,10) A type (1 = bf16), [10,13) B type, bit 15 / 16 A / B major (1 = MN-major),
// [17,23) N >> 3, [24,29) M >> 4.
__host__ __device__ constexpr uint32_t instr_desc(int m, int n, int b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// ---------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ bool mbar_test(uint64_t *bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return done != 0;
}

// MMA with the accumulate flag known at compile time (no predicate set-up per instruction).
template <bool kAccumulate>
__device__ __forceinline__ void tc_mma_c(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "n"(kAccumulate ? 1 : 0)
        : "memory");
}

// MMA / commit executed by a whole converged warp: one elected lane issues the instruction.  The
// descriptors arrive as 32-bit halves so that stepping through a tile is a 32-bit add.
template <bool kAccumulate>
__device__ __forceinline__ void tc_mma_elect(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                             uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "elect.sync _|q, 0xffffffff;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "n"(kAccumulate ? 1 : 0)
        : "memory");
}

__device__ __forceinline__ void tc_commit_elect(uint64_t *bar)
{
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "elect.sync _|q, 0xffffffff;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        ::"r"(smem_u32(bar))
        : "memory");
}

// 16 lanes x 32 columns twice: threads 0-15 of the warp read columns [c, c+32) of lanes 0-15 of
// their quarter, threads 16-31 read columns [c+32, c+64) of the same lanes.  This is how the 64
// rows of an M=64 accumulator (which live in lanes 0-15 of each quarter) are spread over all 32
// threads of the warp that serves the quarter.
__device__ __forceinline__ void tc_ld16x2(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.16x32bx2.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32], 32;"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

__global__ void __launch_bounds__(kTcThreads, 1)
tc_decode_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap kv_map,
                 const __grid_constant__ CUtensorMap kv_page_map, DecodeParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    TcControl *ctl = reinterpret_cast<TcControl *>(smem + kSmemCtl);
    const uint32_t smem_base = smem_u32(smem);

    const int head_groups = (p.heads + kTcHeads - 1) / kTcHeads;
    const int hg = blockIdx.x % head_groups;
    const int s = (blockIdx.x / head_groups) % p.splits;
    const int b = blockIdx.x / (head_groups * p.splits);
    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;  // warp-uniform
    const int h0 = hg * kTcHeads;

    // Programmatic dependent launch, both ways: nothing in global memory is touched until the
    // kernel before this one in the stream has completed, and the kernel after this one (the split
    // merge) may be scheduled as soon as resources allow; it waits in the same way before it reads.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const Selection selection = load_selection(p, b);
    const int n = selection.n;
    const bool bad_len = selection.bad;
    int begin, end;
    split_range(n, p.splits, s, begin, end);
    const int tiles = (end - begin + kTile - 1) / kTile;

    if (tiles == 0) {
        // empty split: zero output / -inf log-sum-exp, no tensor-core work
        if (threadIdx.x == 0 && bad_len) flag_status(p.status, OMNI_DEV_BAD_INDEX);
        for (int r = warp; r < kTcHeads; r += kTcThreads / 32) {
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

    // ---- set-up: barriers, tensor memory ------------------------------------------------
    if (threadIdx.x == 0) {
        mbar_init(&ctl->q_full, 1);
        for (int i = 0; i < kStages; ++i) {
            mbar_init(&ctl->kv_full[i], 1);
            mbar_init(&ctl->kv_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&ctl->s_full[i], 1);
            mbar_init(&ctl->s_empty[i], 128);
        }
        mbar_init(&ctl->p_full, 128);
        mbar_init(&ctl->pv_done, 1);
        ctl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;
    volatile uint32_t *abort_flag = &ctl->abort;

    if (warp == 0) {
        // =========================== producer ===========================================
        const int32_t *pt = p.page_table + (size_t)b * p.max_pages;
        if (lane == 0) {
            mbar_expect_tx(&ctl->q_full, kTileBytes);
            tma_box3d(smem_base + kSmemQ, &q_map, &ctl->q_full, b * p.heads + h0, 0);
        }
        bool any_bad = bad_len;
        // Lane l serves tokens l and l+32 of a tile.  Token positions are fetched two tiles
        // ahead and turned into pool rows one tile ahead, so neither dependent load sits
        // between a freed stage and the copy that refills it.
        auto fetch = [&](int tile, int &t0, int &t1) {
            const int j0 = begin + tile * kTile + lane, j1 = j0 + 32;
            t0 = (tile < tiles && j0 < end) ? selection_at(selection, j0) : 0;
            t1 = (tile < tiles && j1 < end) ? selection_at(selection, j1) : 0;
        };
        auto lookup = [&](int tile, int t0, int t1, int &row_lo, int &row_hi, uint64_t &mask, bool &contig) {
            const int j0 = begin + tile * kTile + lane, j1 = j0 + 32;
            int64_t r0 = -1, r1 = -1;
            if (j0 < end) {
                r0 = resolve_row(pt, t0, p.max_pages, p.num_pages);
                any_bad |= (r0 < 0 && !is_padding(selection, t0));
            }
            if (j1 < end) {
                r1 = resolve_row(pt, t1, p.max_pages, p.num_pages);
                any_bad |= (r1 < 0 && !is_padding(selection, t1));
            }
            const uint32_t m0 = __ballot_sync(0xffffffffu, r0 >= 0), m1 = __ballot_sync(0xffffffffu, r1 >= 0);
            mask = (uint64_t)m0 | ((uint64_t)m1 << 32);
            row_lo = r0 >= 0 ? (int)r0 : 0;      // masked tokens still load a real row (row 0)
            row_hi = r1 >= 0 ? (int)r1 : 0;
            const int base = __shfl_sync(0xffffffffu, row_lo, 0);
            contig = __all_sync(0xffffffffu, r0 == (int64_t)base + lane && r1 == (int64_t)base + 32 + lane);
        };
        int row_lo, row_hi, t0n, t1n;
        uint64_t mask;
        bool contig;
        fetch(0, t0n, t1n);
        lookup(0, t0n, t1n, row_lo, row_hi, mask, contig);
        fetch(1, t0n, t1n);
        int issued = 0;
        for (int i = 0; i < tiles; ++i) {
            const int st = i % kStages;
            bool ok = true;
            if (i >= kStages) ok = mbar_wait(&ctl->kv_empty[st], ((i / kStages) - 1) & 1);
            ok = __all_sync(0xffffffffu, ok) && (*abort_flag == 0);
            if (!ok) {
                if (lane == 0) {
                    flag_status(p.status, OMNI_DEV_TIMEOUT);
                    *abort_flag = 1;
                }
                break;
            }
            if (lane == 0) {
                ctl->valid_mask[st] = mask;
                mbar_expect_tx(&ctl->kv_full[st], kTileBytes);
            }
            __syncwarp();
            const uint32_t stage = smem_base + kSmemKV + st * kTileBytes;
            if (contig) {
                // 64 consecutive pool rows (a whole page in order): the whole tile is one 3-D box
                if (lane == 0) tma_box3d(stage, &kv_page_map, &ctl->kv_full[st], row_lo, 0);
            } else {
                // scattered rows: lane g < 16 gathers tokens 4g..4g+3 into rows 4g..4g+3 of every panel
                int r[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int src = (4 * lane + k) & 31;
                    const int a = __shfl_sync(0xffffffffu, row_lo, src), c = __shfl_sync(0xffffffffu, row_hi, src);
                    r[k] = lane < 8 ? a : c;
                }
                if (lane < 16) {
#pragma unroll
                    for (int c = 0; c < kPanels; ++c)
                        tma_gather4(stage + lane * 512 + c * kPanelBytes, &kv_map, &ctl->kv_full[st], c * 64, r[0], r[1],
                                    r[2], r[3]);
                }
            }
            issued = i + 1;
            if (i + 1 < tiles) lookup(i + 1, t0n, t1n, row_lo, row_hi, mask, contig);
            fetch(i + 2, t0n, t1n);
        }
        if (__any_sync(0xffffffffu, any_bad) && lane == 0) flag_status(p.status, OMNI_DEV_BAD_INDEX);
        if (*abort_flag) {
            // let every copy this warp started land before the CTA can exit
            for (int i = max(0, issued - kStages); i < issued; ++i) mbar_wait(&ctl->kv_full[i % kStages], (i / kStages) & 1);
            mbar_wait(&ctl->q_full, 0);
        }
    } else if (warp == 1) {
        // =========================== MMA issuer =========================================
        // The whole warp runs this loop with warp-uniform control flow (loop bounds broadcast from
        // lane 0, buffer parity a compile-time constant) and one elected lane issues each MMA: the
        // descriptor arithmetic then stays on the uniform datapath and an MMA issues every ~30 clocks,
        // where a lone diverged thread needs ~75.
        {
            constexpr uint32_t idesc_qk = instr_desc(kTcHeads, kTile, 0);
            constexpr uint32_t idesc_pv = instr_desc(kTcHeads, 256, 1);
            const uint64_t q_desc = smem_desc(smem_base + kSmemQ, 16, 1024);
            const uint64_t k_desc = smem_desc(smem_base + kSmemKV, 16, 1024);
            const uint64_t p_desc = smem_desc(smem_base + kSmemP, 16, 1024);
            const uint64_t v_desc = smem_desc(smem_base + kSmemKV, kPanelBytes, 1024);
            const uint32_t q_lo = (uint32_t)q_desc, k_lo = (uint32_t)k_desc, p_lo = (uint32_t)p_desc, v_lo = (uint32_t)v_desc;
            const uint32_t kmaj_hi = (uint32_t)(q_desc >> 32), v_hi = (uint32_t)(v_desc >> 32);
            const int tiles_u = __shfl_sync(0xffffffffu, tiles, 0);
            const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem, 0);
            // S(t) = Q K(t)^T : 36 k-steps of 16 columns; panel c of Q against panel c of the stage
            auto issue_qk = [&](auto par_tag) {
                constexpr int par = decltype(par_tag)::value;
                const uint32_t d = tmem_u + kColS + 64 * par;
                const uint32_t kb = k_lo + ((par * kTileBytes) >> 4);
                tc_mma_elect<false>(d, q_lo, kmaj_hi, kb, kmaj_hi, idesc_qk);
#pragma unroll
                for (int kk = 1; kk < kDqk / 16; ++kk) {
                    const uint32_t off = ((kk >> 2) * kPanelBytes + (kk & 3) * 32) >> 4;
                    tc_mma_elect<true>(d, q_lo + off, kmaj_hi, kb + off, kmaj_hi, idesc_qk);
                }
                tc_commit_elect(&ctl->s_full[par]);
            };
            // O += P(i) V(i) : the stage read N-major (64-column panels 8192 B apart, 8-token groups
            // 1024 B apart); value columns 0..255 and 256..511 go to the two interleaved accumulators
            auto issue_pv = [&](auto par_tag, bool first) {
                constexpr int par = decltype(par_tag)::value;
                const uint32_t vb = v_lo + ((par * kTileBytes) >> 4);
                if (first) {
                    tc_mma_elect<false>(tmem_u + kColO, p_lo, kmaj_hi, vb, v_hi, idesc_pv);
                    tc_mma_elect<false>(tmem_u + kColO + kLane16, p_lo, kmaj_hi, vb + ((4 * kPanelBytes) >> 4), v_hi, idesc_pv);
                } else {
                    tc_mma_elect<true>(tmem_u + kColO, p_lo, kmaj_hi, vb, v_hi, idesc_pv);
                    tc_mma_elect<true>(tmem_u + kColO + kLane16, p_lo, kmaj_hi, vb + ((4 * kPanelBytes) >> 4), v_hi, idesc_pv);
                }
#pragma unroll
                for (int k = 1; k < kTile / 16; ++k) {
                    tc_mma_elect<true>(tmem_u + kColO, p_lo + ((k * 32) >> 4), kmaj_hi, vb + ((k * 2048) >> 4), v_hi, idesc_pv);
                    tc_mma_elect<true>(tmem_u + kColO + kLane16, p_lo + ((k * 32) >> 4), kmaj_hi,
                                       vb + ((4 * kPanelBytes + k * 2048) >> 4), v_hi, idesc_pv);
                }
                tc_commit_elect(&ctl->kv_empty[par]);
                tc_commit_elect(&ctl->pv_done);
            };
            // one tile: Q K^T of the next tile first, then P V of this one
            auto step = [&](auto par_tag, int i) -> bool {
                constexpr int par = decltype(par_tag)::value;
                bool good = true;
                if (i + 1 < tiles_u) {
                    const int t = i + 1;
                    good = mbar_wait(&ctl->kv_full[par ^ 1], (t >> 1) & 1) &&
                           (t < 2 || mbar_wait(&ctl->s_empty[par ^ 1], ((t >> 1) - 1) & 1));
                    good = __all_sync(0xffffffffu, good);
                    if (!good) return false;
                    tc_fence_after();
                    issue_qk(std::integral_constant<int, par ^ 1>{});
                }
                good = mbar_wait(&ctl->p_full, i & 1);
                good = __all_sync(0xffffffffu, good);
                if (!good) return false;
                tc_fence_after();
                issue_pv(par_tag, i == 0);
                return true;
            };
            bool ok = mbar_wait(&ctl->q_full, 0) && mbar_wait(&ctl->kv_full[0], 0);
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                tc_fence_after();
                issue_qk(std::integral_constant<int, 0>{});
            }
            for (int i = 0; ok && i < tiles_u; i += 2) {
                ok = step(std::integral_constant<int, 0>{}, i);
                if (ok && i + 1 < tiles_u) ok = step(std::integral_constant<int, 1>{}, i + 1);
            }
            if (!ok && lane == 0) {
                flag_status(p.status, OMNI_DEV_TIMEOUT);
                *abort_flag = 1;
            }
        }
        __syncwarp();
    } else {
        // =========================== softmax + epilogue =================================
        const int quarter = warp & 3;                       // tensor-memory lane quarter of this warp
        const int row = quarter * 16 + (lane & 15);         // head row within the CTA
        const int half = lane >> 4;                         // token half of S / column half of O
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        uint8_t *p_row = smem + kSmemP + row * 128;
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
            uint32_t sv[32];
            tc_ld16x2(tmem + lane_base + kColS + 64 * buf, sv);
            tc_wait_ld();
            tc_fence_before();
            mbar_arrive(&ctl->s_empty[buf]);
            const uint64_t vm = ctl->valid_mask[i % kStages];
            const uint32_t valid = (uint32_t)(vm >> (32 * half));
            float x[32];
            float mt = -INFINITY;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                x[j] = ((valid >> j) & 1u) ? __uint_as_float(sv[j]) * p.scale_log2 : -INFINITY;
                mt = fmaxf(mt, x[j]);
            }
            mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 16));
            // move the reference only when the tile maximum leaves the window above it
            float factor = 1.f;
            bool moved = false;
            if (mt > m_ref + kRescaleThreshold || (m_ref == -INFINITY && mt > -INFINITY)) {
                factor = exp2f(m_ref - mt);                 // 0 on the first finite maximum
                m_ref = mt;
                moved = true;
            }
            const float mr = (m_ref == -INFINITY) ? 0.f : m_ref;
            float sum = 0.f;
            uint32_t pk[16];
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
                const float e0 = fast_exp2(x[j] - mr), e1 = fast_exp2(x[j + 1] - mr);
                sum += e0 + e1;
                pk[j >> 1] = pack_bf16(e0, e1);
            }
            l = l * factor + sum;
            // P and O may only be touched once the previous tile's P V has finished
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
            // P row: 64 tokens x bf16 = 128 B = eight 16-byte chunks, chunk c stored at c ^ (row % 8)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int chunk = (half * 4 + c) ^ (row & 7);
                *reinterpret_cast<uint4 *>(p_row + chunk * 16) =
                    make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(&ctl->p_full);
        }
        if (ok) {
            ok = mbar_wait(&ctl->pv_done, (tiles - 1) & 1);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            const float lt = l + __shfl_xor_sync(0xffffffffu, l, 16);
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

    // ---- tear-down ----------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------
// host side: tensor maps and launch
// ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            ptr = nullptr;
        return reinterpret_cast<EncodeTiledFn>(ptr);
    }();
    return fn;
}

// Encoding a tensor map costs about a microsecond of host time and a decode step needs up to
// four, more than the launch itself, so encodings are kept (a map depends only on the base
// address and the sizes; nothing in it refers to a call).  Callers that must not pay even the
// lookup build a plan once (omni_sparse_mla_plan_init), which stores the maps themselves.
// The table is direct-mapped on a hash of the key and large enough for the maps of a few
// hundred distinct pools (a model with one KV pool per layer uses three maps per layer); a
// colliding key replaces the older entry.
struct MapCacheEntry {
    const void *base;
    uint64_t rows;
    uint32_t box_rows, box_panels, kind;
    bool used;
    CUtensorMap map;
};

inline bool cached_map(CUtensorMap *out, const void *base, uint64_t rows, uint32_t box_rows, uint32_t box_panels,
                       uint32_t kind, bool (*encode)(CUtensorMap *, const void *, uint64_t, uint32_t, uint32_t))
{
    constexpr uint32_t kEntries = 1024;
    static MapCacheEntry cache[kEntries];
    static std::mutex mu;
    uint64_t h = reinterpret_cast<uintptr_t>(base) * 0x9E3779B97F4A7C15ull;
    h ^= (rows + 0x7F4A7C15ull) * 0xC2B2AE3D27D4EB4Full;
    h ^= ((uint64_t)box_rows << 40) ^ ((uint64_t)box_panels << 20) ^ kind;
    h *= 0x9E3779B97F4A7C15ull;
    MapCacheEntry &e = cache[(h >> 40) % kEntries];
    std::lock_guard<std::mutex> lock(mu);
    if (e.used && e.base == base && e.rows == rows && e.box_rows == box_rows && e.box_panels == box_panels && e.kind == kind) {
        *out = e.map;
        return true;
    }
    if (!encode(out, base, rows, box_rows, box_panels)) return false;
    e.base = base;
    e.rows = rows;
    e.box_rows = box_rows;
    e.box_panels = box_panels;
    e.kind = kind;
    e.map = *out;
    e.used = true;
    return true;
}

// 2-D bf16 row-major [rows, 576] tensor, boxes of 64 columns x box_rows rows, 128-byte swizzle.
inline bool encode_row_map(CUtensorMap *map, const void *base, uint64_t rows, uint32_t box_rows, uint32_t)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)kDqk, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)kDqk * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same tensor seen as [rows, 9 panels of 64 columns]: 3-D boxes {64 columns, box_rows, n panels}
// land in shared memory panel by panel ([64 rows x 128 B] each, 128-byte swizzle), which is the
// operand layout of the MMAs, so one instruction fills up to a whole 72 KiB tile.
inline bool encode_panel_map(CUtensorMap *map, const void *base, uint64_t rows, uint32_t box_rows, uint32_t box_panels)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {64, (cuuint64_t)rows, (cuuint64_t)kPanels};
    const cuuint64_t strides[2] = {(cuuint64_t)kDqk * 2, 128};
    const cuuint32_t box[3] = {64, box_rows, box_panels};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline bool make_row_map(CUtensorMap *map, const void *base, uint64_t rows, uint32_t box_rows)
{
    return cached_map(map, base, rows, box_rows, 0, 0, encode_row_map);
}

inline bool make_panel_map(CUtensorMap *map, const void *base, uint64_t rows, uint32_t box_rows, uint32_t box_panels)
{
    return cached_map(map, base, rows, box_rows, box_panels, 1, encode_panel_map);
}

// Host side of a launch, in three steps so that a plan can do the first two once:
// per-device kernel attributes, the tensor maps, the launch itself.
inline bool tc_prepare_device()
{
    static bool attr_set[64] = {};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    std::lock_guard<std::mutex> lock(mu);
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(tc_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemBytes) !=
            cudaSuccess)
            return false;
        attr_set[dev] = true;
    }
    return true;
}

// maps[0] = q, maps[1] = pool rows (gathers), maps[2] = pool pages (boxes)
inline bool tc_make_maps(const DecodeParams &p, CUtensorMap *maps, bool cached)
{
    const uint64_t rows = (uint64_t)p.num_pages * kPage, qrows = (uint64_t)p.batch * p.heads;
    if (cached)
        return make_panel_map(&maps[0], p.q, qrows, kTcHeads, kPanels) && make_row_map(&maps[1], p.kv, rows, 1) &&
               make_panel_map(&maps[2], p.kv, rows, kTile, kPanels);
    return encode_panel_map(&maps[0], p.q, qrows, kTcHeads, kPanels) && encode_row_map(&maps[1], p.kv, rows, 1, 0) &&
           encode_panel_map(&maps[2], p.kv, rows, kTile, kPanels);
}

inline omni_status_t tc_launch(const CUtensorMap *maps, const DecodeParams &p, cudaStream_t stream)
{
    const int head_groups = (p.heads + kTcHeads - 1) / kTcHeads;
    const unsigned grid = (unsigned)(p.batch * p.splits * head_groups);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = kTcSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;    // see the kernel's first lines
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, tc_decode_kernel, maps[0], maps[1], maps[2], p) == cudaSuccess ? OMNI_OK
                                                                                                   : OMNI_ERR_CUDA;
}

}  // namespace omni
