// Selection producer for token-level sparsity: the positions of the k largest scores of every
// request, written as the sel_idx / sel_len arrays the decode kernels read.
//
// One cluster of up to eight CTAs per request.  Every CTA loads its share of the request's scores
// ONCE, as order-preserving 32-bit keys, into shared memory; everything after that works on
// shared memory.  A most-significant-digit radix select (four passes of 8 bits) finds the key
// T of the k-th largest score: per pass every CTA histograms the digit of its keys that still
// match the prefix, the cluster's histograms are summed through distributed shared memory, and each
// CTA scans the 256 bins for the digit that holds the k-th largest.  Then every key above T is
// selected, and of the keys equal to T the ones at the lowest positions, as many as are still
// missing; positions are written in increasing order, so the output is a deterministic function
// of the scores (ties included).
#pragma once

#include <mutex>

#include "common.cuh"

namespace omni {

constexpr int kTopkCluster = 8;
constexpr int kTopkThreads = 512;
constexpr int kTopkChunk = 24576;                        // most keys a CTA holds in shared memory (96 KiB)
constexpr int kTopkFew = 4096;                           // candidates below which a pass skips the lane-private copies
constexpr int kTopkMaxContext = 131072;                  // positions per request

// float bits -> unsigned key with the same order; NaN sorts below everything
__device__ __forceinline__ uint32_t topk_key(float f)
{
    const uint32_t u = __float_as_uint(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ uint32_t ld_cluster_u32(uint32_t cluster_addr)
{
    uint32_t v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(cluster_addr) : "memory");
    return v;
}

__device__ __forceinline__ uint32_t topk_map(const void *p, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"((uint32_t)__cvta_generic_to_shared(p)), "r"(rank));
    return r;
}

__device__ __forceinline__ void topk_cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

constexpr int kTopkWarps = kTopkThreads / 32;

struct alignas(16) TopkShared {
    uint32_t replicas[256 * 32];     // digit histogram, one copy per lane: entry (digit, lane) at digit * 32 + lane
    uint32_t published[2][256];      // this CTA's histogram of the current pass, read by the whole cluster
    uint32_t counts[2];              // keys above / equal to the threshold in this chunk
    uint32_t prefix, need;           // result of a digit search: the extended prefix, keys still to take in its bin
    uint32_t bin_count;              // ... and the keys of the whole cluster in that bin
    uint32_t warp_sums[kTopkWarps];
    uint32_t warp_gt[kTopkWarps], warp_eq[kTopkWarps];
};
static_assert(sizeof(TopkShared) % 16 == 0, "the keys behind the control block are stored with 16-byte stores");

__global__ void __launch_bounds__(kTopkThreads, 2)
topk_select_kernel(const float *__restrict__ scores, const int32_t *__restrict__ ctx_len, int stride, int k,
                   int32_t *__restrict__ sel_idx, int32_t *__restrict__ sel_len)
{
    extern __shared__ __align__(16) unsigned char topk_smem[];
    TopkShared &sh = *reinterpret_cast<TopkShared *>(topk_smem);
    uint32_t *keys = reinterpret_cast<uint32_t *>(topk_smem + sizeof(TopkShared));     // this CTA's keys: ceil(stride / cluster width) (+ 4 of slack)

    uint32_t crank, nranks;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank));
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(nranks));
    // launched with programmatic stream serialization: nothing of the previous kernel in the stream is
    // read or overwritten before this returns
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int b = blockIdx.x / nranks;
    int m = __ldg(ctx_len + b);
    m = max(0, min(m, stride));
    const int want = min(k, m);
    const int chunk = ((m + (int)nranks - 1) / (int)nranks + 3) & ~3;      // a multiple of four keeps the 16-byte loads aligned
    const int start = min(m, (int)crank * chunk), len = min(m, start + chunk) - start;
    const float *src = scores + (size_t)b * stride + start;
    {
        // scalar head up to a 16-byte boundary, 16-byte loads for the body, scalar tail
        // the keys sit in shared memory at the same offset from a 16-byte boundary as the scores in global
        // memory, so that the body is stored with 16-byte stores too
        const uint32_t misalign = (uint32_t)((reinterpret_cast<uintptr_t>(src) >> 2) & 3u);
        keys += misalign;
        const int head = min(len, (int)((4u - misalign) & 3u));
        const int body = (len - head) >> 2;
        const float4 *src4 = reinterpret_cast<const float4 *>(src + head);
#pragma unroll 8
        for (int j = threadIdx.x; j < body; j += kTopkThreads) {
            const float4 v = __ldg(src4 + j);
            *reinterpret_cast<uint4 *>(keys + head + 4 * j) =
                make_uint4(topk_key(v.x), topk_key(v.y), topk_key(v.z), topk_key(v.w));
        }
        if ((int)threadIdx.x < head) keys[threadIdx.x] = topk_key(__ldg(src + threadIdx.x));
        const int tail = head + 4 * body;
        if (tail + (int)threadIdx.x < len) keys[tail + threadIdx.x] = topk_key(__ldg(src + tail + threadIdx.x));
    }
    for (int i = threadIdx.x; i < 256 * 32; i += kTopkThreads) sh.replicas[i] = 0;

    uint32_t prefix = 0, mask = 0, need = (uint32_t)want;
    bool few = false;                                      // at most kTopkFew keys of the cluster still match the prefix
    int pass = 0;
    for (int shift = 24; shift >= 0; shift -= 8, ++pass) {
        __syncthreads();                                   // keys stored (first pass), histogram copies zeroed
        if (few) {
            // few keys are left in the cluster: they go straight into the published histogram
            if (threadIdx.x < 256) sh.published[pass & 1][threadIdx.x] = 0;
            __syncthreads();
#pragma unroll 8
            for (int i = threadIdx.x; i < len; i += kTopkThreads) {
                const uint32_t key = keys[i];
                if ((key & mask) == prefix) atomicAdd(&sh.published[pass & 1][(key >> shift) & 255u], 1u);
            }
            topk_cluster_sync();
        } else {
            // every lane adds into its own copy of the histogram: no two lanes of a warp ever meet on a
            // word or a bank, however the digits are distributed
#pragma unroll 8
            for (int i = threadIdx.x; i < len; i += kTopkThreads) {
                const uint32_t key = keys[i];
                if ((key & mask) == prefix) atomicAdd(&sh.replicas[((key >> shift) & 255u) * 32 + lane], 1u);
            }
            __syncthreads();
            {
                // thread t sums half of the 32 copies of bin t / 2 (rotated start keeps the banks apart)
                const int bin = threadIdx.x >> 1, half = threadIdx.x & 1;
                uint32_t c = 0;
#pragma unroll
                for (int j = 0; j < 16; ++j) c += sh.replicas[bin * 32 + half * 16 + ((j + bin) & 15)];
                c += __shfl_xor_sync(0xffffffffu, c, 1);
                if (half == 0) sh.published[pass & 1][bin] = c;
            }
            __syncthreads();                                   // all copies read: they can be cleared for the next pass
            asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
            for (int i = threadIdx.x; i < 256 * 32; i += kTopkThreads) sh.replicas[i] = 0;
            asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");      // every CTA's histogram is visible
        }
        {
            // threads 0..255: bin t of the histogram summed over the cluster, then the bin that holds
            // the need-th largest key: keys in higher bins < need <= keys in this and higher bins
            uint32_t c = 0;
            if (threadIdx.x < 256) {
                uint32_t part[kTopkCluster];               // all remote loads in flight before the first use
#pragma unroll
                for (uint32_t r = 0; r < kTopkCluster; ++r)
                    part[r] = r < nranks ? ld_cluster_u32(topk_map(&sh.published[pass & 1][threadIdx.x], r)) : 0u;
#pragma unroll
                for (uint32_t r = 0; r < kTopkCluster; ++r) c += part[r];
            }
            uint32_t inc = c;                              // inclusive suffix sum within the warp
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t o = __shfl_down_sync(0xffffffffu, inc, d);
                if (lane + d < 32) inc += o;
            }
            if (lane == 0) sh.warp_sums[warp] = inc;
            __syncthreads();
            uint32_t above = 0;                            // keys in the bins of higher warps
            for (int w = warp + 1; w < 8; ++w) above += sh.warp_sums[w];
            const uint32_t with_me = above + inc, higher = with_me - c;
            if (threadIdx.x < 256 && higher < need && need <= with_me) {
                sh.prefix = prefix | ((uint32_t)threadIdx.x << shift);
                sh.need = need - higher;
                sh.bin_count = c;
            }
            if (need == 0 && threadIdx.x == 0) {
                sh.prefix = prefix | (255u << shift);      // nothing to select: any threshold will do
                sh.need = 0;
                sh.bin_count = 0;
            }
        }
        __syncthreads();
        prefix = sh.prefix;
        need = sh.need;
        few = sh.bin_count <= (uint32_t)kTopkFew;
        mask |= 255u << shift;
        // published[] alternates between passes, and the next pass's cluster barrier comes before
        // anybody overwrites the copy read here
        if (need == sh.bin_count) break;                   // every key left under the prefix is taken: the lower digits decide nothing
    }
    // Keys above the prefix's range are selected, keys inside it (all digits searched: keys equal to the
    // threshold) tie for the `need` places left, lowest positions first.
    // Warp w owns the contiguous keys [w * per_warp, (w + 1) * per_warp) of the chunk.
    const uint32_t T = prefix | ~mask;                     // largest key under the prefix
    const int per_warp = ((len + kTopkWarps - 1) / kTopkWarps + 127) & ~127;
    const int w_begin = min(len, warp * per_warp), w_end = min(len, w_begin + per_warp);
    uint32_t gt = 0, eq = 0;
#pragma unroll 8
    for (int i = w_begin + lane; i < w_end; i += 32) {
        gt += keys[i] > T;
        eq += (keys[i] & mask) == prefix;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        gt += __shfl_xor_sync(0xffffffffu, gt, d);
        eq += __shfl_xor_sync(0xffffffffu, eq, d);
    }
    if (lane == 0) {
        sh.warp_gt[warp] = gt;
        sh.warp_eq[warp] = eq;
    }
    __syncthreads();
    uint32_t gt_before = 0, eq_before = 0, gt_all = 0, eq_all = 0;       // within this chunk, before this warp
    for (int w = 0; w < kTopkWarps; ++w) {
        const uint32_t g = sh.warp_gt[w], e = sh.warp_eq[w];
        if (w < warp) {
            gt_before += g;
            eq_before += e;
        }
        gt_all += g;
        eq_all += e;
    }
    if (threadIdx.x == 0) {
        sh.counts[0] = gt_all;
        sh.counts[1] = eq_all;
    }
    topk_cluster_sync();
    // threshold ties and keys above the threshold in the chunks before this one
    {
        uint32_t g[kTopkCluster], e[kTopkCluster];         // all remote loads in flight before the first use
#pragma unroll
        for (uint32_t r = 0; r < kTopkCluster; ++r) {
            g[r] = r < crank ? ld_cluster_u32(topk_map(&sh.counts[0], r)) : 0u;
            e[r] = r < crank ? ld_cluster_u32(topk_map(&sh.counts[1], r)) : 0u;
        }
#pragma unroll
        for (uint32_t r = 0; r < kTopkCluster; ++r) {
            gt_before += g[r];
            eq_before += e[r];
        }
    }
    // entries written before this warp's first key: everything above T, and the first `need` ties
    uint32_t run_eq = eq_before, run_out = gt_before + min(eq_before, need);
    int32_t *dst = sel_idx + (size_t)b * k;
    const uint32_t lanes_below = (1u << lane) - 1u;
    for (int base = w_begin; base < w_end && want > 0; base += 128) {
        uint32_t key[4];
        bool at_least[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = base + 32 * j + lane;
            key[j] = i < w_end ? keys[i] : 0u;
            at_least[j] = i < w_end && key[j] >= prefix;
        }
        if (!__any_sync(0xffffffffu, at_least[0] || at_least[1] || at_least[2] || at_least[3])) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const bool is_eq = at_least[j] && (key[j] & mask) == prefix;
            const uint32_t eq_ballot = __ballot_sync(0xffffffffu, is_eq);
            const uint32_t eq_rank = run_eq + __popc(eq_ballot & lanes_below);
            const bool sel = at_least[j] && (!is_eq || eq_rank < need);
            const uint32_t sel_ballot = __ballot_sync(0xffffffffu, sel);
            const uint32_t pos = run_out + __popc(sel_ballot & lanes_below);
            if (sel && pos < (uint32_t)want) dst[pos] = start + base + 32 * j + lane;
            run_eq += __popc(eq_ballot);
            run_out += __popc(sel_ballot);
        }
    }
    if (crank == 0 && threadIdx.x == 0) sel_len[b] = want;
    topk_cluster_sync();                                   // nobody leaves while its counts may still be read
}

// Launch shape.  A CTA costs about 4 us plus 0.4 us per CTA of its cluster, plus 0.6 us per 1024 keys
// when it has its SM to itself and 0.85 us per 1024 keys when two CTAs share an SM (fitted to
// measurements).  Every width from 1 to 8 that holds the context is priced with the number of clusters
// of that width the device keeps resident, alone on their SMs or two to an SM, and the cheapest wins.
struct TopkShape {
    int width;
    size_t smem;
};

constexpr size_t kTopkSmemAlone = 120 * 1024;            // more than half an SM's shared memory: one CTA per SM
constexpr size_t kTopkSmemPair = 112 * 1024;             // two CTAs of up to this much fit one SM

inline size_t topk_smem_need(int chunk) { return sizeof(TopkShared) + (size_t)(chunk + 4) * sizeof(uint32_t); }

inline void topk_launch_config(cudaLaunchConfig_t &cfg, cudaLaunchAttribute *attr, int batch, int width, size_t smem,
                               cudaStream_t stream)
{
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = dim3((unsigned)(batch * width));
    cfg.blockDim = dim3(kTopkThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)width;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
}

// Clusters of `width` resident at once (asked once per device, width and mode; at least 1).
inline int topk_resident_clusters(int dev, int width, bool alone)
{
    static std::mutex lock;                                // callers on several host threads share the table
    static int cache[64][kTopkCluster + 1][2] = {};
    std::lock_guard<std::mutex> guard(lock);
    int &slot = cache[dev][width][alone ? 1 : 0];
    if (slot == 0) {
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attr[2];
        topk_launch_config(cfg, attr, 1, width, alone ? kTopkSmemAlone : kTopkSmemPair, nullptr);
        cfg.numAttrs = 1;                                  // the cluster shape is all the query needs
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, topk_select_kernel, &cfg) != cudaSuccess) n = 0;
        slot = n > 0 ? n : 1;
    }
    return slot;
}

inline TopkShape topk_shape(int dev, int batch, int stride)
{
    TopkShape best = {kTopkCluster, topk_smem_need(kTopkChunk)};
    double best_cost = 1e30;
    for (int width = kTopkCluster; width >= 1; --width) {
        const int chunk = ((stride + width - 1) / width + 3) & ~3;
        if (chunk > kTopkChunk) break;                     // narrower clusters cannot hold the context
        const size_t need = topk_smem_need(chunk);
        const double per_key = chunk / 1024.0;
        const int alone = topk_resident_clusters(dev, width, true);
        const double fixed = 4.0 + 0.4 * width + ((width & (width - 1)) ? 0.5 : 0.0);   // odd widths measured slightly slower
        const double cost_alone = ((batch + alone - 1) / alone) * (fixed + 0.6 * per_key);
        if (cost_alone < best_cost) {
            best_cost = cost_alone;
            best = {width, need > kTopkSmemAlone ? need : kTopkSmemAlone};
        }
        if (need <= kTopkSmemPair) {
            const int paired = topk_resident_clusters(dev, width, false);
            const double cost_pair = ((batch + paired - 1) / paired) * (fixed + 0.85 * per_key);
            if (cost_pair < best_cost) {
                best_cost = cost_pair;
                best = {width, need};
            }
        }
    }
    return best;
}

inline omni_status_t launch_topk_select(const float *scores, const int32_t *ctx_len, int batch, int stride, int k,
                                        int32_t *sel_idx, int32_t *sel_len, cudaStream_t stream)
{
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return OMNI_ERR_CUDA;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(topk_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)topk_smem_need(kTopkChunk)) != cudaSuccess)
            return OMNI_ERR_CUDA;
        attr_set[dev] = true;
    }
    const TopkShape shape = topk_shape(dev, batch, stride);
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    topk_launch_config(cfg, attr, batch, shape.width, shape.smem, stream);
    return cudaLaunchKernelEx(&cfg, topk_select_kernel, scores, ctx_len, stride, k, sel_idx, sel_len) == cudaSuccess
               ? OMNI_OK
               : OMNI_ERR_CUDA;
}

}  // namespace omni
