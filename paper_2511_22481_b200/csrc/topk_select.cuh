// Selection producer for token-level sparsity: the positions of the k largest scores of every
// request, written as the sel_idx / sel_len arrays the decode kernels read.
//
// One cluster of eight CTAs per request.  Every CTA loads an eighth of the request's scores
// ONCE, as order-preserving 32-bit keys, into shared memory; everything after that works on
// shared memory.  A most-significant-digit radix select (four passes of 8 bits) finds the key
// T of the k-th largest score: per pass every CTA histograms the digit of its keys that still
// match the prefix, the eight histograms are summed through distributed shared memory, and each
// CTA scans the 256 bins for the digit that holds the k-th largest.  Then every key above T is
// selected, and of the keys equal to T the ones at the lowest positions, as many as are still
// missing; positions are written in increasing order, so the output is a deterministic function
// of the scores (ties included).
#pragma once

#include "common.cuh"

namespace omni {

constexpr int kTopkCluster = 8;
constexpr int kTopkThreads = 512;
constexpr int kTopkChunk = 16384;                        // keys per CTA held in shared memory
constexpr int kTopkMaxContext = kTopkCluster * kTopkChunk;   // 131072 positions per request

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

// Exclusive prefix sum of one value per thread over the block (512 threads); also returns the total.
__device__ __forceinline__ int topk_block_scan(int v, int *warp_sums, int &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += o;
    }
    __syncthreads();                                      // warp_sums may still be read from the last call
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    int base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kTopkThreads / 32; ++w) {
        const int s = warp_sums[w];
        if (w < warp) base += s;
        tot += s;
    }
    total = tot;
    return base + inc - v;
}

__global__ void __launch_bounds__(kTopkThreads, 1)
topk_select_kernel(const float *__restrict__ scores, const int32_t *__restrict__ ctx_len, int stride, int k,
                   int32_t *__restrict__ sel_idx, int32_t *__restrict__ sel_len)
{
    extern __shared__ uint32_t keys[];                    // kTopkChunk keys of this CTA
    __shared__ uint32_t hist[256];                         // this CTA's digit histogram (read by the whole cluster)
    __shared__ uint32_t counts[2];                         // keys above / equal to the threshold in this chunk
    __shared__ uint32_t sh_prefix, sh_need;
    __shared__ int warp_sums[kTopkThreads / 32];

    uint32_t crank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank));
    const int b = blockIdx.x / kTopkCluster;
    int m = __ldg(ctx_len + b);
    m = max(0, min(m, stride));
    const int want = min(k, m);
    const int chunk = (m + kTopkCluster - 1) / kTopkCluster;
    const int start = min(m, (int)crank * chunk), len = min(m, start + chunk) - start;
    const float *src = scores + (size_t)b * stride + start;
    for (int i = threadIdx.x; i < len; i += kTopkThreads) keys[i] = topk_key(__ldg(src + i));

    uint32_t prefix = 0, mask = 0, need = (uint32_t)want;
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (threadIdx.x < 256) hist[threadIdx.x] = 0;
        __syncthreads();
        for (int i = threadIdx.x; i < len; i += kTopkThreads) {
            const uint32_t key = keys[i];
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        topk_cluster_sync();                               // every CTA's histogram is complete and visible
        if (threadIdx.x < 32) {
            // lane l owns bins 8l .. 8l+7 of the summed histogram; find the bin of the need-th largest
            uint32_t bins[8], mine = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                uint32_t c = 0;
                for (uint32_t r = 0; r < kTopkCluster; ++r) c += ld_cluster_u32(topk_map(&hist[8 * threadIdx.x + j], r));
                bins[j] = c;
                mine += c;
            }
            // above = keys in bins of higher lanes
            uint32_t above = 0;
            for (int l = 31; l >= 1; --l) {
                const uint32_t other = __shfl_sync(0xffffffffu, mine, l);
                if (l > (int)threadIdx.x) above += other;
            }
            const bool here = above < need && above + mine >= need;      // exactly one lane when need >= 1
            if (here) {
                uint32_t cum = above;
                int digit = 8 * threadIdx.x;
#pragma unroll
                for (int j = 7; j >= 0; --j) {
                    if (cum + bins[j] >= need) {
                        digit = 8 * threadIdx.x + j;
                        break;
                    }
                    cum += bins[j];
                }
                sh_prefix = prefix | ((uint32_t)digit << shift);
                sh_need = need - cum;
            }
            if (need == 0 && threadIdx.x == 0) {
                sh_prefix = prefix | (255u << shift);      // nothing to select: any threshold above all keys will do
                sh_need = 0;
            }
        }
        __syncthreads();
        prefix = sh_prefix;
        need = sh_need;
        mask |= 255u << shift;
        topk_cluster_sync();                               // all CTAs have read this pass's histograms
    }
    // prefix is now the key T of the want-th largest score, need the number of keys equal to T still to take
    const uint32_t T = prefix;
    uint32_t gt = 0, eq = 0;
    for (int i = threadIdx.x; i < len; i += kTopkThreads) {
        gt += keys[i] > T;
        eq += keys[i] == T;
    }
    if (threadIdx.x < 2) counts[threadIdx.x] = 0;
    __syncthreads();
    if (want > 0) {
        atomicAdd(&counts[0], gt);
        atomicAdd(&counts[1], eq);
    }
    __syncthreads();
    topk_cluster_sync();
    // selected entries and threshold ties in the chunks before this one
    uint32_t out_base = 0, eq_before = 0;
    for (uint32_t r = 0; r < crank; ++r) {
        const uint32_t g = ld_cluster_u32(topk_map(&counts[0], r)), e = ld_cluster_u32(topk_map(&counts[1], r));
        const uint32_t take = eq_before < need ? min(e, need - eq_before) : 0u;
        out_base += g + take;
        eq_before += e;
    }
    int32_t *dst = sel_idx + (size_t)b * k;
    int run_out = (int)out_base, run_eq = (int)eq_before;
    for (int base = 0; base < len && want > 0; base += kTopkThreads) {
        const int i = base + threadIdx.x;
        const uint32_t key = i < len ? keys[i] : 0u;
        const int is_eq = (i < len && key == T) ? 1 : 0;
        int eq_total, sel_total;
        const int eq_rank = run_eq + topk_block_scan(is_eq, warp_sums, eq_total);
        const int sel = (i < len && (key > T || (is_eq && (uint32_t)eq_rank < need))) ? 1 : 0;
        const int pos = run_out + topk_block_scan(sel, warp_sums, sel_total);
        if (sel && pos < want) dst[pos] = start + i;
        run_eq += eq_total;
        run_out += sel_total;
    }
    if (crank == 0 && threadIdx.x == 0) sel_len[b] = want;
    topk_cluster_sync();                                   // nobody leaves while its counts may still be read
}

inline omni_status_t launch_topk_select(const float *scores, const int32_t *ctx_len, int batch, int stride, int k,
                                        int32_t *sel_idx, int32_t *sel_len, cudaStream_t stream)
{
    const size_t smem = (size_t)kTopkChunk * sizeof(uint32_t);
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return OMNI_ERR_CUDA;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(topk_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return OMNI_ERR_CUDA;
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(batch * kTopkCluster));
    cfg.blockDim = dim3(kTopkThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kTopkCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, topk_select_kernel, scores, ctx_len, stride, k, sel_idx, sel_len) == cudaSuccess
               ? OMNI_OK
               : OMNI_ERR_CUDA;
}

}  // namespace omni
