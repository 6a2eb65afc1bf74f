// Nucleus sampling (Sec. 3.2 names it as the alternative to the top-1 token) on logits that a
// head kernel has written to global memory: one thread-block cluster per path (as many CTAs as
// the SMs allow at the call's path count, up to eight).  A CTA takes a contiguous share of the
// vocabulary and keeps as much of it as fits in shared memory, so that the row is read from
// global memory once; every decision (maximum, boundary bin, boundary token) is taken by every
// CTA of the cluster on merged data read through distributed shared memory, hence identically,
// and the CTAs meet at the hardware cluster barrier only.
//
//   p = Softmax(l / temperature);  nucleus = tokens in order of decreasing p (equal p: increasing
//   id) up to and including the one whose cumulative probability reaches top_p;  the token is the
//   argmax over the nucleus of l[v] / temperature + Gumbel noise (dm_common.cuh: gumbel_noise).
//
// No sort of the vocabulary: the boundary of the nucleus is found by mass.  Probabilities are
// summed as 40-bit fixed-point integers, so that every sum is exact and independent of the order
// in which threads add (the result of a call depends on its inputs only).
//   1. m = max z, z = l / temperature
//   2. histogram of q_v = floor(exp(z_v - m) * 2^40) over 2048 bins of (m - z) (bin width 1/64,
//      the last bin takes the rest); Q = its total; the bin in which the running mass from the
//      top reaches top_p * Q holds the boundary
//   3. if that bin holds more tokens than the sort below takes: the same once more inside it
//   4. the tokens of the boundary bin are sorted by (z, id) in shared memory and walked until
//      the mass is reached: the last one taken is the boundary token
//   5. Gumbel-max over all tokens that do not come after the boundary token
#include <cooperative_groups.h>

#include "dm_internal.h"

namespace dm {

namespace {

namespace cg = cooperative_groups;

constexpr int kNsThreads = 1024;
constexpr int kNsBins = 2048;
constexpr int kNsList = 1024;
constexpr float kNsBinsPerUnit = 64.0f;            // level-0 bins per unit of z
constexpr float kNsFixedOne = 1099511627776.0f;    // 2^40

__device__ __forceinline__ unsigned long long block_sum_u64(unsigned long long x, unsigned long long* red) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, off);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
    __syncthreads();
    unsigned long long t = 0;
    for (int w = 0; w < kNsThreads / 32; ++w) t += red[w];
    return t;
}
__device__ __forceinline__ unsigned long long block_max_u64(unsigned long long x, unsigned long long* red) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, x, off);
        x = o > x ? o : x;
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
    __syncthreads();
    unsigned long long t = 0;
    for (int w = 0; w < kNsThreads / 32; ++w) t = red[w] > t ? red[w] : t;
    return t;
}

// Exclusive prefix sum over the block's threads (thread order); `red` holds one word per warp.
__device__ __forceinline__ unsigned long long block_exclusive_scan_u64(unsigned long long x, unsigned long long* red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long incl = x;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned long long o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += o;
    }
    __syncthreads();
    if (lane == 31) red[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        unsigned long long t = red[lane], ti = t;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned long long o = __shfl_up_sync(0xFFFFFFFFu, ti, off);
            if (lane >= off) ti += o;
        }
        red[lane] = ti - t;   // exclusive over the warps
    }
    __syncthreads();
    return red[warp] + incl - x;
}

// Order of the nucleus walk: larger z first, equal z: smaller id first.
__device__ __forceinline__ unsigned long long walk_key(float z, int v) {
    return ((unsigned long long)float_key(z) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)v);
}


// Shared memory of a CTA (dynamic): the three histogram arrays, the CTA's own list of boundary-bin
// tokens, the cluster's merged list, then the stash of z values.
constexpr size_t kNsFixedSmem = 3 * kNsBins * sizeof(unsigned int) + 4 * kNsList * sizeof(unsigned long long);

__global__ void __launch_bounds__(kNsThreads)
nucleus_sample_kernel(const float* __restrict__ logits, int V, int chunk, int stash_len, RowMap map, uint32_t key0,
                      uint32_t key1, float inv_temp, float top_p, int v_offset,
                      unsigned long long* __restrict__ out_packed) {
    extern __shared__ __align__(16) unsigned char ns_smem[];
    unsigned int* hist_lo = reinterpret_cast<unsigned int*>(ns_smem);   // 64-bit mass per bin as two words (32-bit shared atomics are native)
    unsigned int* hist_hi = hist_lo + kNsBins;
    unsigned int* cnt = hist_hi + kNsBins;
    unsigned long long* list_key = reinterpret_cast<unsigned long long*>(cnt + kNsBins);   // this CTA's boundary-bin tokens
    unsigned long long* list_q = list_key + kNsList;
    unsigned long long* all_key = list_q + kNsList;                                         // the cluster's, merged
    unsigned long long* all_q = all_key + kNsList;
    float* stash = reinterpret_cast<float*>(all_q + kNsList);
    __shared__ unsigned long long red[kNsThreads / 32];
    __shared__ unsigned long long x_word;      // what this CTA shows the others: its maximum, later its best candidate
    __shared__ int x_count;                    // ... and the length of its list
    __shared__ int s_bin, s_count, s_level;
    __shared__ unsigned long long s_above, s_boundary;
    __shared__ float s_lo;   // distance m - z at which the level-1 bins start

    cg::cluster_group cluster = cg::this_cluster();
    const int n_cta = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
    const int row = blockIdx.x / n_cta, tid = threadIdx.x;
    const int v0 = rank * chunk, n = max(0, min(V, v0 + chunk) - v0);   // this CTA's share of the vocabulary
    const float* l = logits + (size_t)row * V + v0;
    RowKey k;
    row_key(map, row, k);
    // z of local entry x: from the stash where it fits, else from global memory again
    auto zval = [&](int x) { return x < stash_len ? stash[x] : l[x] * inv_temp; };

    // 1. maximum (and the stash)
    float mx = -INFINITY;
#pragma unroll 8
    for (int x = tid; x < n; x += kNsThreads) {
        const float z = l[x] * inv_temp;
        if (x < stash_len) stash[x] = z;
        mx = fmaxf(mx, z);
    }
    {
        const unsigned long long mine = block_max_u64((unsigned long long)float_key(mx), red);
        if (tid == 0) x_word = mine;
    }
    cluster.sync();
    unsigned long long mkey = 0ull;
    for (int r = 0; r < n_cta; ++r) {
        const unsigned long long o = *cluster.map_shared_rank(&x_word, r);
        mkey = o > mkey ? o : mkey;
    }
    const float m = key_float((uint32_t)mkey);

    // 2./3. the bin that holds the boundary: level 0 over m - z, level 1 inside the level-0 bin.
    // The level-0 histogram also gives the total mass Q (its sum) and the bins' token counts.
    if (tid == 0) { s_level = 0; s_above = 0; s_lo = 0.0f; s_bin = 0; }
    unsigned long long target = 0;
    __syncthreads();
    for (int level = 0; level < 2; ++level) {
        for (int b = tid; b < kNsBins; b += kNsThreads) { hist_lo[b] = 0u; hist_hi[b] = 0u; cnt[b] = 0u; }
        __syncthreads();
        const float lo = s_lo;
        const int bin0 = s_bin;   // level 1: the level-0 bin being refined
#pragma unroll 4
        for (int x = tid; x < n; x += kNsThreads) {
            const float z = zval(x);
            const float dist = m - z;
            int b = min(kNsBins - 1, (int)(dist * kNsBinsPerUnit));
            if (level == 1) {
                if (b != bin0) continue;
                b = min(kNsBins - 1, max(0, (int)((dist - lo) * (kNsBinsPerUnit * kNsBins))));
            }
            const unsigned long long q = (unsigned long long)(expf(z - m) * kNsFixedOne);
            const uint32_t q_lo = (uint32_t)q;
            const uint32_t old = atomicAdd(&hist_lo[b], q_lo);
            const uint32_t q_hi = (uint32_t)(q >> 32) + ((uint32_t)(old + q_lo) < q_lo ? 1u : 0u);   // carry out of the low word
            if (q_hi) atomicAdd(&hist_hi[b], q_hi);
            atomicAdd(&cnt[b], 1u);
        }
        cluster.sync();   // every CTA's histogram is complete
        {   // the first bin at which the running mass reaches the target (the last bin if none does):
            // two bins per thread, summed over the CTAs, then a prefix sum over the threads
            unsigned long long h0 = 0, h1 = 0;
            unsigned int c0 = 0, c1 = 0;
            for (int r = 0; r < n_cta; ++r) {
                const unsigned int* rlo = cluster.map_shared_rank(hist_lo, r);
                const unsigned int* rhi = cluster.map_shared_rank(hist_hi, r);
                const unsigned int* rc = cluster.map_shared_rank(cnt, r);
                h0 += ((unsigned long long)rhi[2 * tid] << 32) + rlo[2 * tid];
                h1 += ((unsigned long long)rhi[2 * tid + 1] << 32) + rlo[2 * tid + 1];
                c0 += rc[2 * tid];
                c1 += rc[2 * tid + 1];
            }
            if (level == 0) {
                const unsigned long long Q = block_sum_u64(h0 + h1, red);
                const double target_d = (double)top_p * (double)Q;
                target = (unsigned long long)target_d;
                if ((double)target < target_d) ++target;     // the running mass must reach top_p * Q
            }
            const unsigned long long base = s_above;
            const unsigned long long before = base + block_exclusive_scan_u64(h0 + h1, red);
            int b = -1;
            unsigned long long above = 0;
            unsigned int cb = 0;
            if (before < target) {
                if (before + h0 >= target) { b = 2 * tid; above = before; cb = c0; }
                else if (before + h0 + h1 >= target || tid == kNsThreads - 1) { b = 2 * tid + 1; above = before + h0; cb = c1; }
            }
            __syncthreads();
            if (b >= 0) {             // exactly one thread: the running mass is non-decreasing
                s_above = above;      // mass of everything before the boundary bin
                if (level == 0) s_bin = b; else s_level = 1 + b;   // level 1: remember the sub-bin
                s_count = (int)cb;    // tokens in the boundary bin, over the whole cluster
            }
        }
        cluster.sync();   // everybody has read everybody's histogram (and this CTA's decision is in shared memory)
        if (s_count <= kNsList || level == 1) break;
        if (tid == 0) s_lo = (float)s_bin / kNsBinsPerUnit;
        __syncthreads();
    }

    // 4. the boundary token: the boundary bin's tokens of all CTAs, sorted by (z, id) and walked
    const int b0 = s_bin, b1 = s_level - 1;
    const float lo1 = s_lo;
    const bool refined = s_level > 0;
    for (int i = tid; i < kNsList; i += kNsThreads) { all_key[i] = 0ull; all_q[i] = 0ull; }
    if (tid == 0) x_count = 0;
    __syncthreads();
#pragma unroll 8
    for (int x = tid; x < n; x += kNsThreads) {
        const float z = zval(x);
        const float dist = m - z;
        if (min(kNsBins - 1, (int)(dist * kNsBinsPerUnit)) != b0) continue;
        if (refined && min(kNsBins - 1, max(0, (int)((dist - lo1) * (kNsBinsPerUnit * kNsBins)))) != b1) continue;
        const int slot = atomicAdd(&x_count, 1);
        if (slot < kNsList) {
            list_key[slot] = walk_key(z, v0 + x);
            list_q[slot] = (unsigned long long)(expf(z - m) * kNsFixedOne);
        }
    }
    cluster.sync();   // every CTA's list is complete
    int total = 0;
    for (int r = 0; r < n_cta; ++r) {     // the merged list, in every CTA (order does not matter: it is sorted next)
        const int c = *cluster.map_shared_rank(&x_count, r);
        const int take = min(c, kNsList);
        const unsigned long long* rk = cluster.map_shared_rank(list_key, r);
        const unsigned long long* rq = cluster.map_shared_rank(list_q, r);
        for (int i = tid; i < take; i += kNsThreads)
            if (total + i < kNsList) { all_key[total + i] = rk[i]; all_q[total + i] = rq[i]; }
        total += c;
    }
    __syncthreads();
    const int n_list = min(total, kNsList);
    // bitonic sort, descending by key (empty slots have key 0 and sink to the end)
    for (int size = 2; size <= kNsList; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const int i = tid, j = i ^ stride;
            if (j > i && i < kNsList) {
                const bool descending = (i & size) == 0;
                const unsigned long long a = all_key[i], b = all_key[j];
                if ((a < b) == descending) {
                    all_key[i] = b; all_key[j] = a;
                    const unsigned long long qa = all_q[i]; all_q[i] = all_q[j]; all_q[j] = qa;
                }
            }
            __syncthreads();
        }
    }
    {   // walk the sorted list: the first entry at which the running mass reaches the target
        if (tid == 0) s_boundary = n_list > 0 ? all_key[n_list - 1] : 0ull;   // (none does: all of them are in)
        const unsigned long long q = tid < n_list ? all_q[tid] : 0ull;
        const unsigned long long before = s_above + block_exclusive_scan_u64(q, red);
        if (tid < n_list && before < target && before + q >= target) s_boundary = all_key[tid];
    }
    __syncthreads();
    const unsigned long long boundary = s_boundary;
    const bool overflow = total > kNsList;   // more tokens of (nearly) one value than the sort takes: all of them are in

    // 5. Gumbel-max over the nucleus
    unsigned long long best = 0ull;
#pragma unroll 8
    for (int x = tid; x < n; x += kNsThreads) {
        const float z = zval(x);
        const int v = v0 + x;
        bool in;
        if (!overflow) {
            in = walk_key(z, v) >= boundary;
        } else {
            const float dist = m - z;
            const int b = min(kNsBins - 1, (int)(dist * kNsBinsPerUnit));
            in = b < b0 || (b == b0 && (!refined || min(kNsBins - 1, max(0, (int)((dist - lo1) * (kNsBinsPerUnit * kNsBins)))) <= b1));
        }
        if (!in) continue;
        const float val = z + gumbel_noise((uint32_t)(v + v_offset), k, key0, key1);
        const unsigned long long cand = pack_best(float_key(val), (uint32_t)(v + v_offset));
        best = cand > best ? cand : best;
    }
    best = block_max_u64(best, red);
    if (tid == 0) x_word = best;   // (the maxima exchanged through this word were read before the first histogram barrier)
    cluster.sync();
    if (rank == 0 && tid == 0) {
        unsigned long long b = 0ull;
        for (int r = 0; r < n_cta; ++r) {
            const unsigned long long o = *cluster.map_shared_rank(&x_word, r);
            b = o > b ? o : b;
        }
        out_packed[row] = b;
    }
    cluster.sync();   // nobody leaves while its shared memory may still be read
}

}  // namespace

int launch_nucleus_sample(const float* logits, int V, int rows, const RowMap& map, const MaskKey& mk, float top_p,
                          int v_offset, unsigned long long* out_packed, cudaStream_t stream) {
    if (rows < 1 || rows > 0x7FFFFFFF / 8) return DM_EINVAL;
    int sms = 148, dev = 0, smem_max = 227 * 1024;
    if (cudaGetDevice(&dev) != cudaSuccess) return DM_ECUDA;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    // As many CTAs per path as one wave of the SMs allows (a CTA fills an SM), eight at most
    // (the portable cluster size), and no more than the vocabulary has 1024-entry pieces.
    int n_cta = sms / rows;
    if (n_cta > 8) n_cta = 8;
    if (n_cta > (V + 1023) / 1024) n_cta = (V + 1023) / 1024;
    if (n_cta < 1) n_cta = 1;
    const int chunk = (V + n_cta - 1) / n_cta;
    const size_t room = (size_t)smem_max - kNsFixedSmem - 1024;   // static arrays and slack
    const int stash_len = (size_t)chunk * sizeof(float) <= room ? chunk : (int)(room / sizeof(float));
    const size_t smem = kNsFixedSmem + (size_t)stash_len * sizeof(float);
    // the attribute belongs to the kernel on one device: remembered per device (the first 64)
    static unsigned long long attr_set_on = 0ull;
    const unsigned long long dev_bit = dev >= 0 && dev < 64 ? 1ull << dev : 0ull;
    if ((attr_set_on & dev_bit) == 0ull) {
        if (cudaFuncSetAttribute(nucleus_sample_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max - 1024) != cudaSuccess) {
            cudaGetLastError();
            return DM_ECUDA;
        }
        attr_set_on |= dev_bit;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(rows * n_cta));
    cfg.blockDim = dim3(kNsThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = (unsigned)n_cta; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, nucleus_sample_kernel, logits, V, chunk, stash_len, map, mk.key0, mk.key1, mk.inv_temp,
                           top_p, v_offset, out_packed) != cudaSuccess) {
        cudaGetLastError();
        return DM_ECUDA;
    }
    return cudaGetLastError() == cudaSuccess ? DM_OK : DM_ECUDA;
}

}  // namespace dm
