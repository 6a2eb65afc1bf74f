// Nucleus sampling (Sec. 3.2 names it as the alternative to the top-1 token) on logits that a
// head kernel has written to global memory: one block per path.
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
#include "dm_internal.h"

namespace dm {

namespace {

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

__global__ void __launch_bounds__(kNsThreads)
nucleus_sample_kernel(const float* __restrict__ logits, int V, RowMap map, uint32_t key0, uint32_t key1,
                      float inv_temp, float top_p, int v_offset, unsigned long long* __restrict__ out_packed) {
    __shared__ unsigned int hist_lo[kNsBins], hist_hi[kNsBins];   // 64-bit mass per bin as two words (32-bit shared atomics are native)
    __shared__ unsigned int cnt[kNsBins];
    __shared__ unsigned long long list_key[kNsList];
    __shared__ unsigned long long list_q[kNsList];
    __shared__ unsigned long long red[kNsThreads / 32];
    __shared__ int s_bin, s_count, s_level;
    __shared__ unsigned long long s_above, s_boundary;
    __shared__ float s_lo;   // distance m - z at which the level-1 bins start

    const int row = blockIdx.x, tid = threadIdx.x;
    const float* l = logits + (size_t)row * V;
    RowKey k;
    row_key(map, row, k);

    // 1. maximum
    float mx = -INFINITY;
#pragma unroll 8
    for (int v = tid; v < V; v += kNsThreads) mx = fmaxf(mx, l[v] * inv_temp);
    const float m = key_float((uint32_t)(block_max_u64((unsigned long long)float_key(mx), red)));

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
        for (int v = tid; v < V; v += kNsThreads) {
            const float z = l[v] * inv_temp;
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
        __syncthreads();
        {   // the first bin at which the running mass reaches the target (the last bin if none does):
            // two bins per thread, a prefix sum over the threads
            const unsigned long long h0 = ((unsigned long long)hist_hi[2 * tid] << 32) | hist_lo[2 * tid];
            const unsigned long long h1 = ((unsigned long long)hist_hi[2 * tid + 1] << 32) | hist_lo[2 * tid + 1];
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
            if (before < target) {
                if (before + h0 >= target) { b = 2 * tid; above = before; }
                else if (before + h0 + h1 >= target || tid == kNsThreads - 1) { b = 2 * tid + 1; above = before + h0; }
            }
            __syncthreads();
            if (b >= 0) {             // exactly one thread: the running mass is non-decreasing
                s_above = above;      // mass of everything before the boundary bin
                if (level == 0) s_bin = b; else s_level = 1 + b;   // level 1: remember the sub-bin
                s_count = (int)cnt[b];   // tokens in the boundary bin
            }
        }
        __syncthreads();
        if (s_count <= kNsList || level == 1) break;
        if (tid == 0) s_lo = (float)s_bin / kNsBinsPerUnit;
        __syncthreads();
    }

    // 4. the boundary token: sort the boundary bin's tokens by (z, id) and walk them
    const int b0 = s_bin, b1 = s_level - 1;
    const float lo1 = s_lo;
    const bool refined = s_level > 0;
    for (int i = tid; i < kNsList; i += kNsThreads) { list_key[i] = 0ull; list_q[i] = 0ull; }
    if (tid == 0) s_count = 0;
    __syncthreads();
#pragma unroll 8
    for (int v = tid; v < V; v += kNsThreads) {
        const float z = l[v] * inv_temp;
        const float dist = m - z;
        if (min(kNsBins - 1, (int)(dist * kNsBinsPerUnit)) != b0) continue;
        if (refined && min(kNsBins - 1, max(0, (int)((dist - lo1) * (kNsBinsPerUnit * kNsBins)))) != b1) continue;
        const int slot = atomicAdd(&s_count, 1);
        if (slot < kNsList) {
            list_key[slot] = walk_key(z, v);
            list_q[slot] = (unsigned long long)(expf(z - m) * kNsFixedOne);
        }
    }
    __syncthreads();
    const int n_list = min(s_count, kNsList);
    // bitonic sort, descending by key (empty slots have key 0 and sink to the end)
    for (int size = 2; size <= kNsList; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const int i = tid, j = i ^ stride;
            if (j > i && i < kNsList) {
                const bool descending = (i & size) == 0;
                const unsigned long long a = list_key[i], b = list_key[j];
                if ((a < b) == descending) {
                    list_key[i] = b; list_key[j] = a;
                    const unsigned long long qa = list_q[i]; list_q[i] = list_q[j]; list_q[j] = qa;
                }
            }
            __syncthreads();
        }
    }
    {   // walk the sorted list: the first entry at which the running mass reaches the target
        if (tid == 0) s_boundary = n_list > 0 ? list_key[n_list - 1] : 0ull;   // (none does: all of them are in)
        const unsigned long long q = tid < n_list ? list_q[tid] : 0ull;
        const unsigned long long before = s_above + block_exclusive_scan_u64(q, red);
        if (tid < n_list && before < target && before + q >= target) s_boundary = list_key[tid];
    }
    __syncthreads();
    const unsigned long long boundary = s_boundary;
    const bool overflow = s_count > kNsList;   // more tokens of (nearly) one value than the sort takes: all of them are in

    // 5. Gumbel-max over the nucleus
    unsigned long long best = 0ull;
#pragma unroll 8
    for (int v = tid; v < V; v += kNsThreads) {
        const float z = l[v] * inv_temp;
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
    if (tid == 0) out_packed[row] = best;
}

}  // namespace

int launch_nucleus_sample(const float* logits, int V, int rows, const RowMap& map, const MaskKey& mk, float top_p,
                          int v_offset, unsigned long long* out_packed, cudaStream_t stream) {
    if (rows < 1 || rows > 0x7FFFFFFF / 2) return DM_EINVAL;
    nucleus_sample_kernel<<<rows, kNsThreads, 0, stream>>>(logits, V, map, mk.key0, mk.key1, mk.inv_temp, top_p, v_offset,
                                                          out_packed);
    return cudaGetLastError() == cudaSuccess ? DM_OK : DM_ECUDA;
}

}  // namespace dm
