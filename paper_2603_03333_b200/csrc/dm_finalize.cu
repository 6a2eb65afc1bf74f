// Split-V merge, token histogram and acceptance (Sec. 3.2: naive token matching, Eq. 6
// majority; left-to-right rule; tree drafts of Sec. 4.4), plus the debug mask dump (Eq. 1).
// One block per sequence; everything after the merge is integer work on <= T*K tokens.
#include "dm_internal.h"

namespace dm {

// Does `draft` pass `rule` against the K tokens of one hidden row (shared memory)?
__device__ __forceinline__ bool position_ok(const int32_t* toks, int K, int32_t draft, int rule,
                                            int* hits_out) {
    int hits = 0;
    for (int i = 0; i < K; ++i) hits += (toks[i] == draft);
    if (hits_out) *hits_out = hits;
    if (rule == DM_RULE_NAIVE) return hits >= 1;
    // Eq. 6: draft must be the most frequent token; equal frequencies -> smallest id wins.
    if (hits == 0) return false;
    for (int i = 0; i < K; ++i) {
        int32_t y = toks[i];
        if (y == draft) continue;
        int c = 0;
        for (int i2 = 0; i2 < K; ++i2) c += (toks[i2] == y);
        if (c > hits || (c == hits && y < draft)) return false;
    }
    return true;
}

__global__ void __launch_bounds__(256)
finalize_kernel(const unsigned long long* __restrict__ partials, int n_slices, int rows,
                FinalizeArgs a) {
    extern __shared__ int32_t sm[];
    const int TK = a.T * a.K;
    int32_t* toks = sm;            // [T*K]
    int32_t* flag = sm + TK;       // chain: ok[T]; tree: test[N] then ok/depth packed [N]
    const int b = blockIdx.x;
    const size_t row0 = (size_t)b * TK;

    // split-V merge: the packed (key, inverted index) maximum over slices is the argmax with
    // the smallest index on ties.  One warp per row: lanes stride over the slices.
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
    for (int x = warp; x < TK; x += n_warps) {
        unsigned long long best = 0ull;
        for (int s = lane; s < n_slices; s += 32) {
            unsigned long long c = partials[(size_t)s * rows + row0 + x];
            best = c > best ? c : best;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, best, off);
            best = o > best ? o : best;
        }
        if (lane == 0) {
            int32_t tok = (int32_t)best_index(best);
            toks[x] = tok;
            a.out_tokens[row0 + x] = tok;
        }
    }
    __syncthreads();

    // empirical distribution: multiplicity of every sampled token within its position
    for (int x = threadIdx.x; x < TK; x += blockDim.x) {
        const int32_t* row = toks + (x / a.K) * a.K;
        int32_t y = toks[x];
        int c = 0;
        for (int i = 0; i < a.K; ++i) c += (row[i] == y);
        a.out_counts[row0 + x] = c;
    }

    if (a.N == 0) {
        for (int t = threadIdx.x; t < a.T; t += blockDim.x) {
            int hits;
            bool ok = position_ok(toks + t * a.K, a.K, a.draft[(size_t)b * a.T + t], a.rule, &hits);
            flag[t] = ok;
            if (a.out_hits) a.out_hits[(size_t)b * a.T + t] = hits;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int len = 0;
            while (len < a.T && flag[len]) ++len;   // first rejection ends acceptance
            a.out_accept_len[b] = len;
        }
        return;
    }

    // tree: per-node test in parallel, then one serial topological walk
    const size_t n0 = (size_t)b * a.N;
    int32_t* depth = flag + a.N;
    for (int n = threadIdx.x; n < a.N; n += blockDim.x) {
        int h = a.node_hrow[n0 + n];
        bool ok = false;
        if (h >= 0 && h < a.T) ok = position_ok(toks + h * a.K, a.K, a.node_token[n0 + n], a.rule, nullptr);
        flag[n] = ok;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int best_depth = 0, best = -1;
        for (int n = 0; n < a.N; ++n) {
            int par = a.node_parent[n0 + n];
            bool par_ok = par < 0 ? true : (par < n ? flag[par] != 0 : false);
            int dep = (par < 0 || par >= n) ? 1 : depth[par] + 1;
            bool ok = par_ok && flag[n];
            flag[n] = ok;
            depth[n] = dep;
            if (ok && dep > best_depth) { best_depth = dep; best = n; }
        }
        a.out_accept_len[b] = best_depth;
        a.out_best_node[b] = best;
    }
    __syncthreads();
    if (a.out_node_ok)
        for (int n = threadIdx.x; n < a.N; n += blockDim.x) a.out_node_ok[n0 + n] = flag[n];
}

size_t finalize_smem_bytes(int T, int K, int N) {
    size_t extra = N > 0 ? 2 * (size_t)N : (size_t)T;
    return ((size_t)T * K + extra) * sizeof(int32_t);
}

int launch_finalize(const unsigned long long* partials, int n_slices, int rows,
                    const FinalizeArgs& a, cudaStream_t stream) {
    const size_t smem = finalize_smem_bytes(a.T, a.K, a.N);
    if (smem > 200 * 1024) return DM_EUNSUPPORTED;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(finalize_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return DM_ECUDA;
    finalize_kernel<<<a.B, 256, smem, stream>>>(partials, n_slices, rows, a);
    return cudaGetLastError() == cudaSuccess ? DM_OK : DM_ECUDA;
}

// Eq. 1 keep bits, one 32-bit word (eight Philox quads) per thread.
__global__ void debug_masks_kernel(int n_paths, int K, int T, int d, MaskKey mk, uint32_t seq_base_lo,
                                   uint32_t* __restrict__ out_bits) {
    const int words = (d + 31) / 32;
    const long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= (long long)n_paths * words) return;
    const int r = (int)(x / words), w = (int)(x - (long long)r * words);
    RowMap map{nullptr, K, T, 0, seq_base_lo};
    RowKey k;
    row_key(map, r, k);
    uint32_t bits = 0;
    for (int n = 0; n < 8; ++n) {
        int quad = w * 8 + n;
        if (quad * 4 >= d) break;
        uint32_t keep = keep4((uint32_t)quad, k, mk.key0, mk.key1, mk.thr);
        int left = d - quad * 4;
        if (left < 4) keep &= (1u << left) - 1u;
        bits |= keep << (4 * n);
    }
    out_bits[x] = bits;
}

int launch_debug_masks(int B, int T, int K, int d, const MaskKey& mk, uint32_t seq_base_lo,
                       uint32_t* out_bits, cudaStream_t stream) {
    const long long n_paths = (long long)B * T * K;
    const long long total = n_paths * ((d + 31) / 32);
    if (total > (1ll << 40)) return DM_EUNSUPPORTED;
    const long long blocks = (total + 255) / 256;
    if (blocks > 0x7FFFFFFFll) return DM_EUNSUPPORTED;
    debug_masks_kernel<<<(unsigned)blocks, 256, 0, stream>>>((int)n_paths, K, T, d, mk, seq_base_lo, out_bits);
    return cudaGetLastError() == cudaSuccess ? DM_OK : DM_ECUDA;
}

}  // namespace dm
