// Split-V merge, token histogram and acceptance of one sequence (Sec. 3.2: naive token matching,
// Eq. 6 majority; left-to-right rule; tree drafts of Sec. 4.4), as a device routine that a group
// of threads runs together: the finalize kernel (one block per sequence) and the last CTA of
// the fused head kernel (its four epilogue warps, sequence after sequence) both call it.
#pragma once
#include "dm_internal.h"

namespace dm {

// Bytes of scratch finalize_sequence needs (the host's finalize_smem_bytes, for device code).
__host__ __device__ __forceinline__ size_t finalize_smem_bytes_dev(int T, int K, int N) {
    const size_t extra = N > 0 ? 2 * (size_t)N : (size_t)T;
    return ((size_t)T * K + extra) * sizeof(int32_t);
}

struct BlockSync {
    __device__ __forceinline__ void operator()() const { __syncthreads(); }
};
// bar.sync on a named barrier among `threads` threads (a multiple of 32, whole warps).
struct NamedSync {
    int id, threads;
    __device__ __forceinline__ void operator()() const {
        asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
    }
};

// __syncwarp: one warp runs finalize_sequence on its own (nthreads = 32).
struct WarpSync {
    __device__ __forceinline__ void operator()() const { __syncwarp(); }
};

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

// Sequence b of a call of `rows` paths whose per-slice partial argmaxes are partials[slice][row].
// `sm` is scratch shared memory of finalize_smem_bytes(T, K, N) bytes; thread `tid` of `nthreads`.
template <class Sync>
__device__ __forceinline__ void finalize_sequence(const unsigned long long* partials, int n_slices, int rows,
                                                  const FinalizeArgs& a, int b, int32_t* sm, int tid,
                                                  int nthreads, Sync sync) {
    // Kp paths per hidden row: the K dropout paths and, if a.plain, one unmasked path after them
    // (the target's own greedy token).  Outputs are compact [T][K]; the scratch keeps [T][Kp].
    const int Kp = a.K + a.plain;
    const int Td = a.T_draft > 0 ? a.T_draft : a.T;   // draft positions that are scanned (<= T)
    const int TK = a.T * Kp;
    int32_t* toks = sm;            // [T*Kp]
    int32_t* flag = sm + TK;       // chain: ok[T]; tree: test[N] then ok/depth packed [N]
    const size_t row0 = (size_t)b * TK;
    const size_t out0 = (size_t)b * a.T * a.K;
    // The first loads of the routine do not depend on one another: the per-row word and the draft
    // token of this thread are requested together with the error word (one round trip, not three).
    const bool one_slice = n_slices == 1;
    unsigned long long first_word = 0ull;
    int32_t first_draft = 0;
    if (one_slice && tid < TK) first_word = __ldcg(partials + row0 + tid);
    if (a.N == 0 && a.draft != nullptr && tid < Td) first_draft = a.draft[(size_t)b * Td + tid];
    // A kernel of this call gave up on a wait (device error word set): the partial maxima are
    // incomplete.  Nothing may then look accepted to a consumer further down the stream: no token
    // (-1), empty histogram, accepted length 0 (the left-to-right rule rejects everything).
    if (a.err != nullptr && *reinterpret_cast<const volatile uint32_t*>(a.err) != 0u) {
        for (int x = tid; x < a.T * a.K; x += nthreads) { a.out_tokens[out0 + x] = -1; a.out_counts[out0 + x] = 0; }
        for (int t = tid; t < a.T; t += nthreads)
            if (a.out_plain) a.out_plain[(size_t)b * a.T + t] = -1;
        if (a.N == 0) {
            for (int t = tid; t < Td; t += nthreads)
                if (a.out_hits) a.out_hits[(size_t)b * Td + t] = 0;
        } else {
            for (int n = tid; n < a.N; n += nthreads)
                if (a.out_node_ok) a.out_node_ok[(size_t)b * a.N + n] = 0;
        }
        if (tid == 0) {
            a.out_accept_len[b] = 0;
            if (a.N > 0) a.out_best_node[b] = -1;
            if (a.out_next) a.out_next[b] = -1;
        }
        sync();
        return;
    }
    auto store_token = [&](int x, int32_t tok) {
        toks[x] = tok;
        const int t = x / Kp, i = x - t * Kp;
        if (i < a.K) a.out_tokens[out0 + (size_t)t * a.K + i] = tok;
        else if (a.out_plain) a.out_plain[(size_t)b * a.T + t] = tok;
    };

    // split-V merge: the packed (key, inverted index) maximum over slices is the argmax with
    // the smallest index on ties.  Many slices: one warp per row, lanes stride over the slices.
    // Few slices (the fused kernel's CTAs have already reduced into one): one thread per row, so
    // that all loads of a sequence are in flight together.
    const int warp = tid >> 5, lane = tid & 31, n_warps = nthreads >> 5;
    if (n_slices < 32) {
        for (int x = tid; x < TK; x += nthreads) {
            unsigned long long best = 0ull;
            if (one_slice && x == tid) {
                best = first_word;
            } else {
                for (int s = 0; s < n_slices; ++s) {
                    unsigned long long c = __ldcg(partials + (size_t)s * rows + row0 + x);
                    best = c > best ? c : best;
                }
            }
            store_token(x, (int32_t)best_index(best));
        }
    } else {
        for (int x0 = warp * 4; x0 < TK; x0 += n_warps * 4) {   // four rows at a time: their loads overlap
            unsigned long long best[4] = {0ull, 0ull, 0ull, 0ull};
            for (int s = lane; s < n_slices; s += 32) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (x0 + u < TK) {
                        unsigned long long c = __ldcg(partials + (size_t)s * rows + row0 + x0 + u);
                        best[u] = c > best[u] ? c : best[u];
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) {
                    unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, best[u], off);
                    best[u] = o > best[u] ? o : best[u];
                }
                if (lane == 0 && x0 + u < TK) store_token(x0 + u, (int32_t)best_index(best[u]));
            }
        }
    }
    sync();

    // empirical distribution: multiplicity of every sampled token within its position
    for (int x = tid; x < a.T * a.K; x += nthreads) {
        const int t = x / a.K;
        const int32_t* row = toks + t * Kp;
        int32_t y = row[x - t * a.K];
        int c = 0;
        for (int i = 0; i < a.K; ++i) c += (row[i] == y);
        a.out_counts[out0 + x] = c;
    }

    if (a.N == 0) {
        for (int t = tid; t < Td; t += nthreads) {
            int hits;
            bool ok = position_ok(toks + t * Kp, a.K, t == tid ? first_draft : a.draft[(size_t)b * Td + t], a.rule, &hits);
            flag[t] = ok;
            if (a.out_hits) a.out_hits[(size_t)b * Td + t] = hits;
        }
        sync();
        if (tid == 0) {
            int len = 0;
            while (len < Td && flag[len]) ++len;   // first rejection ends acceptance
            a.out_accept_len[b] = len;
            // the token the engine emits next: the target's greedy token at the first position
            // that was not accepted (a correction), or after all of them if that row was given
            if (a.out_next) a.out_next[b] = (a.plain && len < a.T) ? toks[len * Kp + a.K] : -1;
        }
        sync();   // the scratch may be reused for the next sequence
        return;
    }

    // tree: per-node test in parallel, then one serial topological walk
    const size_t n0 = (size_t)b * a.N;
    int32_t* depth = flag + a.N;
    for (int n = tid; n < a.N; n += nthreads) {
        int h = a.node_hrow[n0 + n];
        bool ok = false;
        if (h >= 0 && h < a.T) ok = position_ok(toks + h * Kp, a.K, a.node_token[n0 + n], a.rule, nullptr);
        flag[n] = ok;
        depth[n] = a.node_parent[n0 + n];   // staged here so that the serial walk stays in shared memory
    }
    sync();
    if (tid == 0) {
        int best_depth = 0, best = -1;
        for (int n = 0; n < a.N; ++n) {
            int par = depth[n];             // still the parent: entries below n already hold depths
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
    sync();
    if (a.out_node_ok)
        for (int n = tid; n < a.N; n += nthreads) a.out_node_ok[n0 + n] = flag[n];
    sync();   // the scratch may be reused for the next sequence
}

}  // namespace dm
