// JS-divergence acceptance (Sec. 3.2: Eq. 4 centroid, Eq. 5 test, Algorithm 1) on the logits that
// a head kernel has written to global memory: [n_pos][K][V] fp32 (20 MB for the Llama-3-8B head at
// 40 paths; the head kernel streams W with an evict-first policy, so they are still in L2).
// Up to 32 paths per position, js_sweep_kernel does the work, a block per (position, vocabulary
// chunk) that holds its chunk in shared memory:
//   first sweep    the chunk's part of the log-sum-exp of each of the K paths and of the centroid
//                  logits (their mean over the paths); the last block of a position to finish
//                  merges the parts
//   second sweep   the chunk's share of JS(p_i || pbar) for every path and of JS(phat || pbar);
//                  the last block of the grid sums the shares and runs Algorithm 1 and the scan
// either as one cooperative launch (calls whose logits fit the shared memory of the GPU: the
// chunk stays where it is between the sweeps) or as two launches.  More paths than that: three
// plain kernels that take one series at a time (js_lse_kernel, js_sum_kernel, js_accept_kernel).
// Probabilities are never stored: p = exp(l - lse) is recomputed where it is needed.
#include "dm_finalize.cuh"
#include "dm_internal.h"

namespace dm {

namespace {

constexpr int kJsThreads = 256;

__device__ __forceinline__ float block_reduce_sum(float x, float* red) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, off);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
    __syncthreads();
    float t = 0.0f;
    for (int w = 0; w < kJsThreads / 32; ++w) t += red[w];
    return t;
}
__device__ __forceinline__ float block_reduce_max(float x, float* red) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) x = fmaxf(x, __shfl_xor_sync(0xFFFFFFFFu, x, off));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
    __syncthreads();
    float t = red[0];
    for (int w = 1; w < kJsThreads / 32; ++w) t = fmaxf(t, red[w]);
    return t;
}

// Logit of series s at vocabulary entry v of one position: path s for s < K, else the centroid.
__device__ __forceinline__ float series_logit(const float* __restrict__ pos_logits, int V, int K, int s, int v) {
    if (s < K) return pos_logits[(size_t)s * V + v];
    float acc = 0.0f;
    for (int i = 0; i < K; ++i) acc += pos_logits[(size_t)i * V + v];
    return acc / (float)K;
}

// part[(pos*(K+1) + s)*n_chunks + chunk] = (max, sum of exp(l - max)) over the chunk
__global__ void __launch_bounds__(kJsThreads)
js_lse_kernel(const float* __restrict__ logits, int V, int K, int chunk_len, int n_chunks,
              float2* __restrict__ part) {
    extern __shared__ float cen[];   // [chunk_len] centroid logits of the chunk (Eq. 4 before the softmax)
    __shared__ float red[kJsThreads / 32];
    const int pos = blockIdx.y, chunk = blockIdx.x;
    const int v0 = chunk * chunk_len, v1 = min(V, v0 + chunk_len);
    const float* pl = logits + (size_t)pos * K * V;
    for (int v = v0 + threadIdx.x; v < v1; v += kJsThreads) cen[v - v0] = series_logit(pl, V, K, K, v);
    __syncthreads();
    for (int s = 0; s <= K; ++s) {
        float mx = -INFINITY;
        for (int v = v0 + threadIdx.x; v < v1; v += kJsThreads)
            mx = fmaxf(mx, s < K ? pl[(size_t)s * V + v] : cen[v - v0]);
        mx = block_reduce_max(mx, red);
        float sum = 0.0f;
        for (int v = v0 + threadIdx.x; v < v1; v += kJsThreads)
            sum += expf((s < K ? pl[(size_t)s * V + v] : cen[v - v0]) - mx);
        sum = block_reduce_sum(sum, red);
        if (threadIdx.x == 0) part[((size_t)pos * (K + 1) + s) * n_chunks + chunk] = make_float2(mx, sum);
    }
}

// One term of 2*JS(P||Q) at an outcome with log-probabilities lp, lq (natural logarithm):
// P log(P/M) + Q log(Q/M), M = (P+Q)/2.  A vanishing probability contributes nothing.
// Written around the log-ratio a = lo - hi <= 0 of the smaller to the larger probability, so that
// nothing is lost to cancellation between large log-probabilities: log(hi/M) = -log((1+e^a)/2).
__device__ __forceinline__ float js_term(float lp, float lq) {
    const float hi = fmaxf(lp, lq), lo = fminf(lp, lq);
    if (hi == -INFINITY) return 0.0f;
    const float a = lo - hi;                                  // may be -inf
    // fast intrinsics: the logarithm's argument lies in [0.5, 1], where __logf is good to ~4e-7
    // absolute, and every exponent is <= 0; the errors are weighted by probabilities that sum to 1
    const float r = -__logf(0.5f + 0.5f * __expf(a));         // log(P_hi / M), in [0, log 2]
    float t = __expf(hi) * r;
    if (a > -INFINITY) t += __expf(lo) * (a + r);             // log(P_lo / M) = a + r
    return t;
}

// share[(pos*(K+1) + s)*n_chunks + chunk] = this chunk's part of JS(series s || centroid) for
// s < K, and of JS(draft || centroid) for s = K.
__global__ void __launch_bounds__(kJsThreads)
js_sum_kernel(const float* __restrict__ logits, const float* __restrict__ draft_prob, int V, int K, int chunk_len,
              int n_chunks, const float2* __restrict__ part, float* __restrict__ share) {
    extern __shared__ float js_smem[];
    float* lse = js_smem;            // [K+1]
    float* lqs = js_smem + K + 1;    // [chunk_len] log pbar of the chunk
    __shared__ float red[kJsThreads / 32];
    const int pos = blockIdx.y, chunk = blockIdx.x;
    for (int s = threadIdx.x; s <= K; s += kJsThreads) {
        const float2* ps = part + ((size_t)pos * (K + 1) + s) * n_chunks;
        float mx = -INFINITY;
        for (int c = 0; c < n_chunks; ++c) mx = fmaxf(mx, ps[c].x);
        float sum = 0.0f;
        for (int c = 0; c < n_chunks; ++c) sum += ps[c].y * expf(ps[c].x - mx);
        lse[s] = mx + logf(sum);
    }
    __syncthreads();
    const int v0 = chunk * chunk_len, v1 = min(V, v0 + chunk_len);
    const float* pl = logits + (size_t)pos * K * V;
    const float* dp = draft_prob + (size_t)pos * V;
    const float lse_c = lse[K];
    for (int v = v0 + threadIdx.x; v < v1; v += kJsThreads) lqs[v - v0] = series_logit(pl, V, K, K, v) - lse_c;
    __syncthreads();
    for (int s = 0; s <= K; ++s) {
        float acc = 0.0f;
        for (int v = v0 + threadIdx.x; v < v1; v += kJsThreads) {
            float lp;
            if (s < K) lp = pl[(size_t)s * V + v] - lse[s];                   // log p_s[v]
            else { const float P = dp[v]; lp = P > 0.0f ? logf(P) : -INFINITY; }
            acc += js_term(lp, lqs[v - v0]);
        }
        acc = block_reduce_sum(acc, red);
        if (threadIdx.x == 0) share[((size_t)pos * (K + 1) + s) * n_chunks + chunk] = 0.5f * acc;
    }
}

// Algorithm 1 and the left-to-right scan for sequence b, run by one block of kJsThreads threads;
// also exports the divergences.  `ok` is shared scratch of T ints.
struct JsAcceptArgs {
    const float* share;
    int n_chunks, B, T, K;
    const int32_t* tokens;
    const int32_t* draft;
    float* out_js;
    int32_t* out_js_ok;
    int32_t* out_accept_len;
    const uint32_t* err;
};

__device__ __forceinline__ void js_accept_sequence(const JsAcceptArgs& a, int b, int32_t* ok) {
    const int T = a.T, K = a.K, n_chunks = a.n_chunks;
    // a kernel of this call gave up on a wait: the logits are incomplete, nothing may be accepted
    const bool failed = a.err != nullptr && *reinterpret_cast<const volatile uint32_t*>(a.err) != 0u;
    // divergences: one warp per (position, series), lanes over the chunks, summed in double
    for (int x = threadIdx.x >> 5; x < T * (K + 1); x += kJsThreads / 32) {
        const size_t idx = (size_t)b * T * (K + 1) + x;
        double acc = 0.0;
        for (int c = threadIdx.x & 31; c < n_chunks; c += 32) acc += (double)__ldcg(a.share + idx * n_chunks + c);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
        if ((threadIdx.x & 31) == 0) a.out_js[idx] = (float)acc;
    }
    __syncthreads();
    for (int t = threadIdx.x; t < T; t += kJsThreads) {
        const size_t q = (size_t)b * T + t;
        const float* js = a.out_js + q * (K + 1);
        float max_heads = js[0];
        for (int i = 1; i < K; ++i) max_heads = fmaxf(max_heads, js[i]);
        const bool eq5 = js[K] <= max_heads;                                   // Eq. 5
        const bool eq6 = position_ok(a.tokens + q * K, K, a.draft[q], DM_RULE_MAJORITY, nullptr);   // Eq. 6
        if (a.out_js_ok) a.out_js_ok[q] = eq5 && !failed;
        ok[t] = (eq5 || eq6) && !failed;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int len = 0;
        while (len < T && ok[len]) ++len;
        a.out_accept_len[b] = len;
    }
    __syncthreads();
}

// ---- the two sweeps for up to 32 paths per position ---------------------------------------------
// A block copies its chunk of the K logit rows of its position and of the draft distribution
// into shared memory (asynchronous copies, all in flight at once) and adds the centroid logits
// (Eq. 4 before the softmax) as one more row.
// MODE 0: both sweeps.  Launched cooperatively (every block resident): after the first sweep the
//         blocks of a position meet at a counter in global memory (bounded waits); the last to
//         arrive merges the parts and publishes the K+1 log-sum-exps, the others wait for its
//         flag; the second sweep then runs on the copy in shared memory: the logits cross the
//         memory system once, and there is one launch.
// MODE 1: the first sweep alone (nobody waits: the last block of a position merges).
// MODE 2: the second sweep alone, on a fresh copy, with the log-sum-exps that MODE 1 published.
// In modes 0 and 2 the last block of the grid runs Algorithm 1 and leaves the counters at zero.
__device__ __forceinline__ float ex2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float lg2_fast(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;

// One term of 2*JS(P||Q) from lp = log P, lq = log Q and Q itself (which the series of an entry
// share).  With E = exp(-|lp - lq|) and r = -log((1 + E)/2) = log(max(P,Q)/M), M = (P+Q)/2:
//   P log(P/M) + Q log(Q/M) = max(P,Q) * (r + E*(r - |lp - lq|)),
// all of it on [0, log 2] and [0, 1]: nothing cancels.  A vanishing P (lp = -inf) gives Q log 2.
// The logarithm's argument lies in [0.5, 1], where the fast form is good to ~4e-7 absolute, and
// every exponent is <= 0; the errors are weighted by probabilities that sum to 1.
__device__ __forceinline__ float js_term_q(float lp, float lq, float Q) {
    const float a = fminf(fabsf(lp - lq), 126.0f);            // beyond that E is zero in fp32 anyway
    const float E = ex2_fast(-kLog2e * a);
    const float r = -kLn2 * lg2_fast(fmaf(0.5f, E, 0.5f));
    return fmaxf(ex2_fast(kLog2e * lp), Q) * fmaf(E, r - a, r);
}

__device__ __forceinline__ void cp_async_f1(float* dst_smem, const float* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_f4(float* dst_smem, const float* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}

// Algorithm 1 and the scan for every sequence of the call by one block of kJsThreads threads, for
// K <= 32: shares, tokens and drafts are staged in `scratch` (shared memory) in one sweep of
// loads; a half-warp sums the shares of a series (in double), a warp tests a position.
__device__ __forceinline__ int js_accept_scratch_floats(int n_pos, int K, int n_chunks) {
    return n_pos * (K + 1) * n_chunks + n_pos * (K + 1) + n_pos * K + 2 * n_pos;
}

__device__ __forceinline__ void js_accept_staged(const JsAcceptArgs& a, float* scratch) {
    const int T = a.T, K = a.K, n_chunks = a.n_chunks, n_pos = a.B * a.T;
    const int S = n_pos * (K + 1), total = S * n_chunks;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* jsv = scratch + total;                                   // [S]
    int32_t* tok = reinterpret_cast<int32_t*>(jsv + S);             // [n_pos][K]
    int32_t* drf = tok + n_pos * K;                                 // [n_pos]
    int32_t* ok = drf + n_pos;                                      // [n_pos]
    for (int x = threadIdx.x; x < total; x += kJsThreads) scratch[x] = __ldcg(a.share + x);
    for (int x = threadIdx.x; x < n_pos * K; x += kJsThreads) tok[x] = a.tokens[x];
    for (int x = threadIdx.x; x < n_pos; x += kJsThreads) drf[x] = a.draft[x];
    // a kernel of this call gave up on a wait: the logits are incomplete, nothing may be accepted
    const bool failed = a.err != nullptr && *reinterpret_cast<const volatile uint32_t*>(a.err) != 0u;
    __syncthreads();
    const int hw = threadIdx.x >> 4, hl = threadIdx.x & 15;
    for (int s0 = 0; s0 < S; s0 += kJsThreads / 16) {
        const int s = s0 + hw;
        double acc = 0.0;
        if (s < S)
            for (int c = hl; c < n_chunks; c += 16) acc += (double)scratch[(size_t)s * n_chunks + c];
#pragma unroll
        for (int off = 8; off > 0; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
        if (s < S && hl == 0) { jsv[s] = (float)acc; a.out_js[s] = (float)acc; }
    }
    __syncthreads();
    for (int q = warp; q < n_pos; q += kJsThreads / 32) {
        float mh = lane < K ? jsv[(size_t)q * (K + 1) + lane] : -INFINITY;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mh = fmaxf(mh, __shfl_xor_sync(0xFFFFFFFFu, mh, off));
        const bool eq5 = jsv[(size_t)q * (K + 1) + K] <= mh;                   // Eq. 5
        // Eq. 6: the draft must be the most frequent path token; equal frequencies -> smallest id wins
        const int32_t d = drf[q];
        const int32_t my = lane < K ? tok[q * K + lane] : -2 - lane;          // padding lanes match nobody
        const int hits = __popc(__ballot_sync(0xFFFFFFFFu, lane < K && my == d));
        const int cnt = __popc(__match_any_sync(0xFFFFFFFFu, my));
        const bool beats = lane < K && my != d && (cnt > hits || (cnt == hits && my < d));
        const bool eq6 = hits > 0 && __ballot_sync(0xFFFFFFFFu, beats) == 0u;
        if (lane == 0) {
            if (a.out_js_ok) a.out_js_ok[q] = eq5 && !failed;
            ok[q] = (eq5 || eq6) && !failed;
        }
    }
    __syncthreads();
    for (int b = threadIdx.x; b < a.B; b += kJsThreads) {
        int len = 0;
        while (len < T && ok[b * T + len]) ++len;
        a.out_accept_len[b] = len;
    }
}

// words: [0] ticket of the grid, [1 + pos] arrivals of a position, [1 + n_pos + pos] "log-sum-exps
// published" flag of a position; lse_out[pos][K+1] in global memory.
template <int KMAX, int MODE>
__global__ void __launch_bounds__(kJsThreads)
js_sweep_kernel(const float* __restrict__ logits, const float* __restrict__ draft_prob, int V, int K, int chunk_len,
                int n_chunks, int vec, float2* __restrict__ part, float* __restrict__ share, float* __restrict__ lse_out,
                unsigned int* __restrict__ words, long long wait_limit, uint32_t* __restrict__ err, int scratch_floats,
                JsAcceptArgs accept) {
    extern __shared__ __align__(16) float xs[];   // [K+2][chunk_len]: logits, centroid logits, draft probabilities
    __shared__ unsigned int s_ticket, s_last;
    __shared__ float bm[KMAX + 1], lse[KMAX + 1];
    __shared__ float red[kJsThreads / 32][KMAX + 1];
    const int pos = blockIdx.y, chunk = blockIdx.x, n_pos = gridDim.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int v0 = chunk * chunk_len, n = min(V, v0 + chunk_len) - v0;   // may be <= 0 for a trailing chunk
    const float* pl = logits + (size_t)pos * K * V + v0;
    const float* dp = draft_prob + (size_t)pos * V + v0;
    float* xc = xs + (size_t)K * chunk_len;         // centroid row
    float* xd = xs + (size_t)(K + 1) * chunk_len;   // draft row
    // ---- copy the chunk: every load of the block in flight at once
    const int n_rows = MODE == 1 ? K : K + 1;       // the first sweep alone has no use for the draft row
    if (vec) {
        for (int i = 0; i < n_rows; ++i) {
            const float* src = i < K ? pl + (size_t)i * V : dp;
            float* dst = i < K ? xs + (size_t)i * chunk_len : xd;
            for (int x = 4 * threadIdx.x; x < n; x += 4 * kJsThreads) cp_async_f4(dst + x, src + x);
        }
    } else {
        for (int i = 0; i < n_rows; ++i) {
            const float* src = i < K ? pl + (size_t)i * V : dp;
            float* dst = i < K ? xs + (size_t)i * chunk_len : xd;
            for (int x = threadIdx.x; x < n; x += kJsThreads) cp_async_f1(dst + x, src + x);
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    // ---- centroid logits (and, for the first sweep, the chunk's maxima)
    const float inv_k = 1.0f / (float)K;
    float mx[KMAX + 1];
#pragma unroll
    for (int i = 0; i <= KMAX; ++i) mx[i] = -INFINITY;
    for (int x = threadIdx.x; x < n; x += kJsThreads) {
        float c = 0.0f;
#pragma unroll
        for (int i = 0; i < KMAX; ++i)
            if (i < K) {
                const float val = xs[i * chunk_len + x];
                c += val;
                mx[i] = fmaxf(mx[i], val);
            }
        c *= inv_k;
        xc[x] = c;
        mx[KMAX] = fmaxf(mx[KMAX], c);
    }
    float acc[KMAX + 1];
    if (MODE != 2) {
        // ---- first sweep: the sums of exponentials around the chunk's maxima
#pragma unroll
        for (int i = 0; i <= KMAX; ++i)
            if (i < K || i == KMAX) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xFFFFFFFFu, mx[i], off));
                if (lane == 0) red[warp][i] = mx[i];
            }
        __syncthreads();
        for (int i = threadIdx.x; i <= KMAX; i += kJsThreads)
            if (i < K || i == KMAX) {
                float t = red[0][i];
                for (int w = 1; w < kJsThreads / 32; ++w) t = fmaxf(t, red[w][i]);
                bm[i] = t;   // (-inf for an empty chunk)
            }
        __syncthreads();
#pragma unroll
        for (int i = 0; i <= KMAX; ++i) acc[i] = 0.0f;
        for (int x = threadIdx.x; x < n; x += kJsThreads) {    // the thread reads back its own centroid entries
#pragma unroll
            for (int i = 0; i < KMAX; ++i)
                if (i < K) acc[i] += ex2_fast((xs[i * chunk_len + x] - bm[i]) * kLog2e);
            acc[KMAX] += ex2_fast((xc[x] - bm[KMAX]) * kLog2e);
        }
#pragma unroll
        for (int i = 0; i <= KMAX; ++i)
            if (i < K || i == KMAX) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) acc[i] += __shfl_xor_sync(0xFFFFFFFFu, acc[i], off);
                if (lane == 0) red[warp][i] = acc[i];
            }
        __syncthreads();
        for (int i = threadIdx.x; i <= KMAX; i += kJsThreads)
            if (i < K || i == KMAX) {
                float t = 0.0f;
                for (int w = 0; w < kJsThreads / 32; ++w) t += red[w][i];
                part[((size_t)pos * (K + 1) + (i == KMAX ? K : i)) * n_chunks + chunk] = make_float2(bm[i], t);
                __threadfence();
            }
        __syncthreads();
        // ---- the blocks of this position meet
        if (threadIdx.x == 0) s_last = atomicAdd(words + 1 + pos, 1u) == (unsigned int)(n_chunks - 1) ? 1u : 0u;
        __syncthreads();
        if (s_last) {
            // the last to arrive: every part of this position is in global memory
            __threadfence();
            // a half-warp per series: its loads all in flight, then the maximum, then one rescaled sum
            const int hw = threadIdx.x >> 4, hl = threadIdx.x & 15;
            for (int s0 = 0; s0 <= K; s0 += kJsThreads / 16) {
                const int series = s0 + hw;
                const bool valid = series <= K;
                const float2* ps = part + ((size_t)pos * (K + 1) + (valid ? series : 0)) * n_chunks;
                float mm = -INFINITY, ss = 0.0f;
                for (int c0 = 0; c0 < n_chunks; c0 += 128) {
                    float2 pr[8];
                    float m8 = -INFINITY;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const int c = c0 + 16 * u + hl;
                        pr[u] = (valid && c < n_chunks) ? __ldcg(ps + c) : make_float2(-INFINITY, 0.0f);
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) m8 = fmaxf(m8, pr[u].x);
                    const float M = fmaxf(mm, m8);
                    float t = ss == 0.0f ? 0.0f : ss * ex2_fast((mm - M) * kLog2e);
#pragma unroll
                    for (int u = 0; u < 8; ++u) t += pr[u].y == 0.0f ? 0.0f : pr[u].y * ex2_fast((pr[u].x - M) * kLog2e);
                    mm = M;
                    ss = t;
                }
                float M = mm;
#pragma unroll
                for (int off = 8; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, off));
                float t = ss == 0.0f ? 0.0f : ss * ex2_fast((mm - M) * kLog2e);
#pragma unroll
                for (int off = 8; off > 0; off >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, off);
                if (valid && hl == 0) {
                    const float l = M + logf(t);
                    lse[series == K ? KMAX : series] = l;
                    lse_out[(size_t)pos * (K + 1) + series] = l;
                    __threadfence();
                }
            }
            __syncthreads();
            if (MODE == 0 && threadIdx.x == 0) atomicExch(words + 1 + n_pos + pos, 1u);
        } else if (MODE == 0) {
            if (threadIdx.x == 0) {
                volatile unsigned int* flag = words + 1 + n_pos + pos;
                const long long t0 = clock64();
                while (*flag == 0u) {
                    if (clock64() - t0 > wait_limit) {     // give up: the call then accepts nothing (the error word is set)
                        atomicCAS(err, 0u, (uint32_t)ERR_WAIT_JS);
                        break;
                    }
                    __nanosleep(32);
                }
                __threadfence();
            }
            __syncthreads();
            for (int i = threadIdx.x; i <= K; i += kJsThreads) lse[i == K ? KMAX : i] = __ldcg(lse_out + (size_t)pos * (K + 1) + i);
            __syncthreads();
        }
        if (MODE == 1) return;
    } else {
        for (int i = threadIdx.x; i <= K; i += kJsThreads) lse[i == K ? KMAX : i] = __ldcg(lse_out + (size_t)pos * (K + 1) + i);
        __syncthreads();
    }
    // ---- second sweep: this chunk's share of every divergence, from shared memory
#pragma unroll
    for (int i = 0; i <= KMAX; ++i) acc[i] = 0.0f;
    const float lse_c = lse[KMAX];
    for (int x = threadIdx.x; x < n; x += kJsThreads) {
        const float lq = xc[x] - lse_c;          // log pbar[v]
        const float Q = ex2_fast(kLog2e * lq);
        const float P = xd[x];
#pragma unroll
        for (int i = 0; i < KMAX; ++i)
            if (i < K) acc[i] += js_term_q(xs[i * chunk_len + x] - lse[i], lq, Q);
        acc[KMAX] += js_term_q(P > 0.0f ? logf(P) : -INFINITY, lq, Q);
    }
#pragma unroll
    for (int i = 0; i <= KMAX; ++i)
        if (i < K || i == KMAX) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc[i] += __shfl_xor_sync(0xFFFFFFFFu, acc[i], off);
            if (lane == 0) red[warp][i] = acc[i];
        }
    __syncthreads();
    for (int i = threadIdx.x; i <= KMAX; i += kJsThreads)
        if (i < K || i == KMAX) {
            float t = 0.0f;
            for (int w = 0; w < kJsThreads / 32; ++w) t += red[w][i];
            share[((size_t)pos * (K + 1) + (i == KMAX ? K : i)) * n_chunks + chunk] = 0.5f * t;
            __threadfence();
        }
    __syncthreads();
    if (threadIdx.x == 0) s_ticket = atomicAdd(words, 1u);
    __syncthreads();
    if (s_ticket == gridDim.x * gridDim.y - 1) {
        __threadfence();
        if (js_accept_scratch_floats(n_pos, K, n_chunks) <= scratch_floats) js_accept_staged(accept, xs);
        else
            for (int b = 0; b < accept.B; ++b) js_accept_sequence(accept, b, reinterpret_cast<int32_t*>(xs));
        for (int x = threadIdx.x; x < 1 + 2 * n_pos; x += kJsThreads) words[x] = 0u;   // ticket, counters, flags
    }
}

__global__ void __launch_bounds__(kJsThreads)
js_accept_kernel(JsAcceptArgs a) {
    extern __shared__ int32_t ok[];   // [T]
    js_accept_sequence(a, (int)blockIdx.x, ok);
}

}  // namespace

// Vocabulary chunks per position.  The two sweeps are short kernels: they must fit the GPU in one
// wave (four blocks of 256 threads per SM at their register count), so the chunk count follows
// from the number of positions; chunks of about 1024 entries at most.
int js_chunks(int V, int n_pos) {
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int n = (V + 1023) / 1024;
    const int fit = (4 * sms) / (n_pos < 1 ? 1 : n_pos);
    if (n > fit) n = fit;
    return n < 1 ? 1 : n;
}

size_t js_words_offset(int V, int max_rows, int max_hidden) {
    // partial (max, sum) pairs and JS shares for every (position, series, chunk), at the largest
    // chunk count (chunks of 512 entries, which the two-launch form takes from 17 paths up)
    return (size_t)(max_rows + max_hidden) * ((V + 511) / 512) * 3;
}

size_t js_workspace_floats(int V, int max_rows, int max_hidden) {
    // ... then the ticket word of the last sweep, an arrival counter and a flag per position (all
    // zero between calls), and the K+1 merged log-sum-exps of every position
    return js_words_offset(V, max_rows, max_hidden) + 4 + 2 * (size_t)max_hidden + (size_t)(max_rows + max_hidden);
}

namespace {

// The two sweeps for K <= KMAX: one cooperative launch if the call's logits fit the shared memory of
// the SMs with every block resident, else two plain launches with chunks of about 1024 entries.
template <int KMAX>
int launch_js_sweeps(const float* logits, const float* draft_prob, float* workspace, float* lse_out, unsigned int* words,
                     int V, int n_pos, int K, int T, const JsAcceptArgs& acc_in, long long wait_limit, uint32_t* err,
                     cudaStream_t stream, int* launches_out) {
    int sms = 148, dev = 0, coop = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return DM_ECUDA;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    // the attribute belongs to the kernel on one device: remembered per device (the first 64)
    static unsigned long long attr_set_on = 0ull;
    const unsigned long long dev_bit = dev >= 0 && dev < 64 ? 1ull << dev : 0ull;
    const int smem_cap = 200 * 1024;
    if ((attr_set_on & dev_bit) == 0ull) {
        if (cudaFuncSetAttribute(js_sweep_kernel<KMAX, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_cap) != cudaSuccess ||
            cudaFuncSetAttribute(js_sweep_kernel<KMAX, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_cap) != cudaSuccess ||
            cudaFuncSetAttribute(js_sweep_kernel<KMAX, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_cap) != cudaSuccess) {
            cudaGetLastError();
            return DM_ECUDA;
        }
        attr_set_on |= dev_bit;
    }
    float2* part = reinterpret_cast<float2*>(workspace);
    JsAcceptArgs acc = acc_in;
    // 16-byte copies where every row of every chunk starts on a 16-byte boundary
    int vec = (V % 4 == 0 && (reinterpret_cast<uintptr_t>(logits) & 15u) == 0 &&
               (reinterpret_cast<uintptr_t>(draft_prob) & 15u) == 0) ? 1 : 0;
    for (int per_sm = coop ? 4 : 0; per_sm >= 1; --per_sm) {   // more resident blocks hide more latency
        int n_chunks = (V + 1023) / 1024;
        const int fit = (per_sm * sms) / n_pos;
        if (n_chunks > fit) n_chunks = fit;
        if (n_chunks < 1) continue;
        int chunk_len = (((V + n_chunks - 1) / n_chunks) + 3) & ~3;   // rows of the copy start 16-byte aligned
        size_t smem = (size_t)(K + 2) * chunk_len * sizeof(float);
        if (smem < (size_t)T * sizeof(int32_t)) smem = (size_t)T * sizeof(int32_t);
        if (smem > (size_t)smem_cap) continue;
        int resident = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, js_sweep_kernel<KMAX, 0>, kJsThreads, smem) != cudaSuccess) {
            cudaGetLastError();
            break;
        }
        if ((long long)resident * sms < (long long)n_chunks * n_pos) continue;
        float* share = workspace + (size_t)n_pos * (K + 1) * n_chunks * 2;
        acc.share = share;
        acc.n_chunks = n_chunks;
        int scratch_floats = (int)(smem / sizeof(float));
        void* args[] = {(void*)&logits, (void*)&draft_prob, (void*)&V, (void*)&K, (void*)&chunk_len, (void*)&n_chunks,
                        (void*)&vec, (void*)&part, (void*)&share, (void*)&lse_out, (void*)&words, (void*)&wait_limit,
                        (void*)&err, (void*)&scratch_floats, (void*)&acc};
        if (cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(js_sweep_kernel<KMAX, 0>),
                                        dim3((unsigned)n_chunks, (unsigned)n_pos), dim3(kJsThreads), args, smem,
                                        stream) != cudaSuccess) {
            cudaGetLastError();
            return DM_ECUDA;
        }
        *launches_out = 1;
        return DM_OK;
    }
    // Two launches.  Chunks of 1024 entries, 512 from 17 paths up (two blocks per SM either way).
    const int chunk_len = KMAX <= 16 ? 1024 : 512;
    int n_chunks = (V + chunk_len - 1) / chunk_len;
    size_t smem = (size_t)(K + 2) * chunk_len * sizeof(float);
    if (smem < (size_t)T * sizeof(int32_t)) smem = (size_t)T * sizeof(int32_t);
    if (smem > (size_t)smem_cap) return DM_EUNSUPPORTED;
    float* share = workspace + (size_t)n_pos * (K + 1) * n_chunks * 2;
    acc.share = share;
    acc.n_chunks = n_chunks;
    const int scratch_floats = (int)(smem / sizeof(float));
    const dim3 grid((unsigned)n_chunks, (unsigned)n_pos);
    js_sweep_kernel<KMAX, 1><<<grid, kJsThreads, smem, stream>>>(logits, draft_prob, V, K, chunk_len, n_chunks, vec, part,
                                                              share, lse_out, words, wait_limit, err, scratch_floats, acc);
    js_sweep_kernel<KMAX, 2><<<grid, kJsThreads, smem, stream>>>(logits, draft_prob, V, K, chunk_len, n_chunks, vec, part,
                                                              share, lse_out, words, wait_limit, err, scratch_floats, acc);
    *launches_out = 2;
    return cudaGetLastError() == cudaSuccess ? DM_OK : DM_ECUDA;
}

}  // namespace

int launch_js(const float* logits, const float* draft_prob, float* workspace, size_t words_offset, int max_hidden, int V, int B, int T,
              int K, const int32_t* tokens, const int32_t* draft, float* out_js, int32_t* out_js_ok,
              int32_t* out_accept_len, uint32_t* err, long long wait_limit, cudaStream_t stream, int* launches_out) {
    const int n_pos = B * T;
    if (n_pos > kJsMaxPositions) return DM_EUNSUPPORTED;   // positions are the grid's second dimension
    int launches = 0;
    if (K <= 32) {
        unsigned int* words = reinterpret_cast<unsigned int*>(workspace + words_offset);
        float* lse_out = workspace + words_offset + 4 + 2 * (size_t)max_hidden;
        const JsAcceptArgs a1{nullptr, 0, B, T, K, tokens, draft, out_js, out_js_ok, out_accept_len, err};
        const long long limit = wait_limit > 0 ? wait_limit : 2000000000ll;
        const int st = K <= 8    ? launch_js_sweeps<8>(logits, draft_prob, workspace, lse_out, words, V, n_pos, K, T, a1, limit, err, stream, &launches)
                       : K <= 16 ? launch_js_sweeps<16>(logits, draft_prob, workspace, lse_out, words, V, n_pos, K, T, a1, limit, err, stream, &launches)
                                 : launch_js_sweeps<32>(logits, draft_prob, workspace, lse_out, words, V, n_pos, K, T, a1, limit, err, stream, &launches);
        if (launches_out) *launches_out = launches;
        return st;
    }
    // More paths than the sweep kernel keeps in registers: one series at a time, acceptance in a kernel of its own.
    if (launches_out) *launches_out = 3;
    const int n_chunks = js_chunks(V, n_pos);
    const int chunk_len = (V + n_chunks - 1) / n_chunks;
    float2* part = reinterpret_cast<float2*>(workspace);
    float* share = workspace + (size_t)n_pos * (K + 1) * n_chunks * 2;
    if ((size_t)(K + 1 + chunk_len) * sizeof(float) > 40 * 1024 || (size_t)T * sizeof(int32_t) > 40 * 1024) return DM_EUNSUPPORTED;
    dim3 grid((unsigned)n_chunks, (unsigned)n_pos);
    const JsAcceptArgs acc{share, n_chunks, B, T, K, tokens, draft, out_js, out_js_ok, out_accept_len, err};
    const size_t ok_bytes = (size_t)T * sizeof(int32_t);
    js_lse_kernel<<<grid, kJsThreads, chunk_len * sizeof(float), stream>>>(logits, V, K, chunk_len, n_chunks, part);
    js_sum_kernel<<<grid, kJsThreads, (K + 1 + chunk_len) * sizeof(float), stream>>>(logits, draft_prob, V, K,
                                                                                  chunk_len, n_chunks, part, share);
    if (cudaGetLastError() != cudaSuccess) return DM_ECUDA;
    js_accept_kernel<<<B, kJsThreads, ok_bytes, stream>>>(acc);
    return cudaGetLastError() == cudaSuccess ? DM_OK : DM_ECUDA;
}

}  // namespace dm
