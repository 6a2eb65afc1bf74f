// JS-divergence acceptance (Sec. 3.2: Eq. 4 centroid, Eq. 5 test, Algorithm 1) on the logits that
// a head kernel has written to global memory.  Three small kernels over [n_pos][K][V] fp32
// logits (20 MB for the Llama-3-8B head at 40 paths, L2-resident right after the head kernel):
//   js_lse_kernel      per (position, vocabulary chunk): partial log-sum-exp of each of the K
//                      paths and of the centroid logits (their mean over the paths)
//   js_sum_kernel      per (position, chunk): merges the partial log-sum-exps, then the chunk's
//                      share of JS(p_i || pbar) for every path and of JS(phat || pbar)
//   js_accept_kernel   per sequence: sums the shares, Eq. 5, else Eq. 6, left-to-right scan
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

// ---- the same two sweeps for K <= KMAX paths with every series kept in registers --------------
// A thread takes vocabulary entries v0 + tid, v0 + tid + 256, ...: it loads the K logits of an
// entry once (coalesced across the block), forms the centroid and updates all K+1 running
// results; the block is reduced once at the end.  Slot KMAX holds the centroid (first sweep) or
// the draft distribution (second sweep).

__device__ __forceinline__ void lse_merge(float& m, float& s, float m2, float s2) {
    const float M = fmaxf(m, m2);
    if (M == -INFINITY) { m = M; s = 0.0f; return; }
    // fast exponentials: relative error ~1e-7 per term of a sum of positive terms, far inside the
    // tolerance of the divergences (the arguments are <= 0)
    s = s * __expf(m - M) + s2 * __expf(m2 - M);
    m = M;
}

template <int KMAX>
__global__ void __launch_bounds__(kJsThreads)
js_lse_reg_kernel(const float* __restrict__ logits, int V, int K, int chunk_len, int n_chunks,
                  float2* __restrict__ part) {
    __shared__ float2 red[kJsThreads / 32][KMAX + 1];
    const int pos = blockIdx.y, chunk = blockIdx.x;
    const int v0 = chunk * chunk_len, v1 = min(V, v0 + chunk_len);
    const float* pl = logits + (size_t)pos * K * V;
    float m[KMAX + 1], s[KMAX + 1];
#pragma unroll
    for (int i = 0; i <= KMAX; ++i) { m[i] = -INFINITY; s[i] = 0.0f; }
    const float inv_k = 1.0f / (float)K;
    for (int v = v0 + threadIdx.x; v < v1; v += kJsThreads) {
        float c = 0.0f;
#pragma unroll
        for (int i = 0; i < KMAX; ++i)
            if (i < K) {
                const float x = pl[(size_t)i * V + v];
                c += x;
                lse_merge(m[i], s[i], x, 1.0f);
            }
        lse_merge(m[KMAX], s[KMAX], c * inv_k, 1.0f);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
    for (int i = 0; i <= KMAX; ++i) {
        if (i < K || i == KMAX) {
            float M = m[i];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, off));
            float t = M == -INFINITY ? 0.0f : s[i] * __expf(m[i] - M);   // one rescale, then a plain sum
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, off);
            if (lane == 0) red[warp][i] = make_float2(M, t);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i <= KMAX; i += kJsThreads) {
        if (i < K || i == KMAX) {
            float mm = red[0][i].x, ss = red[0][i].y;
            for (int w = 1; w < kJsThreads / 32; ++w) lse_merge(mm, ss, red[w][i].x, red[w][i].y);
            const int series = i == KMAX ? K : i;
            part[((size_t)pos * (K + 1) + series) * n_chunks + chunk] = make_float2(mm, ss);
        }
    }
}

// The block that finishes last (a ticket counter in global memory, left at zero) also runs
// Algorithm 1 and the scan for every sequence: no third kernel.
template <int KMAX>
__global__ void __launch_bounds__(kJsThreads)
js_sum_reg_kernel(const float* __restrict__ logits, const float* __restrict__ draft_prob, int V, int K,
                  int chunk_len, int n_chunks, const float2* __restrict__ part, float* __restrict__ share,
                  unsigned int* __restrict__ ticket, JsAcceptArgs accept) {
    extern __shared__ int32_t ok_scratch[];   // [T], for the last block
    __shared__ unsigned int s_ticket;
    __shared__ float lse[KMAX + 1];
    __shared__ float red[kJsThreads / 32][KMAX + 1];
    const int pos = blockIdx.y, chunk = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int series = warp; series <= K; series += kJsThreads / 32) {   // merge the chunks' partial log-sum-exps
        const float2* ps = part + ((size_t)pos * (K + 1) + series) * n_chunks;
        float mm = -INFINITY, ss = 0.0f;
        for (int c = lane; c < n_chunks; c += 32) lse_merge(mm, ss, ps[c].x, ps[c].y);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1)
            lse_merge(mm, ss, __shfl_xor_sync(0xFFFFFFFFu, mm, off), __shfl_xor_sync(0xFFFFFFFFu, ss, off));
        if (lane == 0) lse[series == K ? KMAX : series] = mm + logf(ss);
    }
    __syncthreads();
    const int v0 = chunk * chunk_len, v1 = min(V, v0 + chunk_len);
    const float* pl = logits + (size_t)pos * K * V;
    const float* dp = draft_prob + (size_t)pos * V;
    float acc[KMAX + 1];
#pragma unroll
    for (int i = 0; i <= KMAX; ++i) acc[i] = 0.0f;
    const float inv_k = 1.0f / (float)K, lse_c = lse[KMAX];
    for (int v = v0 + threadIdx.x; v < v1; v += kJsThreads) {
        float x[KMAX];
        float c = 0.0f;
#pragma unroll
        for (int i = 0; i < KMAX; ++i)
            if (i < K) { x[i] = pl[(size_t)i * V + v]; c += x[i]; }
        const float lq = c * inv_k - lse_c;                       // log pbar[v]
#pragma unroll
        for (int i = 0; i < KMAX; ++i)
            if (i < K) acc[i] += js_term(x[i] - lse[i], lq);
        const float P = dp[v];
        acc[KMAX] += js_term(P > 0.0f ? logf(P) : -INFINITY, lq);
    }
#pragma unroll
    for (int i = 0; i <= KMAX; ++i) {
        if (i < K || i == KMAX) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc[i] += __shfl_xor_sync(0xFFFFFFFFu, acc[i], off);
            if (lane == 0) red[warp][i] = acc[i];
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i <= KMAX; i += kJsThreads) {
        if (i < K || i == KMAX) {
            float t = 0.0f;
            for (int w = 0; w < kJsThreads / 32; ++w) t += red[w][i];
            const int series = i == KMAX ? K : i;
            share[((size_t)pos * (K + 1) + series) * n_chunks + chunk] = 0.5f * t;
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_ticket = atomicAdd(ticket, 1u);
    __syncthreads();
    if (s_ticket == gridDim.x * gridDim.y - 1) {
        __threadfence();
        for (int b = 0; b < accept.B; ++b) js_accept_sequence(accept, b, ok_scratch);
        if (threadIdx.x == 0) *ticket = 0u;
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

size_t js_workspace_floats(int V, int max_rows, int max_hidden) {
    // partial (max, sum) pairs and JS shares for every (position, series, chunk), at the largest
    // chunk count; then the ticket word of the second sweep
    return (size_t)(max_rows + max_hidden) * ((V + 1023) / 1024) * 3 + 4;
}

int launch_js(const float* logits, const float* draft_prob, float* workspace, size_t ticket_offset, int V, int B, int T,
              int K, const int32_t* tokens, const int32_t* draft, float* out_js, int32_t* out_js_ok,
              int32_t* out_accept_len, const uint32_t* err, cudaStream_t stream) {
    const int n_pos = B * T, n_chunks = js_chunks(V, n_pos);
    if (n_pos > kJsMaxPositions) return DM_EUNSUPPORTED;   // positions are the grid's second dimension
    const int chunk_len = (V + n_chunks - 1) / n_chunks;
    float2* part = reinterpret_cast<float2*>(workspace);
    float* share = workspace + (size_t)n_pos * (K + 1) * n_chunks * 2;
    unsigned int* ticket = reinterpret_cast<unsigned int*>(workspace + ticket_offset);
    if ((size_t)(K + 1 + chunk_len) * sizeof(float) > 40 * 1024 || (size_t)T * sizeof(int32_t) > 40 * 1024) return DM_EUNSUPPORTED;
    dim3 grid((unsigned)n_chunks, (unsigned)n_pos);
    const JsAcceptArgs acc{share, n_chunks, B, T, K, tokens, draft, out_js, out_js_ok, out_accept_len, err};
    const size_t ok_bytes = (size_t)T * sizeof(int32_t);
    if (K <= 8) {
        js_lse_reg_kernel<8><<<grid, kJsThreads, 0, stream>>>(logits, V, K, chunk_len, n_chunks, part);
        js_sum_reg_kernel<8><<<grid, kJsThreads, ok_bytes, stream>>>(logits, draft_prob, V, K, chunk_len, n_chunks, part, share, ticket, acc);
    } else if (K <= 16) {
        js_lse_reg_kernel<16><<<grid, kJsThreads, 0, stream>>>(logits, V, K, chunk_len, n_chunks, part);
        js_sum_reg_kernel<16><<<grid, kJsThreads, ok_bytes, stream>>>(logits, draft_prob, V, K, chunk_len, n_chunks, part, share, ticket, acc);
    } else if (K <= 32) {
        js_lse_reg_kernel<32><<<grid, kJsThreads, 0, stream>>>(logits, V, K, chunk_len, n_chunks, part);
        js_sum_reg_kernel<32><<<grid, kJsThreads, ok_bytes, stream>>>(logits, draft_prob, V, K, chunk_len, n_chunks, part, share, ticket, acc);
    } else {   // more paths than fit in registers: one series at a time, acceptance in a kernel of its own
        js_lse_kernel<<<grid, kJsThreads, chunk_len * sizeof(float), stream>>>(logits, V, K, chunk_len, n_chunks, part);
        js_sum_kernel<<<grid, kJsThreads, (K + 1 + chunk_len) * sizeof(float), stream>>>(logits, draft_prob, V, K,
                                                                                      chunk_len, n_chunks, part, share);
        if (cudaGetLastError() != cudaSuccess) return DM_ECUDA;
        js_accept_kernel<<<B, kJsThreads, ok_bytes, stream>>>(acc);
    }
    return cudaGetLastError() == cudaSuccess ? DM_OK : DM_ECUDA;
}

}  // namespace dm
