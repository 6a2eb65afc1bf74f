/*
 * DropMatch verification oracle -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, obviously-correct CPU statement of what the MC-dropout
 * LM-head verification step computes (paper Sec. 3.1 "Multi-Sample LM Head via
 * MC Dropout" and Sec. 3.2 "Acceptance Criteria").  Every floating-point
 * quantity is accumulated in fp64, in index order, with no blocking, fusion or
 * reordering.  Only tests, the smoke check and the benchmark's cpu-baseline leg
 * may call this file; the CUDA library never does, and the two share no code.
 *
 * Steps, in the paper's order:
 *   Eq. 1  mask      m^(i)_j ~ iid Bernoulli(1 - p_drop), one mask per
 *                    (sequence, position, path); the random bits come from the
 *                    counter-based Philox4x32-10 generator (Salmon et al.,
 *                    SC'11) so that they can be reproduced from indices alone.
 *   Eq. 2  dropout   h^(i) = h (.) m^(i) / (1 - p_drop)
 *   Eq. 3  logits    l^(i) = W h^(i)
 *   Sec. 3.2         y^(i) = argmax softmax(l^(i)) = argmax l^(i)
 *   Eq. 3' (naive)   accept iff draft token is one of the K path tokens
 *   Eq. 6 (majority) accept iff draft token equals the most frequent path token
 *   Sec. 2 ("Lossless Speculative Decoding" paragraph): a rejection rejects all
 *                    later positions -> accepted length = leading run of accepts.
 *   Eq. 4, Eq. 5, Algorithm 1: centroid distribution, Jensen-Shannon test, JS-else-majority.
 *   Sec. 4.4         tree drafts: candidates under one parent share that parent's
 *                    target distribution; naive rule per node; the result is the
 *                    longest accepted root-to-leaf path.
 *
 * Pins (tests/test_oracle_*.py): cuRAND host Philox4_32_10 stream, an
 * independent Python-integer Philox, Bernoulli closed forms, p=0 == fp64 GEMV
 * + greedy verification, K=1 single path, brute force over all 16 masks at d=4,
 * linearity identity, scale invariance, first-reject-stops, nested-K
 * monotonicity, batched == singles, chain == path-shaped tree.  JS criterion (Eq. 4, Eq. 5,
 * Algorithm 1): scipy's Jensen-Shannon distance, relative entropy and softmax, closed forms,
 * a scipy restatement of Algorithm 1 with both outcomes, p=0 collapse onto the centroid.
 * Next-token call: library fp64 GEMV argmax and a brute-force scan.  Shared masks: equal hidden
 * rows decode alike path by path, position t equals a one-position call.
 * Sampling decode: the uniform variates against the Python-integer Philox; the nucleus against a
 * numpy sort-and-cut; sampled tokens against a numpy Gumbel-max; token frequencies over many
 * paths against the renormalised nucleus probabilities (chi-square) on vocabularies of up to 8;
 * temperature -> 0 and top_p -> 0 reduce to the argmax.
 * Parity unpinned: the paper's printed aggregates (tau, agreement ratios) need
 * the authors' models and datasets and cannot pin anything here.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_F32 0
#define ORACLE_BF16 1
#define ORACLE_RULE_NAIVE 0
#define ORACLE_RULE_MAJORITY 1

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (published algorithm: 10 rounds of two 32x32->64 multiplies, */
/* a fixed word permutation with key injection, Weyl key schedule).           */
/* ------------------------------------------------------------------------- */

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint64_t mult_a = 0xD2511F53u; /* multiplier applied to word 0 */
    const uint64_t mult_b = 0xCD9E8D57u; /* multiplier applied to word 2 */
    const uint32_t weyl_a = 0x9E3779B9u; /* key[0] increment per round   */
    const uint32_t weyl_b = 0xBB67AE85u; /* key[1] increment per round   */
    uint32_t x0 = ctr[0], x1 = ctr[1], x2 = ctr[2], x3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t pa = mult_a * (uint64_t)x0;
        uint64_t pb = mult_b * (uint64_t)x2;
        uint32_t y0 = (uint32_t)(pb >> 32) ^ x1 ^ k0;
        uint32_t y1 = (uint32_t)pb;
        uint32_t y2 = (uint32_t)(pa >> 32) ^ x3 ^ k1;
        uint32_t y3 = (uint32_t)pa;
        x0 = y0; x1 = y1; x2 = y2; x3 = y3;
        k0 += weyl_a;
        k1 += weyl_b;
    }
    out[0] = x0; out[1] = x1; out[2] = x2; out[3] = x3;
}

/* Eq. 1: P(drop) = thr / 2^32 with thr = floor(p * 2^32); p is the float the
 * caller passes, widened exactly to double. */
uint32_t oracle_drop_threshold(float p)
{
    double scaled = floor((double)p * 4294967296.0);
    if (scaled < 0.0) scaled = 0.0;
    if (scaled > 4294967295.0) scaled = 4294967295.0;
    return (uint32_t)scaled;
}

/* Eq. 1: keep bit of element j for (sequence s, position t, path i).
 * counter = (j / 4, i, t, s mod 2^32), key = (seed low word, seed high word);
 * element j uses output word j mod 4; the element is dropped iff word < thr. */
int oracle_mask_keep(uint64_t seed, uint64_t s, uint32_t t, uint32_t i, uint32_t j, uint32_t thr)
{
    uint32_t ctr[4] = { j >> 2, i, t, (uint32_t)s };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t w[4];
    oracle_philox4x32_10(ctr, key, w);
    return w[j & 3u] >= thr;
}

/* All masks of a call, bit-packed: out_bits[((b*T+t)*K+i)*ceil(d/32) + j/32]
 * has bit (j mod 32) set iff element j is kept. */
void oracle_masks(int B, int T, int K, int d, float p, uint64_t seed, uint64_t seq_base,
                  uint32_t *out_bits)
{
    const uint32_t thr = oracle_drop_threshold(p);
    const int words = (d + 31) / 32;
    memset(out_bits, 0, (size_t)B * T * K * words * sizeof(uint32_t));
    for (int b = 0; b < B; ++b)
        for (int t = 0; t < T; ++t)
            for (int i = 0; i < K; ++i) {
                uint32_t *row = out_bits + (((size_t)b * T + t) * K + i) * words;
                for (int j = 0; j < d; ++j)
                    if (oracle_mask_keep(seed, seq_base + (uint64_t)b, (uint32_t)t, (uint32_t)i,
                                         (uint32_t)j, thr))
                        row[j >> 5] |= 1u << (j & 31);
            }
}

/* ------------------------------------------------------------------------- */
/* Eq. 2 - Eq. 3: masked hidden state and logits of one path                  */
/* ------------------------------------------------------------------------- */

/* Exact widening of a stored element (fp32, or bf16 = the upper 16 bits of an
 * fp32) to double. */
static double load_elem(const void *base, int dtype, size_t idx)
{
    if (dtype == ORACLE_F32)
        return (double)((const float *)base)[idx];
    uint32_t bits = (uint32_t)((const uint16_t *)base)[idx] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* Eq. 2 without the scale: hm[j] = h[j] if kept else 0 (exact). */
void oracle_masked_hidden(const void *h_row, int dtype, int d, float p, uint64_t seed, uint64_t s,
                          int t, int i, double *hm)
{
    const uint32_t thr = oracle_drop_threshold(p);
    for (int j = 0; j < d; ++j) {
        int keep = oracle_mask_keep(seed, s, (uint32_t)t, (uint32_t)i, (uint32_t)j, thr);
        hm[j] = keep ? load_elem(h_row, dtype, (size_t)j) : 0.0;
    }
}

/* Eq. 3 with Eq. 2's scale applied to the finished sum:
 * l[v] = (sum_j W[v,j] * hm[j]) * 1/(1-p), j ascending, all in fp64. */
void oracle_logits_row(const void *W, int dtype, int V, int d, const void *h_row, float p,
                       uint64_t seed, uint64_t s, int t, int i, double *logits)
{
    double *hm = (double *)malloc((size_t)d * sizeof(double));
    oracle_masked_hidden(h_row, dtype, d, p, seed, s, t, i, hm);
    const double scale = 1.0 / (1.0 - (double)p);
#pragma omp parallel for schedule(static)
    for (int v = 0; v < V; ++v) {
        double acc = 0.0;
        for (int j = 0; j < d; ++j)
            acc += load_elem(W, dtype, (size_t)v * d + j) * hm[j];
        logits[v] = acc * scale;
    }
    free(hm);
}

/* Sec. 3.2: y = argmax_v l[v]; ties go to the smallest index.  Also reports
 * gap = l[y] - (largest logit at any other index), used only to flag near-ties. */
int oracle_argmax(const double *logits, int V, double *gap)
{
    int best = 0;
    for (int v = 1; v < V; ++v)
        if (logits[v] > logits[best]) best = v;
    double second = -INFINITY;
    for (int v = 0; v < V; ++v)
        if (v != best && logits[v] > second) second = logits[v];
    if (gap) *gap = (V > 1) ? logits[best] - second : INFINITY;
    return best;
}

/* ------------------------------------------------------------------------- */
/* Sec. 3.2: empirical token distribution and per-position tests              */
/* ------------------------------------------------------------------------- */

/* counts[i] = how many of the K path tokens equal tokens[i];
 * returns hits = how many equal the draft token. */
int oracle_counts(const int32_t *tokens, int K, int32_t draft, int32_t *counts)
{
    int hits = 0;
    for (int i = 0; i < K; ++i) {
        int c = 0;
        for (int i2 = 0; i2 < K; ++i2)
            if (tokens[i2] == tokens[i]) ++c;
        if (counts) counts[i] = c;
        if (tokens[i] == draft) ++hits;
    }
    return hits;
}

/* Eq. 6: the most frequent path token (plurality); equal frequencies resolve to
 * the smallest token id. */
int32_t oracle_majority_token(const int32_t *tokens, int K)
{
    int32_t mode = tokens[0];
    int mode_count = 0;
    for (int i = 0; i < K; ++i) {
        int c = 0;
        for (int i2 = 0; i2 < K; ++i2)
            if (tokens[i2] == tokens[i]) ++c;
        if (c > mode_count || (c == mode_count && tokens[i] < mode)) {
            mode = tokens[i];
            mode_count = c;
        }
    }
    return mode;
}

/* Per-position acceptance: naive = set membership (Eq. 3'), majority = Eq. 6. */
int oracle_position_ok(const int32_t *tokens, int K, int32_t draft, int rule)
{
    if (rule == ORACLE_RULE_MAJORITY)
        return oracle_majority_token(tokens, K) == draft;
    return oracle_counts(tokens, K, draft, NULL) >= 1;
}

/* Left-to-right acceptance: number of leading accepted positions. */
int oracle_accept_chain(const int32_t *tokens /*[T,K]*/, const int32_t *draft /*[T]*/, int T, int K,
                        int rule)
{
    int len = 0;
    while (len < T && oracle_position_ok(tokens + (size_t)len * K, K, draft[len], rule)) ++len;
    return len;
}

/* Tree acceptance.  Nodes are in topological order (parent[n] < n; -1 = child of
 * the committed prefix).  Node n is tested against the K tokens sampled from
 * hidden row hrow[n].  node_ok[n] = (parent is the prefix or parent ok) and the
 * node's own test.  Result: depth of the deepest ok node (0 if none) and the
 * smallest-index ok node of that depth (-1 if none). */
int oracle_accept_tree(const int32_t *tokens /*[N_h,K]*/, const int32_t *node_token,
                       const int32_t *node_parent, const int32_t *node_hrow, int N, int K, int rule,
                       int32_t *node_ok /*[N] or NULL*/, int32_t *best_node)
{
    int *ok = (int *)malloc((size_t)(N > 0 ? N : 1) * sizeof(int));
    int *depth = (int *)malloc((size_t)(N > 0 ? N : 1) * sizeof(int));
    int best_depth = 0, best = -1;
    for (int n = 0; n < N; ++n) {
        int par = node_parent[n];
        int par_ok = (par < 0) ? 1 : ok[par];
        depth[n] = (par < 0) ? 1 : depth[par] + 1;
        ok[n] = par_ok &&
                oracle_position_ok(tokens + (size_t)node_hrow[n] * K, K, node_token[n], rule);
        if (node_ok) node_ok[n] = ok[n];
        if (ok[n] && depth[n] > best_depth) {
            best_depth = depth[n];
            best = n;
        }
    }
    if (best_node) *best_node = best;
    free(ok);
    free(depth);
    return best_depth;
}

/* ------------------------------------------------------------------------- */
/* Whole verification calls                                                   */
/* ------------------------------------------------------------------------- */

/* Tokens (and top-2 gaps) of every path of n_bt hidden rows.  Hidden row q
 * belongs to sequence q / rows_per_seq and has position index q % rows_per_seq;
 * path (q, i) is written at out_tokens[q*K + i]. */
static void sample_tokens(const void *W, int dtype, int V, int d, const void *H, int n_bt,
                          int rows_per_seq, int K, float p, uint64_t seed, uint64_t seq_base,
                          int shared_masks, int32_t *out_tokens, double *out_gap)
{
    const size_t elem = (dtype == ORACLE_F32) ? 4 : 2;
    double *logits = (double *)malloc((size_t)V * sizeof(double));
    for (int q = 0; q < n_bt; ++q) {
        const uint64_t s = seq_base + (uint64_t)(q / rows_per_seq);
        /* shared masks: path i uses one mask m^(i) at every position, i.e. position 0's key */
        const int t = shared_masks ? 0 : q % rows_per_seq;
        const void *h_row = (const char *)H + (size_t)q * d * elem;
        for (int i = 0; i < K; ++i) {
            double gap;
            oracle_logits_row(W, dtype, V, d, h_row, p, seed, s, t, i, logits);
            out_tokens[(size_t)q * K + i] = oracle_argmax(logits, V, &gap);
            if (out_gap) out_gap[(size_t)q * K + i] = gap;
        }
    }
    free(logits);
}

/* shared_masks = 1 is the other reading of Eq. 1 (m^(i) carries no position index): the K paths
 * are K persistent heads, each with one mask for all positions of a sequence.
 * Chain verification of B independent sequences (sequence b has id seq_base+b).
 * H[B,T,d], draft[B,T] -> tokens[B,T,K], gap[B,T,K] (may be NULL),
 * counts[B,T,K], hits[B,T], accept_len[B]. */
void oracle_verify_batched_ex(const void *W, int dtype, int V, int d, const void *H,
                              const int32_t *draft, int B, int T, int K, float p, uint64_t seed,
                              uint64_t seq_base, int rule, int shared_masks, int32_t *out_tokens,
                              double *out_gap, int32_t *out_counts, int32_t *out_hits,
                              int32_t *out_accept_len)
{
    sample_tokens(W, dtype, V, d, H, B * T, T, K, p, seed, seq_base, shared_masks, out_tokens, out_gap);
    for (int b = 0; b < B; ++b) {
        for (int t = 0; t < T; ++t) {
            size_t q = (size_t)b * T + t;
            int hits = oracle_counts(out_tokens + q * K, K, draft[q], out_counts + q * K);
            if (out_hits) out_hits[q] = hits;
        }
        out_accept_len[b] = oracle_accept_chain(out_tokens + (size_t)b * T * K,
                                                draft + (size_t)b * T, T, K, rule);
    }
}

/* The default reading (R1): an independent mask per (sequence, position, path). */
void oracle_verify_batched(const void *W, int dtype, int V, int d, const void *H,
                           const int32_t *draft, int B, int T, int K, float p, uint64_t seed,
                           uint64_t seq_base, int rule, int32_t *out_tokens, double *out_gap,
                           int32_t *out_counts, int32_t *out_hits, int32_t *out_accept_len)
{
    oracle_verify_batched_ex(W, dtype, V, d, H, draft, B, T, K, p, seed, seq_base, rule, 0, out_tokens,
                             out_gap, out_counts, out_hits, out_accept_len);
}

/* Tree verification of B sequences: H[B,N_h,d]; per sequence N nodes
 * (token, parent, hrow).  counts are multiplicities per hidden row. */
void oracle_verify_tree(const void *W, int dtype, int V, int d, const void *H,
                        const int32_t *node_token, const int32_t *node_parent,
                        const int32_t *node_hrow, int B, int N_h, int N, int K, float p,
                        uint64_t seed, uint64_t seq_base, int rule, int32_t *out_tokens,
                        double *out_gap, int32_t *out_counts, int32_t *out_node_ok,
                        int32_t *out_best_node, int32_t *out_accept_len)
{
    sample_tokens(W, dtype, V, d, H, B * N_h, N_h, K, p, seed, seq_base, 0, out_tokens, out_gap);
    for (int b = 0; b < B; ++b) {
        for (int q = 0; q < N_h; ++q) {
            size_t row = (size_t)b * N_h + q;
            oracle_counts(out_tokens + row * K, K, -1, out_counts + row * K);
        }
        out_accept_len[b] = oracle_accept_tree(
            out_tokens + (size_t)b * N_h * K, node_token + (size_t)b * N, node_parent + (size_t)b * N,
            node_hrow + (size_t)b * N, N, K, rule, out_node_ok ? out_node_ok + (size_t)b * N : NULL,
            out_best_node + b);
    }
}

/* ------------------------------------------------------------------------- */
/* Sampling decode rule (Sec. 3.2: the per-path token is the top-1 token "or"  */
/* a token selected by nucleus sampling; the paper gives no parameters)        */
/* ------------------------------------------------------------------------- */

/* Uniform variate of vocabulary entry v for (sequence s, position t, path i): Philox4x32-10 at
 * counter (v / 4, i + 2^31, t, s mod 2^32), key = seed, word v mod 4.  Path indices stay below
 * 2^31, so these counters never meet the mask counters of Eq. 1.  The top 23 bits k of the word
 * give u = (k + 0.5) / 2^23, which lies strictly inside (0,1) and is exact in fp32 and fp64. */
double oracle_sample_uniform(uint64_t seed, uint64_t s, uint32_t t, uint32_t i, uint32_t v)
{
    uint32_t ctr[4] = { v >> 2, i | 0x80000000u, t, (uint32_t)s };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t w[4];
    oracle_philox4x32_10(ctr, key, w);
    return ((double)(w[v & 3u] >> 9) + 0.5) / 8388608.0;
}

/* Standard Gumbel variate g = -log(-log(u)). */
double oracle_gumbel(double u)
{
    return -log(-log(u));
}

struct prob_index { double p; int v; };
static int by_prob_desc(const void *a, const void *b)
{
    const struct prob_index *x = (const struct prob_index *)a, *y = (const struct prob_index *)b;
    if (x->p > y->p) return -1;
    if (x->p < y->p) return 1;
    return x->v - y->v;   /* equal probabilities: smaller token id first */
}

/* Nucleus of a logit row: p = Softmax(l / temperature); tokens in order of decreasing p (equal p:
 * increasing id) are taken until their cumulative probability reaches top_p, the token that
 * crosses it included; top_p >= 1 keeps every token.  in_nucleus[v] = 1/0.  Returns the size. */
int oracle_nucleus(const double *logits, int V, double temperature, double top_p, unsigned char *in_nucleus)
{
    if (top_p >= 1.0) {
        memset(in_nucleus, 1, (size_t)V);
        return V;
    }
    struct prob_index *ord = (struct prob_index *)malloc((size_t)V * sizeof *ord);
    double zmax = -INFINITY, sum = 0.0;
    for (int v = 0; v < V; ++v)
        if (logits[v] / temperature > zmax) zmax = logits[v] / temperature;
    for (int v = 0; v < V; ++v) {
        ord[v].p = exp(logits[v] / temperature - zmax);
        ord[v].v = v;
        sum += ord[v].p;
    }
    for (int v = 0; v < V; ++v) ord[v].p /= sum;
    qsort(ord, (size_t)V, sizeof *ord, by_prob_desc);
    memset(in_nucleus, 0, (size_t)V);
    double cum = 0.0;
    int n = 0;
    while (n < V) {
        in_nucleus[ord[n].v] = 1;
        cum += ord[n].p;
        ++n;
        if (cum >= top_p) break;
    }
    free(ord);
    return n;
}

/* One sampled token: y = argmax over the nucleus of l[v] / temperature + g[v] (the Gumbel-max
 * form of drawing from the renormalised nucleus distribution); equal keys go to the smaller id.
 * gap = winning key - runner-up key within the nucleus (infinite if the nucleus is one token). */
int oracle_sample_row(const double *logits, int V, double temperature, double top_p, uint64_t seed,
                      uint64_t s, uint32_t t, uint32_t i, double *gap)
{
    unsigned char *in = (unsigned char *)malloc((size_t)V);
    oracle_nucleus(logits, V, temperature, top_p, in);
    int best = -1;
    double best_key = -INFINITY, second = -INFINITY;
    for (int v = 0; v < V; ++v) {
        if (!in[v]) continue;
        double key = logits[v] / temperature + oracle_gumbel(oracle_sample_uniform(seed, s, t, i, (uint32_t)v));
        if (best < 0 || key > best_key) {
            if (best >= 0) second = best_key;
            best_key = key;
            best = v;
        } else if (key > second) {
            second = key;
        }
    }
    if (gap) *gap = best_key - second;
    free(in);
    return best;
}

/* Chain verification with the sampling decode rule in place of the argmax of Sec. 3.2: Eq. 1-3 as
 * before, y^(i) drawn as above, then counts, per-position test and left-to-right scan unchanged.
 * H[B,T,d], draft[B,T] -> tokens[B,T,K], gap[B,T,K] (may be NULL), counts, hits[B,T], accept_len[B]. */
void oracle_verify_batched_sampled(const void *W, int dtype, int V, int d, const void *H,
                                   const int32_t *draft, int B, int T, int K, float p, uint64_t seed,
                                   uint64_t seq_base, int rule, double temperature, double top_p,
                                   int32_t *out_tokens, double *out_gap, int32_t *out_counts,
                                   int32_t *out_hits, int32_t *out_accept_len)
{
    const size_t elem = dtype == ORACLE_F32 ? 4 : 2;
    double *logits = (double *)malloc((size_t)V * sizeof(double));
    for (int b = 0; b < B; ++b) {
        for (int t = 0; t < T; ++t) {
            size_t q = (size_t)b * T + t;
            const void *h_row = (const char *)H + q * d * elem;
            for (int i = 0; i < K; ++i) {
                double gap;
                oracle_logits_row(W, dtype, V, d, h_row, p, seed, seq_base + (uint64_t)b, t, i, logits);
                out_tokens[q * K + i] = oracle_sample_row(logits, V, temperature, top_p, seed,
                                                          seq_base + (uint64_t)b, (uint32_t)t, (uint32_t)i, &gap);
                if (out_gap) out_gap[q * K + i] = gap;
            }
            int hits = oracle_counts(out_tokens + q * K, K, draft[q], out_counts + q * K);
            if (out_hits) out_hits[q] = hits;
        }
        out_accept_len[b] = oracle_accept_chain(out_tokens + (size_t)b * T * K, draft + (size_t)b * T, T, K, rule);
    }
    free(logits);
}

/* ------------------------------------------------------------------------- */
/* JS-divergence criterion (Sec. 3.2, Eq. 4, Eq. 5, Algorithm 1)              */
/* ------------------------------------------------------------------------- */

/* Softmax of V logits, in place into prob[] (max-subtracted, fp64). */
static void softmax_f64(const double *logits, int V, double *prob)
{
    double mx = logits[0];
    for (int v = 1; v < V; ++v)
        if (logits[v] > mx) mx = logits[v];
    double sum = 0.0;
    for (int v = 0; v < V; ++v) {
        prob[v] = exp(logits[v] - mx);
        sum += prob[v];
    }
    for (int v = 0; v < V; ++v) prob[v] /= sum;
}

/* Jensen-Shannon divergence of two distributions over V outcomes, natural
 * logarithm: JS(P||Q) = KL(P||M)/2 + KL(Q||M)/2 with M = (P+Q)/2; terms with a
 * zero probability contribute zero. */
double oracle_js_divergence(const double *P, const double *Q, int V)
{
    double acc = 0.0;
    for (int v = 0; v < V; ++v) {
        double m = 0.5 * (P[v] + Q[v]);
        if (P[v] > 0.0) acc += 0.5 * P[v] * log(P[v] / m);
        if (Q[v] > 0.0) acc += 0.5 * Q[v] * log(Q[v] / m);
    }
    return acc;
}

/* Eq. 4 and both sides of Eq. 5 from explicit logits.  logits[K][V] are the K
 * head logits of one position, draft_prob[V] the draft model's distribution.
 * out_js[i] = JS(p^(i) || pbar) for i < K and out_js[K] = JS(phat || pbar),
 * where pbar = Softmax(mean_i logits[i]) and p^(i) = Softmax(logits[i]).
 * Returns 1 iff Eq. 5 holds: out_js[K] <= max_i out_js[i]. */
int oracle_js_from_logits(const double *logits, int K, int V, const double *draft_prob,
                          double *out_js)
{
    double *centroid = (double *)malloc((size_t)V * sizeof(double));
    double *pbar = (double *)malloc((size_t)V * sizeof(double));
    double *pi = (double *)malloc((size_t)V * sizeof(double));
    for (int v = 0; v < V; ++v) {
        double s = 0.0;
        for (int i = 0; i < K; ++i) s += logits[(size_t)i * V + v];
        centroid[v] = s / (double)K;
    }
    softmax_f64(centroid, V, pbar);
    double max_heads = -INFINITY;
    for (int i = 0; i < K; ++i) {
        softmax_f64(logits + (size_t)i * V, V, pi);
        out_js[i] = oracle_js_divergence(pi, pbar, V);
        if (out_js[i] > max_heads) max_heads = out_js[i];
    }
    out_js[K] = oracle_js_divergence(draft_prob, pbar, V);
    free(centroid);
    free(pbar);
    free(pi);
    return out_js[K] <= max_heads;
}

/* Algorithm 1 for B chains: per position Eq. 5, else the majority rule of
 * Eq. 6, else reject; then the left-to-right scan.  draft_prob[B,T,V] is fp32
 * (the draft model's probabilities), widened exactly.
 * Outputs: tokens[B,T,K], counts[B,T,K], js[B,T,K+1], js_ok[B,T] (Eq. 5 alone),
 * accept_len[B]. */
void oracle_verify_js(const void *W, int dtype, int V, int d, const void *H, const int32_t *draft,
                      const float *draft_prob, int B, int T, int K, float p, uint64_t seed,
                      uint64_t seq_base, int32_t *out_tokens, int32_t *out_counts, double *out_js,
                      int32_t *out_js_ok, int32_t *out_accept_len)
{
    const size_t elem = (dtype == ORACLE_F32) ? 4 : 2;
    double *logits = (double *)malloc((size_t)K * V * sizeof(double));
    double *dp = (double *)malloc((size_t)V * sizeof(double));
    for (int b = 0; b < B; ++b) {
        int len = 0, open = 1;
        for (int t = 0; t < T; ++t) {
            const size_t q = (size_t)b * T + t;
            const void *h_row = (const char *)H + q * d * elem;
            for (int i = 0; i < K; ++i) {
                oracle_logits_row(W, dtype, V, d, h_row, p, seed, seq_base + (uint64_t)b, t, i,
                                  logits + (size_t)i * V);
                out_tokens[q * K + i] = oracle_argmax(logits + (size_t)i * V, V, NULL);
            }
            oracle_counts(out_tokens + q * K, K, draft[q], out_counts + q * K);
            for (int v = 0; v < V; ++v) dp[v] = (double)draft_prob[q * V + v];
            int js_ok = oracle_js_from_logits(logits, K, V, dp, out_js + q * (K + 1));
            out_js_ok[q] = js_ok;
            int ok = js_ok || oracle_majority_token(out_tokens + q * K, K) == draft[q];
            if (open && ok) ++len;
            else open = 0;
        }
        out_accept_len[b] = len;
    }
    free(logits);
    free(dp);
}

/* ------------------------------------------------------------------------- */
/* Token emitted after the accepted prefix                                    */
/* ------------------------------------------------------------------------- */

/* Chain verification as oracle_verify_batched, on H[B, T_h, d] with T_h = T + bonus_row hidden
 * rows per sequence (only the first T are scanned against draft[B,T]), plus the target's own
 * greedy token of every hidden row, plain[b,q] = argmax_v (W h_{b,q})[v] (no dropout), and
 * next[b] = plain[b, accept_len[b]] if that row exists, else -1.  The paper leaves the choice of
 * this token open; this is greedy verification's.  plain_gap may be NULL. */
void oracle_verify_batched_next(const void *W, int dtype, int V, int d, const void *H,
                                const int32_t *draft, int B, int T, int bonus_row, int K, float p,
                                uint64_t seed, uint64_t seq_base, int rule, int32_t *out_tokens,
                                double *out_gap, int32_t *out_counts, int32_t *out_hits,
                                int32_t *out_accept_len, int32_t *out_plain, double *plain_gap,
                                int32_t *out_next)
{
    const int T_h = T + (bonus_row ? 1 : 0);
    const size_t elem = (dtype == ORACLE_F32) ? 4 : 2;
    sample_tokens(W, dtype, V, d, H, B * T_h, T_h, K, p, seed, seq_base, 0, out_tokens, out_gap);
    double *logits = (double *)malloc((size_t)V * sizeof(double));
    for (int b = 0; b < B; ++b) {
        for (int q = 0; q < T_h; ++q) {
            const size_t row = (size_t)b * T_h + q;
            const char *h_row = (const char *)H + row * d * elem;
#pragma omp parallel for schedule(static)
            for (int v = 0; v < V; ++v) {
                double acc = 0.0;
                for (int j = 0; j < d; ++j)
                    acc += load_elem(W, dtype, (size_t)v * d + j) * load_elem(h_row, dtype, (size_t)j);
                logits[v] = acc;
            }
            double gap;
            out_plain[row] = oracle_argmax(logits, V, &gap);
            if (plain_gap) plain_gap[row] = gap;
            int hits = oracle_counts(out_tokens + row * K, K, q < T ? draft[(size_t)b * T + q] : -1,
                                     out_counts + row * K);
            if (out_hits && q < T) out_hits[(size_t)b * T + q] = hits;
        }
        /* scan the T draft positions; the token rows of a sequence are T_h apart */
        int len = 0;
        while (len < T && oracle_position_ok(out_tokens + ((size_t)b * T_h + len) * K, K,
                                             draft[(size_t)b * T + len], rule))
            ++len;
        out_accept_len[b] = len;
        out_next[b] = (len < T_h) ? out_plain[(size_t)b * T_h + len] : -1;
    }
    free(logits);
}
