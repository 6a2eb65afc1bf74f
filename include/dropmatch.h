/*
 * dropmatch.h -- C ABI of the B200 (sm_100a) DropMatch verification library.
 *
 * DropMatch (arXiv 2603.03333) verifies draft tokens of speculative decoding by
 * Monte-Carlo dropout on the LM head only.  For every draft position t the target
 * model's final hidden state h_t[d] is copied K times, each copy multiplied by an
 * independent Bernoulli(1-p) keep mask and rescaled by 1/(1-p) (Eq. 1, Eq. 2);
 * each copy is projected through the shared head W[V,d] (Eq. 3) and decoded to its
 * argmax token (Sec. 3.2).  The K tokens of a position form an empirical token
 * distribution; a draft token is accepted when it is one of them (naive
 * token-matching criterion, Sec. 3.2) or when it is their most frequent token
 * (majority criterion, Eq. 6).  Positions are accepted left to right and the first
 * rejection rejects everything after it (Sec. 2, lossless-decoding paragraph);
 * for draft trees (Sec. 4.4) the result is the longest accepted root-to-leaf path.
 *
 * Conventions that hold for every entry point
 *   - Unless a parameter says "host", every tensor pointer is a DEVICE pointer on
 *     the context's device, owned by the caller, dense row-major, and must stay
 *     valid until the work queued on `stream` has finished.
 *   - H (and W) must be 16-byte aligned (DM_EINVAL otherwise).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Device-pointer entry points only enqueue work: they never
 *     synchronise, never allocate and never free.
 *     The context-based verify calls (dropmatch_verify, _batched, _tree, _batched_next, _js)
 *     can therefore be captured into a CUDA graph; the seed and all sizes are then fixed.
 *   - The library allocates device memory only in dm_create, dm_set_head and
 *     dm_enable_js (its workspace) and frees it in dm_set_head / dm_destroy.
 *   - Every function returns DM_OK or a negative status; nothing throws, aborts
 *     or prints.  A CUDA error raised by earlier asynchronous work is reported by
 *     the next call as DM_ECUDA.  A kernel that gives up on an internal wait sets
 *     the context's device error word, which dm_device_error() reads.
 *   - Masks: element j of path i at position t of sequence s is dropped iff word
 *     (j mod 4) of Philox4x32-10(counter = (j/4, i, t, s mod 2^32),
 *     key = (seed low 32 bits, seed high 32 bits)) is < floor(p * 2^32).
 *     Results depend on (seed, s, t, i, j) only, never on batching or launch shape.
 *     (dm_set_mask_mode can take t out of the key.)
 *   - Row order: path i of hidden row q (q = b*T + t) is "row" q*K + i.
 *   - A context is not thread-safe; use one per host thread or lock around it.
 */
#ifndef DROPMATCH_H_
#define DROPMATCH_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dm_ctx dm_ctx; /* opaque: device id, head description, workspace, TMA descriptors */

enum {
    DM_OK = 0,
    DM_EINVAL = -1,       /* bad argument (null pointer, size < 1, p outside [0,1), bad enum)   */
    DM_EUNSUPPORTED = -2, /* shape the kernels cannot handle (see dm_set_head)                  */
    DM_ECUDA = -3,        /* a CUDA runtime or driver call failed                               */
    DM_EWORKSPACE = -4,   /* call needs more rows than dm_set_head reserved                     */
    DM_EDEVICE = -5,      /* device is not compute capability 10.x                              */
    DM_ENOHEAD = -6,      /* dm_set_head has not been called                                    */
    DM_ESTATICLIMIT = -7  /* call exceeds DM_STATIC_MAX_ROWS of dropmatch_verify_batched_static */
};
enum { DM_F32 = 0, DM_BF16 = 1 };             /* storage type of W and H (accumulation is fp32) */
enum { DM_RULE_NAIVE = 0, DM_RULE_MAJORITY = 1 };
enum { DM_IMPL_AUTO = 0, DM_IMPL_SIMT = 1, DM_IMPL_TCGEN05 = 2 };
enum { DM_MASK_PER_POSITION = 0, DM_MASK_PER_PATH = 1 };

/* Create a context on CUDA device `device` (must be sm_100).  *out is set on success. */
int dm_create(dm_ctx** out, int device);
/* Free the context and its workspace.  Synchronises the device first.  NULL is allowed. */
int dm_destroy(dm_ctx* ctx);

/* Describe the LM head (Eq. 3): W is a device pointer to V*d elements, row-major [V,d],
 * 16-byte aligned, caller-owned; it is read, never written, by every verify call until the
 * next dm_set_head, and it must be complete before a call is enqueued: the tensor-core kernel
 * is launched with programmatic stream serialization and starts streaming W while the kernel
 * ahead of it in the stream is still finishing (H, the drafts and all outputs are only touched
 * after that kernel has completed).  Reserves workspace for calls of up to `max_rows` rows (rows = B*T*K, or
 * B*N_h*K for trees) and `max_hidden_rows` = rows/K hidden rows (used only by the *_host entry
 * point's staging buffers).  Requirements: V >= 1; d >= 4 and d % 4 == 0 (fp32) or d % 8 == 0
 * (bf16), else DM_EUNSUPPORTED.  bf16 heads with d % 64 == 0 run on the tcgen05 tensor-core
 * kernel, everything else on the CUDA-core kernel, which also needs one hidden row to fit
 * 200 KB of shared memory (d <= 51200 fp32, 102400 bf16; verify calls report DM_EUNSUPPORTED
 * beyond).  Synchronises the device (re-allocation); pins host memory for the *_host call. */
int dm_set_head(dm_ctx* ctx, const void* W, int V, int d, int dtype, int max_rows, int max_hidden_rows);

/* Programmatic stream serialization of the tensor-core kernel, on by default: the kernel starts
 * streaming W while the kernel ahead of it in the stream is still finishing, which is only right
 * if nothing ahead in the stream writes W.  A caller that refreshes W in stream order (a weight
 * reload, a dequantisation into the head buffer) and verifies right behind it on the same stream
 * switches it off with dm_set_pdl(ctx, 0): every verify kernel then starts after all earlier work
 * of the stream has completed, at the cost of about 2 us of launch latency per call. */
int dm_set_pdl(dm_ctx* ctx, int enable);

/* Force a kernel family (DM_IMPL_*) for later calls; DM_IMPL_AUTO restores the default choice.
 * DM_IMPL_TCGEN05 on a head it cannot handle makes verify calls return DM_EUNSUPPORTED. */
int dm_set_impl(dm_ctx* ctx, int impl);

/* How Eq. 1's masks are keyed for later calls.  DM_MASK_PER_POSITION (default): an independent
 * mask per (sequence, position, path).  DM_MASK_PER_PATH: the position is left out of the key, so
 * path i of a sequence applies one and the same mask m^(i) at every position (for trees: at every
 * hidden row) -- the K paths then behave as K persistent heads, which is how Eq. 1 and the
 * per-head table of Sec. 3.1 can also be read.  Everything else is unchanged. */
int dm_set_mask_mode(dm_ctx* ctx, int mode);

/* Verify one chain of T draft tokens (sequence id 0): Eq. 1-3, per-path argmax, token counts,
 * acceptance scan.
 *   H[T,d]           hidden state whose head output predicts draft[t] (storage type of the head)
 *   draft[T]         draft token ids (ids outside [0,V) simply never match)
 *   K                paths per position, 1 <= K <= 1024;  p in [0,1): drop probability;  seed: Philox key
 *   rule             DM_RULE_NAIVE (Sec. 3.2 token matching) or DM_RULE_MAJORITY (Eq. 6)
 *   out_tokens[T,K]  argmax token of every path (ties: smallest id)
 *   out_counts[T,K]  out_counts[t,i] = number of paths i' with out_tokens[t,i'] == out_tokens[t,i]
 *   out_accept_len[1] number of leading accepted draft tokens, in [0,T] */
int dropmatch_verify(dm_ctx* ctx, const void* H, const int32_t* draft, int T, int K, float p,
                     uint64_t seed, int rule, int32_t* out_tokens, int32_t* out_counts,
                     int32_t* out_accept_len, void* stream);

/* B independent chains in one pass over W; sequence b has id seq_base + b.
 *   H[B,T,d], draft[B,T] -> out_tokens[B,T,K], out_counts[B,T,K], out_accept_len[B];
 *   out_draft_hits[B,T] (may be NULL) = number of paths whose token equals draft[b,t].
 * Equals B calls of dropmatch_verify with the matching sequence ids, bit for bit. */
int dropmatch_verify_batched(dm_ctx* ctx, const void* H, const int32_t* draft, int B, int T, int K,
                             float p, uint64_t seed, uint64_t seq_base, int rule,
                             int32_t* out_tokens, int32_t* out_counts, int32_t* out_draft_hits,
                             int32_t* out_accept_len, void* stream);

/* dropmatch_verify_batched with the sampling decode rule: Sec. 3.2 lets the per-path token be the
 * top-1 token "or" one selected by nucleus sampling, without giving parameters.  Here path i of
 * position t draws y from Softmax(l / temperature) by the Gumbel-max construction,
 *   y = argmax_v ( l[v] / temperature - log(-log(u[v])) ),   equal keys -> smaller id,
 * with u[v] = (n + 0.5) / 2^23, n = top 23 bits of word (v mod 4) of
 * Philox4x32-10(counter = (v/4, i + 2^31, t, s mod 2^32), key = seed): the same generator as the
 * masks, on counters the masks never use, so a call is reproducible from (seed, s, t, i) alone.
 *   temperature > 0;  top_p in (0,1]: the nucleus mass.
 * top_p = 1 (temperature sampling): the noise is generated in the epilogue of the head kernel (one
 * Philox call and two logarithms per logit); no logit is written to memory.
 * top_p < 1 (nucleus sampling): the nucleus is the tokens in order of decreasing
 * Softmax(l / temperature) (equal probabilities: increasing id) up to and including the one whose
 * cumulative probability reaches top_p, and the draw is restricted to it.  The cut needs all logits
 * of a path at once: the head kernel writes them to the buffer that dm_enable_js reserves (call it
 * first with room for B*T*K rows, else DM_EWORKSPACE), and a second kernel, one thread-block cluster per path,
 * finds the boundary by mass (fixed-point sums: the result does not depend on the order of
 * additions) and draws the token.  Sharded heads (dm_set_vocab_offset) are not supported here: the
 * nucleus is taken over this context's head.
 * Counts, per-position test and scan are unchanged; everything else as for dropmatch_verify_batched. */
int dropmatch_verify_batched_sampled(dm_ctx* ctx, const void* H, const int32_t* draft, int B, int T, int K,
                                     float p, uint64_t seed, uint64_t seq_base, int rule, float temperature,
                                     float top_p, int32_t* out_tokens, int32_t* out_counts,
                                     int32_t* out_draft_hits, int32_t* out_accept_len, void* stream);

/* dropmatch_verify_batched plus the token the engine emits after the accepted prefix.  Every
 * hidden row gets, in the same pass over W, one more path without dropout: the target model's own
 * greedy token (the paper does not say how DropMatch picks the correction or bonus token; this
 * is the choice of plain speculative decoding with greedy verification).
 *   H[B, T + bonus_row, d]   bonus_row = 1: one more hidden row per sequence, the state after the
 *                            last draft token, so that a fully accepted draft yields a bonus token
 *   draft[B,T]               as before; positions 0..T-1 are scanned
 *   out_tokens, out_counts   [B, T + bonus_row, K] (the extra row's paths are computed too)
 *   out_draft_hits           [B,T] or NULL
 *   out_plain_tokens         [B, T + bonus_row]: argmax of the undropped head per hidden row
 *   out_next_token[B]        out_plain_tokens[b, accept_len[b]], or -1 if that row does not exist
 * Counts B*(T+bonus_row)*(K+1) rows against max_rows of dm_set_head.  K <= 1023. */
int dropmatch_verify_batched_next(dm_ctx* ctx, const void* H, const int32_t* draft, int B, int T, int bonus_row,
                                  int K, float p, uint64_t seed, uint64_t seq_base, int rule,
                                  int32_t* out_tokens, int32_t* out_counts, int32_t* out_draft_hits,
                                  int32_t* out_accept_len, int32_t* out_plain_tokens, int32_t* out_next_token,
                                  void* stream);

/* Same as dropmatch_verify_batched, but H, draft and all outputs are HOST pointers (pinned or
 * pageable).  Pinned buffers (cudaHostAlloc, cudaHostRegister, torch pin_memory) are used where
 * they are: the first kernel of the call (the mask pass, or a small copy kernel) fetches the
 * inputs over the host link while the head kernel already streams W, and the results are
 * written by the device straight into the caller's arrays.  Pageable buffers go through the
 * context's own pinned buffers (one memcpy each way).  The call returns once every result is in
 * place: the block that finishes the call writes a word into host memory behind its results and
 * the host waits for that word (or, where several blocks finish the call, for `stream` to
 * drain), so the call's last kernel may still be retiring on `stream` for a few microseconds
 * after the return; work queued on `stream` afterwards is ordered behind it as usual.  Whether a pointer is pinned is
 * looked up once and remembered (the last eight pointers): do not unpin or free a buffer and
 * reuse its address as pageable memory without a dm_set_head in between.  Needs
 * B*T <= max_hidden_rows of dm_set_head; H_host 16-byte aligned.  out_draft_hits may be NULL. */
int dropmatch_verify_batched_host(dm_ctx* ctx, const void* H_host, const int32_t* draft_host, int B,
                                  int T, int K, float p, uint64_t seed, uint64_t seq_base, int rule,
                                  int32_t* out_tokens_host, int32_t* out_counts_host,
                                  int32_t* out_draft_hits_host, int32_t* out_accept_len_host,
                                  void* stream);

/* JS-divergence criterion (Sec. 3.2: Eq. 4, Eq. 5, Algorithm 1).  dm_enable_js reserves, after
 * dm_set_head, the buffers this criterion needs for calls of up to max_rows = B*T*K paths and
 * max_hidden_rows = B*T positions: fp32 logits of every path (max_rows * V * 4 bytes) and small
 * partial sums.  Allocates; synchronises the device; a later dm_set_head drops the buffers. */
int dm_enable_js(dm_ctx* ctx, int max_rows, int max_hidden_rows);

/* Chain verification under Algorithm 1: position t is accepted iff
 *   JS(phat_t || pbar_t) <= max_i JS(p_t^(i) || pbar_t)                         (Eq. 5), or
 *   draft[t] is the most frequent of the K path tokens                           (Eq. 6),
 * where p_t^(i) = Softmax(l_t^(i)), pbar_t = Softmax(mean_i l_t^(i)) (Eq. 4) and phat_t is the
 * draft model's distribution; then the left-to-right rule.  Natural logarithm; fp32 arithmetic
 * on fp32 logits.
 *   draft_prob[B,T,V]   device, fp32 probabilities of the draft model (used as given)
 *   out_js[B,T,K+1]     device, fp32: JS(p^(i) || pbar) for i < K, then JS(phat || pbar)
 *   out_js_ok[B,T]      device, 1 iff Eq. 5 holds (may be NULL)
 *   the rest            as for dropmatch_verify_batched
 * Needs dm_enable_js with room for the call, else DM_EWORKSPACE; B*T <= 65535, else
 * DM_EUNSUPPORTED (checked before anything is launched).  Only enqueues work. */
int dropmatch_verify_js(dm_ctx* ctx, const void* H, const int32_t* draft, const float* draft_prob, int B, int T,
                        int K, float p, uint64_t seed, uint64_t seq_base, int32_t* out_tokens,
                        int32_t* out_counts, float* out_js, int32_t* out_js_ok, int32_t* out_accept_len,
                        void* stream);

/* Vocabulary-sharded heads (the deployment of Sec. 4.1 is tensor-parallel: every GPU holds a
 * slice of the LM head).  A context whose head is rows [offset, offset+V) of the full head reports
 * global token ids after dm_set_vocab_offset(ctx, offset) (call it after dm_set_head; default 0).
 * The masks are keyed on indices only, so every shard draws the same masks without any exchange.
 *
 * dropmatch_partial_best runs Eq. 1-3 and the vocabulary reduction on this context's head and
 * writes one packed word per path, out_packed[B*T*K] (device): (ordered fp32 key of the best logit
 * << 32) | (2^32-1 - token id).  The elementwise maximum of such arrays from all shards is the
 * result for the full head (equal logits resolve to the smaller token id).
 *
 * dropmatch_finalize_packed takes n_parts such arrays back to back, packed[n_parts][B*T*K]
 * (device) -- the layout an all-gather over the shards produces -- merges them and runs the
 * histogram and the acceptance scan as dropmatch_verify_batched does.  Needs no head.
 * Both only enqueue work on `stream`. */
int dm_set_vocab_offset(dm_ctx* ctx, int offset);
int dropmatch_partial_best(dm_ctx* ctx, const void* H, int B, int T, int K, float p, uint64_t seed,
                           uint64_t seq_base, uint64_t* out_packed, void* stream);
int dropmatch_finalize_packed(dm_ctx* ctx, const uint64_t* packed, int n_parts, const int32_t* draft, int B, int T,
                              int K, int rule, int32_t* out_tokens, int32_t* out_counts, int32_t* out_draft_hits,
                              int32_t* out_accept_len, void* stream);

/* The paper has no counterpart to this entry point; it exists for the way the library gets
 * deployed.  Some hosts of this code cannot ask CUDA for device memory at the time they verify:
 * a serving process that hands all of HBM to its own pool at start-up (a later cudaMalloc fails
 * or eats into the KV cache), a latency-critical decode loop (cudaMalloc and cudaFree stall the
 * whole device), or a plug-in that is handed tensors but may not set up a context with a
 * workspace of its own.  For them this call does what dropmatch_verify_batched does on the
 * CUDA-core kernel family, for fp32 and bf16 heads alike, but needs no dm_ctx and never
 * allocates or frees: the per-slice partial argmaxes go to a fixed array inside the library
 * image (about 0.6 MB, held by every GPU that loads the library until the process exits).
 *   device           CUDA device of all the pointers (compute capability 10.x)
 *   W[V,d], dtype    the LM head, as for dm_set_head (device pointer, 16-byte aligned)
 *   the rest         as for dropmatch_verify_batched; out_draft_hits may be NULL
 * Limits and rules:
 *   - B*T*K <= DM_STATIC_MAX_ROWS, else DM_ESTATICLIMIT and nothing is launched.
 *   - The first call on a device looks the array's device address up (once per device and
 *     process).  With CUDA's lazy module loading that first call is also when the driver loads
 *     the code and sets the 0.6 MB array aside, which can fail (DM_ECUDA) once a pool owns all
 *     of the device's memory: make one call per device at start-up, before the pool takes the
 *     memory and before any stream capture begins.  The remembered address does not survive a
 *     cudaDeviceReset.
 *   - All calls on a device share the one array, which keeps the previous call's contents; the
 *     call itself clears the part that must start at zero.  Two calls whose kernels can overlap
 *     on the GPU (different streams, or host threads racing on one device) corrupt each other:
 *     issue them on one stream, or order them with events.
 *   - Only enqueues work on `stream`; results are ready when the stream reaches that point. */
#define DM_STATIC_MAX_ROWS 256
int dropmatch_verify_batched_static(int device, const void* W, int V, int d, int dtype, const void* H,
                                    const int32_t* draft, int B, int T, int K, float p, uint64_t seed,
                                    uint64_t seq_base, int rule, int32_t* out_tokens, int32_t* out_counts,
                                    int32_t* out_draft_hits, int32_t* out_accept_len, void* stream);

/* Draft trees (Sec. 4.4).  Per sequence: N_h hidden rows H[b,q,:] and N nodes in topological
 * order.  Node n has a token, a parent node (node_parent[n] < n; -1 = child of the committed
 * prefix) and node_hrow[n] in [0,N_h): the hidden row whose head output predicts it (children
 * of one parent share one row).  Paths of hidden row q use position index t = q in the mask key.
 *   node_ok[n] = (parent is the prefix or node_ok[parent]) and token[n] passes `rule` against the
 *                K tokens of row node_hrow[n];
 *   out_accept_len[b] = depth of the deepest ok node (0 if none);
 *   out_best_node[b]  = smallest-index ok node of that depth (-1 if none).
 *   out_tokens[B,N_h,K], out_counts[B,N_h,K]; out_node_ok[B,N] may be NULL.
 * Node arrays are not validated on the device beyond clamping out-of-range indices to "rejected". */
int dropmatch_verify_tree(dm_ctx* ctx, const void* H, const int32_t* node_token,
                          const int32_t* node_parent, const int32_t* node_hrow, int B, int N_h, int N,
                          int K, float p, uint64_t seed, uint64_t seq_base, int rule,
                          int32_t* out_tokens, int32_t* out_counts, int32_t* out_node_ok,
                          int32_t* out_best_node, int32_t* out_accept_len, void* stream);

/* dropmatch_verify_tree plus, in the same pass over W, the target's own greedy token of every
 * hidden row (one more path without dropout, as in dropmatch_verify_batched_next):
 * out_plain_tokens[B,N_h].  The token to emit after the accepted path is the entry of the hidden
 * row that the best node owns (the caller knows which row that is; it need not exist for a leaf).
 * Counts B*N_h*(K+1) rows against max_rows.  K <= 1023. */
int dropmatch_verify_tree_next(dm_ctx* ctx, const void* H, const int32_t* node_token, const int32_t* node_parent,
                               const int32_t* node_hrow, int B, int N_h, int N, int K, float p, uint64_t seed,
                               uint64_t seq_base, int rule, int32_t* out_tokens, int32_t* out_counts,
                               int32_t* out_node_ok, int32_t* out_best_node, int32_t* out_accept_len,
                               int32_t* out_plain_tokens, void* stream);

/* Debug: full logits (Eq. 3 with Eq. 2's scale) of selected paths, computed by the same kernel
 * family a verify call would use.  H[B,T,d]; row_sel[n_sel,3] holds (b, t, i) triples with
 * 0 <= b < B, 0 <= t < T, i >= 0 (checked on the device: a bad triple yields a row of NaN);
 * sequence b has id seq_base + b.  out_logits[n_sel,V] fp32.  1 <= n_sel <= max_rows. */
int dm_debug_logits(dm_ctx* ctx, const void* H, int B, int T, const int32_t* row_sel, int n_sel,
                    float p, uint64_t seed, uint64_t seq_base, float* out_logits, void* stream);

/* Debug: the keep masks of Eq. 1, bit-packed.  out_bits[B,T,K,ceil(d/32)]: bit (j mod 32) of
 * word j/32 is 1 iff element j is kept.  Needs no head. */
int dm_debug_masks(dm_ctx* ctx, int B, int T, int K, int d, float p, uint64_t seed,
                   uint64_t seq_base, uint32_t* out_bits, void* stream);

/* Debug: the masked hidden rows themselves (Eq. 1 and Eq. 2 without the 1/(1-p) factor), exactly
 * as the tensor-core kernel stages them for calls of more than 64 paths or so: out[B*T*K, d] in
 * the head's storage type, row (b*T+t)*K+i = H[b,t,:] with the dropped elements set to zero.
 * bf16 heads only (DM_EUNSUPPORTED otherwise); out is a device pointer, 16-byte aligned. */
int dm_debug_masked_operand(dm_ctx* ctx, const void* H, int B, int T, int K, float p, uint64_t seed,
                            uint64_t seq_base, void* out, void* stream);

/* Measurement aid: enqueues one read-only pass over `bytes` bytes at device pointer `ptr` (16-byte
 * aligned; the bytes beyond a multiple of 16 are not read).  Timed over a buffer much larger than
 * L2 it gives the read-only HBM rate of the part, the ceiling of any kernel that streams W. */
int dm_debug_read_stream(dm_ctx* ctx, const void* ptr, size_t bytes, void* stream);

/* Reads and clears the context's device error word (0 = none); synchronises `stream` first.
 * Non-zero means a kernel abandoned an internal wait.  The outputs of that call, and of every
 * later call until this function has cleared the word, are then the fail-safe values written on
 * the device, so that no consumer further down the stream mistakes them for results:
 * tokens -1, counts and hits 0, accepted length 0, best node -1, node_ok 0, plain/next tokens -1
 * (the left-to-right rule of Sec. 2 with nothing accepted). */
int dm_device_error(dm_ctx* ctx, void* stream, uint32_t* out_code);

/* Debug: how many clock cycles a kernel of this context waits on one of its internal barriers
 * before it gives up, sets the device error word and winds down (0 restores the default, about
 * one second; the time a call spends queued behind the kernel ahead of it counts).  A limit of
 * a few cycles makes the first wait that is not satisfied at once run out: the tests use that
 * to exercise the wind-down and the fail-safe outputs without hanging or faulting anything. */
int dm_debug_set_wait_limit(dm_ctx* ctx, uint64_t cycles);

/* Timing of the head kernel alone (the dominant kernel).  While enabled, every verify call
 * records a CUDA event on `stream` before and after its masked-head kernel launch(es) (not
 * around the finalize kernel); at most 4096 calls are kept between reads, later ones are not
 * recorded.  dm_profile_read waits for the recorded events, returns the summed elapsed time in
 * milliseconds and the number of calls it covers, and clears the record.  Creating the events
 * allocates driver resources, so enable it outside latency-critical code. */
int dm_profile_head(dm_ctx* ctx, int enable);
int dm_profile_read(dm_ctx* ctx, double* out_ms_total, int* out_calls);

/* Bytes of device workspace the context holds; which kernel family the last verify call used
 * (DM_IMPL_SIMT or DM_IMPL_TCGEN05, 0 before any call); kernels launched by the last call. */
size_t dm_workspace_bytes(const dm_ctx* ctx);
int dm_last_impl(const dm_ctx* ctx);
int dm_last_launches(const dm_ctx* ctx);

const char* dm_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* DROPMATCH_H_ */
