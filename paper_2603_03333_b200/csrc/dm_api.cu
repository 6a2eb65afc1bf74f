// C ABI of libdropmatch: argument checks, workspace, kernel choice.  See include/dropmatch.h.
#include <math.h>
#include <string.h>
#include <atomic>
#include <new>
#include <vector>

#include "dm_internal.h"

using namespace dm;

struct dm_ctx {
    int device = 0;
    HeadDesc head{nullptr, 0, 0, 0, 0};
    bool has_head = false;
    int max_rows = 0, max_hidden = 0;
    int impl = DM_IMPL_AUTO;
    int mask_mode = DM_MASK_PER_POSITION;
    bool pdl = true;                         // head kernel launched with programmatic stream serialization (dm_set_pdl)
    long long wait_limit = 0;                // clock cycles a kernel waits on a barrier before it gives up; 0 = default
    int last_impl = 0, last_launches = 0;
    // workspace (device)
    unsigned long long* partials = nullptr;  // [kMaxSlices][max_rows]
    uint32_t* err = nullptr;                 // device error word
    // staging of the host-buffer entry point: one device buffer and one pinned host buffer with
    // the same layout, H then the draft tokens; and a pinned, device-mapped buffer that the
    // kernels write the results into (tokens | counts | hits | accept_len)
    unsigned char* stage_in = nullptr;       // device
    unsigned char* pin_in = nullptr;         // pinned host, mapped
    unsigned char* pin_in_dev = nullptr;     // the same memory as the device sees it
    int32_t* pin_out = nullptr;              // pinned host, mapped
    int32_t* pin_out_dev = nullptr;          // the same memory as the device sees it
    size_t done_off = 0;                     // the "results written" word of host-buffer calls: pin_out[done_off]
    uint32_t done_seq = 0;                   // its value for the latest host-buffer call
    const HostInputs* host_in = nullptr;     // set while a host-buffer call is being launched
    bool done_armed = false;                 // did the latest launch hand the word to a single finishing block?
    size_t ws_bytes = 0;
    // host pointers the host-buffer entry point has already looked up: device alias, or null if pageable
    struct HostAlias { const void* host = nullptr; void* dev = nullptr; };
    HostAlias aliases[8];
    int alias_next = 0;
    FusedState* fused = nullptr;             // tensor maps etc. of the tcgen05 kernel
    // JS criterion (dm_enable_js): logits of every path of a call, and the kernels' partial sums
    float* js_logits = nullptr;              // [js_max_rows][V]
    float* js_ws = nullptr;
    int js_max_rows = 0, js_max_hidden = 0;
    // optional timing of the head kernel alone (dm_profile_head)
    bool profile = false;
    std::vector<cudaEvent_t> prof_events;    // begin/end pairs, grown on demand
    size_t prof_used = 0;                    // events recorded since the last dm_profile_read
};

namespace {

constexpr size_t kMaxProfileEvents = 8192;

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        target = dev;
    }
    ~DeviceGuard() { if (prev >= 0 && prev != target) cudaSetDevice(prev); }
    int target = -1;
};

void free_workspace(dm_ctx* c) {
    cudaFree(c->partials); c->partials = nullptr;
    cudaFree(c->stage_in); c->stage_in = nullptr;
    cudaFreeHost(c->pin_in); c->pin_in = nullptr;
    c->pin_in_dev = nullptr;
    cudaFreeHost(c->pin_out); c->pin_out = nullptr;
    c->pin_out_dev = nullptr;
    if (c->fused) { fused_destroy(c->fused); c->fused = nullptr; }
    cudaFree(c->js_logits); c->js_logits = nullptr;
    cudaFree(c->js_ws); c->js_ws = nullptr;
    c->js_max_rows = c->js_max_hidden = 0;
    c->ws_bytes = 0;
}

// Device-side alias of a host pointer if the memory is pinned (page-locked and readable and writable by the
// device), else null.  Looked up once per pointer and remembered: the lookup costs about a microsecond.
void* device_alias(dm_ctx* c, const void* host) {
    for (const dm_ctx::HostAlias& a : c->aliases)
        if (a.host == host) return a.dev;
    cudaPointerAttributes attr{};
    void* dev = nullptr;
    if (cudaPointerGetAttributes(&attr, host) == cudaSuccess && attr.type == cudaMemoryTypeHost)
        dev = attr.devicePointer;
    cudaGetLastError();
    c->aliases[c->alias_next] = dm_ctx::HostAlias{host, dev};
    c->alias_next = (c->alias_next + 1) % 8;
    return dev;
}

bool make_mask_key(float p, uint64_t seed, MaskKey* mk) {
    if (!(p >= 0.0f) || !(p < 1.0f)) return false;
    double scaled = floor((double)p * 4294967296.0);
    if (scaled > 4294967295.0) scaled = 4294967295.0;
    mk->thr = (uint32_t)scaled;
    mk->key0 = (uint32_t)seed;
    mk->key1 = (uint32_t)(seed >> 32);
    mk->scale = (float)(1.0 / (1.0 - (double)p));
    mk->sample = 0;
    mk->inv_temp = 1.0f;
    return true;
}

// Which kernel family serves this head under the context's override?
int pick_impl(const dm_ctx* c, int rows, int* impl) {
    const bool tc_ok = c->fused != nullptr && fused_supported(c->head, rows);
    if (c->impl == DM_IMPL_TCGEN05) {
        if (!tc_ok) return DM_EUNSUPPORTED;
        *impl = DM_IMPL_TCGEN05;
    } else if (c->impl == DM_IMPL_SIMT) {
        *impl = DM_IMPL_SIMT;
    } else {
        *impl = tc_ok ? DM_IMPL_TCGEN05 : DM_IMPL_SIMT;
    }
    return DM_OK;
}

// Masked head + per-slice argmax for `rows` rows, then merge/histogram/acceptance.
int run_verify(dm_ctx* c, const void* H, int rows, const RowMap& map, const MaskKey& mk,
               const FinalizeArgs& fa_in, cudaStream_t stream, float* logits_out = nullptr) {
    FinalizeArgs fa = fa_in;
    fa.err = c->err;   // results are replaced by "nothing accepted" if a kernel of the call gives up on a wait
    const HostInputs* host = c->host_in;
    if (host != nullptr) {
        fa.done = reinterpret_cast<uint32_t*>(c->pin_out_dev + c->done_off);
        fa.done_value = c->done_seq;
    }
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return DM_ECUDA; }
    if (rows > c->max_rows) return DM_EWORKSPACE;
    if (finalize_smem_bytes(fa.T, fa.K + fa.plain, fa.N) > 200 * 1024) return DM_EUNSUPPORTED;
    int impl;
    int st = pick_impl(c, rows, &impl);
    if (st != DM_OK) return st;
    int n_slices = 0, launches = 0;
    cudaEvent_t ev_begin = nullptr, ev_end = nullptr;
    if (c->profile && c->prof_used + 2 <= kMaxProfileEvents) {
        while (c->prof_events.size() < c->prof_used + 2) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); return DM_ECUDA; }
            c->prof_events.push_back(e);
        }
        ev_begin = c->prof_events[c->prof_used];
        ev_end = c->prof_events[c->prof_used + 1];
        cudaEventRecord(ev_begin, stream);
    }
    bool folded = false, best_reduced = false;
    unsigned long long* best = c->partials + (size_t)kMaxSlices * c->max_rows;   // one word per path, zero between calls
    if (impl == DM_IMPL_TCGEN05)
        st = fused_launch(c->fused, c->head, H, fa.B * fa.T, rows, map, mk, &n_slices, c->partials,
                          logits_out, c->err, stream, &launches, &fa, c->err + 1, best, &folded, nullptr,
                          c->wait_limit, c->pdl, host, &best_reduced);
    else {
        if (host != nullptr) {
            st = launch_host_gather(host->h_src, host->h_bytes, host->draft_src, host->n_draft, host->h_dst,
                                    host->draft_dst, stream);
            if (st != DM_OK) return st;
            H = host->h_dst;
            ++launches;
        }
        st = launch_simt(c->head, H, rows, map, mk, &n_slices, c->partials, logits_out, c->err, stream);
        ++launches;
    }
    if (ev_end != nullptr) {
        cudaEventRecord(ev_end, stream);
        c->prof_used += 2;
    }
    if (st != DM_OK) return st;
    if (!folded) {   // calls of several launches, and the CUDA-core family, finish in a kernel of their own
        st = best_reduced ? launch_finalize(best, 1, rows, fa, stream) : launch_finalize(c->partials, n_slices, rows, fa, stream);
        if (st != DM_OK) return st;
        ++launches;
        if (best_reduced && cudaMemsetAsync(best, 0, (size_t)rows * sizeof(unsigned long long), stream) != cudaSuccess) {
            cudaGetLastError();
            return DM_ECUDA;
        }
    }
    c->done_armed = host != nullptr && (folded || fa.B == 1);   // one block finishes the call and writes the word
    c->last_impl = impl;
    c->last_launches = launches;
    return DM_OK;
}

int check_common(const dm_ctx* c, const void* H, int B, int T, int K) {
    if (c == nullptr || H == nullptr) return DM_EINVAL;
    if ((reinterpret_cast<uintptr_t>(H) & 15u) != 0) return DM_EINVAL;
    if (!c->has_head) return DM_ENOHEAD;
    if (B < 1 || T < 1 || K < 1 || K > kMaxK) return DM_EINVAL;
    if ((long long)B * T * K > 0x3FFFFFFFll) return DM_EINVAL;
    return DM_OK;
}

}  // namespace

extern "C" {

int dm_create(dm_ctx** out, int device) {
    if (out == nullptr) return DM_EINVAL;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess) { cudaGetLastError(); return DM_ECUDA; }
    if (device < 0 || device >= count) return DM_EINVAL;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) return DM_ECUDA;
    if (major != 10) return DM_EDEVICE;
    DeviceGuard g(device);
    if (!g.ok) return DM_ECUDA;
    dm_ctx* c = new (std::nothrow) dm_ctx();
    if (c == nullptr) return DM_ECUDA;
    c->device = device;
    // the device error word, the finished-CTA ticket of the fused kernel, a sink for dm_debug_read_stream
    if (cudaMalloc(&c->err, 4 * sizeof(uint32_t)) != cudaSuccess ||
        cudaMemset(c->err, 0, 4 * sizeof(uint32_t)) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(c->err);
        delete c;
        return DM_ECUDA;
    }
    *out = c;
    return DM_OK;
}

int dm_destroy(dm_ctx* c) {
    if (c == nullptr) return DM_OK;
    DeviceGuard g(c->device);
    cudaDeviceSynchronize();
    free_workspace(c);
    cudaFree(c->err);
    for (cudaEvent_t e : c->prof_events) cudaEventDestroy(e);
    cudaGetLastError();
    delete c;
    return DM_OK;
}

int dm_set_head(dm_ctx* c, const void* W, int V, int d, int dtype, int max_rows, int max_hidden_rows) {
    if (c == nullptr || W == nullptr) return DM_EINVAL;
    if (dtype != DM_F32 && dtype != DM_BF16) return DM_EINVAL;
    if (V < 1 || d < 1 || max_rows < 1 || max_hidden_rows < 1) return DM_EINVAL;
    if (max_rows > (1 << 24) || max_hidden_rows > max_rows) return DM_EINVAL;
    if ((reinterpret_cast<uintptr_t>(W) & 15u) != 0) return DM_EINVAL;
    const int vec = dtype == DM_F32 ? 4 : 8;
    if (d < 4 || d % vec != 0) return DM_EUNSUPPORTED;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return DM_ECUDA; }
    free_workspace(c);
    c->has_head = false;
    const size_t elem = dtype == DM_F32 ? 4 : 2;
    // per-slice partial argmaxes [kMaxSlices][max_rows], then the per-row running best [max_rows]
    // that the fused kernel's CTAs reduce into when one launch covers the call (zero between calls)
    const size_t n_part = ((size_t)kMaxSlices + 1) * max_rows * sizeof(unsigned long long);
    const size_t n_in = (size_t)max_hidden_rows * d * elem + 16 + (size_t)max_hidden_rows * sizeof(int32_t);
    c->done_off = (((size_t)2 * max_hidden_rows + 2 * (size_t)max_rows) + 15) & ~static_cast<size_t>(15);
    const size_t n_out = (c->done_off + 16) * sizeof(int32_t);
    void* out_dev = nullptr;
    void* in_dev = nullptr;
    if (cudaMalloc(&c->partials, n_part) != cudaSuccess || cudaMalloc(&c->stage_in, n_in) != cudaSuccess ||
        cudaHostAlloc(reinterpret_cast<void**>(&c->pin_in), n_in, cudaHostAllocMapped) != cudaSuccess ||
        cudaHostAlloc(reinterpret_cast<void**>(&c->pin_out), n_out, cudaHostAllocMapped) != cudaSuccess ||
        cudaHostGetDevicePointer(&out_dev, c->pin_out, 0) != cudaSuccess ||
        cudaHostGetDevicePointer(&in_dev, c->pin_in, 0) != cudaSuccess ||
        cudaMemset(c->partials + (size_t)kMaxSlices * max_rows, 0, (size_t)max_rows * sizeof(unsigned long long)) !=
            cudaSuccess) {
        cudaGetLastError();
        free_workspace(c);
        return DM_ECUDA;
    }
    c->pin_out_dev = static_cast<int32_t*>(out_dev);
    c->pin_out[c->done_off] = 0;
    c->done_seq = 0;
    c->pin_in_dev = static_cast<unsigned char*>(in_dev);
    for (dm_ctx::HostAlias& a : c->aliases) a = dm_ctx::HostAlias{};
    c->ws_bytes = n_part + n_in;
    c->head = HeadDesc{W, V, d, dtype, 0};
    c->max_rows = max_rows;
    c->max_hidden = max_hidden_rows;
    size_t fused_bytes = 0;
    int st = fused_create(&c->fused, c->head, max_rows, max_hidden_rows, &fused_bytes);
    if (st != DM_OK) { free_workspace(c); return st; }
    c->ws_bytes += fused_bytes;
    c->has_head = true;
    return DM_OK;
}

int dm_set_impl(dm_ctx* c, int impl) {
    if (c == nullptr || impl < DM_IMPL_AUTO || impl > DM_IMPL_TCGEN05) return DM_EINVAL;
    c->impl = impl;
    return DM_OK;
}

int dm_set_vocab_offset(dm_ctx* c, int offset) {
    if (c == nullptr) return DM_EINVAL;
    if (!c->has_head) return DM_ENOHEAD;
    if (offset < 0 || (long long)offset + c->head.V > 0x7FFFFFFFll) return DM_EINVAL;
    c->head.v_offset = offset;
    return DM_OK;
}

int dropmatch_partial_best(dm_ctx* c, const void* H, int B, int T, int K, float p, uint64_t seed,
                           uint64_t seq_base, uint64_t* out_packed, void* stream) {
    int st = check_common(c, H, B, T, K);
    if (st != DM_OK) return st;
    if (out_packed == nullptr) return DM_EINVAL;
    MaskKey mk;
    if (!make_mask_key(p, seed, &mk)) return DM_EINVAL;
    const int rows = B * T * K;
    if (rows > c->max_rows) return DM_EWORKSPACE;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return DM_ECUDA; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    RowMap map{nullptr, K, T, B, (uint32_t)seq_base, c->mask_mode};
    int impl;
    st = pick_impl(c, rows, &impl);
    if (st != DM_OK) return st;
    int n_slices = 0, launches = 1;
    bool reduced = false;
    unsigned long long* out = reinterpret_cast<unsigned long long*>(out_packed);
    if (impl == DM_IMPL_TCGEN05) {
        // A call of one launch: the CTAs reduce straight into the caller's array (zero first), no
        // second kernel.  Larger calls leave per-slice partials that a small kernel merges.
        if (cudaMemsetAsync(out, 0, (size_t)rows * sizeof(unsigned long long), s) != cudaSuccess) {
            cudaGetLastError();
            return DM_ECUDA;
        }
        st = fused_launch(c->fused, c->head, H, B * T, rows, map, mk, &n_slices, c->partials, nullptr, c->err, s,
                          &launches, nullptr, nullptr, nullptr, &reduced, out, c->wait_limit, c->pdl);
    } else {
        st = launch_simt(c->head, H, rows, map, mk, &n_slices, c->partials, nullptr, c->err, s);
    }
    if (st != DM_OK) return st;
    if (!reduced) {
        st = launch_merge_partials(c->partials, n_slices, rows, out, s);
        if (st != DM_OK) return st;
        ++launches;
    }
    c->last_impl = impl;
    c->last_launches = launches;
    return DM_OK;
}

int dropmatch_finalize_packed(dm_ctx* c, const uint64_t* packed, int n_parts, const int32_t* draft, int B, int T,
                              int K, int rule, int32_t* out_tokens, int32_t* out_counts, int32_t* out_draft_hits,
                              int32_t* out_accept_len, void* stream) {
    if (c == nullptr || packed == nullptr || draft == nullptr || out_tokens == nullptr || out_counts == nullptr ||
        out_accept_len == nullptr)
        return DM_EINVAL;
    if (n_parts < 1 || n_parts > 4096 || B < 1 || T < 1 || K < 1 || K > kMaxK) return DM_EINVAL;
    if ((long long)B * T * K > 0x3FFFFFFFll) return DM_EINVAL;
    if (rule != DM_RULE_NAIVE && rule != DM_RULE_MAJORITY) return DM_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    FinalizeArgs fa{};
    fa.B = B; fa.T = T; fa.K = K; fa.rule = rule;
    fa.draft = draft; fa.out_hits = out_draft_hits;
    fa.N = 0;
    fa.out_tokens = out_tokens; fa.out_counts = out_counts; fa.out_accept_len = out_accept_len;
    fa.err = c->err;
    return launch_finalize(reinterpret_cast<const unsigned long long*>(packed), n_parts, B * T * K, fa,
                           static_cast<cudaStream_t>(stream));
}

int dm_set_pdl(dm_ctx* c, int enable) {
    if (c == nullptr) return DM_EINVAL;
    c->pdl = enable != 0;
    return DM_OK;
}

int dm_debug_set_wait_limit(dm_ctx* c, uint64_t cycles) {
    if (c == nullptr || cycles > (1ull << 40)) return DM_EINVAL;
    c->wait_limit = (long long)cycles;
    return DM_OK;
}

int dm_set_mask_mode(dm_ctx* c, int mode) {
    if (c == nullptr || (mode != DM_MASK_PER_POSITION && mode != DM_MASK_PER_PATH)) return DM_EINVAL;
    c->mask_mode = mode;
    return DM_OK;
}

int dropmatch_verify_batched(dm_ctx* c, const void* H, const int32_t* draft, int B, int T, int K,
                             float p, uint64_t seed, uint64_t seq_base, int rule, int32_t* out_tokens,
                             int32_t* out_counts, int32_t* out_draft_hits, int32_t* out_accept_len,
                             void* stream) {
    int st = check_common(c, H, B, T, K);
    if (st != DM_OK) return st;
    if (draft == nullptr || out_tokens == nullptr || out_counts == nullptr || out_accept_len == nullptr)
        return DM_EINVAL;
    if (rule != DM_RULE_NAIVE && rule != DM_RULE_MAJORITY) return DM_EINVAL;
    MaskKey mk;
    if (!make_mask_key(p, seed, &mk)) return DM_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    RowMap map{nullptr, K, T, B, (uint32_t)seq_base, c->mask_mode};
    FinalizeArgs fa{};
    fa.B = B; fa.T = T; fa.K = K; fa.rule = rule;
    fa.draft = draft; fa.out_hits = out_draft_hits;
    fa.N = 0;
    fa.out_tokens = out_tokens; fa.out_counts = out_counts; fa.out_accept_len = out_accept_len;
    return run_verify(c, H, B * T * K, map, mk, fa, static_cast<cudaStream_t>(stream));
}

int dropmatch_verify_batched_sampled(dm_ctx* c, const void* H, const int32_t* draft, int B, int T, int K, float p,
                                     uint64_t seed, uint64_t seq_base, int rule, float temperature, float top_p,
                                     int32_t* out_tokens, int32_t* out_counts, int32_t* out_draft_hits,
                                     int32_t* out_accept_len, void* stream) {
    int st = check_common(c, H, B, T, K);
    if (st != DM_OK) return st;
    if (draft == nullptr || out_tokens == nullptr || out_counts == nullptr || out_accept_len == nullptr)
        return DM_EINVAL;
    if (rule != DM_RULE_NAIVE && rule != DM_RULE_MAJORITY) return DM_EINVAL;
    if (!(temperature > 0.0f) || !(temperature < 1e30f) || !(top_p > 0.0f) || !(top_p <= 1.0f)) return DM_EINVAL;
    MaskKey mk;
    if (!make_mask_key(p, seed, &mk)) return DM_EINVAL;
    mk.inv_temp = 1.0f / temperature;
    const int rows = B * T * K;
    if (top_p < 1.0f && (c->js_logits == nullptr || rows > c->js_max_rows)) return DM_EWORKSPACE;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    RowMap map{nullptr, K, T, B, (uint32_t)seq_base, c->mask_mode};
    FinalizeArgs fa{};
    fa.B = B; fa.T = T; fa.K = K; fa.rule = rule;
    fa.draft = draft; fa.out_hits = out_draft_hits;
    fa.N = 0;
    fa.out_tokens = out_tokens; fa.out_counts = out_counts; fa.out_accept_len = out_accept_len;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (top_p >= 1.0f) {   // temperature sampling: Gumbel-max in the epilogue of the head kernel, no logits in memory
        mk.sample = 1;
        return run_verify(c, H, rows, map, mk, fa, s);
    }
    // Nucleus: the cut needs all logits of a path at once.  The head kernel writes them to the
    // context's logits buffer (its own argmax is not used), one cluster of blocks per path finds the nucleus
    // and draws the token, the finalize kernel does the rest.
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return DM_ECUDA; }
    if (rows > c->max_rows) return DM_EWORKSPACE;
    int impl;
    st = pick_impl(c, rows, &impl);
    if (st != DM_OK) return st;
    int n_slices = 0, launches = 1;
    if (impl == DM_IMPL_TCGEN05)
        st = fused_launch(c->fused, c->head, H, B * T, rows, map, mk, &n_slices, c->partials, c->js_logits, c->err, s,
                          &launches, nullptr, nullptr, nullptr, nullptr, nullptr, c->wait_limit, c->pdl);
    else
        st = launch_simt(c->head, H, rows, map, mk, &n_slices, c->partials, c->js_logits, c->err, s);
    if (st != DM_OK) return st;
    unsigned long long* packed = c->partials;   // the per-slice partials are not needed: reuse their first row
    st = launch_nucleus_sample(c->js_logits, c->head.V, rows, map, mk, top_p, c->head.v_offset, packed, s);
    if (st != DM_OK) return st;
    fa.err = c->err;
    st = launch_finalize(packed, 1, rows, fa, s);
    if (st != DM_OK) return st;
    c->last_impl = impl;
    c->last_launches = launches + 2;
    return DM_OK;
}

int dropmatch_verify_batched_next(dm_ctx* c, const void* H, const int32_t* draft, int B, int T, int bonus_row,
                                  int K, float p, uint64_t seed, uint64_t seq_base, int rule,
                                  int32_t* out_tokens, int32_t* out_counts, int32_t* out_draft_hits,
                                  int32_t* out_accept_len, int32_t* out_plain_tokens, int32_t* out_next_token,
                                  void* stream) {
    if (bonus_row != 0 && bonus_row != 1) return DM_EINVAL;
    const int T_h = T + bonus_row;   // hidden rows per sequence
    int st = check_common(c, H, B, T_h, K);
    if (st != DM_OK) return st;
    if (T < 1 || K + 1 > kMaxK) return DM_EINVAL;
    if (draft == nullptr || out_tokens == nullptr || out_counts == nullptr || out_accept_len == nullptr ||
        out_plain_tokens == nullptr || out_next_token == nullptr)
        return DM_EINVAL;
    if (rule != DM_RULE_NAIVE && rule != DM_RULE_MAJORITY) return DM_EINVAL;
    if ((long long)B * T_h * (K + 1) > 0x3FFFFFFFll) return DM_EINVAL;
    MaskKey mk;
    if (!make_mask_key(p, seed, &mk)) return DM_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    RowMap map{nullptr, K, T_h, B, (uint32_t)seq_base, c->mask_mode, 1};
    FinalizeArgs fa{};
    fa.B = B; fa.T = T_h; fa.K = K; fa.rule = rule;
    fa.plain = 1; fa.T_draft = T;
    fa.out_plain = out_plain_tokens; fa.out_next = out_next_token;
    fa.draft = draft; fa.out_hits = out_draft_hits;
    fa.N = 0;
    fa.out_tokens = out_tokens; fa.out_counts = out_counts; fa.out_accept_len = out_accept_len;
    return run_verify(c, H, B * T_h * (K + 1), map, mk, fa, static_cast<cudaStream_t>(stream));
}

int dropmatch_verify(dm_ctx* c, const void* H, const int32_t* draft, int T, int K, float p,
                     uint64_t seed, int rule, int32_t* out_tokens, int32_t* out_counts,
                     int32_t* out_accept_len, void* stream) {
    return dropmatch_verify_batched(c, H, draft, 1, T, K, p, seed, 0, rule, out_tokens, out_counts,
                                    nullptr, out_accept_len, stream);
}

int dropmatch_verify_batched_host(dm_ctx* c, const void* H_host, const int32_t* draft_host, int B, int T,
                                  int K, float p, uint64_t seed, uint64_t seq_base, int rule,
                                  int32_t* out_tokens_host, int32_t* out_counts_host,
                                  int32_t* out_draft_hits_host, int32_t* out_accept_len_host,
                                  void* stream) {
    int st = check_common(c, H_host, B, T, K);
    if (st != DM_OK) return st;
    if (draft_host == nullptr || out_tokens_host == nullptr || out_counts_host == nullptr ||
        out_accept_len_host == nullptr)
        return DM_EINVAL;
    const long long hidden = (long long)B * T, rows = hidden * K;
    if (hidden > c->max_hidden || rows > c->max_rows) return DM_EWORKSPACE;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t elem = c->head.dtype == DM_F32 ? 4 : 2;
    const size_t h_bytes = (size_t)hidden * c->head.d * elem;
    const size_t draft_off = (h_bytes + 15) & ~static_cast<size_t>(15);
    // Inputs.  Pinned caller buffers are read by the device where they are; pageable ones are
    // first gathered in the context's pinned buffer.  A small kernel then brings them over the
    // host link into the device staging buffer while the head kernel already streams W.
    const void* h_src = device_alias(c, H_host);
    const void* d_src = device_alias(c, draft_host);
    if (h_src == nullptr) {
        memcpy(c->pin_in, H_host, h_bytes);
        h_src = c->pin_in_dev;
    }
    if (d_src == nullptr) {
        memcpy(c->pin_in + draft_off, draft_host, (size_t)hidden * sizeof(int32_t));
        d_src = c->pin_in_dev + draft_off;
    }
    int32_t* draft_dev = reinterpret_cast<int32_t*>(c->stage_in + draft_off);
    const HostInputs host{h_src, h_bytes, static_cast<const int32_t*>(d_src), (int)hidden, c->stage_in, draft_dev};
    // Outputs.  The kernels write them into host memory the device can reach (a few hundred bytes
    // crossing to the host), so that no device-to-host copy is queued behind the call: straight into
    // the caller's arrays if those are pinned, else into the context's mapped buffer.
    int32_t* o_tok = static_cast<int32_t*>(device_alias(c, out_tokens_host));
    int32_t* o_cnt = static_cast<int32_t*>(device_alias(c, out_counts_host));
    int32_t* o_len = static_cast<int32_t*>(device_alias(c, out_accept_len_host));
    int32_t* o_hits = out_draft_hits_host ? static_cast<int32_t*>(device_alias(c, out_draft_hits_host)) : nullptr;
    int32_t* d_out = c->pin_out_dev;
    c->host_in = &host;   // the first kernel of the call fetches the inputs
    ++c->done_seq;
    c->done_armed = false;
    st = dropmatch_verify_batched(c, c->stage_in, draft_dev, B, T, K, p, seed, seq_base, rule,
                                  o_tok ? o_tok : d_out, o_cnt ? o_cnt : d_out + rows,
                                  o_hits ? o_hits : d_out + 2 * rows, o_len ? o_len : d_out + 2 * rows + hidden, stream);
    c->host_in = nullptr;
    if (st != DM_OK) return st;
    // The block that finishes the call writes a word into host memory behind the results: poll it
    // rather than wait for the stream to report the kernel retired.  The stream is asked now and
    // then all the same, so that a launch that failed, or a call whose end no single block sees,
    // ends the loop too.
    bool seen = false;
    if (c->done_armed) {
        const volatile uint32_t* word = reinterpret_cast<const volatile uint32_t*>(c->pin_out + c->done_off);
        for (unsigned spins = 1;; ++spins) {
            if (*word == c->done_seq) { seen = true; break; }
            if ((spins & 2047u) == 0) {
                if (cudaStreamQuery(s) != cudaErrorNotReady) break;
                cudaGetLastError();   // "not ready" is no error: do not leave it for the next call to find
            }
#if defined(__x86_64__)
            __builtin_ia32_pause();
#endif
        }
        std::atomic_thread_fence(std::memory_order_acquire);
    }
    if (!seen && cudaStreamSynchronize(s) != cudaSuccess) { cudaGetLastError(); return DM_ECUDA; }
    if (!o_tok) memcpy(out_tokens_host, c->pin_out, (size_t)rows * sizeof(int32_t));
    if (!o_cnt) memcpy(out_counts_host, c->pin_out + rows, (size_t)rows * sizeof(int32_t));
    if (!o_len) memcpy(out_accept_len_host, c->pin_out + 2 * rows + hidden, (size_t)B * sizeof(int32_t));
    if (out_draft_hits_host && !o_hits) memcpy(out_draft_hits_host, c->pin_out + 2 * rows, (size_t)hidden * sizeof(int32_t));
    return DM_OK;
}

int dm_enable_js(dm_ctx* c, int max_rows, int max_hidden_rows) {
    if (c == nullptr) return DM_EINVAL;
    if (!c->has_head) return DM_ENOHEAD;
    if (max_rows < 1 || max_hidden_rows < 1 || max_rows > c->max_rows || max_hidden_rows > max_rows) return DM_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return DM_ECUDA; }
    cudaFree(c->js_logits); c->js_logits = nullptr;
    cudaFree(c->js_ws); c->js_ws = nullptr;
    c->js_max_rows = c->js_max_hidden = 0;
    const size_t n_logits = (size_t)max_rows * c->head.V * sizeof(float);
    const size_t n_ws = js_workspace_floats(c->head.V, max_rows, max_hidden_rows) * sizeof(float);
    if (cudaMalloc(&c->js_logits, n_logits) != cudaSuccess || cudaMalloc(&c->js_ws, n_ws) != cudaSuccess ||
        cudaMemset(c->js_ws, 0, n_ws) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(c->js_logits); c->js_logits = nullptr;
        cudaFree(c->js_ws); c->js_ws = nullptr;
        return DM_ECUDA;
    }
    c->js_max_rows = max_rows;
    c->js_max_hidden = max_hidden_rows;
    c->ws_bytes += n_logits + n_ws;
    return DM_OK;
}

int dropmatch_verify_js(dm_ctx* c, const void* H, const int32_t* draft, const float* draft_prob, int B, int T,
                        int K, float p, uint64_t seed, uint64_t seq_base, int32_t* out_tokens,
                        int32_t* out_counts, float* out_js, int32_t* out_js_ok, int32_t* out_accept_len,
                        void* stream) {
    int st = check_common(c, H, B, T, K);
    if (st != DM_OK) return st;
    if (draft == nullptr || draft_prob == nullptr || out_tokens == nullptr || out_counts == nullptr ||
        out_js == nullptr || out_accept_len == nullptr)
        return DM_EINVAL;
    const long long hidden = (long long)B * T, rows = hidden * K;
    if (hidden > kJsMaxPositions) return DM_EUNSUPPORTED;   // before anything is launched or overwritten
    if (c->js_logits == nullptr || rows > c->js_max_rows || hidden > c->js_max_hidden) return DM_EWORKSPACE;
    MaskKey mk;
    if (!make_mask_key(p, seed, &mk)) return DM_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the ordinary call (tokens, counts; its own accepted length is the majority rule's and is
    // overwritten below) with every logit of every path kept in the context's buffer
    RowMap map{nullptr, K, T, B, (uint32_t)seq_base, c->mask_mode};
    FinalizeArgs fa{};
    fa.B = B; fa.T = T; fa.K = K; fa.rule = DM_RULE_MAJORITY;
    fa.draft = draft; fa.out_hits = nullptr;
    fa.N = 0;
    fa.out_tokens = out_tokens; fa.out_counts = out_counts; fa.out_accept_len = out_accept_len;
    st = run_verify(c, H, (int)rows, map, mk, fa, s, c->js_logits);
    if (st != DM_OK) return st;
    int js_launches = 0;
    st = launch_js(c->js_logits, draft_prob, c->js_ws, js_words_offset(c->head.V, c->js_max_rows, c->js_max_hidden),
                   c->js_max_hidden, c->head.V, B, T, K, out_tokens, draft, out_js, out_js_ok, out_accept_len, c->err, c->wait_limit, s,
                   &js_launches);
    if (st != DM_OK) return st;
    c->last_launches += js_launches;
    return DM_OK;
}

int dropmatch_verify_tree(dm_ctx* c, const void* H, const int32_t* node_token, const int32_t* node_parent,
                          const int32_t* node_hrow, int B, int N_h, int N, int K, float p, uint64_t seed,
                          uint64_t seq_base, int rule, int32_t* out_tokens, int32_t* out_counts,
                          int32_t* out_node_ok, int32_t* out_best_node, int32_t* out_accept_len,
                          void* stream) {
    int st = check_common(c, H, B, N_h, K);
    if (st != DM_OK) return st;
    if (N < 1 || N > (1 << 20)) return DM_EINVAL;
    if (node_token == nullptr || node_parent == nullptr || node_hrow == nullptr || out_tokens == nullptr ||
        out_counts == nullptr || out_best_node == nullptr || out_accept_len == nullptr)
        return DM_EINVAL;
    if (rule != DM_RULE_NAIVE && rule != DM_RULE_MAJORITY) return DM_EINVAL;
    MaskKey mk;
    if (!make_mask_key(p, seed, &mk)) return DM_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    RowMap map{nullptr, K, N_h, B, (uint32_t)seq_base, c->mask_mode};
    FinalizeArgs fa{};
    fa.B = B; fa.T = N_h; fa.K = K; fa.rule = rule;
    fa.N = N; fa.node_token = node_token; fa.node_parent = node_parent; fa.node_hrow = node_hrow;
    fa.out_node_ok = out_node_ok; fa.out_best_node = out_best_node;
    fa.out_tokens = out_tokens; fa.out_counts = out_counts; fa.out_accept_len = out_accept_len;
    return run_verify(c, H, B * N_h * K, map, mk, fa, static_cast<cudaStream_t>(stream));
}

int dropmatch_verify_tree_next(dm_ctx* c, const void* H, const int32_t* node_token, const int32_t* node_parent,
                               const int32_t* node_hrow, int B, int N_h, int N, int K, float p, uint64_t seed,
                               uint64_t seq_base, int rule, int32_t* out_tokens, int32_t* out_counts,
                               int32_t* out_node_ok, int32_t* out_best_node, int32_t* out_accept_len,
                               int32_t* out_plain_tokens, void* stream) {
    int st = check_common(c, H, B, N_h, K);
    if (st != DM_OK) return st;
    if (N < 1 || N > (1 << 20) || K + 1 > kMaxK) return DM_EINVAL;
    if (node_token == nullptr || node_parent == nullptr || node_hrow == nullptr || out_tokens == nullptr ||
        out_counts == nullptr || out_best_node == nullptr || out_accept_len == nullptr || out_plain_tokens == nullptr)
        return DM_EINVAL;
    if (rule != DM_RULE_NAIVE && rule != DM_RULE_MAJORITY) return DM_EINVAL;
    if ((long long)B * N_h * (K + 1) > 0x3FFFFFFFll) return DM_EINVAL;
    MaskKey mk;
    if (!make_mask_key(p, seed, &mk)) return DM_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    RowMap map{nullptr, K, N_h, B, (uint32_t)seq_base, c->mask_mode, 1};
    FinalizeArgs fa{};
    fa.B = B; fa.T = N_h; fa.K = K; fa.rule = rule;
    fa.plain = 1; fa.out_plain = out_plain_tokens;
    fa.N = N; fa.node_token = node_token; fa.node_parent = node_parent; fa.node_hrow = node_hrow;
    fa.out_node_ok = out_node_ok; fa.out_best_node = out_best_node;
    fa.out_tokens = out_tokens; fa.out_counts = out_counts; fa.out_accept_len = out_accept_len;
    return run_verify(c, H, B * N_h * (K + 1), map, mk, fa, static_cast<cudaStream_t>(stream));
}

int dm_debug_logits(dm_ctx* c, const void* H, int B, int T, const int32_t* row_sel, int n_sel, float p,
                    uint64_t seed, uint64_t seq_base, float* out_logits, void* stream) {
    if (c == nullptr || H == nullptr || row_sel == nullptr || out_logits == nullptr) return DM_EINVAL;
    if ((reinterpret_cast<uintptr_t>(H) & 15u) != 0) return DM_EINVAL;
    if (!c->has_head) return DM_ENOHEAD;
    if (B < 1 || T < 1 || n_sel < 1) return DM_EINVAL;
    if (n_sel > c->max_rows) return DM_EWORKSPACE;
    MaskKey mk;
    if (!make_mask_key(p, seed, &mk)) return DM_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return DM_ECUDA; }
    RowMap map{row_sel, 1, T, B, (uint32_t)seq_base, c->mask_mode};
    int impl;
    int st = pick_impl(c, n_sel, &impl);
    if (st != DM_OK) return st;
    int n_slices = 0, launches = 1;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (impl == DM_IMPL_TCGEN05)
        st = fused_launch(c->fused, c->head, H, B * T, n_sel, map, mk, &n_slices, c->partials, out_logits,
                          c->err, s, &launches);
    else
        st = launch_simt(c->head, H, n_sel, map, mk, &n_slices, c->partials, out_logits, c->err, s);
    if (st != DM_OK) return st;
    c->last_impl = impl;
    c->last_launches = launches;
    return DM_OK;
}

int dm_debug_masks(dm_ctx* c, int B, int T, int K, int d, float p, uint64_t seed, uint64_t seq_base,
                   uint32_t* out_bits, void* stream) {
    if (c == nullptr || out_bits == nullptr) return DM_EINVAL;
    if (B < 1 || T < 1 || K < 1 || d < 1) return DM_EINVAL;
    if ((long long)B * T * K > 0x3FFFFFFFll) return DM_EINVAL;
    MaskKey mk;
    if (!make_mask_key(p, seed, &mk)) return DM_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    return launch_debug_masks(B, T, K, d, mk, (uint32_t)seq_base, c->mask_mode, out_bits, static_cast<cudaStream_t>(stream));
}

int dm_debug_masked_operand(dm_ctx* c, const void* H, int B, int T, int K, float p, uint64_t seed,
                            uint64_t seq_base, void* out, void* stream) {
    int st = check_common(c, H, B, T, K);
    if (st != DM_OK) return st;
    if (out == nullptr || (reinterpret_cast<uintptr_t>(out) & 15u) != 0) return DM_EINVAL;
    MaskKey mk;
    if (!make_mask_key(p, seed, &mk)) return DM_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    RowMap map{nullptr, K, T, B, (uint32_t)seq_base, c->mask_mode};
    return fused_debug_operand(c->head, H, B * T * K, map, mk, out, c->err, static_cast<cudaStream_t>(stream));
}

int dm_debug_read_stream(dm_ctx* c, const void* ptr, size_t bytes, void* stream) {
    if (c == nullptr || ptr == nullptr || bytes < 16 || (reinterpret_cast<uintptr_t>(ptr) & 15u) != 0) return DM_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess) return DM_ECUDA;
    // the sink is the ticket word's neighbour: it is only ever written with a value nobody reads
    return launch_read_stream(ptr, bytes, c->err + 2, sms, static_cast<cudaStream_t>(stream));
}

int dm_device_error(dm_ctx* c, void* stream, uint32_t* out_code) {
    if (c == nullptr || out_code == nullptr) return DM_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint32_t code = 0;
    if (cudaMemcpyAsync(&code, c->err, sizeof code, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaMemsetAsync(c->err, 0, 2 * sizeof code, s) != cudaSuccess || cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return DM_ECUDA;
    }
    if (code != 0 && c->partials != nullptr) {   // a call that gave up may have left partial maxima behind
        if (cudaMemsetAsync(c->partials + (size_t)kMaxSlices * c->max_rows, 0,
                            (size_t)c->max_rows * sizeof(unsigned long long), s) != cudaSuccess ||
            cudaStreamSynchronize(s) != cudaSuccess) {
            cudaGetLastError();
            return DM_ECUDA;
        }
    }
    *out_code = code;
    return DM_OK;
}

int dm_profile_head(dm_ctx* c, int enable) {
    if (c == nullptr) return DM_EINVAL;
    c->profile = enable != 0;
    return DM_OK;
}

int dm_profile_read(dm_ctx* c, double* out_ms_total, int* out_calls) {
    if (c == nullptr || out_ms_total == nullptr || out_calls == nullptr) return DM_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return DM_ECUDA;
    double total = 0.0;
    int calls = 0;
    for (size_t n = 0; n + 1 < c->prof_used; n += 2) {
        float ms = 0.0f;
        if (cudaEventSynchronize(c->prof_events[n + 1]) != cudaSuccess ||
            cudaEventElapsedTime(&ms, c->prof_events[n], c->prof_events[n + 1]) != cudaSuccess) {
            cudaGetLastError();
            c->prof_used = 0;
            return DM_ECUDA;
        }
        total += ms;
        ++calls;
    }
    c->prof_used = 0;
    *out_ms_total = total;
    *out_calls = calls;
    return DM_OK;
}

size_t dm_workspace_bytes(const dm_ctx* c) { return c ? c->ws_bytes : 0; }
int dm_last_impl(const dm_ctx* c) { return c ? c->last_impl : 0; }
int dm_last_launches(const dm_ctx* c) { return c ? c->last_launches : 0; }

const char* dm_strerror(int status) {
    switch (status) {
        case DM_OK: return "ok";
        case DM_EINVAL: return "invalid argument";
        case DM_EUNSUPPORTED: return "unsupported shape";
        case DM_ECUDA: return "CUDA error";
        case DM_EWORKSPACE: return "call exceeds the rows reserved by dm_set_head";
        case DM_EDEVICE: return "device is not compute capability 10.x";
        case DM_ENOHEAD: return "dm_set_head has not been called";
        case DM_ESTATICLIMIT: return "call exceeds the fixed scratch of dropmatch_verify_batched_static";
        default: return "unknown status";
    }
}

}  // extern "C"
