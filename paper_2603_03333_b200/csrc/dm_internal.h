// Internal host-side declarations shared by the translation units of libdropmatch.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/dropmatch.h"
#include "dm_common.cuh"

namespace dm {

constexpr int kSimtMaxSlices = 296;   // vocabulary slices of the CUDA-core kernel
constexpr int kMaxSlices = 296;       // rows of the partial-argmax workspace
constexpr int kMaxK = 1024;

struct HeadDesc {
    const void* W;
    int V, d, dtype;
    int v_offset;   // added to every token id: first vocabulary row of this head within a sharded one
};

// Per-call mask parameters (Eq. 1, Eq. 2).
struct MaskKey {
    uint32_t key0, key1;  // Philox key = seed
    uint32_t thr;         // drop iff word < thr; thr = floor(p * 2^32)
    float scale;          // 1 / (1 - p)
    int sample;           // 0: argmax decode; 1: draw from Softmax(logits / temperature) by Gumbel-max
    float inv_temp;       // 1 / temperature (sample == 1)
};

// Acceptance inputs/outputs handed to the finalize kernel.
struct FinalizeArgs {
    int B, T, K, rule;     // T hidden rows per sequence, K dropout paths per row
    int plain;             // 1: every hidden row has one more, unmasked path after its K dropout paths
    int T_draft;           // draft positions scanned per sequence (0 = T); T - T_draft extra hidden rows
    int32_t* out_plain;    // [B,T] token of the unmasked path, or null
    int32_t* out_next;     // [B] unmasked token at position accept_len (-1 if there is no such row), or null
    // chain
    const int32_t* draft;        // [B,T] or null (tree)
    int32_t* out_hits;           // [B,T] or null
    // tree
    int N;                       // nodes per sequence (0 = chain)
    const int32_t* node_token;   // [B,N]
    const int32_t* node_parent;  // [B,N]
    const int32_t* node_hrow;    // [B,N]
    int32_t* out_node_ok;        // [B,N] or null
    int32_t* out_best_node;      // [B]
    // both
    int32_t* out_tokens;         // [B,T,K]
    int32_t* out_counts;         // [B,T,K]
    int32_t* out_accept_len;     // [B]
    // device error word of the call's context (or null): if it is set when the results are about to
    // be written, a kernel of the call gave up on a wait and the partial maxima mean nothing
    const uint32_t* err;
    // Host-buffer calls: a word in host memory that receives `done_value` once every result of the
    // call has been written (only when one block finishes the whole call), or null.
    uint32_t* done;
    uint32_t done_value;
};

// Reduce the per-slice partial argmaxes to one packed word per row (no histogram, no acceptance).
int launch_merge_partials(const unsigned long long* partials, int n_slices, int rows,
                          unsigned long long* out_packed, cudaStream_t stream);

int launch_simt(const HeadDesc& head, const void* H, int rows, const RowMap& map, const MaskKey& mk,
                int* n_slices_out, unsigned long long* partials, float* dbg_logits, uint32_t* err,
                cudaStream_t stream);

// Merge the per-slice partial argmaxes into tokens, count them, run the acceptance scan.
int launch_finalize(const unsigned long long* partials, int n_slices, int rows,
                    const FinalizeArgs& a, cudaStream_t stream);
size_t finalize_smem_bytes(int T, int K, int N);

// tcgen05 tensor-core kernel (bf16 heads).  FusedState owns the TMA descriptors.
struct FusedState;
bool fused_supported(const HeadDesc& head, int rows);
int fused_create(FusedState** out, const HeadDesc& head, int max_rows, int max_hidden_rows, size_t* bytes);
void fused_destroy(FusedState* fs);
// Inputs of a host-buffer call: where the device can read them (pinned host memory) and where
// the kernels of the call expect them (device staging).
struct HostInputs {
    const void* h_src;
    size_t h_bytes;
    const int32_t* draft_src;
    int n_draft;
    void* h_dst;
    int32_t* draft_dst;
};

int fused_launch(FusedState* fs, const HeadDesc& head, const void* H, int n_hidden, int rows,
                 const RowMap& map, const MaskKey& mk, int* n_slices_out, unsigned long long* partials,
                 float* dbg_logits, uint32_t* err, cudaStream_t stream, int* launches_out,
                 const FinalizeArgs* fin = nullptr, unsigned int* ticket = nullptr,
                 unsigned long long* best = nullptr, bool* folded_out = nullptr,
                 unsigned long long* packed_out = nullptr, long long wait_limit = 0, bool allow_pdl = true,
                 const HostInputs* host = nullptr, bool* best_reduced_out = nullptr);

// The staged masked operand of the tensor-core kernel (Eq. 1 and the numerator of Eq. 2), written to `out`.
int fused_debug_operand(const HeadDesc& head, const void* H, int rows, const RowMap& map, const MaskKey& mk,
                        void* out, uint32_t* err, cudaStream_t stream);

// Copy a call's inputs from device-readable host memory into the device staging buffer (a kernel, not a DMA copy).
int launch_host_gather(const void* src_h, size_t h_bytes, const int32_t* src_draft, int n_draft, void* dst_h,
                       int32_t* dst_draft, cudaStream_t stream);

int launch_read_stream(const void* ptr, size_t bytes, unsigned int* sink, int sms, cudaStream_t stream);

// JS-divergence acceptance (Eq. 4, Eq. 5, Algorithm 1) on logits [B*T*K][V] written by a head kernel.
int js_chunks(int V, int n_pos);
size_t js_workspace_floats(int V, int max_rows, int max_hidden);
size_t js_words_offset(int V, int max_rows, int max_hidden);       // where the ticket and counter words start (zero between calls)
constexpr int kJsMaxPositions = 65535;   // B*T of one JS call (a grid dimension)
int launch_js(const float* logits, const float* draft_prob, float* workspace, size_t words_offset, int max_hidden, int V, int B, int T,
              int K, const int32_t* tokens, const int32_t* draft, float* out_js, int32_t* out_js_ok,
              int32_t* out_accept_len, uint32_t* err, long long wait_limit, cudaStream_t stream, int* launches_out);

// Nucleus sampling on logits [rows][V] in global memory: one packed (key, inverted token id) word per path.
int launch_nucleus_sample(const float* logits, int V, int rows, const RowMap& map, const MaskKey& mk, float top_p,
                          int v_offset, unsigned long long* out_packed, cudaStream_t stream);

int launch_debug_masks(int B, int T, int K, int d, const MaskKey& mk, uint32_t seq_base_lo, int shared_masks,
                       uint32_t* out_bits, cudaStream_t stream);

}  // namespace dm
