// dropmatch_verify_batched_static: the chain verification call for callers that may not
// allocate device memory.  Same kernels as the CUDA-core path of dropmatch_verify_batched
// (masked head with per-slice argmax, then merge / histogram / acceptance); the only difference
// is where the per-slice partial argmaxes live: in a fixed array that is part of the library
// image instead of a cudaMalloc'ed workspace owned by a context.
#include <math.h>
#include <mutex>

#include "dm_internal.h"

using namespace dm;

namespace {

// Largest call the fixed scratch array serves: rows = B*T*K paths.
constexpr int kStaticMaxRows = DM_STATIC_MAX_ROWS;
constexpr size_t kPartialBytes = (size_t)kSimtMaxSlices * kStaticMaxRows * sizeof(unsigned long long);
constexpr size_t kScratchBytes = kPartialBytes + 256;   // + one 256-byte line holding the error word
constexpr int kMaxDevices = 64;

// The scratch itself.  Every device that loads the library carries one copy (about 0.6 MB) from
// load to exit.  Layout: partial argmaxes [slice][rows of the call], then the error word.
// In host code this name is only a handle for cudaGetSymbolAddress, never a pointer to pass on.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

// Start-of-call reset of what must begin at zero: the error word (the partial argmaxes are
// overwritten in full by every call before they are read).  Device code may name the array.
__global__ void static_scratch_reset_kernel() {
    *reinterpret_cast<uint32_t*>(g_static_scratch + kPartialBytes) = 0u;
}

std::mutex g_setup_lock;
unsigned char* g_scratch_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device

// Device address of the scratch on `device`, which must be the current device.  The first call
// per device asks the runtime for it; later calls only read the cached value.
int scratch_address(int device, unsigned char** out) {
    if (device < 0 || device >= kMaxDevices) return DM_EINVAL;
    std::lock_guard<std::mutex> hold(g_setup_lock);
    if (g_scratch_addr[device] == nullptr) {
        unsigned char* addr = nullptr;
        if (cudaGetSymbolAddress((void**)&addr, g_static_scratch) != cudaSuccess || addr == nullptr) {
            cudaGetLastError();
            return DM_ECUDA;
        }
        g_scratch_addr[device] = addr;
    }
    *out = g_scratch_addr[device];
    return DM_OK;
}

}  // namespace

extern "C" int dropmatch_verify_batched_static(int device, const void* W, int V, int d, int dtype,
                                               const void* H, const int32_t* draft, int B, int T, int K,
                                               float p, uint64_t seed, uint64_t seq_base, int rule,
                                               int32_t* out_tokens, int32_t* out_counts,
                                               int32_t* out_draft_hits, int32_t* out_accept_len,
                                               void* stream) {
    if (W == nullptr || H == nullptr || draft == nullptr || out_tokens == nullptr || out_counts == nullptr ||
        out_accept_len == nullptr)
        return DM_EINVAL;
    if (dtype != DM_F32 && dtype != DM_BF16) return DM_EINVAL;
    if (rule != DM_RULE_NAIVE && rule != DM_RULE_MAJORITY) return DM_EINVAL;
    if (((reinterpret_cast<uintptr_t>(W) | reinterpret_cast<uintptr_t>(H)) & 15u) != 0) return DM_EINVAL;
    if (V < 1 || B < 1 || T < 1 || K < 1 || K > kMaxK) return DM_EINVAL;
    if (!(p >= 0.0f) || !(p < 1.0f)) return DM_EINVAL;
    const int vec = dtype == DM_F32 ? 4 : 8;
    if (d < 4 || d % vec != 0) return DM_EUNSUPPORTED;
    const long long rows = (long long)B * T * K;
    if (rows > kStaticMaxRows) return DM_ESTATICLIMIT;   // the fixed scratch cannot hold this call

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) { cudaGetLastError(); return DM_ECUDA; }
    if (prev != device && cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return DM_ECUDA; }
    int st = DM_OK;
    do {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) { st = DM_ECUDA; break; }
        if (major != 10) { st = DM_EDEVICE; break; }
        unsigned char* scratch = nullptr;
        st = scratch_address(device, &scratch);
        if (st != DM_OK) break;
        if (finalize_smem_bytes(T, K, 0) > 200 * 1024) { st = DM_EUNSUPPORTED; break; }
        unsigned long long* partials = reinterpret_cast<unsigned long long*>(scratch);
        uint32_t* err = reinterpret_cast<uint32_t*>(scratch + kPartialBytes);
        cudaStream_t s = static_cast<cudaStream_t>(stream);

        MaskKey mk;
        double scaled = floor((double)p * 4294967296.0);
        if (scaled > 4294967295.0) scaled = 4294967295.0;
        mk.thr = (uint32_t)scaled;
        mk.key0 = (uint32_t)seed;
        mk.key1 = (uint32_t)(seed >> 32);
        mk.scale = (float)(1.0 / (1.0 - (double)p));
        mk.sample = 0;
        mk.inv_temp = 1.0f;

        static_scratch_reset_kernel<<<1, 1, 0, s>>>();
        if (cudaGetLastError() != cudaSuccess) { st = DM_ECUDA; break; }
        HeadDesc head{W, V, d, dtype, 0};
        RowMap map{nullptr, K, T, B, (uint32_t)seq_base};
        int n_slices = 0;
        st = launch_simt(head, H, (int)rows, map, mk, &n_slices, partials, nullptr, err, s);
        if (st != DM_OK) break;
        FinalizeArgs fa{};
        fa.B = B; fa.T = T; fa.K = K; fa.rule = rule;
        fa.draft = draft; fa.out_hits = out_draft_hits;
        fa.N = 0;
        fa.out_tokens = out_tokens; fa.out_counts = out_counts; fa.out_accept_len = out_accept_len;
        fa.err = err;
        st = launch_finalize(partials, n_slices, (int)rows, fa, s);
    } while (false);
    if (st == DM_ECUDA) cudaGetLastError();
    if (prev != device) cudaSetDevice(prev);
    return st;
}
