// Split-V merge, token histogram and acceptance (Sec. 3.2: naive token matching, Eq. 6
// majority; left-to-right rule; tree drafts of Sec. 4.4), plus the debug mask dump (Eq. 1).
// One block per sequence; everything after the merge is integer work on <= T*K tokens.
#include "dm_finalize.cuh"

namespace dm {

__global__ void __launch_bounds__(256)
finalize_kernel(const unsigned long long* __restrict__ partials, int n_slices, int rows, FinalizeArgs a) {
    extern __shared__ int32_t sm[];
    finalize_sequence(partials, n_slices, rows, a, (int)blockIdx.x, sm, (int)threadIdx.x, (int)blockDim.x, BlockSync{});
    if (a.done != nullptr && gridDim.x == 1) {   // one block wrote every result: tell the waiting host
        __threadfence_system();
        __syncthreads();
        if (threadIdx.x == 0) *reinterpret_cast<volatile uint32_t*>(a.done) = a.done_value;
    }
}

// One packed word per row: the maximum over the slices (argmax with the smallest index on ties).
__global__ void __launch_bounds__(256)
merge_partials_kernel(const unsigned long long* __restrict__ partials, int n_slices, int rows,
                      unsigned long long* __restrict__ out_packed) {
    const int warp = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
    const int x0 = warp * 4;   // four rows per warp: their loads overlap
    if (x0 >= rows) return;
    unsigned long long best[4] = {0ull, 0ull, 0ull, 0ull};
    for (int s = lane; s < n_slices; s += 32)
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (x0 + u < rows) {
                unsigned long long c = __ldcg(partials + (size_t)s * rows + x0 + u);
                best[u] = c > best[u] ? c : best[u];
            }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, best[u], off);
            best[u] = o > best[u] ? o : best[u];
        }
        if (lane == 0 && x0 + u < rows) out_packed[x0 + u] = best[u];
    }
}

int launch_merge_partials(const unsigned long long* partials, int n_slices, int rows,
                          unsigned long long* out_packed, cudaStream_t stream) {
    const int warps = (rows + 3) / 4;
    merge_partials_kernel<<<(warps * 32 + 255) / 256, 256, 0, stream>>>(partials, n_slices, rows, out_packed);
    return cudaGetLastError() == cudaSuccess ? DM_OK : DM_ECUDA;
}

size_t finalize_smem_bytes(int T, int K, int N) { return finalize_smem_bytes_dev(T, K, N); }

int launch_finalize(const unsigned long long* partials, int n_slices, int rows,
                    const FinalizeArgs& a, cudaStream_t stream) {
    const size_t smem = finalize_smem_bytes(a.T, a.K + a.plain, a.N);   // the scratch keeps the unmasked path too
    if (smem > 200 * 1024) return DM_EUNSUPPORTED;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(finalize_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return DM_ECUDA;
    finalize_kernel<<<a.B, 256, smem, stream>>>(partials, n_slices, rows, a);
    return cudaGetLastError() == cudaSuccess ? DM_OK : DM_ECUDA;
}

// Host-buffer entry point: fetch a call's inputs (a few tens of KB) from pinned host memory that
// the device can read and put them where the head kernel expects them.  The head kernel behind
// this one may be scheduled at once: it streams W until its builders need H, and they wait for
// this kernel to finish, so the trip over the host link hides behind the fill of the W ring.
__global__ void __launch_bounds__(256)
host_gather_kernel(const uint4* __restrict__ src_h, size_t n16, const int32_t* __restrict__ src_draft, int n_draft,
                   uint4* __restrict__ dst_h, int32_t* __restrict__ dst_draft) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t x = (size_t)blockIdx.x * blockDim.x + threadIdx.x; x < n16; x += stride) dst_h[x] = src_h[x];
    for (size_t x = (size_t)blockIdx.x * blockDim.x + threadIdx.x; x < (size_t)n_draft; x += stride)
        dst_draft[x] = src_draft[x];
}

int launch_host_gather(const void* src_h, size_t h_bytes, const int32_t* src_draft, int n_draft, void* dst_h,
                       int32_t* dst_draft, cudaStream_t stream) {
    const size_t n16 = h_bytes / 16;
    size_t blocks = (n16 + 255) / 256;
    if (blocks < 1) blocks = 1;
    if (blocks > 592) blocks = 592;
    host_gather_kernel<<<(unsigned)blocks, 256, 0, stream>>>(static_cast<const uint4*>(src_h), n16, src_draft, n_draft,
                                                           static_cast<uint4*>(dst_h), dst_draft);
    return cudaGetLastError() == cudaSuccess ? DM_OK : DM_ECUDA;
}

// Measurement aid: a plain read-only stream over a buffer (16-byte loads, grid-stride, XOR-folded
// so that the loads cannot be dropped).  Its rate is the read-only HBM ceiling of the part.
__global__ void __launch_bounds__(1024, 2)
read_stream_kernel(const uint4* __restrict__ p, size_t n16, unsigned int* __restrict__ sink) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    unsigned int acc = 0;
    for (; i + 3 * stride < n16; i += 4 * stride) {
        const uint4 a = __ldcs(p + i), b = __ldcs(p + i + stride), c = __ldcs(p + i + 2 * stride),
                    e = __ldcs(p + i + 3 * stride);
        acc ^= a.x ^ a.y ^ a.z ^ a.w ^ b.x ^ b.y ^ b.z ^ b.w ^ c.x ^ c.y ^ c.z ^ c.w ^ e.x ^ e.y ^ e.z ^ e.w;
    }
    for (; i < n16; i += stride) { const uint4 a = __ldcs(p + i); acc ^= a.x ^ a.y ^ a.z ^ a.w; }
    if (acc == 0x9E3779B9u) atomicExch(sink, acc);   // practically never: keeps the loads alive
}

int launch_read_stream(const void* ptr, size_t bytes, unsigned int* sink, int sms, cudaStream_t stream) {
    read_stream_kernel<<<sms * 4, 1024, 0, stream>>>(static_cast<const uint4*>(ptr), bytes / 16, sink);
    return cudaGetLastError() == cudaSuccess ? DM_OK : DM_ECUDA;
}

// Eq. 1 keep bits, one 32-bit word (eight Philox quads) per thread.
__global__ void debug_masks_kernel(int n_paths, int K, int T, int d, MaskKey mk, uint32_t seq_base_lo, int shared_masks,
                                   uint32_t* __restrict__ out_bits) {
    const int words = (d + 31) / 32;
    const long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= (long long)n_paths * words) return;
    const int r = (int)(x / words), w = (int)(x - (long long)r * words);
    RowMap map{nullptr, K, T, 0, seq_base_lo, shared_masks};
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

int launch_debug_masks(int B, int T, int K, int d, const MaskKey& mk, uint32_t seq_base_lo, int shared_masks,
                       uint32_t* out_bits, cudaStream_t stream) {
    const long long n_paths = (long long)B * T * K;
    const long long total = n_paths * ((d + 31) / 32);
    if (total > (1ll << 40)) return DM_EUNSUPPORTED;
    const long long blocks = (total + 255) / 256;
    if (blocks > 0x7FFFFFFFll) return DM_EUNSUPPORTED;
    debug_masks_kernel<<<(unsigned)blocks, 256, 0, stream>>>((int)n_paths, K, T, d, mk, seq_base_lo, shared_masks, out_bits);
    return cudaGetLastError() == cudaSuccess ? DM_OK : DM_ECUDA;
}

}  // namespace dm
