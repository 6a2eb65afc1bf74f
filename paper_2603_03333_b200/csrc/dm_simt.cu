// CUDA-core (fp32 FMA) kernel for the masked LM head: Eq. 1-3 and the per-slice argmax of
// Sec. 3.2.  It serves fp32 heads (tensor cores have no fp32-exact mode), bf16 heads whose
// hidden size the tensor-core kernel cannot tile, and the debug-logits entry point.
//
// Each block owns a contiguous vocabulary slice.  Rows (paths) are processed RC at a time:
// the block first builds the RC masked hidden rows in shared memory (exact zeroing, storage
// type), then each warp walks vocabulary rows of the slice, streaming W[v,:] with 16-byte
// loads and accumulating RC dot products in fp32.  Eq. 2's 1/(1-p) is applied to the sum.
#include "dm_internal.h"

namespace dm {

template <typename T> struct Vec;
template <> struct Vec<float> {
    static constexpr int N = 4;
    __device__ static void load(const float* p, float (&out)[4]) {
        float4 v = *reinterpret_cast<const float4*>(p);
        out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    }
};
template <> struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ static void load(const __nv_bfloat16* p, float (&out)[8]) {
        uint4 v = *reinterpret_cast<const uint4*>(p);
        uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int n = 0; n < 4; ++n) {  // bf16 -> fp32 is a 16-bit shift
            out[2 * n] = __uint_as_float(w[n] << 16);
            out[2 * n + 1] = __uint_as_float(w[n] & 0xFFFF0000u);
        }
    }
};

template <typename T, int RC>
__global__ void __launch_bounds__(256)
simt_head_kernel(const T* __restrict__ W, const T* __restrict__ H, int V, int d, int rows,
                 RowMap map, uint32_t key0, uint32_t key1, uint32_t thr, float scale, int sample, float inv_temp,
                 int v_per_block, int v_offset, unsigned long long* __restrict__ partials,
                 float* __restrict__ dbg_logits, uint32_t* __restrict__ err) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* hm = reinterpret_cast<T*>(smem_raw);  // [RC][d] masked hidden rows
    __shared__ unsigned long long warp_best[8][RC];
    __shared__ int row_valid[RC];

    constexpr int VEC = Vec<T>::N;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int v_begin = blockIdx.x * v_per_block;
    const int v_end = min(V, v_begin + v_per_block);
    const int quads = d >> 2;

    for (int r0 = 0; r0 < rows; r0 += RC) {
        const int nrr = min(RC, rows - r0);
        // Eq. 1 + Eq. 2 numerator: masked copies of the hidden rows, four elements per Philox call
        for (int w = threadIdx.x; w < nrr * quads; w += blockDim.x) {
            int rr = w / quads, quad = w - rr * quads;
            RowKey k;
            bool ok = row_key(map, r0 + rr, k);
            if (quad == 0) {
                row_valid[rr] = ok;
                if (!ok) atomicExch(err, (uint32_t)ERR_BAD_ROW);
            }
            uint32_t keep = keep4((uint32_t)quad, k, key0, key1, thr);
            const T* src = H + (size_t)k.q * d + 4 * quad;
            T* dst = hm + (size_t)rr * d + 4 * quad;
#pragma unroll
            for (int n = 0; n < 4; ++n) dst[n] = ((keep >> n) & 1u) ? src[n] : T(0.0f);
        }
        __syncthreads();

        unsigned long long best = 0ull;  // lane rr tracks row r0+rr; key 0 is below every float key
        for (int v = v_begin + warp; v < v_end; v += 8) {
            float acc[RC];
#pragma unroll
            for (int rr = 0; rr < RC; ++rr) acc[rr] = 0.0f;
            const T* wrow = W + (size_t)v * d;
            for (int j = lane * VEC; j < d; j += 32 * VEC) {
                float wv[VEC];
                Vec<T>::load(wrow + j, wv);
#pragma unroll
                for (int rr = 0; rr < RC; ++rr) {
                    if (rr < nrr) {
                        float hv[VEC];
                        Vec<T>::load(hm + (size_t)rr * d + j, hv);
#pragma unroll
                        for (int n = 0; n < VEC; ++n) acc[rr] = fmaf(wv[n], hv[n], acc[rr]);
                    }
                }
            }
#pragma unroll
            for (int rr = 0; rr < RC; ++rr) {
                float s = acc[rr];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
                s *= scale;
                if (rr < nrr) {
                    if (dbg_logits != nullptr && lane == 0)
                        dbg_logits[(size_t)(r0 + rr) * V + v] =
                            row_valid[rr] ? s : __uint_as_float(0x7FC00000u);
                    if (lane == rr) {
                        if (sample) {   // sampling decode: Gumbel-max on logit / temperature
                            RowKey k;
                            row_key(map, r0 + rr, k);
                            s = fmaf(s, inv_temp, gumbel_noise((uint32_t)(v + v_offset), k, key0, key1));
                        }
                        unsigned long long cand = pack_best(float_key(s), (uint32_t)(v + v_offset));
                        best = cand > best ? cand : best;
                    }
                }
            }
        }
        if (lane < RC) warp_best[warp][lane] = best;
        __syncthreads();
        if (threadIdx.x < nrr) {
            unsigned long long b = warp_best[0][threadIdx.x];
#pragma unroll
            for (int w = 1; w < 8; ++w) b = warp_best[w][threadIdx.x] > b ? warp_best[w][threadIdx.x] : b;
            partials[(size_t)blockIdx.x * rows + r0 + threadIdx.x] = b;
        }
        __syncthreads();
    }
}

template <typename T, int RC>
static int launch_simt_rc(const HeadDesc& head, const void* H, int rows, const RowMap& map,
                          const MaskKey& mk, int* n_slices_out, unsigned long long* partials,
                          float* dbg_logits, uint32_t* err, cudaStream_t stream) {
    const size_t smem = (size_t)RC * head.d * sizeof(T);
    int v_per_block = (head.V + kSimtMaxSlices - 1) / kSimtMaxSlices;
    if (v_per_block < 8) v_per_block = 8;
    const int n_slices = (head.V + v_per_block - 1) / v_per_block;
    auto kern = simt_head_kernel<T, RC>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return DM_ECUDA;
    kern<<<n_slices, 256, smem, stream>>>(static_cast<const T*>(head.W), static_cast<const T*>(H),
                                          head.V, head.d, rows, map, mk.key0, mk.key1, mk.thr,
                                          mk.scale, mk.sample, mk.inv_temp, v_per_block, head.v_offset, partials, dbg_logits, err);
    if (cudaGetLastError() != cudaSuccess) return DM_ECUDA;
    *n_slices_out = n_slices;
    return DM_OK;
}

// Eight masked rows at a time fit shared memory up to d = 12800 (bf16) or 6400 (fp32); longer
// hidden sizes take four, two or one row at a time (W is then re-read from L2 more often).
template <typename T>
static int launch_simt_t(const HeadDesc& head, const void* H, int rows, const RowMap& map,
                         const MaskKey& mk, int* n_slices_out, unsigned long long* partials,
                         float* dbg_logits, uint32_t* err, cudaStream_t stream) {
    const size_t row_bytes = (size_t)head.d * sizeof(T), limit = 200 * 1024;
    if (8 * row_bytes <= limit)
        return launch_simt_rc<T, 8>(head, H, rows, map, mk, n_slices_out, partials, dbg_logits, err, stream);
    if (4 * row_bytes <= limit)
        return launch_simt_rc<T, 4>(head, H, rows, map, mk, n_slices_out, partials, dbg_logits, err, stream);
    if (2 * row_bytes <= limit)
        return launch_simt_rc<T, 2>(head, H, rows, map, mk, n_slices_out, partials, dbg_logits, err, stream);
    if (row_bytes <= limit)
        return launch_simt_rc<T, 1>(head, H, rows, map, mk, n_slices_out, partials, dbg_logits, err, stream);
    return DM_EUNSUPPORTED;
}

int launch_simt(const HeadDesc& head, const void* H, int rows, const RowMap& map, const MaskKey& mk,
                int* n_slices_out, unsigned long long* partials, float* dbg_logits, uint32_t* err,
                cudaStream_t stream) {
    if (head.dtype == DM_F32)
        return launch_simt_t<float>(head, H, rows, map, mk, n_slices_out, partials, dbg_logits, err, stream);
    return launch_simt_t<__nv_bfloat16>(head, H, rows, map, mk, n_slices_out, partials, dbg_logits, err, stream);
}

}  // namespace dm
