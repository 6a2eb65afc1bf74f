// Shared device helpers of the DropMatch CUDA library: mask generator (Eq. 1), row
// indexing, ordered float keys for the argmax (Sec. 3.2), partial-result layout.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace dm {

// Device error word codes (dm_device_error).
enum : uint32_t {
    ERR_NONE = 0,
    ERR_WAIT_FULL = 1,      // consumer gave up waiting for a TMA stage
    ERR_WAIT_EMPTY = 2,     // producer gave up waiting for a free stage
    ERR_WAIT_OPERAND = 3,   // MMA issuer gave up waiting for the masked operand
    ERR_WAIT_ACC_FULL = 4,  // epilogue gave up waiting for an accumulator
    ERR_WAIT_ACC_EMPTY = 5, // MMA issuer gave up waiting for a drained accumulator
    ERR_BAD_ROW = 6,        // debug row selection out of range
    ERR_WAIT_JS = 7         // a block of the one-kernel JS sweep gave up waiting for the other blocks of its position
};

// One path ("row") of a call: which hidden row it masks and its mask key words.
struct RowKey {
    int q;        // hidden row index into H
    uint32_t s;   // sequence id (low 32 bits)
    uint32_t t;   // position index in the mask key (0 when masks are shared across positions)
    uint32_t i;   // path index
};

// How rows map to (hidden row, sequence, position, path).
// sel == nullptr: row r -> q = r / K, i = r % K, s = seq_base + q / T, t = q % T.
// sel != nullptr: (b, t, i) triples; q = b*T + t.
struct RowMap {
    const int32_t* sel;
    int K, T, B;
    uint32_t seq_base_lo;
    int shared_masks;   // 1: the mask key ignores the position (one mask per sequence and path)
    int plain_extra;    // 1: K+1 paths per hidden row, the last one unmasked (path index kPlainPath)
};
constexpr uint32_t kPlainPath = 0xFFFFFFFFu;   // RowKey.i of a path that keeps every element

__device__ __forceinline__ bool row_key(const RowMap& m, int r, RowKey& k) {
    if (m.sel == nullptr) {
        const int kp = m.K + m.plain_extra;
        int q = r / kp;
        k.q = q;
        k.i = (uint32_t)(r - q * kp);
        if (m.plain_extra && k.i == (uint32_t)m.K) k.i = kPlainPath;
        int b = q / m.T;
        k.t = m.shared_masks ? 0u : (uint32_t)(q - b * m.T);
        k.s = m.seq_base_lo + (uint32_t)b;
        return true;
    }
    int b = m.sel[3 * r], t = m.sel[3 * r + 1], i = m.sel[3 * r + 2];
    bool ok = b >= 0 && b < m.B && t >= 0 && t < m.T && i >= 0;
    k.q = ok ? b * m.T + t : 0;
    k.t = m.shared_masks ? 0u : (uint32_t)t;
    k.i = (uint32_t)i;
    k.s = m.seq_base_lo + (uint32_t)b;
    return ok;
}

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): ten rounds; each round multiplies
// words 0 and 2 by fixed odd constants, mixes the high halves with words 1 and 3 and the
// round key, and the key advances by Weyl constants.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1) {
    constexpr uint32_t MA = 0xD2511F53u, MB = 0xCD9E8D57u;
    constexpr uint32_t WA = 0x9E3779B9u, WB = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        // one widening multiply per product (both halves from a single 32x32->64 instruction)
        const unsigned long long pa = (unsigned long long)MA * c.x, pb = (unsigned long long)MB * c.z;
        const uint32_t hi_a = (uint32_t)(pa >> 32), lo_a = (uint32_t)pa;
        const uint32_t hi_b = (uint32_t)(pb >> 32), lo_b = (uint32_t)pb;
        c = make_uint4(hi_b ^ c.y ^ k0, lo_b, hi_a ^ c.w ^ k1, lo_a);
        k0 += WA;
        k1 += WB;
    }
    return c;
}

// Keep flags (bit n = element 4*quad + n kept) of one Philox quad of a path.
__device__ __forceinline__ uint32_t keep4(uint32_t quad, const RowKey& k, uint32_t key0,
                                          uint32_t key1, uint32_t thr) {
    if (k.i == kPlainPath) return 0xFu;   // the unmasked path of a hidden row
    uint4 w = philox4x32_10(make_uint4(quad, k.i, k.t, k.s), key0, key1);
    return (w.x >= thr ? 1u : 0u) | (w.y >= thr ? 2u : 0u) | (w.z >= thr ? 4u : 0u) |
           (w.w >= thr ? 8u : 0u);
}

// Sampling decode rule (Sec. 3.2 names nucleus sampling as the alternative to the top-1 token):
// Gumbel noise of vocabulary entry v for the path with key k.  Philox counter (v / 4, i + 2^31,
// t, s), word v mod 4: path indices stay below 2^31, so these counters never meet the mask
// counters.  The top 23 bits n of the word give u = (n + 0.5) / 2^23, exact in fp32 and strictly
// inside (0,1); g = -log(-log(u)) is a standard Gumbel variate, and the argmax of
// logit / temperature + g is a draw from Softmax(logits / temperature).
__device__ __forceinline__ float gumbel_noise(uint32_t v, const RowKey& k, uint32_t key0, uint32_t key1) {
    const uint4 w = philox4x32_10(make_uint4(v >> 2, k.i | 0x80000000u, k.t, k.s), key0, key1);
    const uint32_t word = (v & 2u) ? ((v & 1u) ? w.w : w.z) : ((v & 1u) ? w.y : w.x);
    const float u = ((float)(word >> 9) + 0.5f) * 1.1920928955078125e-07f;   // 2^-23
    return -logf(-logf(u));
}

// Monotone map float -> uint32 (larger float <=> larger key); -0 is folded into +0 first so
// that equal logits get equal keys.  NaN inputs are not expected (finite W and H).
__device__ __forceinline__ uint32_t float_key(float x) {
    uint32_t b = __float_as_uint(x + 0.0f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t key) {
    uint32_t b = (key & 0x80000000u) ? (key & 0x7FFFFFFFu) : ~key;
    return __uint_as_float(b);
}

// Partial argmax of one vocabulary slice for one row: (ordered key of the max logit, its index).
// A larger packed value wins; on equal keys the SMALLER index wins, hence the inverted index.
__device__ __forceinline__ unsigned long long pack_best(uint32_t key, uint32_t idx) {
    return ((unsigned long long)key << 32) | (unsigned long long)(0xFFFFFFFFu - idx);
}
__device__ __forceinline__ uint32_t best_index(unsigned long long packed) {
    return 0xFFFFFFFFu - (uint32_t)(packed & 0xFFFFFFFFull);
}

}  // namespace dm
