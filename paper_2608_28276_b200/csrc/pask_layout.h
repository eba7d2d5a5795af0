// Physical packing of K/V inside cache pages.  Shared by the append kernels (writers), the
// decode-attention kernel (reader) and the host-side canonical dump.
//
// The packing is "fragment-major": bytes are ordered the way the attention kernel's warps
// consume them, so that every 128-bit shared-memory load of a warp is one contiguous 512-byte
// run (no bank conflicts, no padding, and the tile can be brought in with one linear bulk copy)
// and lands directly in the register layout of the m16n8k16 tensor-core fragments.
//
// Lane numbering: lane = 4*g + t, g = lane / 4 (0..7), t = lane % 4 (0..3).
//
// HIGH page  : [kv head][K tile 4096 B][V tile 4096 B]            (n_kv * 8192 B)
//   K tile   : 8 rounds i of 512 B; round i = 2*j + hi holds, for lane (g,t), the 16-byte chunk
//              (dims 8c .. 8c+7, c = 4*j + t) of token g + 8*hi.  QK^T uses tokens as the M
//              rows: lane (g,t) owns rows g and g+8 and the k-slots of its own t.
//   V tile   : 8 rounds i = 4*e + k of 512 B; lane (g,t) holds for token
//              {2t, 2t+1, 2t+8, 2t+9}[k] the 8-byte pieces dims 32*(2e)+4g .. +3 and
//              32*(2e+1)+4g .. +3.  P.V uses head dims as the M rows and tokens as k-slots.
// LOW page   : [kv head][K codes 1024][K scales 128][V codes 1024][V scales 128]   (n_kv * 2304 B)
//   K codes  : 2 rounds hi of 512 B; lane (g,t) holds 4 words w (one per 32-dim group) for token
//              g + 8*hi; word w packs dims 32w + 8t + e, e = 0..7, at nibble (e>>1) + 4*(e&1),
//              so that (word >> 4s) & 0x000F000F yields dims (2s, 2s+1) as a 16-bit pair.
//   V codes  : 2 rounds ps of 512 B; lane (g,t) holds 4 words q; word q packs, for dims
//              32q + 4g + i (i = 0..3), token 2t + 8*ps in nibble i and token 2t + 1 + 8*ps in
//              nibble i + 4, so the same mask yields (even token, odd token) pairs per dim.
//   scales   : [token 16][group 4] fp16.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define PASK_HD __host__ __device__ __forceinline__
#else
#define PASK_HD inline
#endif

namespace pask {

constexpr int kHeadDim = 128;
constexpr int kPageTokens = 16;
constexpr int kQGroup = 32;
constexpr int kGroupsPerHead = 4;
constexpr int kHighTileBytes = 4096;
constexpr int kHighHeadBytes = 8192;
constexpr int kLowCodesBytes = 1024;
constexpr int kLowScalesBytes = 128;
constexpr int kLowHalfBytes = 1152;  // codes + scales of K (or of V)
constexpr int kLowHeadBytes = 2304;
// cost of streaming one page (all heads), in units of n_kv * 256 bytes
constexpr uint32_t kCostHighPage = 32;
constexpr uint32_t kCostLowPage = 9;

// HIGH K tile: offset of the 16-byte chunk c (dims 8c..8c+7) of token tau.
PASK_HD int high_k_chunk_off(int tau, int c) {
    const int g = tau & 7, hi = tau >> 3, t = c & 3, j = c >> 2;
    return (2 * j + hi) * 512 + (4 * g + t) * 16;
}

// HIGH V tile: offset of the 8-byte piece holding dims 32q + 4g .. 32q + 4g + 3 of token tau.
PASK_HD int high_v_piece_off(int tau, int q, int g) {
    const int t = (tau & 7) >> 1, k = (tau & 1) + 2 * (tau >> 3);
    return (4 * (q >> 1) + k) * 512 + (4 * g + t) * 16 + 8 * (q & 1);
}

// LOW K codes: offset of the 32-bit word holding dims 32w + 8t .. +7 of token tau.
PASK_HD int low_k_word_off(int tau, int w, int t) {
    return (tau >> 3) * 512 + (4 * (tau & 7) + t) * 16 + 4 * w;
}
// nibble index of dim offset e (0..7) inside that word
PASK_HD int low_k_nibble(int e) { return (e >> 1) + 4 * (e & 1); }

// LOW V codes (relative to the V half): offset of the 16-bit half-word holding dims
// 32q + 4g .. +3 of token tau (nibble i = dim i).
PASK_HD int low_v_half_off(int tau, int q, int g) {
    const int t = (tau & 7) >> 1;
    return (tau >> 3) * 512 + (4 * g + t) * 16 + 4 * q + 2 * (tau & 1);
}

// scales (relative to the K or V half): fp16 of (token tau, group w)
PASK_HD int low_scale_off(int tau, int w) { return kLowCodesBytes + tau * 8 + w * 2; }

// ---- work partition of decode attention -------------------------------------------------
// Sequences are laid end to end in "cost space" (a HIGH page costs kCostHighPage, a LOW page
// kCostLowPage); CTA b of G owns [C*b/G, C*(b+1)/G).  A cut at local offset x of a sequence whose
// cost is cs splits BOTH of its page lists at the same fraction x / cs, so every CTA gets the
// sequence's own mix of HIGH and LOW pages (the two kinds differ in time per byte, and a CTA
// that received only one kind would finish early or late).  Both neighbours of a cut apply the
// same rule, so every page is processed exactly once.

// number of pages (of a list of n_pages) that lie before local cost offset x of a sequence of cost cs
PASK_HD uint32_t cut_pages(uint32_t x, uint32_t cs, uint32_t n_pages) {
    return x >= cs ? n_pages : (uint32_t)(((uint64_t)x * n_pages) / cs);
}

}  // namespace pask
