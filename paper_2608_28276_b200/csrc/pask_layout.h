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
//   K tile   : 8 rounds i of 512 B, one per MMA of the tile's QK^T; round i = 2*j + h holds, for
//              lane (g,t), the four A registers of that MMA in order: with d = 8*(4j+t) + 4h,
//              {token g dims d,d+1 | token g+8 dims d,d+1 | token g dims d+2,d+3 | token g+8 dims
//              d+2,d+3}.  QK^T uses tokens as the M rows: lane (g,t) owns rows g and g+8 and the
//              k-slots of its own t, so one 128-bit load is one operand quad, no register moves.
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
// LOW page, 8-bit codes (policy low_bits = 8):
//              [kv head][K codes 2048][K scales 128][V codes 2048][V scales 128]   (n_kv * 4352 B)
//   K codes  : 4 rounds of 512 B; round rr holds, for lane (g,t), the 16 dims of k-chunks 2rr and
//              2rr+1 as two 8-byte pieces; the piece of chunk c is {token g dims 16c+2t,+1 | token g+8
//              same dims | token g dims 16c+2t+8,+9 | token g+8 same dims}, one byte per code: two PRMTs
//              per 32-bit word turn it into the fp16 pairs 1024 + code of an m16n8k16 A operand.
//   V codes  : 4 rounds of 512 B, one per 32-dim group q; lane (g,t) holds for r = 0,1 the piece
//              {dim D tokens 2t,2t+1 | dim D+1 tokens 2t,2t+1 | dim D tokens 2t+8,+9 | dim D+1 tokens
//              2t+8,+9} with D = 32q + 4g + 2r: the A operand of the P.V tile whose rows g, g+8 are
//              dims D, D+1 (the row order the bf16 and 4-bit paths use too).
// LOW page, 2-bit codes (policy low_bits = 2):
//              [kv head][K codes 512][K scales 128][V codes 512][V scales 128]     (n_kv * 1280 B)
//   K codes  : one round of 512 B; lane (g,t) holds 4 words j (one per 32-dim group); in word j the
//              low half-word holds even dims and the high one odd dims, byte 0 of either token g and
//              byte 1 token g+8, and the field at bits 2i of a byte dims 32j + 8t + 2i (+1): so
//              ((word >> 8 hi) & (0x00030003 << 2i)) | 0x64006400 is the fp16 pair 1024 + 4^i code of an
//              A register, and the eight dims of a token's 16-byte chunk fill two whole bytes.
//   V codes  : one round of 512 B; lane (g,t) holds 4 words q; low half-word token 2t (+8 in byte 1),
//              high half-word token 2t+1 (+8 in byte 1); the field at bits 2i of a byte is dim
//              32q + 4g + i: fields 0, 1 are rows g, g+8 of P.V tile 2q, fields 2, 3 of tile 2q+1
//              (the row order of the other formats).
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
constexpr int kLow8CodesBytes = 2048;
constexpr int kLow8HalfBytes = 2176;  // codes + scales of K (or of V), 8-bit codes
constexpr int kLow8HeadBytes = 4352;
constexpr int kLow2CodesBytes = 512;
constexpr int kLow2HalfBytes = 640;   // codes + scales of K (or of V), 2-bit codes
constexpr int kLow2HeadBytes = 1280;
// cost of streaming one page (all heads), in units of n_kv * 256 bytes
constexpr uint32_t kCostHighPage = 32;
constexpr uint32_t kCostLowPage = 9;
constexpr uint32_t kCostLow8Page = 17;
constexpr uint32_t kCostLow2Page = 5;

// HIGH K tile: offset of the 4-byte piece holding dims 2p, 2p+1 (p = 0..63) of token tau.
PASK_HD int high_k_pair_off(int tau, int p) {
    const int c = p >> 2, h = (p >> 1) & 1, second = p & 1;   // chunk of 8 dims, half of it, pair within the half
    const int g = tau & 7, hi = tau >> 3, t = c & 3, j = c >> 2;
    return (2 * j + h) * 512 + (4 * g + t) * 16 + second * 8 + hi * 4;
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

// 8-bit LOW K codes: byte offset of the code of (token tau, dim d) within the K codes
PASK_HD int low8_k_off(int tau, int d) {
    const int c = d >> 4, within = d & 15, t = (within & 7) >> 1, upper = within >> 3;
    return (c >> 1) * 512 + (4 * (tau & 7) + t) * 16 + (c & 1) * 8 + upper * 4 + (tau >> 3) * 2 + (within & 1);
}
// 8-bit LOW V codes (relative to the V half)
PASK_HD int low8_v_off(int tau, int d) {
    const int q = d >> 5, g = (d & 31) >> 2, i = d & 3, t = (tau & 7) >> 1;
    return q * 512 + (4 * g + t) * 16 + (i >> 1) * 8 + (tau >> 3) * 4 + (i & 1) * 2 + (tau & 1);
}
PASK_HD int low8_scale_off(int tau, int w) { return kLow8CodesBytes + tau * 8 + w * 2; }

// 2-bit LOW K codes: byte offset of the byte holding dims {8c + 2i + e, i = 0..3} (c = 0..15 the
// 16-byte chunk of the token's row, e = 0 even / 1 odd dims) of token tau; dim 8c + 2i + e sits at bits 2i
PASK_HD int low2_k_byte_off(int tau, int c, int e) {
    return (4 * (tau & 7) + (c & 3)) * 16 + (c >> 2) * 4 + e * 2 + (tau >> 3);
}
// 2-bit LOW V codes (relative to the V half): byte holding dims 4u .. 4u+3 (u = 0..31) of token tau; dim 4u + i at bits 2i
PASK_HD int low2_v_byte_off(int tau, int u) {
    return (4 * (u & 7) + ((tau & 7) >> 1)) * 16 + (u >> 3) * 4 + (tau & 1) * 2 + (tau >> 3);
}
PASK_HD int low2_scale_off(int tau, int w) { return kLow2CodesBytes + tau * 8 + w * 2; }

// ---- work partition of decode attention -------------------------------------------------
// Every sequence's pages are visited in one fixed order that interleaves its HIGH and LOW pages
// evenly: position v (0 <= v < n = nH + nL) is a HIGH page iff floor((v+1) nH / n) > floor(v nH / n).
// HIGH pages are bandwidth-heavy and LOW pages instruction-heavy; taking them in turn keeps both
// the memory system and the issue slots busy, and any run of consecutive positions has the
// sequence's own mix.  Sequences are laid end to end in "cost space" (a HIGH page costs
// kCostHighPage, a LOW page kCostLowPage); CTA b of G owns [C*b/G, C*(b+1)/G); a cut at local cost
// offset x of a sequence of cost cs falls before position floor(x n / cs).  Both neighbours of a
// cut apply the same rule, so every page is processed exactly once.

// which page sits at position v: returns true and the HIGH page index, or false and the LOW page index
PASK_HD bool page_at(uint32_t v, uint32_t nh, uint32_t nl, uint32_t &idx) {
    const uint32_t n = nh + nl;
    uint32_t h0, h1;
    if (n < 65536u) {   // products fit 32 bits (streams below a million tokens): cheap division
        h0 = (v * nh) / n;
        h1 = ((v + 1) * nh) / n;
    } else {
        h0 = (uint32_t)(((uint64_t)v * nh) / n);
        h1 = (uint32_t)(((uint64_t)(v + 1) * nh) / n);
    }
    idx = h1 > h0 ? h0 : v - h0;
    return h1 > h0;
}

// number of positions (of n) that lie before local cost offset x of a sequence of cost cs
PASK_HD uint32_t cut_positions(uint32_t x, uint32_t cs, uint32_t n) {
    return x >= cs ? n : (uint32_t)(((uint64_t)x * n) / cs);
}

// A small batch (at least kSnapCtasPerSeq CTAs per sequence): the cost line is replaced by one on which every
// non-empty sequence covers a whole number of CTA shares -- cost[s] becomes the first CTA of sequence s and
// cost[n_seqs] the grid -- so that no CTA's range crosses from one sequence into the next (a second segment costs a
// CTA a fresh set-up of about two microseconds, which a short kernel feels as a straggler).  Every non-empty
// sequence gets one CTA, and the others are shared out by cost (rounded cumulatively, so the error does not add up):
// no CTA then carries more than grid / (grid - sequences) <= 16/15 of an even share.  Inside a sequence the cuts fall
// at equal numbers of positions of its order list as before.  Everything that reads the prefix (the streaming
// kernel's ranges, the merge's list of CTAs per sequence) works from it unchanged.
constexpr uint32_t kSnapCtasPerSeq = 16;
PASK_HD void snap_cost_prefix(uint32_t *cost, int n_seqs, uint32_t n_ctas) {
    const uint32_t total = cost[n_seqs];
    if (total == 0 || (uint64_t)n_seqs * kSnapCtasPerSeq > n_ctas) return;
    uint32_t n_ne = 0;                       // non-empty sequences
    for (int s = 0; s < n_seqs; s++) n_ne += cost[s + 1] > cost[s];
    const uint32_t rest = n_ctas - n_ne;     // CTAs shared out by cost
    uint32_t old_lo = cost[0], at = 0, given = 0;      // old cost[s]; new cost[s]; of `rest`, given to the sequences before
    for (int s = 0; s < n_seqs; s++) {
        const uint32_t old_hi = cost[s + 1];
        if (old_hi > old_lo) {
            const uint32_t upto = (uint32_t)(((uint64_t)old_hi * rest + total / 2) / total);
            at += 1 + (upto - given);
            given = upto;
        }
        cost[s + 1] = at;
        old_lo = old_hi;
    }
}

// entries of the per-call page order list built by the plan kernel
constexpr uint32_t kOrderHigh = 0x80000000u;   // the page has the HIGH (bf16) format (else LOW)
constexpr int kOrderValidShift = 27;           // bits 27..30: tokens of the page to attend, 0 meaning all 16
constexpr uint32_t kOrderIdMask = 0x07ffffffu;

}  // namespace pask
