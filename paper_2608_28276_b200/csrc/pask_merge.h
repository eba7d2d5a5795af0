// The merge step of a planned-ahead decode step (device code of the kernel that ends such a step).
#pragma once
#include <cuda_fp16.h>

#include "pask_internal.h"

namespace pask {

__device__ __forceinline__ float merge_bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float merge_bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// What the merge kernel of a planned-ahead step needs to attend each sequence's new token from the call's inputs.
struct NewTokens {
    const uint2 *k, *v;            // bf16 [n_seqs][n_kv][128] viewed as 8-byte pieces (4 dims)
    const uint2 *q;                // bf16 [n_seqs][n_q][128]
    const uint8_t *tags;           // [n_seqs]
    const uint8_t *decided;        // [n_seqs][n_groups] or null
    const int32_t *seq_ids, *planned_ids;   // this call's list and the one the plan was made for
    uint32_t *status;
    int group, n_groups, n_kv, low_bits;
};

// Partial (m, l = 1, o = v) of one new token for one query head: the token at the precision it is stored at.
// lane = 4 consecutive head dims; a 32-dim group is 8 adjacent lanes.
__device__ __forceinline__ void quantise_like_append(float (&x)[4], int low_bits) {
    float amax = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 4));
    const float qmax = low_bits == 8 ? 127.0f : low_bits == 2 ? 1.0f : 7.0f;
    __half sh = __float2half_rn(low_bits == 2 ? amax : __fdiv_rn(amax, qmax));
    if (__hisinf(sh)) sh = __ushort_as_half((unsigned short)0x7BFF);
    const float s = __half2float(sh);
    const float inv = s == 0.0f ? 0.0f : __fdiv_rn(1.0f, s);
#pragma unroll
    for (int i = 0; i < 4; i++) {
        float r = rintf(__fmul_rn(x[i], inv));
        r = fminf(fmaxf(r, -qmax), qmax);
        x[i] = __fmul_rn(r, s);          // (code - zero) * scale, exact
    }
}

// How many warps share the partials of one (sequence, query head) row.  A row has about n_ctas / n_seqs partials, and a
// warp takes eight per round trip to L2: small batches, whose rows have dozens, are split so that one round trip does.
inline int merge_split(int n_seqs, int n_ctas) {
    int split = 1;
    while (split < 8 && n_ctas / n_seqs + 2 > 8 * split) split *= 2;
    return split;
}

constexpr int kMergeThreads = 256;     // CTA of the kernels that merge: 8 warps = 8 / split rows

// Online merge of the partials b_first + sub, b_first + sub + split, ... <= b_last of row (s, h) into (o, M, L); lane = 4
// output dims.  Eight partials per round trip.
__device__ __forceinline__ void merge_share(const float2 *__restrict__ part_ml, const float *__restrict__ part_o, int s, int h,
                                            int n_q, uint32_t b_first, uint32_t b_last, uint32_t sub, uint32_t split, int lane,
                                            float4 &o, float &M, float &L) {
    for (uint32_t b = b_first + sub; b <= b_last; b += 8 * split) {
        float2 ml[8];
        float4 v[8];
#pragma unroll
        for (int u = 0; u < 8; u++) {
            const bool have = b + u * split <= b_last;
            const size_t row = ((size_t)b + u * split + s) * n_q + h;
            ml[u] = have ? part_ml[row] : make_float2(-INFINITY, 0.f);
            v[u] = have ? *reinterpret_cast<const float4 *>(part_o + row * kHeadDim + lane * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 8; u++) {
            if (ml[u].x == -INFINITY) continue;      // a CTA whose share of this sequence was empty
            const float Mn = fmaxf(M, ml[u].x);
            const float fo = exp2f(M - Mn), fn = exp2f(ml[u].x - Mn);   // exp2f(-inf) = 0 on the first one
            o.x = fmaf(fn, v[u].x, o.x * fo); o.y = fmaf(fn, v[u].y, o.y * fo);
            o.z = fmaf(fn, v[u].z, o.z * fo); o.w = fmaf(fn, v[u].w, o.w * fo);
            L = fmaf(fn, ml[u].y, L * fo);
            M = Mn;
        }
    }
}

// The `split` warps of a row (adjacent warps of one CTA; every thread of the CTA calls this) hand their shares to the
// row's first warp, which merges them in warp order: the result is the same whatever the timing.
__device__ __forceinline__ void merge_across_warps(uint32_t sub, uint32_t split, int lane, float4 &o, float &M, float &L) {
    __shared__ float4 s_o[kMergeThreads / 32][32];
    __shared__ float2 s_ml[kMergeThreads / 32];
    if (split == 1) return;
    const int warp = threadIdx.x >> 5;
    if (sub != 0) {
        s_o[warp][lane] = o;
        if (lane == 0) s_ml[warp] = make_float2(M, L);
    }
    __syncthreads();
    if (sub != 0) return;
    for (uint32_t w = 1; w < split; w++) {
        const float2 ml = s_ml[warp + w];
        if (ml.x == -INFINITY) continue;
        const float4 v = s_o[warp + w][lane];
        const float Mn = fmaxf(M, ml.x);
        const float fo = exp2f(M - Mn), fn = exp2f(ml.x - Mn);
        o.x = fmaf(fn, v.x, o.x * fo); o.y = fmaf(fn, v.y, o.y * fo);
        o.z = fmaf(fn, v.z, o.z * fo); o.w = fmaf(fn, v.w, o.w * fo);
        L = fmaf(fn, ml.y, L * fo);
        M = Mn;
    }
}

// The merge of a planned-ahead step for the (sequence, query head) rows of this CTA's warps (`split` adjacent warps a
// row, lane = 4 output dims): the partials of the history (streamed from the plan of the cache before this call's
// append) and, as one more partial, the sequence's new token taken from the call's k / v.  Everything that does not
// come from the kernels before is fetched first; the function then executes the kernel's dependency wait itself.
// Every thread of the CTA must call it (it holds a block-wide barrier when split > 1).  The CTAs that merge are those
// from first_cta on.
__device__ __forceinline__ void merge_rows_with_new_token(const uint32_t *__restrict__ prefix, const float2 *__restrict__ part_ml,
                                                          const float *__restrict__ part_o, float *__restrict__ out,
                                                          float *__restrict__ lse, int n_seqs, int n_q, uint32_t n_ctas,
                                                          uint32_t split, const NewTokens &nt, const SmallLut &lut,
                                                          uint32_t first_cta) {
    const int wid = ((blockIdx.x - first_cta) * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int row_id = wid / (int)split;
    const uint32_t sub = (uint32_t)wid % split;
    const int s = row_id / n_q, h = row_id % n_q;
    const bool mine = row_id < n_seqs * n_q;
    // everything that does not come from the kernels before is fetched ahead of the dependency wait
    uint32_t p0 = 0, p1 = 0;
    uint64_t total = 0;
    int act = PASK_ACTION_RELEASE;
    float kx[4] = {0.f, 0.f, 0.f, 0.f}, vx[4] = {0.f, 0.f, 0.f, 0.f}, qx[4] = {0.f, 0.f, 0.f, 0.f};
    bool stale = false;
    if (mine) { p0 = __ldg(prefix + s); p1 = __ldg(prefix + s + 1); total = __ldg(prefix + n_seqs); }
    if (mine && sub == 0) {       // the new token is the business of the row's first warp
        act = nt.decided ? nt.decided[(size_t)s * nt.n_groups + nt.group] : lut.action[nt.tags[s]];
        if (act > PASK_ACTION_RETAIN_HIGH) act = PASK_ACTION_RELEASE;      // (the append refuses the call)
        stale = nt.seq_ids[s] != nt.planned_ids[s];
        if (act != PASK_ACTION_RELEASE) {
            const int kv = h / (n_q / nt.n_kv);
            const uint2 kw = nt.k[((size_t)s * nt.n_kv + kv) * 32 + lane], vw = nt.v[((size_t)s * nt.n_kv + kv) * 32 + lane];
            const uint2 qw = nt.q[((size_t)s * n_q + h) * 32 + lane];
            kx[0] = merge_bf_lo(kw.x); kx[1] = merge_bf_hi(kw.x); kx[2] = merge_bf_lo(kw.y); kx[3] = merge_bf_hi(kw.y);
            vx[0] = merge_bf_lo(vw.x); vx[1] = merge_bf_hi(vw.x); vx[2] = merge_bf_lo(vw.y); vx[3] = merge_bf_hi(vw.y);
            qx[0] = merge_bf_lo(qw.x); qx[1] = merge_bf_hi(qw.x); qx[2] = merge_bf_lo(qw.y); qx[3] = merge_bf_hi(qw.y);
        }
    }
    float m_new = -INFINITY;
    if (act == PASK_ACTION_RETAIN_LOW) { quantise_like_append(kx, nt.low_bits); quantise_like_append(vx, nt.low_bits); }
    if (act != PASK_ACTION_RELEASE) {       // (warp-uniform: one sequence and head per warp)
        float dot = fmaf(qx[0], kx[0], fmaf(qx[1], kx[1], fmaf(qx[2], kx[2], qx[3] * kx[3])));
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) dot += __shfl_xor_sync(0xffffffffu, dot, d);
        m_new = dot * (0.088388347648318440550f * 1.4426950408889634074f);      // log2 units, as the partials
    }
    if (stale && lane == 0 && h == 0) atomicOr(nt.status, PASK_DEV_STALE_PLAN);
    // which CTAs hold partials of this sequence: worked out ahead of the wait as well (two 64-bit divisions)
    uint32_t b_first = 1, b_last = 0;
    if (p1 > p0) {
        b_first = (uint32_t)((((uint64_t)p0 + 1) * n_ctas - 1) / total);
        b_last = (uint32_t)(((uint64_t)p1 * n_ctas - 1) / total);
    }
    pdl_wait();
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    float M = -INFINITY, L = 0.f;
    if (p1 > p0) merge_share(part_ml, part_o, s, h, n_q, b_first, b_last, sub, split, lane, o, M, L);
    merge_across_warps(sub, split, lane, o, M, L);
    if (!mine || sub != 0) return;
    if (m_new != -INFINITY) {                // the new token: weight 1 at its own score
        const float Mn = fmaxf(M, m_new);
        const float fo = exp2f(M - Mn), fn = exp2f(m_new - Mn);
        o.x = fmaf(fn, vx[0], o.x * fo); o.y = fmaf(fn, vx[1], o.y * fo);
        o.z = fmaf(fn, vx[2], o.z * fo); o.w = fmaf(fn, vx[3], o.w * fo);
        L = fmaf(fn, 1.0f, L * fo);
        M = Mn;
    }
    const size_t orow = (size_t)s * n_q + h;
    if (L > 0.f) {
        const float inv = 1.0f / L;
        o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
    }
    *reinterpret_cast<float4 *>(out + orow * kHeadDim + lane * 4) = o;
    if (lse && lane == 0) lse[orow] = L > 0.f ? (M + log2f(L)) * 0.69314718055994530942f : -INFINITY;
}


}  // namespace pask
