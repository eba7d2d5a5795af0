// pask_append_kv: table lookup, per-stream compaction, deterministic page allocation, budget
// accounting (plan kernel) and the drop / int4-quantise / bf16-keep writes (write kernel).
//
// Algorithm 2 of the paper, steps 1-2 (lookup, a = max(a0, floor)), 7 (persist) and 8 (budget
// recurrence), applied to a ragged batch of tokens for one layer.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "pask_internal.h"
#include "pask_merge.h"

namespace pask {

namespace {

constexpr int kPlanThreads = 256;      // threads of the one-launch append (and of its three-value scan)
constexpr int kBulkThreads = 1024;     // threads of the bulk append's plan kernel: 4096 tokens of a sequence per round

// Plan records are written by other CTAs of the same launch: read them through L2.
__device__ __forceinline__ AppendPlan load_plan_cg(const AppendPlan *p) {
    union { AppendPlan plan; uint4 q[4]; } u;
    const uint4 *src = reinterpret_cast<const uint4 *>(p);
#pragma unroll
    for (int i = 0; i < 4; i++) u.q[i] = __ldcg(src + i);
    return u.plan;
}

__device__ __forceinline__ void budget_add(uint64_t *p, uint64_t v) {
    if (v) atomicAdd(reinterpret_cast<unsigned long long *>(p), (unsigned long long)v);
}

// pages of a stream that an append of cnt tokens at length old writes into (the first may be a page
// the stream already holds)
__device__ __forceinline__ uint32_t pages_touched(uint32_t old, uint32_t cnt) {
    return cnt ? ((old + cnt - 1) >> 4) - (old >> 4) + 1 : 0u;
}

// exclusive scan of one value per thread over a block of kBulkThreads; returns the block total too
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t *s_warp, uint32_t *total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t o = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += o;
    }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    uint32_t before = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kBulkThreads / 32; w++) {
        const uint32_t x = s_warp[w];
        if (w < warp) before += x;
        tot += x;
    }
    __syncthreads();
    *total = tot;
    return before + inc - v;
}

// the same for three values per thread at once (one barrier; the per-warp slots are used once per kernel)
__device__ __forceinline__ void block_excl_scan3(uint32_t (&v)[3], uint32_t (*s_warp)[3], uint32_t (&total)[3]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc[3] = {v[0], v[1], v[2]};
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
#pragma unroll
        for (int k = 0; k < 3; k++) {
            const uint32_t o = __shfl_up_sync(0xffffffffu, inc[k], d);
            if (lane >= d) inc[k] += o;
        }
    }
    if (lane == 31) { s_warp[warp][0] = inc[0]; s_warp[warp][1] = inc[1]; s_warp[warp][2] = inc[2]; }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 3; k++) {
        uint32_t before = 0, tot = 0;
#pragma unroll
        for (int w = 0; w < kPlanThreads / 32; w++) {
            const uint32_t x = s_warp[w][k];
            if (w < warp) before += x;
            tot += x;
        }
        total[k] = tot;
        v[k] = before + inc[k] - v[k];
    }
}

// One CTA per sequence of the call: decide every token, rank it inside its stream, record the
// per-sequence plan; the CTA that arrives last allocates pages for the whole call (exclusive scan
// over sequences in call order, so ids do not depend on scheduling) and commits all counters --
// or refuses the whole call.
__global__ void __launch_bounds__(kBulkThreads)
append_plan_kernel(DevCache c, int layer, int n_seqs, int total_tokens, const int32_t *__restrict__ seq_ids,
                   const int32_t *__restrict__ cu_tokens, const uint8_t *__restrict__ tags,
                   const uint8_t *__restrict__ decided, uint8_t *__restrict__ actions_out) {
    __shared__ uint8_t s_lut[256];
    __shared__ uint32_t s_wh[2 * (kBulkThreads / 32)], s_wb[2 * (kBulkThreads / 32)];
    __shared__ uint32_t s_scan[kBulkThreads / 32];
    __shared__ uint32_t s_first_h[PASK_MAX_SEQS_PER_CALL], s_first_l[PASK_MAX_SEQS_PER_CALL];
    __shared__ int s_flag;
    const int i = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int group = c.layer_group[layer];
    if (tid < 256) s_lut[tid] = tid < c.n_tags ? c.lut[tid * c.n_groups + group] : (uint8_t)PASK_ACTION_RETAIN_HIGH;
    // this launch's serial: every CTA reads it before its arrival ticket, the CTA arriving last stores it back
    uint32_t serial = c.ctrl[kCtrlSerial] + 1u;
    if (serial == 0) serial = 1;
    const int seq = seq_ids[i];
    const int t0 = cu_tokens[i], t1 = cu_tokens[i + 1];
    uint32_t err = 0;
    if (t0 < 0 || t1 < t0 || t1 > total_tokens || (i == 0 && t0 != 0) || (i == n_seqs - 1 && t1 != total_tokens))
        err |= PASK_DEV_BAD_RAGGED;
    if (seq < 0 || seq >= c.max_seqs) err |= PASK_DEV_BAD_SEQ;
    if (tid == 0) {
        if (!(err & PASK_DEV_BAD_SEQ) && atomicExch(&c.seq_mark[seq], serial) == serial) s_flag = 1;  // named twice
        else s_flag = 0;
    }
    __syncthreads();
    if (s_flag) err |= PASK_DEV_BAD_SEQ;

    // Four consecutive tokens per thread and round; counts of a round travel packed (HIGH in the low
    // half-word, LOW in the high one; at most 1024 each), running totals stay in registers (every
    // thread adds the same round totals), and the per-warp slots alternate between rounds, so a
    // round costs one barrier.
    int bad_action = 0;
    uint32_t run_h = 0, run_l = 0, run_b = 0;
    if (!err) {
        int buf = 0;
        for (int base = t0; base < t1; base += 4 * kBulkThreads, buf ^= 1) {
            const int tb = base + 4 * tid;
            int a[4];
            uint32_t cnt = 0, nbad = 0;
#pragma unroll
            for (int e = 0; e < 4; e++) {
                const int t = tb + e;
                a[e] = 3;
                if (t < t1) {
                    const int tag = tags[t];
                    a[e] = s_lut[tag];
                    nbad += tag != PASK_TAG_PROTECTED && tag >= c.n_tags;
                    if (decided) {   // Algorithm 2 step 7 on the actions pask_decide chose
                        a[e] = decided[(size_t)t * c.n_groups + group];
                        if (a[e] > PASK_ACTION_RETAIN_HIGH) { bad_action = 1; a[e] = PASK_ACTION_RELEASE; }
                    }
                }
                cnt += (a[e] == PASK_ACTION_RETAIN_HIGH ? 1u : 0u) + (a[e] == PASK_ACTION_RETAIN_LOW ? 0x10000u : 0u);
            }
            uint32_t inc = cnt;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t o = __shfl_up_sync(0xffffffffu, inc, d);
                if (lane >= d) inc += o;
            }
            nbad = __reduce_add_sync(0xffffffffu, nbad);
            if (lane == 31) { s_wh[buf * (kBulkThreads / 32) + warp] = inc; s_wb[buf * (kBulkThreads / 32) + warp] = nbad; }
            __syncthreads();
            uint32_t before = 0, tot = 0, tot_b = 0;
#pragma unroll
            for (int w = 0; w < kBulkThreads / 32; w++) {
                const uint32_t x = s_wh[buf * (kBulkThreads / 32) + w];
                if (w < warp) before += x;
                tot += x;
                tot_b += s_wb[buf * (kBulkThreads / 32) + w];
            }
            const uint32_t excl = before + inc - cnt;
            uint32_t pos_h = run_h + (excl & 0xffffu), pos_l = run_l + (excl >> 16);
#pragma unroll
            for (int e = 0; e < 4; e++) {
                const int t = tb + e;
                if (t >= t1) break;
                // stream-ordered token lists for the write kernel: HIGH from the front of the
                // sequence's token range, LOW from its back
                if (a[e] == PASK_ACTION_RETAIN_HIGH) c.tok_list[t0 + pos_h++] = (uint32_t)t;
                else if (a[e] == PASK_ACTION_RETAIN_LOW) c.tok_list[t1 - 1 - pos_l++] = (uint32_t)t;
                if (actions_out) actions_out[t] = (uint8_t)a[e];
            }
            run_h += tot & 0xffffu;
            run_l += tot >> 16;
            run_b += tot_b;
        }
    }

    if (__syncthreads_or(bad_action)) err |= PASK_DEV_BAD_ACTION;
    if (tid == 0) {
        AppendPlan p{};
        p.seq = err ? -1 : seq;
        if (!err) {
            const size_t sl = (size_t)seq * c.n_layers + layer;
            p.old_high = c.n_high[sl];
            p.old_low = c.n_low[sl];
            p.old_tok = c.n_tok[sl];
            p.cnt_high = run_h;
            p.cnt_low = run_l;
            p.cnt_drop = (uint32_t)(t1 - t0) - run_h - run_l;
            p.bad_tags = run_b;
            const uint32_t ph0 = (p.old_high + kPageTokens - 1) / kPageTokens, ph1 = (p.old_high + p.cnt_high + kPageTokens - 1) / kPageTokens;
            const uint32_t pl0 = (p.old_low + kPageTokens - 1) / kPageTokens, pl1 = (p.old_low + p.cnt_low + kPageTokens - 1) / kPageTokens;
            p.new_pages_high = ph1 - ph0;
            p.new_pages_low = pl1 - pl0;
            p.tok0 = t0;
            p.tok1 = t1;
            if (ph1 > (uint32_t)c.max_pages || pl1 > (uint32_t)c.max_pages) { err |= PASK_DEV_SEQ_OVERFLOW; p.seq = -1; }
        }
        if (err) atomicOr(&c.ctrl[kCtrlStatus], err);
        c.plan[i] = p;
        __threadfence();
        s_flag = (atomicAdd(&c.ctrl[kCtrlTicket], 1u) == (uint32_t)(n_seqs - 1));
    }
    __syncthreads();
    if (!s_flag) return;

    // ---- last CTA: allocate for the whole call and commit, or refuse
    __threadfence();
    constexpr int kPer = PASK_MAX_SEQS_PER_CALL / kBulkThreads;  // sequences per thread, blocked
    uint32_t nh[kPer], nl[kPer], ni[kPer];
    uint32_t sum_h = 0, sum_l = 0, sum_i = 0;
    int any_bad = 0;
#pragma unroll
    for (int r = 0; r < kPer; r++) {
        const int j = tid * kPer + r;
        nh[r] = nl[r] = ni[r] = 0;
        if (j < n_seqs) {
            const AppendPlan p = load_plan_cg(&c.plan[j]);
            if (p.seq < 0) any_bad = 1;
            nh[r] = p.new_pages_high;
            nl[r] = p.new_pages_low;
            ni[r] = pages_touched(p.old_high, p.cnt_high) + pages_touched(p.old_low, p.cnt_low);
        }
        sum_h += nh[r];
        sum_l += nl[r];
        sum_i += ni[r];
    }
    uint32_t need_h, need_l, n_items;
    uint32_t base_h = block_excl_scan(sum_h, s_scan, &need_h);
    uint32_t base_l = block_excl_scan(sum_l, s_scan, &need_l);
    uint32_t base_i = block_excl_scan(sum_i, s_scan, &n_items);
    any_bad = __syncthreads_or(any_bad);
    const uint32_t free_h = c.ctrl[kCtrlHighFree], next_h = c.ctrl[kCtrlHighNext];
    const uint32_t free_l = c.ctrl[kCtrlLowFree], next_l = c.ctrl[kCtrlLowNext];
    const bool fits = need_h <= free_h + (c.cap_high - next_h) && need_l <= free_l + (c.cap_low - next_l);
    __syncthreads();
    if (any_bad || !fits) {
        if (tid == 0) {
            if (!fits && !any_bad) atomicOr(&c.ctrl[kCtrlStatus], PASK_DEV_POOL_EXHAUSTED);
            c.ctrl[kCtrlPlanOk] = 0;
            c.ctrl[kCtrlSerial] = serial;
            c.ctrl[kCtrlTicket] = 0;
        }
        return;
    }
    const int grp = group;
#pragma unroll
    for (int r = 0; r < kPer; r++) {
        const int j = tid * kPer + r;
        if (j >= n_seqs) break;
        const AppendPlan p = load_plan_cg(&c.plan[j]);
        const size_t sl = (size_t)p.seq * c.n_layers + layer;
        s_first_h[j] = base_h;                     // where this sequence's new pages start in the call's numbering
        s_first_l[j] = base_l;
        base_h += nh[r];
        base_l += nl[r];
        c.item_base[j] = base_i;
        base_i += ni[r];
        c.n_high[sl] = p.old_high + p.cnt_high;
        c.n_low[sl] = p.old_low + p.cnt_low;
        pask_budget_state_t &b = c.budget[p.seq];
        const uint64_t n_tok = (uint64_t)p.cnt_high + p.cnt_low + p.cnt_drop;
        if (c.window) c.n_tok[sl] = p.old_tok + (uint32_t)n_tok;
        b.n_seen[grp] += n_tok;
        b.n_high[grp] += p.cnt_high;
        b.n_low[grp] += p.cnt_low;
        b.n_drop[grp] += p.cnt_drop;
        b.retained_bytes += (uint64_t)p.cnt_high * c.bytes_h + (uint64_t)p.cnt_low * c.bytes_l;
        b.full_bytes += n_tok * c.bytes_h;
        b.bad_tags += p.bad_tags;
        b.pages_high += nh[r];
        b.pages_low += nl[r];
    }
    // page tables: a warp per sequence, its lanes over the sequence's new pages (a prefill hands
    // out hundreds of pages per sequence)
    __syncthreads();
    for (int j = warp; j < n_seqs; j += kBulkThreads / 32) {
        const AppendPlan p = load_plan_cg(&c.plan[j]);
        const size_t sl = (size_t)p.seq * c.n_layers + layer;
        const uint32_t ph0 = (p.old_high + kPageTokens - 1) / kPageTokens, pl0 = (p.old_low + kPageTokens - 1) / kPageTokens;
        for (uint32_t x = lane; x < p.new_pages_high; x += 32) {
            const uint32_t kk = s_first_h[j] + x;
            c.tbl_high[sl * c.max_pages + ph0 + x] = kk < free_h ? c.free_high[free_h - 1 - kk] : next_h + (kk - free_h);
        }
        for (uint32_t x = lane; x < p.new_pages_low; x += 32) {
            const uint32_t kk = s_first_l[j] + x;
            c.tbl_low[sl * c.max_pages + pl0 + x] = kk < free_l ? c.free_low[free_l - 1 - kk] : next_l + (kk - free_l);
        }
    }
    if (tid == 0) {
        const uint32_t pop_h = need_h < free_h ? need_h : free_h, pop_l = need_l < free_l ? need_l : free_l;
        c.ctrl[kCtrlHighFree] = free_h - pop_h;
        c.ctrl[kCtrlHighNext] = next_h + (need_h - pop_h);
        c.ctrl[kCtrlLowFree] = free_l - pop_l;
        c.ctrl[kCtrlLowNext] = next_l + (need_l - pop_l);
        c.ctrl[kCtrlItems] = n_items;
        c.item_base[n_seqs] = n_items;
        c.ctrl[kCtrlPlanOk] = 1;
        c.ctrl[kCtrlSerial] = serial;
        c.ctrl[kCtrlTicket] = 0;
    }
}

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Persist one 16-byte chunk (8 head dims; chunk cch of KV head `head`, K if !which else V) of a token
// that takes action a (RETAIN-HIGH or RETAIN-LOW) at position `at` of its stream, which lives in
// pool page `page`.  The four lanes that hold the chunks of one 32-dim group must call together
// (RETAIN-LOW reduces the group's amax across them); the whole warp must be converged.
__device__ __forceinline__ void persist_chunk(const DevCache &c, uint32_t a, uint32_t at, uint32_t page, size_t sl, int head,
                                              int cch, int which, const uint4 x) {
    const uint32_t tau = at & 15u;
    if (page >= (a == PASK_ACTION_RETAIN_HIGH ? c.high_limit : c.cap_low)) {   // never expected: refuse, do not write
        atomicOr(&c.ctrl[kCtrlStatus], PASK_DEV_INTERNAL);
        return;
    }
    if (a == PASK_ACTION_RETAIN_HIGH) {
        uint8_t *dst = c.pool_high + (size_t)page * c.high_page_bytes + (size_t)head * kHighHeadBytes +
                       (which ? kHighTileBytes : 0);
        if (!which) {
            *reinterpret_cast<uint32_t *>(dst + high_k_pair_off((int)tau, 4 * cch)) = x.x;
            *reinterpret_cast<uint32_t *>(dst + high_k_pair_off((int)tau, 4 * cch + 1)) = x.y;
            *reinterpret_cast<uint32_t *>(dst + high_k_pair_off((int)tau, 4 * cch + 2)) = x.z;
            *reinterpret_cast<uint32_t *>(dst + high_k_pair_off((int)tau, 4 * cch + 3)) = x.w;
        } else {
            const int q = cch >> 2, g0 = 2 * (cch & 3);
            *reinterpret_cast<uint2 *>(dst + high_v_piece_off((int)tau, q, g0)) = make_uint2(x.x, x.y);
            *reinterpret_cast<uint2 *>(dst + high_v_piece_off((int)tau, q, g0 + 1)) = make_uint2(x.z, x.w);
        }
        return;
    }
    float f[8] = {bf16_lo(x.x), bf16_hi(x.x), bf16_lo(x.y), bf16_hi(x.y), bf16_lo(x.z), bf16_hi(x.z), bf16_lo(x.w), bf16_hi(x.w)};
    float amax = 0.0f;
#pragma unroll
    for (int e = 0; e < 8; e++) amax = fmaxf(amax, fabsf(f[e]));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));   // the 4 chunks of a 32-dim group
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));   // sit in 4 adjacent lanes
    if (c.low_bits == 8) {   // eight-bit codes: the same recipe with 127 in place of 7, codes offset by 128
        uint8_t *dst8 = c.pool_low + (size_t)page * c.low_page_bytes + (size_t)head * kLow8HeadBytes + (which ? kLow8HalfBytes : 0);
        __half sh8 = __float2half_rn(__fdiv_rn(amax, 127.0f));
        if (__hisinf(sh8)) sh8 = __ushort_as_half((unsigned short)0x7BFF);
        const float s8 = __half2float(sh8);
        const float inv8 = s8 == 0.0f ? 0.0f : __fdiv_rn(1.0f, s8);
        uint32_t code8[8];
#pragma unroll
        for (int e = 0; e < 8; e++) {   // clamp, then 1.5 * 2^23 + 128 leaves the rounded code in the low byte
            const float cl = fminf(fmaxf(__fmul_rn(f[e], inv8), -127.0f), 127.0f);
            code8[e] = __float_as_uint(__fadd_rn(cl, 12583040.0f)) & 255u;
        }
        if (!which) {
#pragma unroll
            for (int e = 0; e < 8; e += 2)
                *reinterpret_cast<uint16_t *>(dst8 + low8_k_off((int)tau, 8 * cch + e)) = (uint16_t)(code8[e] | (code8[e + 1] << 8));
        } else {
#pragma unroll
            for (int e = 0; e < 8; e++) dst8[low8_v_off((int)tau, 8 * cch + e)] = (uint8_t)code8[e];
        }
        if ((cch & 3) == 0) *reinterpret_cast<__half *>(dst8 + low8_scale_off((int)tau, cch >> 2)) = sh8;
        const uint32_t hb8 = __reduce_max_sync(0xffffffffu, which ? (uint32_t)__half_as_ushort(sh8) : 0u);
        if ((threadIdx.x & 31) == 0 && hb8) atomicMax(&c.low_vmax[sl], hb8);
        return;
    }
    if (c.low_bits == 2) {   // two-bit codes: the levels -s, 0, +s with s = fp16(amax), codes offset by 2
        uint8_t *dst2 = c.pool_low + (size_t)page * c.low_page_bytes + (size_t)head * kLow2HeadBytes + (which ? kLow2HalfBytes : 0);
        __half sh2 = __float2half_rn(amax);
        if (__hisinf(sh2)) sh2 = __ushort_as_half((unsigned short)0x7BFF);
        const float s2 = __half2float(sh2);
        const float inv2 = s2 == 0.0f ? 0.0f : __fdiv_rn(1.0f, s2);
        uint32_t code2[8];
#pragma unroll
        for (int e = 0; e < 8; e++) {   // clamp, then 1.5 * 2^23 + 2 leaves the rounded code in the low two bits
            const float cl = fminf(fmaxf(__fmul_rn(f[e], inv2), -1.0f), 1.0f);
            code2[e] = __float_as_uint(__fadd_rn(cl, 12582914.0f)) & 3u;
        }
        if (!which) {   // even dims in one byte, odd dims in the other
            dst2[low2_k_byte_off((int)tau, cch, 0)] = (uint8_t)(code2[0] | (code2[2] << 2) | (code2[4] << 4) | (code2[6] << 6));
            dst2[low2_k_byte_off((int)tau, cch, 1)] = (uint8_t)(code2[1] | (code2[3] << 2) | (code2[5] << 4) | (code2[7] << 6));
        } else {        // four consecutive dims per byte
            dst2[low2_v_byte_off((int)tau, 2 * cch)] = (uint8_t)(code2[0] | (code2[1] << 2) | (code2[2] << 4) | (code2[3] << 6));
            dst2[low2_v_byte_off((int)tau, 2 * cch + 1)] = (uint8_t)(code2[4] | (code2[5] << 2) | (code2[6] << 4) | (code2[7] << 6));
        }
        if ((cch & 3) == 0) *reinterpret_cast<__half *>(dst2 + low2_scale_off((int)tau, cch >> 2)) = sh2;
        const uint32_t hb2 = __reduce_max_sync(0xffffffffu, which ? (uint32_t)__half_as_ushort(sh2) : 0u);
        if ((threadIdx.x & 31) == 0 && hb2) atomicMax(&c.low_vmax[sl], hb2);
        return;
    }
    uint8_t *dst = c.pool_low + (size_t)page * c.low_page_bytes + (size_t)head * kLowHeadBytes + (which ? kLowHalfBytes : 0);
    const float s32 = __fdiv_rn(amax, 7.0f);
    __half sh = __float2half_rn(s32);
    if (__hisinf(sh)) sh = __ushort_as_half((unsigned short)0x7BFF);  // saturate, never infinite
    const float s = __half2float(sh);
    uint32_t code[8];
    if (s == 0.0f) {
#pragma unroll
        for (int e = 0; e < 8; e++) code[e] = 8u;
    } else {
        const float inv = __fdiv_rn(1.0f, s);
#pragma unroll
        for (int e = 0; e < 8; e++) {
            float r = rintf(__fmul_rn(f[e], inv));
            r = fminf(fmaxf(r, -7.0f), 7.0f);
            code[e] = (uint32_t)((int)r + 8);
        }
    }
    const int w = cch >> 2, u = cch & 3;
    if (!which) {
        uint32_t word = 0;
#pragma unroll
        for (int e = 0; e < 8; e++) word |= code[e] << (4 * low_k_nibble(e));
        *reinterpret_cast<uint32_t *>(dst + low_k_word_off((int)tau, w, u)) = word;
    } else {
        const uint16_t h0 = (uint16_t)(code[0] | (code[1] << 4) | (code[2] << 8) | (code[3] << 12));
        const uint16_t h1 = (uint16_t)(code[4] | (code[5] << 4) | (code[6] << 8) | (code[7] << 12));
        *reinterpret_cast<uint16_t *>(dst + low_v_half_off((int)tau, w, 2 * u)) = h0;
        *reinterpret_cast<uint16_t *>(dst + low_v_half_off((int)tau, w, 2 * u + 1)) = h1;
    }
    if (u == 0) *reinterpret_cast<__half *>(dst + low_scale_off((int)tau, w)) = sh;
    // decode attention forms P * (V scale) in fp16 relative to the stream's largest V scale:
    // keep that maximum per (sequence, layer) -- one atomic per warp, nothing comes back (no round trip)
    const uint32_t hb = __reduce_max_sync(0xffffffffu, which ? (uint32_t)__half_as_ushort(sh) : 0u);
    if ((threadIdx.x & 31) == 0 && hb) atomicMax(&c.low_vmax[sl], hb);
}

// General path, second kernel: page-centric.  The plan kernel left, per sequence, its retained
// tokens in stream order (tok_list) and a prefix over sequences of the stream pages the call
// writes into (item_base).  A work item is one such page; CTA b takes the items
// [T b / G, T (b+1) / G).  A page whose 16 tokens all come from this call -- nearly every page of
// a prefill -- is assembled head by head in shared memory from the 16 source rows and leaves as
// one run of 128-bit stores in the packed layout; a partly filled page (the first and last page of
// a stream's range at most) is written token by token with persist_chunk.
constexpr int kWriteThreads = 256;
constexpr int kRowPad = 16;                       // bytes between two staged rows (bank spread: rows are 2^k bytes)
constexpr long long kWriteWaitCycles = 2000000000LL;   // bound of the wait for a page's staged rows (about a second)

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
// waits for a phase of an mbarrier, at most `limit` clock cycles; false if it gave up
__device__ __noinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, long long limit) {
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; i++) {
            uint32_t done;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(done) : "r"(bar), "r"(parity) : "memory");
            if (done) return true;
        }
        if (clock64() - t0 > limit) return false;
    }
}

__global__ void __launch_bounds__(kWriteThreads, 3)
append_write_kernel(DevCache c, int layer, int n_seqs, const uint4 *__restrict__ k, const uint4 *__restrict__ v) {
    extern __shared__ __align__(16) uint8_t s_dyn[];                    // the page's source rows, see in_row()
    __shared__ __align__(16) uint8_t s_low[4][kLowHeadBytes];           // packed heads of a LOW page (two pairs in turn)
    __shared__ uint32_t s_tok[kPageTokens];
    __shared__ __align__(8) uint64_t s_bar;                             // completion of a page's row copies
    // source rows of the page being written: [K|V][token] whole rows (all heads, as they lie in memory), kRowPad apart
    const int row_bytes = c.n_kv * 2 * kHeadDim, row_stride = row_bytes + kRowPad;
    auto in_row = [&](int head, int which, int tau) -> uint8_t * {
        return s_dyn + (size_t)(which * kPageTokens + tau) * row_stride + head * (2 * kHeadDim);
    };
    if (c.ctrl[kCtrlPlanOk] == 0) return;
    const int tid = threadIdx.x;
    uint32_t bar_parity = 0;
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&s_bar)) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    const uint32_t n_items = c.ctrl[kCtrlItems];
    const uint32_t item0 = (uint32_t)(((uint64_t)n_items * blockIdx.x) / gridDim.x);
    const uint32_t item1 = (uint32_t)(((uint64_t)n_items * (blockIdx.x + 1)) / gridDim.x);
    if (item0 >= item1) return;
    // find the sequence item0 belongs to (base[j] <= item0 < base[j + 1]) with the prefix table staged
    // in the row buffer, which is free until the first page is fetched
    int j = 0;
    uint32_t base_j, base_next;
    {
        uint32_t *s_base = reinterpret_cast<uint32_t *>(s_dyn);
        for (int x = tid; x <= n_seqs; x += kWriteThreads) s_base[x] = c.item_base[x];
        __syncthreads();
        int lo = 0, hi = n_seqs - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (s_base[mid] <= item0) lo = mid; else hi = mid - 1;
        }
        j = lo;
        base_j = s_base[j];
        base_next = s_base[j + 1];
        __syncthreads();
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the buffer is next written by bulk copies
    }
    const int chunks = 16 * c.n_kv;                // 16-byte chunks per token per tensor (a power of two)
    const int chunks_shift = 31 - __clz(chunks);
    AppendPlan p = c.plan[j];
    for (uint32_t item = item0; item < item1; item++) {
        bool moved = false;
        while (item >= base_next) { j++; base_j = base_next; base_next = c.item_base[j + 1]; moved = true; }
        if (moved) p = c.plan[j];
        const uint32_t in_seq = item - base_j;
        const uint32_t items_h = pages_touched(p.old_high, p.cnt_high);
        const bool high = in_seq < items_h;
        const uint32_t old = high ? p.old_high : p.old_low, cnt = high ? p.cnt_high : p.cnt_low;
        const uint32_t pg = (old >> 4) + (high ? in_seq : in_seq - items_h);
        const uint32_t at0 = old > 16u * pg ? old : 16u * pg;
        const uint32_t at1 = old + cnt < 16u * pg + 16u ? old + cnt : 16u * pg + 16u;
        const size_t sl = (size_t)p.seq * c.n_layers + layer;
        const uint32_t page = (high ? c.tbl_high : c.tbl_low)[sl * c.max_pages + pg];
        const uint32_t action = high ? PASK_ACTION_RETAIN_HIGH : PASK_ACTION_RETAIN_LOW;
        __syncthreads();                           // the previous item is done with s_tok
        if ((uint32_t)tid < at1 - at0) {
            const uint32_t r = at0 + tid - old;     // rank among the sequence's tokens of this stream
            s_tok[tid] = c.tok_list[high ? p.tok0 + r : p.tok1 - 1 - r];
        }
        __syncthreads();
        if (at1 - at0 < (uint32_t)kPageTokens || page >= (high ? c.cap_high : c.cap_low)) {
            // partly filled page (or a page id the bounds check refuses): token by token
            if (tid < 2 * chunks) {
                const int which = tid >= chunks, cg = which ? tid - chunks : tid;
                for (uint32_t at = at0; at < at1; at++) {
                    const uint4 x = (which ? v : k)[(size_t)s_tok[at - at0] * chunks + cg];
                    persist_chunk(c, action, at, page, sl, cg >> 4, cg & 15, which, x);
                }
            }
            continue;
        }
        // ---- a full page: the 16 tokens' K rows and V rows (all heads of a token lie together) go to shared memory
        // as 32 bulk copies issued by one warp, completion counted on an mbarrier; then each head leaves as one
        // packed block
        if (tid < 2 * kPageTokens) {
            const int which = tid >> 4, tau = tid & 15;
            const uint32_t bar = smem_addr(&s_bar);
            if (tid == 0)
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(2u * kPageTokens * (uint32_t)row_bytes) : "memory");
            __syncwarp();
            const void *src = (which ? v : k) + (size_t)s_tok[tau] * chunks;
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_addr(in_row(0, which, tau))), "l"(src), "r"((uint32_t)row_bytes), "r"(bar) : "memory");
        }
        {   // bounded wait: rows that never arrive set the sticky time-out bit and end this CTA's work (after one more
            // bounded wait, so that no copy is still on its way into shared memory when the CTA retires)
            const bool ok = mbar_wait_bounded(smem_addr(&s_bar), bar_parity, kWriteWaitCycles);
            if (!__syncthreads_and(ok)) {
                mbar_wait_bounded(smem_addr(&s_bar), bar_parity, kWriteWaitCycles);
                if (tid == 0) atomicOr(&c.ctrl[kCtrlStatus], PASK_DEV_TIMEOUT);
                return;
            }
            bar_parity ^= 1u;
        }
        uint32_t vmax_bits = 0;
        for (int head = 0; head < c.n_kv; head++) {
            if (high) {
                uint4 *dst = reinterpret_cast<uint4 *>(c.pool_high + (size_t)page * c.high_page_bytes + (size_t)head * kHighHeadBytes);
                const int lane = tid & 31, g = lane >> 2, t = lane & 3, i = tid >> 5;
                {   // K tile, round i = 2 jj + hh: the operand quad of lane (g, t), see pask_layout.h
                    const int jj = i >> 1, hh = i & 1, off = 2 * (8 * (4 * jj + t) + 4 * hh);
                    uint4 q;
                    q.x = *reinterpret_cast<const uint32_t *>(in_row(head, 0, g) + off);
                    q.y = *reinterpret_cast<const uint32_t *>(in_row(head, 0, g + 8) + off);
                    q.z = *reinterpret_cast<const uint32_t *>(in_row(head, 0, g) + off + 4);
                    q.w = *reinterpret_cast<const uint32_t *>(in_row(head, 0, g + 8) + off + 4);
                    dst[tid] = q;
                }
                {   // V tile, round i = 4 e + kk: token {2t, 2t+1, 2t+8, 2t+9}[kk], dims 64e + 4g.. and 64e + 32 + 4g..
                    const int e = i >> 2, kk = i & 3, tau = 2 * t + (kk & 1) + 8 * (kk >> 1);
                    const uint2 a = *reinterpret_cast<const uint2 *>(in_row(head, 1, tau) + 128 * e + 8 * g);
                    const uint2 b = *reinterpret_cast<const uint2 *>(in_row(head, 1, tau) + 128 * e + 64 + 8 * g);
                    dst[256 + tid] = make_uint4(a.x, a.y, b.x, b.y);
                }
            } else {
                if (c.low_bits == 4) break;     // four-bit codes: two heads at a time, below
                // thread = (K|V, token, 32-dim group, half of it): 16 values
                const int half = tid & 1, w = (tid >> 1) & 3, tau = (tid >> 3) & 15, which = tid >> 7;
                const uint4 x0 = *reinterpret_cast<const uint4 *>(in_row(head, which, tau) + 64 * w + 32 * half);
                const uint4 x1 = *reinterpret_cast<const uint4 *>(in_row(head, which, tau) + 64 * w + 32 * half + 16);
                const uint32_t xs[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
                // amax on the packed bf16 pairs (abs and max are exact in any format)
                __nv_bfloat162 m2 = __habs2(*reinterpret_cast<const __nv_bfloat162 *>(&xs[0]));
#pragma unroll
                for (int e = 1; e < 8; e++) m2 = __hmax2(m2, __habs2(*reinterpret_cast<const __nv_bfloat162 *>(&xs[e])));
                const uint32_t m2b = *reinterpret_cast<const uint32_t *>(&m2);
                float amax = fmaxf(bf16_lo(m2b), bf16_hi(m2b));
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
                if (c.low_bits == 8) {
                    // eight-bit codes: this thread's 16 values are the k-chunk 2w + half of its token.
                    // One image buffer (both halves of s_low): wait until the previous head has left.
                    __half sh8 = __float2half_rn(__fdiv_rn(amax, 127.0f));
                    if (__hisinf(sh8)) sh8 = __ushort_as_half((unsigned short)0x7BFF);
                    const float s8 = __half2float(sh8);
                    const float inv8 = s8 == 0.0f ? 0.0f : __fdiv_rn(1.0f, s8);
                    uint32_t c8[16];
#pragma unroll
                    for (int e = 0; e < 16; e++) {
                        const float f = (e & 1) ? bf16_hi(xs[e >> 1]) : bf16_lo(xs[e >> 1]);
                        const float cl = fminf(fmaxf(__fmul_rn(f, inv8), -127.0f), 127.0f);
                        c8[e] = __float_as_uint(__fadd_rn(cl, 12583040.0f)) & 255u;
                    }
                    __syncthreads();
                    uint8_t *img8 = &s_low[0][0] + (which ? kLow8HalfBytes : 0);
                    const int d0 = 32 * w + 16 * half;
                    if (!which) {
#pragma unroll
                        for (int e = 0; e < 16; e += 2)
                            *reinterpret_cast<uint16_t *>(img8 + low8_k_off(tau, d0 + e)) = (uint16_t)(c8[e] | (c8[e + 1] << 8));
                    } else {
#pragma unroll
                        for (int e = 0; e < 16; e++) img8[low8_v_off(tau, d0 + e)] = (uint8_t)c8[e];
                        vmax_bits = max(vmax_bits, (uint32_t)__half_as_ushort(sh8));
                    }
                    if (half == 0) *reinterpret_cast<__half *>(img8 + low8_scale_off(tau, w)) = sh8;
                    __syncthreads();
                    uint4 *dst8 = reinterpret_cast<uint4 *>(c.pool_low + (size_t)page * c.low_page_bytes + (size_t)head * kLow8HeadBytes);
                    for (int x = tid; x < kLow8HeadBytes / 16; x += kWriteThreads) dst8[x] = reinterpret_cast<const uint4 *>(&s_low[0][0])[x];
                    continue;
                }
                if (c.low_bits == 2) {
                    // two-bit codes: this thread's 16 values are the chunks 4w + 2 half, +1 of its token's row
                    __half sh2 = __float2half_rn(amax);
                    if (__hisinf(sh2)) sh2 = __ushort_as_half((unsigned short)0x7BFF);
                    const float s2 = __half2float(sh2);
                    const float inv2 = s2 == 0.0f ? 0.0f : __fdiv_rn(1.0f, s2);
                    uint32_t c2[16];
#pragma unroll
                    for (int e = 0; e < 16; e++) {
                        const float f = (e & 1) ? bf16_hi(xs[e >> 1]) : bf16_lo(xs[e >> 1]);
                        const float cl = fminf(fmaxf(__fmul_rn(f, inv2), -1.0f), 1.0f);
                        c2[e] = __float_as_uint(__fadd_rn(cl, 12582914.0f)) & 3u;
                    }
                    uint8_t *img2 = s_low[head & 1] + (which ? kLow2HalfBytes : 0);
                    if (!which) {
#pragma unroll
                        for (int cc = 0; cc < 2; cc++)
#pragma unroll
                            for (int e = 0; e < 2; e++)
                                img2[low2_k_byte_off(tau, 4 * w + 2 * half + cc, e)] =
                                    (uint8_t)(c2[8 * cc + e] | (c2[8 * cc + 2 + e] << 2) | (c2[8 * cc + 4 + e] << 4) | (c2[8 * cc + 6 + e] << 6));
                    } else {
#pragma unroll
                        for (int uu = 0; uu < 4; uu++)
                            img2[low2_v_byte_off(tau, 8 * w + 4 * half + uu)] =
                                (uint8_t)(c2[4 * uu] | (c2[4 * uu + 1] << 2) | (c2[4 * uu + 2] << 4) | (c2[4 * uu + 3] << 6));
                        vmax_bits = max(vmax_bits, (uint32_t)__half_as_ushort(sh2));
                    }
                    if (half == 0) *reinterpret_cast<__half *>(img2 + low2_scale_off(tau, w)) = sh2;
                    __syncthreads();
                    uint4 *dst2 = reinterpret_cast<uint4 *>(c.pool_low + (size_t)page * c.low_page_bytes + (size_t)head * kLow2HeadBytes);
                    if (tid < kLow2HeadBytes / 16) dst2[tid] = reinterpret_cast<const uint4 *>(s_low[head & 1])[tid];
                    continue;
                }
            }
        }
        if (!high && c.low_bits == 4) {
            // Four-bit codes.  thread = (head of a pair, K|V, 32-dim group, token): one whole group, 32 values -- the
            // group's amax, scale and reciprocal are worked out once, by one thread.  A quarter warp reads eight
            // different rows (kRowPad apart: no bank conflicts).
            const int hsel = tid >> 7, which = (tid >> 6) & 1, w = (tid >> 4) & 3, tau = tid & 15;
            for (int hp = 0; hp < c.n_kv; hp += 2) {
                const int head = hp + hsel;
                uint8_t *img = s_low[(hp & 2) + hsel] + (which ? kLowHalfBytes : 0);
                if (head < c.n_kv) {
                    uint32_t xs[16];
#pragma unroll
                    for (int q4 = 0; q4 < 4; q4++) {
                        const uint4 x = *reinterpret_cast<const uint4 *>(in_row(head, which, tau) + 64 * w + 16 * q4);
                        xs[4 * q4] = x.x; xs[4 * q4 + 1] = x.y; xs[4 * q4 + 2] = x.z; xs[4 * q4 + 3] = x.w;
                    }
                    // amax on the packed bf16 pairs (abs and max are exact in any format)
                    __nv_bfloat162 m2 = __habs2(*reinterpret_cast<const __nv_bfloat162 *>(&xs[0]));
#pragma unroll
                    for (int e = 1; e < 16; e++) m2 = __hmax2(m2, __habs2(*reinterpret_cast<const __nv_bfloat162 *>(&xs[e])));
                    const uint32_t m2b = *reinterpret_cast<const uint32_t *>(&m2);
                    const float amax = fmaxf(bf16_lo(m2b), bf16_hi(m2b));
                    const float s32 = __fdiv_rn(amax, 7.0f);
                    __half sh = __float2half_rn(s32);
                    if (__hisinf(sh)) sh = __ushort_as_half((unsigned short)0x7BFF);   // saturate, never infinite
                    const float sc = __half2float(sh);
                    // code = clamp(rint(x * (1/s)), -7, 7) + 8.  Clamping first gives the same integer (the bounds are
                    // integers), and adding 1.5 * 2^23 + 8 to a value in [-7, 7] rounds it to the nearest integer, ties
                    // to even, leaving code in the low 4 bits of the sum.  s == 0 means every value is zero: 1/s is
                    // replaced by 0 and all codes come out 8.
                    const float inv = sc == 0.0f ? 0.0f : __fdiv_rn(1.0f, sc);
                    // The sums are kept as bit patterns, 0x4B400000 + code, and packed by multiply-adds (a nibble per
                    // step, from the top one down) instead of mask, shift and or per code: the constant upper bits add
                    // up to a known word that is taken off at the end (K words, modulo 2^32) or fall outside the result
                    // (V half-words).  A normal, unsaturated fp16 scale is within 2^-11 of amax / 7, so |x / s| < 7.01
                    // and the clamp cannot bite: it is only kept for subnormal scales (rounded coarsely) and the
                    // saturated one.
                    uint32_t raw[32];
                    const uint32_t sbits = __half_as_ushort(sh);
                    if (sbits >= 0x0400u && sbits < 0x7BFFu) {
#pragma unroll
                        for (int e = 0; e < 32; e++) {
                            const float f = (e & 1) ? bf16_hi(xs[e >> 1]) : bf16_lo(xs[e >> 1]);
                            raw[e] = __float_as_uint(__fadd_rn(__fmul_rn(f, inv), 12582920.0f));
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; e++) {
                            const float f = (e & 1) ? bf16_hi(xs[e >> 1]) : bf16_lo(xs[e >> 1]);
                            const float cl = fminf(fmaxf(__fmul_rn(f, inv), -7.0f), 7.0f);
                            raw[e] = __float_as_uint(__fadd_rn(cl, 12582920.0f));
                        }
                    }
                    if (!which) {
                        constexpr uint32_t kRawWord = 0x4B400000u * 0x11111111u;   // what eight constant parts add up to
#pragma unroll
                        for (int t = 0; t < 4; t++) {  // the word of dims 32w + 8t .. +7
                            uint32_t acc = raw[8 * t + 7];          // nibble n holds dim offset 2 (n & 3) + (n >> 2): low_k_nibble inverted
#pragma unroll
                            for (int n = 6; n >= 0; n--) acc = acc * 16u + raw[8 * t + 2 * (n & 3) + (n >> 2)];
                            *reinterpret_cast<uint32_t *>(img + low_k_word_off(tau, w, t)) = acc - kRawWord;
                        }
                    } else {
#pragma unroll
                        for (int g = 0; g < 8; g++) {  // the half-word of dims 32w + 4g .. +3
                            const uint32_t acc = ((raw[4 * g + 3] * 16u + raw[4 * g + 2]) * 16u + raw[4 * g + 1]) * 16u + raw[4 * g];
                            *reinterpret_cast<uint16_t *>(img + low_v_half_off(tau, w, g)) = (uint16_t)acc;
                        }
                        vmax_bits = max(vmax_bits, (uint32_t)__half_as_ushort(sh));
                    }
                    *reinterpret_cast<__half *>(img + low_scale_off(tau, w)) = sh;
                }
                __syncthreads();
                // the two packed heads leave; the next pair is assembled in the other two buffers meanwhile
                for (int x = tid; x < 2 * (kLowHeadBytes / 16); x += kWriteThreads) {
                    const int hh = x >= kLowHeadBytes / 16, r = hh ? x - kLowHeadBytes / 16 : x;
                    if (hp + hh < c.n_kv)
                        reinterpret_cast<uint4 *>(c.pool_low + (size_t)page * c.low_page_bytes + (size_t)(hp + hh) * kLowHeadBytes)[r] =
                            reinterpret_cast<const uint4 *>(s_low[(hp & 2) + hh])[r];
                }
            }
        }
        if (!high) {   // largest V scale of the stream (decode attention forms P * scale relative to it)
            const uint32_t hb = __reduce_max_sync(0xffffffffu, vmax_bits);
            if ((tid & 31) == 0 && hb > c.low_vmax[sl]) atomicMax(&c.low_vmax[sl], hb);
        }
    }
}

// floor(x / n) for x < 2^48 and 0 < n < 2^24 from inv = 1.0 / n: the product is within 2^-4 / n of x / n, a quotient
// that is not whole is at least 1 / n away from the next integer, so truncation is never too high and at most one
// too low (a whole quotient): one correction step makes it exact.
__device__ __forceinline__ uint32_t div_by(uint64_t x, uint32_t n, double inv) {
    uint32_t q = (uint32_t)__double2ll_rz((double)x * inv);
    if ((uint64_t)(q + 1) * n <= x) q++;
    return q;
}
// page_at() of pask_layout.h with the two divisions by n = nh + nl replaced by div_by
__device__ __forceinline__ bool page_at_rcp(uint32_t v, uint32_t nh, uint32_t n, double inv_n, uint32_t &idx) {
    const uint32_t h0 = div_by((uint64_t)v * nh, n, inv_n), h1 = div_by((uint64_t)(v + 1) * nh, n, inv_n);
    idx = h1 > h0 ? h0 : v - h0;
    return h1 > h0;
}

// Small calls (decode: a token or a few per sequence): the whole of pask_append_kv in one launch
// of one CTA per token, built so that the chain of dependent global round trips is as short as it
// can be.  The table column and the layer's group arrive as kernel arguments; every CTA fetches
// every per-sequence word in one round and works out the identical plan for the whole call in
// shared memory (decisions, ranks, page allocation by a scan); then it writes its own token.  All
// CTAs only read the cache state while planning; the CTA that finishes planning last (arrival
// counter, nobody waits) commits the counters, tables and budget states for everybody.
constexpr int kSmallMax = 255;       // at most this many sequences and tokens (one thread each, index n_seqs included)
constexpr int kSmallThreads = 256;

// (the kernel proper is the wrapper below: it places the dependency wait before or after this body)
__device__ __forceinline__ void
append_small_body(const DevCache &c, int layer, int group, int n_seqs, int total, const int32_t *__restrict__ seq_ids,
                  const int32_t *__restrict__ cu_tokens, const uint4 *__restrict__ k, const uint4 *__restrict__ v,
                  const uint8_t *__restrict__ tags, const uint8_t *__restrict__ decided,
                  uint8_t *__restrict__ actions_out, const SmallLut &lut, const int fuse_plan, const Workspace &ws,
                  int32_t *__restrict__ ids_out, const uint32_t n_role) {   // n_role: the CTAs that run this body (one per token)
    __shared__ int s_seq[kSmallMax], s_cu[kSmallMax + 1];
    __shared__ uint32_t s_cost[kSmallMax + 1], s_page[kSmallMax + 1], s_nh[kSmallMax], s_nl[kSmallMax];   // fused attention plan
    __shared__ uint32_t s_old_n[kSmallMax], s_nw[kSmallMax], s_wstart[kSmallMax], s_wlen[kSmallMax];
    __shared__ uint32_t s_old_h[kSmallMax], s_old_l[kSmallMax], s_cnt_h[kSmallMax], s_cnt_l[kSmallMax], s_cnt_bad[kSmallMax];
    __shared__ uint32_t s_new_h[kSmallMax], s_new_l[kSmallMax], s_base_h[kSmallMax], s_base_l[kSmallMax];
    __shared__ uint8_t s_act[kSmallMax], s_tok_seq[kSmallMax], s_tok_bad[kSmallMax];
    __shared__ uint32_t s_pos[kSmallMax], s_ctrl[4], s_err, s_scan3[kSmallThreads / 32][3];
    __shared__ int s_last;
    const int tid = threadIdx.x;
    // this CTA's token and this thread's chunk of it: fetch the data first, it depends on nothing
    const int my_tok = blockIdx.x;
    const int chunks = 16 * c.n_kv;
    const bool writer = tid < 2 * chunks;
    const int which = tid >= chunks, cg = which ? tid - chunks : tid;
    uint4 x = make_uint4(0, 0, 0, 0);
    if (writer) x = (which ? v : k)[(size_t)my_tok * chunks + cg];
    if (tid == 0) s_err = 0;
    if (tid < 4) s_ctrl[tid] = c.ctrl[kCtrlHighNext + tid];     // high next, high free, low next, low free
    if (tid <= n_seqs) s_cu[tid] = cu_tokens[tid];
    if (tid < n_seqs) {
        const int seq = seq_ids[tid];
        s_seq[tid] = seq;
        uint32_t oh = 0, ol = 0, on = 0;
        if (seq >= 0 && seq < c.max_seqs) {
            const size_t sl = (size_t)seq * c.n_layers + layer;
            oh = c.n_high[sl];
            ol = c.n_low[sl];
            if (c.window) on = c.n_tok[sl];
        }
        s_old_h[tid] = oh;
        s_old_l[tid] = ol;
        s_old_n[tid] = on;
    }
    // decide every token (Algorithm 2 steps 1-2, or step 7 on the actions pask_decide chose): needs nothing but the tag
    uint32_t err = 0;
    int my_act = 0;
    if (tid < total) {
        const int my_tag = tags[tid];
        my_act = lut.action[my_tag];
        if (decided) {
            my_act = decided[(size_t)tid * c.n_groups + group];
            if (my_act > PASK_ACTION_RETAIN_HIGH) { err |= PASK_DEV_BAD_ACTION; my_act = PASK_ACTION_RELEASE; }
        }
        s_act[tid] = (uint8_t)my_act;
        s_tok_bad[tid] = my_tag != PASK_TAG_PROTECTED && my_tag >= c.n_tags;
    }
    __syncthreads();

    // ---- validate the call
    if (tid < n_seqs) {
        const int seq = s_seq[tid];
        if (seq < 0 || seq >= c.max_seqs) err |= PASK_DEV_BAD_SEQ;
        if (s_cu[tid] < 0 || s_cu[tid + 1] < s_cu[tid] || (tid == 0 && s_cu[0] != 0) ||
            (tid == n_seqs - 1 && s_cu[n_seqs] != total)) err |= PASK_DEV_BAD_RAGGED;
        // the sequence each token belongs to (offsets are clamped here; a malformed table refuses the call below)
        const int t_end = s_cu[tid + 1] < total ? s_cu[tid + 1] : total;
        for (int t = s_cu[tid] > 0 ? s_cu[tid] : 0; t < t_end; t++) s_tok_seq[t] = (uint8_t)tid;
    }
    {   // a sequence named twice?  Every thread takes one sequence and a share of the distances to the others
        // (with one or two warps per scheduler every dependent instruction costs its full latency, so the work
        // is spread over all 256 threads, by powers of two, four loads at a time).
        const int lg = 32 - __clz(n_seqs - 1);            // n_seqs <= 2^lg <= 256
        const int i = tid & ((1 << lg) - 1), part = tid >> lg, per = kSmallThreads >> lg;
        if (i < n_seqs) {
            const int mine = s_seq[i];
            for (int r0 = part; r0 < n_seqs - 1; r0 += 4 * per) {
                int other[4];
#pragma unroll
                for (int u = 0; u < 4; u++) {
                    int j = i + 1 + r0 + u * per;
                    j = j >= n_seqs ? j - n_seqs : j;
                    other[u] = s_seq[j < n_seqs ? j : i];      // (past the last distance: compares with itself, masked below)
                }
#pragma unroll
                for (int u = 0; u < 4; u++) if (r0 + u * per < n_seqs - 1 && other[u] == mine) err |= PASK_DEV_BAD_SEQ;
            }
        }
    }
    if (err) atomicOr(&s_err, err);
    __syncthreads();
    if (s_err) {   // every CTA sees the same; the last one to get here resets the arrival counter
        if (tid == 0) {
            atomicOr(&c.ctrl[kCtrlStatus], s_err);
            if (atomicAdd(&c.ctrl[kCtrlTicket], 1u) == n_role - 1) { c.ctrl[kCtrlPlanOk] = 0; c.ctrl[kCtrlTicket] = 0; }
        }
        if (fuse_plan && blockIdx.x == 0 && tid <= n_seqs) ws.cost_prefix[tid] = ws.page_prefix[tid] = 0;   // nothing to attend
        return;
    }
    if (actions_out && blockIdx.x == 0 && tid < total) actions_out[tid] = (uint8_t)my_act;

    // ---- per token: rank inside its stream; per sequence: counts and new pages
    if (tid < total) {
        const int i = s_tok_seq[tid], a = s_act[tid];
        uint32_t pos = 0;
        for (int t = s_cu[i]; t < tid; t++) pos += s_act[t] == a;
        s_pos[tid] = pos;
    }
    if (tid < n_seqs) {
        uint32_t ch = 0, cl = 0, cb = 0;
        for (int t = s_cu[tid]; t < s_cu[tid + 1]; t++) {
            ch += s_act[t] == PASK_ACTION_RETAIN_HIGH;
            cl += s_act[t] == PASK_ACTION_RETAIN_LOW;
            cb += s_tok_bad[t];
        }
        s_cnt_h[tid] = ch; s_cnt_l[tid] = cl; s_cnt_bad[tid] = cb;
        const uint32_t oh = s_old_h[tid], ol = s_old_l[tid];
        const uint32_t ph1 = (oh + ch + kPageTokens - 1) / kPageTokens, pl1 = (ol + cl + kPageTokens - 1) / kPageTokens;
        s_new_h[tid] = ph1 - (oh + kPageTokens - 1) / kPageTokens;
        s_new_l[tid] = pl1 - (ol + kPageTokens - 1) / kPageTokens;
        if (ph1 > (uint32_t)c.max_pages || pl1 > (uint32_t)c.max_pages) atomicOr(&s_err, PASK_DEV_SEQ_OVERFLOW);
    }
    __syncthreads();

    // ---- what the fused decode-attention plan needs per sequence (what attn_plan_kernel would compute after this
    // append): tokens attended from the two streams and from the recent-window ring after the call
    const uint32_t W = c.window;
    uint32_t my_cost = 0, my_pages = 0;
    if (fuse_plan) {
        if (tid < n_seqs) {
            uint32_t nh = s_old_h[tid] + s_cnt_h[tid], nl = s_old_l[tid] + s_cnt_l[tid], nw = 0;
            if (W) {
                // The last min(W, tokens seen) tokens are attended from the bf16 ring whatever their action: the
                // streams are shortened by the window's HIGH and LOW members.  Here those among this call's tokens
                // (the last W of the sequence's tokens in the call at most) ...
                const uint32_t n_i = (uint32_t)(s_cu[tid + 1] - s_cu[tid]), n_new = s_old_n[tid] + n_i;
                nw = n_new < W ? n_new : W;
                for (uint32_t r = n_i > W ? n_i - W : 0u; r < n_i; r++) {
                    const uint32_t a = s_act[s_cu[tid] + r];
                    nh -= a == PASK_ACTION_RETAIN_HIGH;
                    nl -= a == PASK_ACTION_RETAIN_LOW;
                }
            }
            s_nh[tid] = nh; s_nl[tid] = nl; s_nw[tid] = nw;
            if (W) {   // ... and where the older members sit in the ring: slots [start, start + len) mod W (token index mod W)
                const uint32_t old_n = s_old_n[tid], n_new = old_n + (uint32_t)(s_cu[tid + 1] - s_cu[tid]);
                const uint32_t lo = n_new > W ? n_new - W : 0u;
                s_wlen[tid] = lo < old_n ? old_n - lo : 0u;
                s_wstart[tid] = lo % W;
            }
        }
        if (W) {
            __syncthreads();
            // ... and here those among the older tokens still in the window: token indices [n_new - W, old_n), whose
            // slots this call does not write.  One thread per 16 slots of a ring; actions are 0, 1, 2, so bit 0 of a byte
            // says LOW and bit 1 HIGH: four bytes are counted with two population counts under a byte mask.
            const int per = (int)W / kPageTokens;
            const uint32_t inv_per = (65536u + per - 1) / per;                    // idx / per for idx < 4096, per <= 16
            for (int idx = tid; idx < n_seqs * per; idx += kSmallThreads) {
                const int sq = (int)(((uint32_t)idx * inv_per) >> 16), i = idx - sq * per;
                const uint32_t len = s_wlen[sq];
                if (len == 0) continue;
                // the members' slots inside this piece [p0, p0 + 16), as a 16-bit mask: [a, b) and, wrapped, [0, b - W)
                const uint32_t a = s_wstart[sq], b = a + len, p0 = 16u * (uint32_t)i;
                auto piece_bits = [&](uint32_t from, uint32_t to) -> uint32_t {   // slots [from, to) clipped to the piece
                    const uint32_t f = from > p0 ? from - p0 : 0u, t = to > p0 ? (to - p0 < 16u ? to - p0 : 16u) : 0u;
                    return f < t ? ((1u << t) - 1u) & ~((1u << f) - 1u) : 0u;
                };
                const uint32_t m16 = piece_bits(a, b < W ? b : W) | (b > W ? piece_bits(0u, b - W) : 0u);
                if (m16 == 0) continue;
                const size_t slw = (size_t)s_seq[sq] * c.n_layers + layer;
                const uint4 a4 = reinterpret_cast<const uint4 *>(c.win_act + slw * W)[i];
                const uint32_t w4[4] = {a4.x, a4.y, a4.z, a4.w};
                uint32_t wh = 0, wl = 0;
#pragma unroll
                for (int k = 0; k < 4; k++) {
                    const uint32_t sel = (((m16 >> (4 * k)) & 15u) * 0x00204081u) & 0x01010101u;   // bit j -> bit 0 of byte j
                    wl += __popc(w4[k] & sel);
                    wh += __popc(w4[k] & (sel << 1));
                }
                if (wh) atomicSub(&s_nh[sq], wh);
                if (wl) atomicSub(&s_nl[sq], wl);
            }
            __syncthreads();
        }
        if (tid < n_seqs) {   // the ring's pages have the HIGH format and count as HIGH pages
            const uint32_t ph = (s_nh[tid] + kPageTokens - 1) / kPageTokens + (s_nw[tid] + kPageTokens - 1) / kPageTokens;
            const uint32_t pl = (s_nl[tid] + kPageTokens - 1) / kPageTokens;
            my_cost = ph * kCostHighPage + pl * c.cost_low_page;
            my_pages = ph + pl;
        }
    }

    // ---- one exclusive scan over the call's sequences for three things: the pages the call allocates
    // (sequence-major like the general path; HIGH pages in the low half-word, LOW pages in the high one: a call
    // of at most 255 tokens allocates fewer than 2^16), and the plan's cost and page prefixes
    uint32_t need_h, need_l;
    {
        uint32_t v3[3] = {tid < n_seqs ? (s_new_h[tid] | (s_new_l[tid] << 16)) : 0u, my_cost, my_pages}, tot3[3];
        block_excl_scan3(v3, s_scan3, tot3);
        need_h = tot3[0] & 0xffffu; need_l = tot3[0] >> 16;
        if (tid < n_seqs) {
            s_base_h[tid] = v3[0] & 0xffffu; s_base_l[tid] = v3[0] >> 16;
            s_cost[tid + 1] = v3[1] + my_cost; s_page[tid + 1] = v3[2] + my_pages;
        }
        if (tid == 0) s_cost[0] = s_page[0] = 0;
        const bool fits = need_h <= s_ctrl[1] + (c.cap_high - s_ctrl[0]) && need_l <= s_ctrl[3] + (c.cap_low - s_ctrl[2]);
        if (tid == 0 && !fits && !s_err) atomicOr(&s_err, PASK_DEV_POOL_EXHAUSTED);
    }
    __syncthreads();
    if (fuse_plan && blockIdx.x == 0) {          // (block 0 writes the prefix)
        if (tid == 0) snap_cost_prefix(s_cost, n_seqs, c.attn_ctas);
        __syncthreads();
    }
    // old page of this CTA's token, if it continues one (page tables are only appended to by the commit)
    uint32_t my_page = 0, my_at = 0;
    const uint32_t my_a = s_act[my_tok];
    const int my_i = s_tok_seq[my_tok];
    const size_t my_sl = (size_t)s_seq[my_i] * c.n_layers + layer;
    if (my_a != PASK_ACTION_RELEASE) {
        const bool high = my_a == PASK_ACTION_RETAIN_HIGH;
        const uint32_t old = high ? s_old_h[my_i] : s_old_l[my_i];
        my_at = old + s_pos[my_tok];
        const uint32_t old_pages = (old + kPageTokens - 1) / kPageTokens, pg = my_at >> 4;
        if (pg < old_pages) {
            my_page = (high ? c.tbl_high : c.tbl_low)[my_sl * c.max_pages + pg];
        } else {   // one of the pages this call allocates: same formula as the commit below
            const uint32_t kk = (high ? s_base_h[my_i] : s_base_l[my_i]) + (pg - old_pages);
            const uint32_t fr = high ? s_ctrl[1] : s_ctrl[3], nx = high ? s_ctrl[0] : s_ctrl[2];
            my_page = kk < fr ? (high ? c.free_high : c.free_low)[fr - 1 - kk] : nx + (kk - fr);
        }
    }
    // ---- the fused plan itself: every CTA knows every sequence's lengths after the call and the ids of the pages
    // the call allocates, so the plan needs nothing that the commit writes
    if (fuse_plan && !s_err) {
        if (blockIdx.x == 0) {
            if (tid <= n_seqs) { ws.cost_prefix[tid] = s_cost[tid]; ws.page_prefix[tid] = s_page[tid]; }
            if (tid < n_seqs) ws.tokens[tid] = make_uint2(s_nh[tid], s_nl[tid]);
            if (ids_out && tid < n_seqs) ids_out[tid] = s_seq[tid];     // whom the plan is for
        }
        // the page-order list, a sequence at a time (CTA b takes sequences b, b + grid, ...): up to four entries per
        // thread and round, the page-table (or free-stack) reads of a round all in flight together
        for (int s = blockIdx.x; s < n_seqs; s += (int)n_role) {
            const uint32_t nh = s_nh[s], nl = s_nl[s], nw = s_nw[s];
            const uint32_t ph = (nh + kPageTokens - 1) / kPageTokens, pl = (nl + kPageTokens - 1) / kPageTokens;
            const uint32_t pw = (nw + kPageTokens - 1) / kPageTokens;
            const uint32_t old_h = (s_old_h[s] + kPageTokens - 1) / kPageTokens, old_l = (s_old_l[s] + kPageTokens - 1) / kPageTokens;
            const size_t slw = (size_t)s_seq[s] * c.n_layers + layer, sl = slw * c.max_pages;
            const uint32_t first = s_page[s], n_pos = ph + pw + pl;
            const double inv_n = 1.0 / (double)n_pos;   // for page_at_rcp: its two divisions by n_pos
            for (uint32_t v0 = tid; v0 < n_pos; v0 += 4 * kSmallThreads) {
                const uint32_t *src[4];    // where the page id is read from, or null when `val` already holds it
                uint32_t val[4], flags[4];
#pragma unroll
                for (int u = 0; u < 4; u++) {
                    const uint32_t v = v0 + u * kSmallThreads;
                    src[u] = nullptr; val[u] = 0; flags[u] = 0;
                    if (v >= n_pos) continue;
                    uint32_t idx;
                    if (page_at_rcp(v, ph + pw, n_pos, inv_n, idx)) {
                        flags[u] = kOrderHigh;
                        if (idx >= ph) {     // a page of the recent-window ring
                            val[u] = c.cap_high + (uint32_t)slw * (W / kPageTokens) + (idx - ph);
                            if (idx - ph == pw - 1) flags[u] |= (nw & (kPageTokens - 1)) << kOrderValidShift;
                        } else {
                            if (idx < old_h) {
                                src[u] = c.tbl_high + sl + idx;
                            } else {         // a page this call allocates: the commit's formula
                                const uint32_t kk = s_base_h[s] + (idx - old_h);
                                if (kk < s_ctrl[1]) src[u] = c.free_high + (s_ctrl[1] - 1 - kk); else val[u] = s_ctrl[0] + (kk - s_ctrl[1]);
                            }
                            if (idx == ph - 1) flags[u] |= (nh & (kPageTokens - 1)) << kOrderValidShift;
                        }
                    } else {
                        if (idx < old_l) {
                            src[u] = c.tbl_low + sl + idx;
                        } else {
                            const uint32_t kk = s_base_l[s] + (idx - old_l);
                            if (kk < s_ctrl[3]) src[u] = c.free_low + (s_ctrl[3] - 1 - kk); else val[u] = s_ctrl[2] + (kk - s_ctrl[3]);
                        }
                        if (idx == pl - 1) flags[u] |= (nl & (kPageTokens - 1)) << kOrderValidShift;
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; u++) if (src[u]) val[u] = *src[u];
#pragma unroll
                for (int u = 0; u < 4; u++) if (v0 + u * kSmallThreads < n_pos) ws.order[first + v0 + u * kSmallThreads] = val[u] | flags[u];
            }
        }
    }
    uint32_t pre_h = 0, pre_l = 0;
    // The token's bytes go out before the arrival ticket: nothing that another CTA still reads is written
    // (pages are only read by later kernels; the ring slots written are those of this call's tokens), the call
    // can no longer be refused (s_err is final), and the stores overlap the ticket's round trip.
    if (!s_err) {
        // ids of the first page each sequence gets from this call, fetched now for the commit
        if (tid < n_seqs) {
            if (s_new_h[tid]) { const uint32_t kk = s_base_h[tid]; pre_h = kk < s_ctrl[1] ? c.free_high[s_ctrl[1] - 1 - kk] : s_ctrl[0] + (kk - s_ctrl[1]); }
            if (s_new_l[tid]) { const uint32_t kk = s_base_l[tid]; pre_l = kk < s_ctrl[3] ? c.free_low[s_ctrl[3] - 1 - kk] : s_ctrl[2] + (kk - s_ctrl[3]); }
        }
        // ---- persist this CTA's token: one thread per 16-byte chunk of K and of V
        if (writer && my_a != PASK_ACTION_RELEASE) persist_chunk(c, my_a, my_at, my_page, my_sl, cg >> 4, cg & 15, which, x);

        // ---- protected recent window: every token, released ones too, also goes to slot (index mod W)
        // of its (sequence, layer) ring as bf16; of a sequence's tokens in this call only the last W can
        // still be in the window afterwards (and they have distinct slots)
        if (c.window) {
            const int W = (int)c.window, r = my_tok - s_cu[my_i], n_i = s_cu[my_i + 1] - s_cu[my_i];
            if (r >= n_i - W) {
                const uint32_t slot = (s_old_n[my_i] + (uint32_t)r) % (uint32_t)W;
                const uint32_t ring_page = c.cap_high + (uint32_t)my_sl * (uint32_t)(W >> 4) + (slot >> 4);
                if (writer) persist_chunk(c, PASK_ACTION_RETAIN_HIGH, slot, ring_page, my_sl, cg >> 4, cg & 15, which, x);
                if (tid == 0) c.win_act[my_sl * (size_t)W + slot] = (uint8_t)my_a;
            }
        }
    }
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(&c.ctrl[kCtrlTicket], 1u) == n_role - 1;   // every read of the old state is done
    __syncthreads();
    if (s_err) {
        if (tid == 0) {
            atomicOr(&c.ctrl[kCtrlStatus], s_err);
            if (s_last) { c.ctrl[kCtrlPlanOk] = 0; c.ctrl[kCtrlTicket] = 0; }
        }
        if (fuse_plan && blockIdx.x == 0 && tid <= n_seqs) ws.cost_prefix[tid] = ws.page_prefix[tid] = 0;   // nothing to attend
        return;
    }

    // ---- commit (last CTA to arrive only): page tables, stream lengths, budget states, pool state
    if (s_last && tid < n_seqs) {
        const int seq = s_seq[tid];
        const size_t sl = (size_t)seq * c.n_layers + layer;
        const uint32_t oh = s_old_h[tid], ol = s_old_l[tid], ch = s_cnt_h[tid], cl = s_cnt_l[tid];
        const uint32_t n_tok = (uint32_t)(s_cu[tid + 1] - s_cu[tid]);
        const uint32_t ph0 = (oh + kPageTokens - 1) / kPageTokens, pl0 = (ol + kPageTokens - 1) / kPageTokens;
        for (uint32_t x = 0; x < s_new_h[tid]; x++) {
            const uint32_t kk = s_base_h[tid] + x;
            c.tbl_high[sl * c.max_pages + ph0 + x] = x == 0 ? pre_h : kk < s_ctrl[1] ? c.free_high[s_ctrl[1] - 1 - kk] : s_ctrl[0] + (kk - s_ctrl[1]);
        }
        for (uint32_t x = 0; x < s_new_l[tid]; x++) {
            const uint32_t kk = s_base_l[tid] + x;
            c.tbl_low[sl * c.max_pages + pl0 + x] = x == 0 ? pre_l : kk < s_ctrl[3] ? c.free_low[s_ctrl[3] - 1 - kk] : s_ctrl[2] + (kk - s_ctrl[3]);
        }
        c.n_high[sl] = oh + ch;
        c.n_low[sl] = ol + cl;
        if (c.window) c.n_tok[sl] = s_old_n[tid] + n_tok;
        // budget state: additions only (no read-modify-write round trip); remaining_bytes is derived
        // from retained_bytes and full_bytes when the state is read
        pask_budget_state_t &b = c.budget[seq];
        budget_add(&b.n_seen[group], n_tok);
        budget_add(&b.n_high[group], ch);
        budget_add(&b.n_low[group], cl);
        budget_add(&b.n_drop[group], n_tok - ch - cl);
        budget_add(&b.retained_bytes, (uint64_t)ch * c.bytes_h + (uint64_t)cl * c.bytes_l);
        budget_add(&b.full_bytes, (uint64_t)n_tok * c.bytes_h);
        budget_add(&b.bad_tags, s_cnt_bad[tid]);
        if (s_new_h[tid]) atomicAdd(&b.pages_high, s_new_h[tid]);
        if (s_new_l[tid]) atomicAdd(&b.pages_low, s_new_l[tid]);
        if (tid == 0) {
            const uint32_t pop_h = need_h < s_ctrl[1] ? need_h : s_ctrl[1], pop_l = need_l < s_ctrl[3] ? need_l : s_ctrl[3];
            c.ctrl[kCtrlHighFree] = s_ctrl[1] - pop_h;
            c.ctrl[kCtrlHighNext] = s_ctrl[0] + (need_h - pop_h);
            c.ctrl[kCtrlLowFree] = s_ctrl[3] - pop_l;
            c.ctrl[kCtrlLowNext] = s_ctrl[2] + (need_l - pop_l);
            c.ctrl[kCtrlPlanOk] = 1;
            c.ctrl[kCtrlTicket] = 0;
        }
    }
}

__global__ void __launch_bounds__(kSmallThreads)
append_small_kernel(DevCache c, int layer, int group, int n_seqs, int total, const int32_t *__restrict__ seq_ids,
                    const int32_t *__restrict__ cu_tokens, const uint4 *__restrict__ k, const uint4 *__restrict__ v,
                    const uint8_t *__restrict__ tags, const uint8_t *__restrict__ decided,
                    uint8_t *__restrict__ actions_out, const SmallLut lut, const int fuse_plan, const Workspace ws) {
    pdl_launch_dependents();
    pdl_wait();
    append_small_body(c, layer, group, n_seqs, total, seq_ids, cu_tokens, k, v, tags, decided, actions_out, lut, fuse_plan, ws,
                      nullptr, gridDim.x);
}

// The kernel that ends a planned-ahead decode step.  Its first n_seqs CTAs run the one-launch append (one token per
// sequence) WITHOUT waiting for the kernel before them in the stream: that is the decode-attention kernel of the same
// layer, which works from a plan of the cache before this append, needs none of its results and touches nothing it
// writes, so the append runs in the shadow of that kernel's tail.  (Everything before that predecessor is complete:
// it has done its own wait before it let this kernel start.)  The other CTAs wait for the predecessor and merge its
// partials, the new tokens included; the kernel is complete when they are -- so whoever comes next in the stream and
// waits for this kernel has waited for both.  (The two roles have CTAs of their own: with a short streaming kernel the
// append, which also writes the next step's plan, ends after the partials are ready, and the merge does not queue
// behind it.)
__global__ void __launch_bounds__(kSmallThreads)
step_tail_kernel(DevCache c, int layer, int group, int n_seqs, const int32_t *__restrict__ seq_ids,
                 const int32_t *__restrict__ cu_tokens, const uint4 *__restrict__ k, const uint4 *__restrict__ v,
                 const uint8_t *__restrict__ tags, const uint8_t *__restrict__ decided, uint8_t *__restrict__ actions_out,
                 const SmallLut lut, const Workspace plan_ws, int32_t *__restrict__ ids_out, const uint32_t *__restrict__ prefix,
                 const float2 *__restrict__ part_ml, const float *__restrict__ part_o, float *__restrict__ out,
                 float *__restrict__ lse, int n_q, uint32_t n_ctas, uint32_t split, const NewTokens nt) {
    pdl_launch_dependents();
    if ((int)blockIdx.x < n_seqs) {
        // (no wait of its own: the kernel is complete only when its merging CTAs are, and those have waited)
        append_small_body(c, layer, group, n_seqs, n_seqs, seq_ids, cu_tokens, k, v, tags, decided, actions_out, lut, 1, plan_ws,
                          ids_out, (uint32_t)n_seqs);
        return;
    }
    merge_rows_with_new_token(prefix, part_ml, part_o, out, lse, n_seqs, n_q, n_ctas, split, nt, lut, (uint32_t)n_seqs);
}

// General path, recent window: CTA (j, y) copies the y-th newest of sequence j's tokens in this call
// (released ones too) into the sequence's ring as bf16 and records its action; only the last W
// tokens of a sequence can still be in the window afterwards, and they have distinct slots.
__global__ void __launch_bounds__(256)
append_window_kernel(DevCache c, int layer, const uint4 *__restrict__ k, const uint4 *__restrict__ v,
                     const uint8_t *__restrict__ tags, const uint8_t *__restrict__ decided) {
    if (c.ctrl[kCtrlPlanOk] == 0) return;
    const AppendPlan p = c.plan[blockIdx.x];
    const int tid = threadIdx.x, chunks = 16 * c.n_kv, W = (int)c.window;
    const int n = p.tok1 - p.tok0, group = c.layer_group[layer];
    if ((int)blockIdx.y >= n) return;
    const int r = n - 1 - (int)blockIdx.y, t = p.tok0 + r;
    const size_t sl = (size_t)p.seq * c.n_layers + layer;
    const int which = tid >= chunks, cg = which ? tid - chunks : tid;
    const uint32_t slot = (p.old_tok + (uint32_t)r) % (uint32_t)W;
    const uint32_t ring_page = c.cap_high + (uint32_t)sl * (uint32_t)(W >> 4) + (slot >> 4);
    if (tid < 2 * chunks) {
        const uint4 x = (which ? v : k)[(size_t)t * chunks + cg];
        persist_chunk(c, PASK_ACTION_RETAIN_HIGH, slot, ring_page, sl, cg >> 4, cg & 15, which, x);
    }
    if (tid == 0) {
        const int tag = tags[t];
        int a = tag < c.n_tags ? c.lut[tag * c.n_groups + group] : PASK_ACTION_RETAIN_HIGH;   // protected, unknown: high
        if (decided) a = decided[(size_t)t * c.n_groups + group];
        c.win_act[sl * (size_t)W + slot] = (uint8_t)a;
    }
}

// Return every page of one sequence to the free stacks and clear its counters.
__global__ void __launch_bounds__(256) seq_reset_kernel(DevCache c, int seq) {
    __shared__ uint32_t s_h, s_l;
    const int tid = threadIdx.x;
    if (tid == 0) { s_h = c.ctrl[kCtrlHighFree]; s_l = c.ctrl[kCtrlLowFree]; }
    __syncthreads();
    for (int layer = 0; layer < c.n_layers; layer++) {
        const size_t sl = (size_t)seq * c.n_layers + layer;
        const uint32_t ph = (c.n_high[sl] + kPageTokens - 1) / kPageTokens, pl = (c.n_low[sl] + kPageTokens - 1) / kPageTokens;
        const uint32_t bh = s_h, bl = s_l;
        for (uint32_t x = tid; x < ph; x += blockDim.x) c.free_high[bh + x] = c.tbl_high[sl * c.max_pages + x];
        for (uint32_t x = tid; x < pl; x += blockDim.x) c.free_low[bl + x] = c.tbl_low[sl * c.max_pages + x];
        __syncthreads();
        if (tid == 0) { s_h = bh + ph; s_l = bl + pl; c.n_high[sl] = 0; c.n_low[sl] = 0; c.low_vmax[sl] = 0; c.n_tok[sl] = 0; }
        __syncthreads();
    }
    if (tid == 0) { c.ctrl[kCtrlHighFree] = s_h; c.ctrl[kCtrlLowFree] = s_l; }
    uint32_t *b = reinterpret_cast<uint32_t *>(&c.budget[seq]);
    for (int x = tid; x < (int)(sizeof(pask_budget_state_t) / 4); x += blockDim.x) b[x] = 0;
}

}  // namespace

pask_status_t launch_append(pask_cache *c, int layer, int n_seqs, int total_tokens, const int32_t *seq_ids,
                            const int32_t *cu_tokens, const void *k, const void *v, const uint8_t *tags,
                            const uint8_t *decided, uint8_t *actions_out, cudaStream_t stream, const Workspace *fuse_ws,
                            bool *fused) {
    if (fused) *fused = false;
    if (n_seqs <= kSmallMax && total_tokens <= kSmallMax) {
        SmallLut lut;
        const int group = c->layer_group[layer];
        fill_small_lut(c, layer, &lut);
        if (total_tokens == 0) return PASK_OK;
        const int fuse = fuse_ws != nullptr;
        if (fused) *fused = fuse != 0;
        const cudaError_t e = launch_pdl(append_small_kernel, dim3(total_tokens), dim3(kSmallThreads), 0, stream, c->dev, layer,
                                         group, n_seqs, total_tokens, seq_ids, cu_tokens, static_cast<const uint4 *>(k),
                                         static_cast<const uint4 *>(v), tags, decided, actions_out, lut, fuse,
                                         fuse ? *fuse_ws : Workspace{});
        return e == cudaSuccess ? PASK_OK : PASK_ERR_CUDA;
    }
    append_plan_kernel<<<n_seqs, kBulkThreads, 0, stream>>>(c->dev, layer, n_seqs, total_tokens, seq_ids, cu_tokens, tags,
                                                           decided, actions_out);
    if (total_tokens > 0) {
        // at most one item per 16 tokens plus two partly filled pages per stream
        const long long bound = (long long)total_tokens / 16 + 4LL * n_seqs;
        const int ctas = bound < (long long)c->sm_count * 3 ? (int)bound : c->sm_count * 3;
        const size_t smem = (size_t)2 * kPageTokens * (c->desc.n_kv_heads * 2 * kHeadDim + kRowPad);
        if (cudaFuncSetAttribute(append_write_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return PASK_ERR_CUDA;
        append_write_kernel<<<ctas, kWriteThreads, smem, stream>>>(c->dev, layer, n_seqs, static_cast<const uint4 *>(k),
                                                                  static_cast<const uint4 *>(v));
    }
    if (c->dev.window && total_tokens > 0)
        append_window_kernel<<<dim3(n_seqs, c->dev.window), 256, 0, stream>>>(c->dev, layer, static_cast<const uint4 *>(k),
                                                        static_cast<const uint4 *>(v), tags, decided);
    return cudaGetLastError() == cudaSuccess ? PASK_OK : PASK_ERR_CUDA;
}

void fill_small_lut(const pask_cache *c, int layer, SmallLut *lut) {
    const int group = c->layer_group[layer];
    for (int z = 0; z < 256; z++)
        lut->action[z] = z < c->dev.n_tags ? c->lut[(size_t)z * c->dev.n_groups + group] : (uint8_t)PASK_ACTION_RETAIN_HIGH;
}

pask_status_t launch_step_tail(pask_cache *c, int layer, int n_seqs, const int32_t *seq_ids, const int32_t *cu_tokens,
                               const void *k, const void *v, const uint8_t *tags, const uint8_t *decided, uint8_t *actions_out,
                               const Workspace &plan_ws, int32_t *ids_out, const uint32_t *prefix, const float2 *part_ml,
                               const float *part_o, float *out, float *lse, const NewTokens &nt, cudaStream_t stream) {
    if (n_seqs < 1 || n_seqs > kSmallMax) return PASK_ERR_UNSUPPORTED_SHAPE;
    SmallLut lut;
    fill_small_lut(c, layer, &lut);
    static_assert(kSmallThreads == kMergeThreads, "the append role and the merge share one CTA shape");
    const int n_q = c->desc.n_q_heads, split = merge_split(n_seqs, c->attn_ctas);
    const int merge_ctas = (n_seqs * n_q * split + 7) / 8;      // `split` warps per (sequence, query head)
    const cudaError_t e = launch_pdl(step_tail_kernel, dim3(n_seqs + merge_ctas), dim3(kSmallThreads), 0,
                                     stream, c->dev, layer, (int)c->layer_group[layer], n_seqs, seq_ids, cu_tokens,
                                     static_cast<const uint4 *>(k), static_cast<const uint4 *>(v), tags, decided, actions_out, lut,
                                     plan_ws, ids_out, prefix, part_ml, part_o, out, lse, n_q, (uint32_t)c->attn_ctas,
                                     (uint32_t)split, nt);
    return e == cudaSuccess ? PASK_OK : PASK_ERR_CUDA;
}

pask_status_t launch_seq_reset(pask_cache *c, int seq, cudaStream_t stream) {
    seq_reset_kernel<<<1, 256, 0, stream>>>(c->dev, seq);
    return cudaGetLastError() == cudaSuccess ? PASK_OK : PASK_ERR_CUDA;
}

}  // namespace pask
