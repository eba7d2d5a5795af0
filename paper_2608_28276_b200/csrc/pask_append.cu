// pask_append_kv: table lookup, per-stream compaction, deterministic page allocation, budget
// accounting (plan kernel) and the drop / int4-quantise / bf16-keep writes (write kernel).
//
// Algorithm 2 of the paper, steps 1-2 (lookup, a = max(a0, floor)), 7 (persist) and 8 (budget
// recurrence), applied to a ragged batch of tokens for one layer.
#include <cuda_fp16.h>

#include "pask_internal.h"

namespace pask {

namespace {

constexpr int kPlanThreads = 256;

// Plan records are written by other CTAs of the same launch: read them through L2.
__device__ __forceinline__ AppendPlan load_plan_cg(const AppendPlan *p) {
    union { AppendPlan plan; uint4 q[4]; } u;
    const uint4 *src = reinterpret_cast<const uint4 *>(p);
#pragma unroll
    for (int i = 0; i < 4; i++) u.q[i] = __ldcg(src + i);
    return u.plan;
}

__device__ __forceinline__ uint32_t lanemask_lt() {
    uint32_t m;
    asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
    return m;
}

// exclusive scan of one value per thread over a 256-thread block; returns the block total too
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
    for (int w = 0; w < kPlanThreads / 32; w++) {
        const uint32_t x = s_warp[w];
        if (w < warp) before += x;
        tot += x;
    }
    __syncthreads();
    *total = tot;
    return before + inc - v;
}

// One CTA per sequence of the call: decide every token, rank it inside its stream, record the
// per-sequence plan; the CTA that arrives last allocates pages for the whole call (exclusive scan
// over sequences in call order, so ids do not depend on scheduling) and commits all counters --
// or refuses the whole call.
__global__ void __launch_bounds__(kPlanThreads)
append_plan_kernel(DevCache c, int layer, int n_seqs, int total_tokens, const int32_t *__restrict__ seq_ids,
                   const int32_t *__restrict__ cu_tokens, const uint8_t *__restrict__ tags,
                   uint8_t *__restrict__ actions_out, uint32_t serial) {
    __shared__ uint8_t s_lut[256];
    __shared__ uint32_t s_wh[kPlanThreads / 32], s_wl[kPlanThreads / 32], s_wb[kPlanThreads / 32];
    __shared__ uint32_t s_scan[kPlanThreads / 32];
    __shared__ uint32_t s_run_h, s_run_l, s_run_b;
    __shared__ int s_flag;
    const int i = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int group = c.layer_group[layer];
    s_lut[tid] = tid < c.n_tags ? c.lut[tid * c.n_groups + group] : (uint8_t)PASK_ACTION_RETAIN_HIGH;
    const int seq = seq_ids[i];
    const int t0 = cu_tokens[i], t1 = cu_tokens[i + 1];
    uint32_t err = 0;
    if (t0 < 0 || t1 < t0 || t1 > total_tokens || (i == 0 && t0 != 0) || (i == n_seqs - 1 && t1 != total_tokens))
        err |= PASK_DEV_BAD_RAGGED;
    if (seq < 0 || seq >= c.max_seqs) err |= PASK_DEV_BAD_SEQ;
    if (tid == 0) {
        s_run_h = s_run_l = s_run_b = 0;
        if (!(err & PASK_DEV_BAD_SEQ) && atomicExch(&c.seq_mark[seq], serial) == serial) s_flag = 1;  // named twice
        else s_flag = 0;
    }
    __syncthreads();
    if (s_flag) err |= PASK_DEV_BAD_SEQ;

    if (!err) {
        for (int base = t0; base < t1; base += kPlanThreads) {
            const int t = base + tid;
            const bool valid = t < t1;
            int a = 3;
            bool bad = false;
            if (valid) {
                const int tag = tags[t];
                a = s_lut[tag];
                bad = tag != PASK_TAG_PROTECTED && tag >= c.n_tags;
            }
            const uint32_t mh = __ballot_sync(0xffffffffu, a == PASK_ACTION_RETAIN_HIGH);
            const uint32_t ml = __ballot_sync(0xffffffffu, a == PASK_ACTION_RETAIN_LOW);
            const uint32_t mb = __ballot_sync(0xffffffffu, bad);
            if (lane == 0) { s_wh[warp] = __popc(mh); s_wl[warp] = __popc(ml); s_wb[warp] = __popc(mb); }
            __syncthreads();
            uint32_t off_h = s_run_h, off_l = s_run_l, tot_h = 0, tot_l = 0, tot_b = 0;
#pragma unroll
            for (int w = 0; w < kPlanThreads / 32; w++) {
                if (w < warp) { off_h += s_wh[w]; off_l += s_wl[w]; }
                tot_h += s_wh[w]; tot_l += s_wl[w]; tot_b += s_wb[w];
            }
            if (valid) {
                uint32_t pos = 0;
                if (a == PASK_ACTION_RETAIN_HIGH) pos = off_h + __popc(mh & lanemask_lt());
                else if (a == PASK_ACTION_RETAIN_LOW) pos = off_l + __popc(ml & lanemask_lt());
                c.tok_scratch[t] = make_uint2((uint32_t)a | (pos << 2), (uint32_t)i);
                if (actions_out) actions_out[t] = (uint8_t)a;
            }
            __syncthreads();
            if (tid == 0) { s_run_h += tot_h; s_run_l += tot_l; s_run_b += tot_b; }
            __syncthreads();
        }
    }

    if (tid == 0) {
        AppendPlan p{};
        p.seq = err ? -1 : seq;
        if (!err) {
            const size_t sl = (size_t)seq * c.n_layers + layer;
            p.old_high = c.n_high[sl];
            p.old_low = c.n_low[sl];
            p.cnt_high = s_run_h;
            p.cnt_low = s_run_l;
            p.cnt_drop = (uint32_t)(t1 - t0) - s_run_h - s_run_l;
            p.bad_tags = s_run_b;
            const uint32_t ph0 = (p.old_high + kPageTokens - 1) / kPageTokens, ph1 = (p.old_high + p.cnt_high + kPageTokens - 1) / kPageTokens;
            const uint32_t pl0 = (p.old_low + kPageTokens - 1) / kPageTokens, pl1 = (p.old_low + p.cnt_low + kPageTokens - 1) / kPageTokens;
            p.new_pages_high = ph1 - ph0;
            p.new_pages_low = pl1 - pl0;
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
    constexpr int kPer = PASK_MAX_SEQS_PER_CALL / kPlanThreads;  // sequences per thread, blocked
    uint32_t nh[kPer], nl[kPer];
    uint32_t sum_h = 0, sum_l = 0;
    int any_bad = 0;
#pragma unroll
    for (int r = 0; r < kPer; r++) {
        const int j = tid * kPer + r;
        nh[r] = nl[r] = 0;
        if (j < n_seqs) {
            const AppendPlan p = load_plan_cg(&c.plan[j]);
            if (p.seq < 0) any_bad = 1;
            nh[r] = p.new_pages_high;
            nl[r] = p.new_pages_low;
        }
        sum_h += nh[r];
        sum_l += nl[r];
    }
    uint32_t need_h, need_l;
    uint32_t base_h = block_excl_scan(sum_h, s_scan, &need_h);
    uint32_t base_l = block_excl_scan(sum_l, s_scan, &need_l);
    any_bad = __syncthreads_or(any_bad);
    const uint32_t free_h = c.ctrl[kCtrlHighFree], next_h = c.ctrl[kCtrlHighNext];
    const uint32_t free_l = c.ctrl[kCtrlLowFree], next_l = c.ctrl[kCtrlLowNext];
    const bool fits = need_h <= free_h + (c.cap_high - next_h) && need_l <= free_l + (c.cap_low - next_l);
    __syncthreads();
    if (any_bad || !fits) {
        if (tid == 0) {
            if (!fits && !any_bad) atomicOr(&c.ctrl[kCtrlStatus], PASK_DEV_POOL_EXHAUSTED);
            c.ctrl[kCtrlPlanOk] = 0;
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
        const uint32_t ph0 = (p.old_high + kPageTokens - 1) / kPageTokens, pl0 = (p.old_low + kPageTokens - 1) / kPageTokens;
        for (uint32_t x = 0; x < nh[r]; x++) {
            const uint32_t kk = base_h + x;
            c.tbl_high[sl * c.max_pages + ph0 + x] = kk < free_h ? c.free_high[free_h - 1 - kk] : next_h + (kk - free_h);
        }
        for (uint32_t x = 0; x < nl[r]; x++) {
            const uint32_t kk = base_l + x;
            c.tbl_low[sl * c.max_pages + pl0 + x] = kk < free_l ? c.free_low[free_l - 1 - kk] : next_l + (kk - free_l);
        }
        base_h += nh[r];
        base_l += nl[r];
        c.n_high[sl] = p.old_high + p.cnt_high;
        c.n_low[sl] = p.old_low + p.cnt_low;
        pask_budget_state_t &b = c.budget[p.seq];
        const uint64_t n_tok = (uint64_t)p.cnt_high + p.cnt_low + p.cnt_drop;
        b.n_seen[grp] += n_tok;
        b.n_high[grp] += p.cnt_high;
        b.n_low[grp] += p.cnt_low;
        b.n_drop[grp] += p.cnt_drop;
        b.retained_bytes += (uint64_t)p.cnt_high * c.bytes_h + (uint64_t)p.cnt_low * c.bytes_l;
        b.full_bytes += n_tok * c.bytes_h;
        b.remaining_bytes = (int64_t)(((uint64_t)c.budget_q16 * b.full_bytes) >> 16) - (int64_t)b.retained_bytes;
        b.bad_tags += p.bad_tags;
        b.pages_high += nh[r];
        b.pages_low += nl[r];
    }
    if (tid == 0) {
        const uint32_t pop_h = need_h < free_h ? need_h : free_h, pop_l = need_l < free_l ? need_l : free_l;
        c.ctrl[kCtrlHighFree] = free_h - pop_h;
        c.ctrl[kCtrlHighNext] = next_h + (need_h - pop_h);
        c.ctrl[kCtrlLowFree] = free_l - pop_l;
        c.ctrl[kCtrlLowNext] = next_l + (need_l - pop_l);
        c.ctrl[kCtrlPlanOk] = 1;
        c.ctrl[kCtrlTicket] = 0;
    }
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// One CTA (32 * n_kv threads) per token at a time; thread = one 16-byte chunk (8 head dims) of
// K (first half of the block) or V (second half).
__global__ void __launch_bounds__(256)
append_write_kernel(DevCache c, int layer, int total_tokens, const uint4 *__restrict__ k, const uint4 *__restrict__ v) {
    if (c.ctrl[kCtrlPlanOk] == 0) return;
    const int tid = threadIdx.x;
    const int chunks = 16 * c.n_kv;            // 16-byte chunks per token per tensor
    const int which = tid >= chunks;           // 0 = K, 1 = V
    const int cg = which ? tid - chunks : tid;
    const int head = cg >> 4, cch = cg & 15;
    const uint4 *src = which ? v : k;
    for (int t = blockIdx.x; t < total_tokens; t += gridDim.x) {
        const uint2 sc = c.tok_scratch[t];
        const uint32_t a = sc.x & 3u, pos = sc.x >> 2;
        if (a == PASK_ACTION_RELEASE) continue;
        const AppendPlan &p = c.plan[sc.y];
        const size_t sl = (size_t)p.seq * c.n_layers + layer;
        const uint4 x = src[(size_t)t * chunks + cg];
        if (a == PASK_ACTION_RETAIN_HIGH) {
            const uint32_t at = p.old_high + pos, tau = at & 15u;
            const uint32_t page = c.tbl_high[sl * c.max_pages + (at >> 4)];
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
        } else {
            const uint32_t at = p.old_low + pos, tau = at & 15u;
            const uint32_t page = c.tbl_low[sl * c.max_pages + (at >> 4)];
            uint8_t *dst = c.pool_low + (size_t)page * c.low_page_bytes + (size_t)head * kLowHeadBytes +
                           (which ? kLowHalfBytes : 0);
            float f[8] = {bf16_lo(x.x), bf16_hi(x.x), bf16_lo(x.y), bf16_hi(x.y),
                          bf16_lo(x.z), bf16_hi(x.z), bf16_lo(x.w), bf16_hi(x.w)};
            float amax = 0.0f;
#pragma unroll
            for (int e = 0; e < 8; e++) amax = fmaxf(amax, fabsf(f[e]));
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));   // the 4 chunks of a 32-dim group
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));   // sit in 4 adjacent lanes
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
            // keep that maximum per (sequence, layer) -- one atomic per warp, and only when it grows
            const uint32_t hb = __reduce_max_sync(0xffffffffu, which ? (uint32_t)__half_as_ushort(sh) : 0u);
            if ((tid & 31) == 0 && hb > c.low_vmax[sl]) atomicMax(&c.low_vmax[sl], hb);
        }
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
        if (tid == 0) { s_h = bh + ph; s_l = bl + pl; c.n_high[sl] = 0; c.n_low[sl] = 0; c.low_vmax[sl] = 0; }
        __syncthreads();
    }
    if (tid == 0) { c.ctrl[kCtrlHighFree] = s_h; c.ctrl[kCtrlLowFree] = s_l; }
    uint32_t *b = reinterpret_cast<uint32_t *>(&c.budget[seq]);
    for (int x = tid; x < (int)(sizeof(pask_budget_state_t) / 4); x += blockDim.x) b[x] = 0;
}

}  // namespace

pask_status_t launch_append(pask_cache *c, int layer, int n_seqs, int total_tokens, const int32_t *seq_ids,
                            const int32_t *cu_tokens, const void *k, const void *v, const uint8_t *tags,
                            uint8_t *actions_out, cudaStream_t stream) {
    if (++c->append_serial == 0) c->append_serial = 1;
    append_plan_kernel<<<n_seqs, kPlanThreads, 0, stream>>>(c->dev, layer, n_seqs, total_tokens, seq_ids, cu_tokens, tags,
                                                           actions_out, c->append_serial);
    if (total_tokens > 0) {
        const int ctas = total_tokens < c->sm_count * 8 ? total_tokens : c->sm_count * 8;
        append_write_kernel<<<ctas, 32 * c->desc.n_kv_heads, 0, stream>>>(c->dev, layer, total_tokens,
                                                                         static_cast<const uint4 *>(k),
                                                                         static_cast<const uint4 *>(v));
    }
    return cudaGetLastError() == cudaSuccess ? PASK_OK : PASK_ERR_CUDA;
}

pask_status_t launch_seq_reset(pask_cache *c, int seq, cudaStream_t stream) {
    seq_reset_kernel<<<1, 256, 0, stream>>>(c->dev, seq);
    return cudaGetLastError() == cudaSuccess ? PASK_OK : PASK_ERR_CUDA;
}

}  // namespace pask
