// pask_decode_attention: split GQA decode attention over the mixed-precision paged cache.
//
// out = softmax(q k^T / sqrt(128)) v over a sequence's retained tokens at one layer: the HIGH
// stream holds bf16 K/V, the LOW stream int4 codes with one fp16 scale per 32 dims, read back
// as (code - 8) * scale.  Released tokens were never stored.
//
// Three kernels per call: plan (tiny), attention (streams every retained byte once), combine (tiny).
//
// Shape of the attention kernel (B200, sm_100a)
//   * The work is HBM-bound streaming with a 4-wide GQA group, not a dense contraction, so the
//     design centres on keeping many bytes in flight and few instructions per byte: every warp
//     owns a 3-stage shared-memory ring fed by cp.async.bulk (TMA bulk copies completing on
//     mbarriers) and is its own producer and consumer -- no block-wide barrier in the loop.
//   * A CTA is n_kv warps; warp w handles KV head w for the CTA's page range, so the four query
//     heads of a group share every K/V byte and no cross-warp reduction exists at all.
//   * The plan kernel writes, per sequence, its pages in the order they will be visited (HIGH and
//     LOW pages interleaved evenly, pask_layout.h) and the cost prefix over sequences.  The grid
//     cuts that cost line into equal spans, so every CTA streams the same bytes and the same
//     HIGH/LOW mix whatever the length mix; a span may cover several sequences, each yields one
//     partial (m, l, o) and the ring is not drained in between.  All per-page bookkeeping of the
//     hot loop is one register shuffle out of a 32-entry window of that list.
//   * Pages are stored fragment-major (pask_layout.h): a 128-bit shared load per lane is exactly
//     a tensor-core operand.  QK^T runs as m16n8k16 MMAs with tokens on M and the four query
//     heads (duplicated to fill N = 8) on N; P.V with head dims on M and tokens on K; fp32
//     accumulation throughout.
//   * HIGH pages use bf16 MMAs: K, V and q are exact, P is split into bf16 hi + lo parts.
//   * LOW pages are bound by the integer/logic pipe that expands nibbles, so that path is built to
//     need the fewest such instructions: fp16 MMAs, codes expanded with one LOP3 per pair of
//     values and one shift per eight (0x6400 | code = 1024 + code, 0x6400 | code << 4 =
//     1024 + 16 code as fp16), the offsets folded into the accumulator's initial value for K and
//     removed by one half2 subtract / fma for V, K scales applied to the per-group partial scores
//     in fp32, V scales folded into P (fp16, relative error 2^-12, formed relative to the largest
//     V scale the stream holds so that no magnitude of V under- or overflows).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "pask_internal.h"
#include "pask_merge.h"

namespace pask {

namespace {

constexpr int kStages = 3;
constexpr int kStageBytes = 4096;
constexpr int kBarBytesPerWarp = 40;          // kStages mbarriers (8 bytes each), then kStages entry words (4 bytes each)
constexpr int kMaxWarps = 8;
constexpr int kScratchBytes = 1152;              // per warp: fp16 query fragments (1024) + accumulator seeds (128)
constexpr int kPlanThreads = 256;

struct AttnParams {
    DevCache c;
    int layer, n_seqs;
    const int32_t *seq_ids;
    const uint4 *q;         // bf16 [n_seqs][n_q][128] viewed as 16-byte chunks
    Workspace ws;
    long long wait_cycles;  // bound of a wait for a bulk copy, in SM clock cycles
    uint32_t overpost;      // test aid: bytes announced beyond what a warp's first copy brings (0 in normal use)
    unsigned long long *span;   // optional: {earliest CTA start, latest CTA end} of this launch in %globaltimer ns, else null
    int early;              // the plan and the pages were written before the kernel's predecessor in the stream started:
                            // range look-up and the first bulk copies need not wait for that predecessor
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---------------------------------------------------------------- PTX helpers

__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// Bounded wait: false if the phase did not complete within `limit` clock cycles.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, long long limit) {
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 256; i++)
            if (mbar_try_wait(bar, parity)) return true;
        if (clock64() - t0 > limit) return false;
    }
}
// adds `bytes` to the barrier's pending transaction count without arriving
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// takes `bytes` off the barrier's pending transaction count, as the arrival of that many copied bytes would
__device__ __forceinline__ void mbar_complete_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.complete_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// expect_tx + TMA bulk copy global -> this CTA's shared memory, completion counted on an mbarrier;
// issued by one elected lane of a converged warp
// (predicated, no divergent branch); the same lane leaves `word` at shared address `note`
// The copy carries an L2 evict-first hint: every page is read exactly once per call.
__device__ __forceinline__ void issue_bulk_elected(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar, uint32_t note,
                                                   uint32_t word, uint64_t policy) {
    asm volatile(
        "{\n\t.reg .pred P;\n\t"
        "elect.sync _|P, 0xffffffff;\n\t"
        "@P st.shared.u32 [%4], %5;\n\t"
        "@P mbarrier.arrive.expect_tx.shared::cta.b64 _, [%3], %2;\n\t"
        "@P cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %6;\n\t}"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "r"(note), "r"(word), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ void sts32(uint32_t a, uint32_t v) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}
__device__ __forceinline__ void sts128(uint32_t a, uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// D = A(16x16, row) * B(16x8, col) + D, fp32 accumulate
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// D = A * B + C with C given as raw register bits (an operand quad straight out of shared memory)
__device__ __forceinline__ void mma_f16_seed(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1, const uint4 &c) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(__uint_as_float(c.x)), "f"(__uint_as_float(c.y)),
          "f"(__uint_as_float(c.z)), "f"(__uint_as_float(c.w)));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
// nibbles at bits 0-3 / 16-19 -> two fp16 values 1024 + code
__device__ __forceinline__ uint32_t nib_even(uint32_t x) {
    uint32_t d;
    asm("lop3.b32 %0, %1, 0x000F000F, 0x64006400, 0xEA;" : "=r"(d) : "r"(x));
    return d;
}
// nibbles at bits 4-7 / 20-23 -> two fp16 values 1024 + 16 * code
__device__ __forceinline__ uint32_t nib_odd(uint32_t x) {
    uint32_t d;
    asm("lop3.b32 %0, %1, 0x00F000F0, 0x64006400, 0xEA;" : "=r"(d) : "r"(x));
    return d;
}
// field i (bits 2i, 2i+1 of byte 0) of both half-words as the fp16 pair 1024 + 4^i code
__device__ __forceinline__ uint32_t two_bit(uint32_t x, int i) { return (x & (0x00030003u << (2 * i))) | 0x64006400u; }
__device__ __forceinline__ uint32_t hsub2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t hmul2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t hfma2(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// two floats -> bf16x2 / f16x2 (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ float2 unpack_f16(uint32_t w) {
    return __half22float2(*reinterpret_cast<const __half2 *>(&w));
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// split x into bf16 hi + bf16 lo (pairs), hi + lo carries 16 mantissa bits
__device__ __forceinline__ void split_pair(float x0, float x1, uint32_t &hi, uint32_t &lo) {
    hi = pack_bf16(x0, x1);
    lo = pack_bf16(x0 - bf_lo(hi), x1 - bf_hi(hi));
}

// ---------------------------------------------------------------- plan kernel

// Cost and page prefixes over the call's sequences, and every sequence's pages in visiting order.
// Every CTA recomputes the (small) prefix tables in shared memory; CTA 0 publishes them; all CTAs
// then fill the order list, one thread per page.
__global__ void __launch_bounds__(kPlanThreads)
attn_plan_kernel(DevCache c, int layer, int n_seqs, const int32_t *__restrict__ seq_ids, Workspace ws, int has_low) {
    extern __shared__ uint32_t s_plan[];
    pdl_launch_dependents();
    pdl_wait();
    uint32_t *s_cost = s_plan, *s_page = s_cost + n_seqs + 1, *s_nh = s_page + n_seqs + 1, *s_nl = s_nh + n_seqs;
    uint32_t *s_nw = s_nl + n_seqs;           // tokens in the protected recent window
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int s = tid; s < n_seqs; s += kPlanThreads) {
        const int sid = seq_ids[s];
        uint32_t nh = 0, nl = 0, nw = 0;
        if (sid >= 0 && sid < c.max_seqs) {
            const size_t sl = (size_t)sid * c.n_layers + layer;
            nh = c.n_high[sl];
            if (has_low) nl = c.n_low[sl];
            if (c.window) { const uint32_t seen = c.n_tok[sl]; nw = seen < c.window ? seen : c.window; }
        }
        s_nh[s] = nh;
        s_nl[s] = nl;
        s_nw[s] = nw;
    }
    if (c.window) {
        // The last min(W, tokens seen) tokens are attended from the bf16 ring whatever their action.
        // Streams are in arrival order, so the window's HIGH and LOW members are the last entries
        // of the two streams: shorten those by as many.  One thread per 16 slots, all loads at once.
        __syncthreads();
        const int per = (int)c.window / kPageTokens;
        for (int idx = tid; idx < n_seqs * per; idx += kPlanThreads) {
            const int s = idx / per, i = idx - s * per;
            const uint32_t nw = s_nw[s];
            if ((uint32_t)i * 16u >= nw) continue;
            const size_t sl = (size_t)seq_ids[s] * c.n_layers + layer;
            const uint4 a4 = reinterpret_cast<const uint4 *>(c.win_act + sl * c.window)[i];
            const uint32_t w4[4] = {a4.x, a4.y, a4.z, a4.w};
            // actions are 0, 1, 2: bit 0 of a byte says LOW, bit 1 HIGH; the piece's first `in` slots are members
            const uint32_t in = nw - (uint32_t)i * 16u < 16u ? nw - (uint32_t)i * 16u : 16u, m16 = (1u << in) - 1u;
            uint32_t wh = 0, wl = 0;
#pragma unroll
            for (int k = 0; k < 4; k++) {
                const uint32_t sel = (((m16 >> (4 * k)) & 15u) * 0x00204081u) & 0x01010101u;   // bit j -> bit 0 of byte j
                wl += __popc(w4[k] & sel);
                wh += __popc(w4[k] & (sel << 1));
            }
            if (wh) atomicSub(&s_nh[s], wh);
            if (wl && has_low) atomicSub(&s_nl[s], wl);
        }
    }
    if (tid == 0) s_cost[0] = s_page[0] = 0;
    __syncthreads();
    if (warp == 0) {
        uint32_t carry_c = 0, carry_p = 0;
        for (int base = 0; base < n_seqs; base += 32) {
            const int idx = base + lane;
            uint32_t ph = 0, pl = 0;
            if (idx < n_seqs) {   // the ring's pages have the HIGH format and count as HIGH pages
                ph = (s_nh[idx] + kPageTokens - 1) / kPageTokens + (s_nw[idx] + kPageTokens - 1) / kPageTokens;
                pl = (s_nl[idx] + kPageTokens - 1) / kPageTokens;
            }
            uint32_t ic = ph * kCostHighPage + pl * c.cost_low_page, ip = ph + pl;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t oc = __shfl_up_sync(0xffffffffu, ic, d), op = __shfl_up_sync(0xffffffffu, ip, d);
                if (lane >= d) { ic += oc; ip += op; }
            }
            if (idx < n_seqs) { s_cost[idx + 1] = carry_c + ic; s_page[idx + 1] = carry_p + ip; }
            carry_c += __shfl_sync(0xffffffffu, ic, 31);
            carry_p += __shfl_sync(0xffffffffu, ip, 31);
        }
    }
    __syncthreads();
    if (tid == 0) snap_cost_prefix(s_cost, n_seqs, c.attn_ctas);
    __syncthreads();
    if (blockIdx.x == 0) {
        for (int s = tid; s <= n_seqs; s += kPlanThreads) { ws.cost_prefix[s] = s_cost[s]; ws.page_prefix[s] = s_page[s]; }
        for (int s = tid; s < n_seqs; s += kPlanThreads) ws.tokens[s] = make_uint2(s_nh[s], s_nl[s]);
    }
    const uint32_t total_pages = s_page[n_seqs];
    for (uint32_t gp = blockIdx.x * kPlanThreads + tid; gp < total_pages; gp += gridDim.x * kPlanThreads) {
        int a = 1, e = n_seqs;   // smallest idx in [1, n_seqs] with s_page[idx] > gp
        while (a < e) {
            const int mid = (a + e) >> 1;
            if (s_page[mid] > gp) e = mid; else a = mid + 1;
        }
        const int s = a - 1;
        const uint32_t nh = s_nh[s], nl = s_nl[s], nw = s_nw[s];
        const uint32_t ph = (nh + kPageTokens - 1) / kPageTokens, pl = (nl + kPageTokens - 1) / kPageTokens;
        const uint32_t pw = (nw + kPageTokens - 1) / kPageTokens;
        const size_t slw = (size_t)seq_ids[s] * c.n_layers + layer, sl = slw * c.max_pages;
        uint32_t idx, entry;
        if (page_at(gp - s_page[s], ph + pw, pl, idx)) {
            if (idx < ph) {
                entry = c.tbl_high[sl + idx] | kOrderHigh;
                if (idx == ph - 1) entry |= (nh & (kPageTokens - 1)) << kOrderValidShift;
            } else {            // a page of the recent-window ring
                entry = (c.cap_high + (uint32_t)slw * (c.window / kPageTokens) + (idx - ph)) | kOrderHigh;
                if (idx - ph == pw - 1) entry |= (nw & (kPageTokens - 1)) << kOrderValidShift;
            }
        } else {
            entry = c.tbl_low[sl + idx];
            if (idx == pl - 1) entry |= (nl & (kPageTokens - 1)) << kOrderValidShift;
        }
        ws.order[gp] = entry;
    }
}

// ---------------------------------------------------------------- attention kernel

// Per-warp pipeline.  The CTA's share of the work is one contiguous range of the page-order list
// (sequences follow one another in it).  The producer side walks that range and issues one bulk
// copy per job (HIGH page: K tile, then V tile; LOW page: K and V halves together), leaving the
// page's list entry next to the stage's mbarrier; the consumer side waits for the jobs in the same
// order and reads the entry back, so it needs no bookkeeping of its own.
// Whatever the kernel was given as a parameter (pools, strides, the order list, the wait limit) is read from the
// parameter block where it is used, not copied into the warp's state: every register the pipeline holds for the
// whole loop is one the MMA operands do not get.
template <int kLow>
struct Pipe {
    static constexpr bool kLowTwo = kLow == 8;     // 8-bit LOW pages come as two jobs (K half, V half)
    static constexpr uint32_t kLowJobBytes = kLow == 8 ? kLow8HalfBytes : kLow == 2 ? kLow2HeadBytes : kLowHeadBytes;
    static constexpr uint32_t kLowHeadStride = kLow == 8 ? kLow8HeadBytes : kLow == 2 ? kLow2HeadBytes : kLowHeadBytes;
    uint64_t policy;          // L2 cache policy of the bulk copies
    int lane, warp;
    uint32_t ring, bars;      // shared-space addresses of this warp's stages and of its mbarriers (the entry words follow those)
    // producer
    uint32_t p_pos, p_end;    // next position and end of the CTA's range
    uint32_t p_sub;           // 0: K tile next, 1: V tile next (HIGH pages)
    uint32_t pw_base, pw_entry;   // window: lane i holds the entry of position pw_base + i
    uint32_t p_stage;
    // consumer
    uint32_t c_stage, c_parity;
    uint32_t outstanding;
    bool dead;

    // Issue the next job into stage p_stage.  Warp-uniform.
    __device__ __forceinline__ void produce(const AttnParams &p) {
        const DevCache &c = p.c;
        if (p_pos == p_end) return;
        if (p_pos - pw_base >= 32u) {
            pw_base = p_pos;
            uint32_t e = p_pos + lane < p_end ? __ldg(p.ws.order + p_pos + lane) : 0u;
            // A page id beyond its pool is never expected (a plan somebody overwrote): flag it and read page 0
            // instead.  Checked here, by the lane that fetches the entry, once per 32 pages -- not per job.
            if ((e & kOrderIdMask) >= ((e & kOrderHigh) ? c.high_limit : c.cap_low)) {
                atomicOr(c.ctrl + kCtrlStatus, PASK_DEV_INTERNAL);
                e &= ~kOrderIdMask;
            }
            pw_entry = e;
        }
        const uint32_t entry = __shfl_sync(0xffffffffu, pw_entry, (int)(p_pos - pw_base));
        const uint32_t id = entry & kOrderIdMask;
        const bool is_high = entry & kOrderHigh;
        const uint8_t *src = is_high ? c.pool_high + ((size_t)id * c.high_page_bytes + (uint32_t)warp * kHighHeadBytes + p_sub * kHighTileBytes)
                                     : c.pool_low + ((size_t)id * c.low_page_bytes + (uint32_t)warp * kLowHeadStride + p_sub * kLowJobBytes);
        const uint32_t bytes = is_high ? (uint32_t)kHighTileBytes : kLowJobBytes;
        issue_bulk_elected(ring + p_stage * kStageBytes, src, bytes, bars + p_stage * 8, bars + kStages * 8 + p_stage * 4, entry, policy);
        p_stage = p_stage + 1 == kStages ? 0 : p_stage + 1;
        outstanding++;
        const bool two = is_high || kLowTwo;               // a HIGH page is two jobs, an 8-bit LOW page too
        const uint32_t page_done = two ? p_sub : 1u;
        p_sub = two ? p_sub ^ 1u : 0u;
        p_pos += page_done;
    }

    __device__ __forceinline__ void wait_for(const AttnParams &p, uint32_t bar, uint32_t parity) {
        if (!mbar_try_wait(bar, parity)) {
            if (dead || !mbar_wait_slow(bar, parity, p.wait_cycles)) {
                if (!dead && lane == 0) atomicOr(p.c.ctrl + kCtrlStatus, PASK_DEV_TIMEOUT);
                dead = true;
            }
        }
    }
    // Wait for the oldest outstanding job; returns the shared address of its stage and the page's entry.
    __device__ __forceinline__ uint32_t acquire(const AttnParams &p, uint32_t &entry) {
        wait_for(p, bars + c_stage * 8, c_parity);
        entry = lds32(bars + kStages * 8 + c_stage * 4);
        return ring + c_stage * kStageBytes;
    }
    // The same for the job after the oldest one, which stays the oldest (two stages are then held at once).
    __device__ __forceinline__ uint32_t acquire_next(const AttnParams &p, uint32_t &entry) {
        uint32_t stage = c_stage + 1, parity = c_parity;
        if (stage == kStages) { stage = 0; parity ^= 1u; }
        wait_for(p, bars + stage * 8, parity);
        entry = lds32(bars + kStages * 8 + stage * 4);
        return ring + stage * kStageBytes;
    }
    // All lanes are done reading the oldest stage: hand it back to the producer.
    __device__ __forceinline__ void release(const AttnParams &p) {
        __syncwarp();
        outstanding--;
        if (++c_stage == kStages) { c_stage = 0; c_parity ^= 1u; }
        if (!dead) produce(p);
    }
};

// kLow: 0 = the LOW stream is compiled out (full high-precision cache), 2 / 4 / 8 = width of its codes
template <int kLow>
__global__ void __launch_bounds__(32 * kMaxWarps, 2) decode_attn_kernel(const __grid_constant__ AttnParams p) {
    constexpr bool kHasLow = kLow != 0;
    extern __shared__ __align__(1024) uint8_t smem[];
    const DevCache &c = p.c;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, n_warps = blockDim.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int n_seqs = p.n_seqs;

    uint32_t *s_cost = reinterpret_cast<uint32_t *>(smem);
    uint32_t *s_page = s_cost + n_seqs + 1;
    size_t off = ((size_t)(2 * n_seqs + 2) * 4 + 127) & ~(size_t)127;
    uint64_t *s_bar = reinterpret_cast<uint64_t *>(smem + off);
    off += 384;                                             // 192 bytes of barriers + 96 bytes of entry words
    off = (off + 1023) & ~(size_t)1023;
    uint8_t *s_ring = smem + off;
    uint8_t *s_scratch = s_ring + (size_t)n_warps * kStages * kStageBytes;

    // Normally everything the kernel reads comes from its predecessor in the stream (the plan).  In a planned-ahead
    // step the plan and every page it names were written a whole step earlier, so the set-up below and the first
    // copies run while the predecessor (the merge kernel of the layer before) is still at work; only the queries,
    // the per-sequence scalars and the partials this kernel writes have to wait.
    if (!p.early) {
        pdl_wait();
        pdl_launch_dependents();   // only now: the combine kernel reads the plan's prefix before its own wait
        if (p.span && tid == 0) atomicMin(p.span, globaltimer_ns());
    }
    for (int s = tid; s <= n_seqs; s += blockDim.x) {
        s_cost[s] = __ldg(p.ws.cost_prefix + s);
        s_page[s] = __ldg(p.ws.page_prefix + s);
    }
    __syncthreads();
    const uint32_t total = s_cost[n_seqs];
    if (total == 0) {
        if (p.early) { pdl_wait(); pdl_launch_dependents(); }
        return;
    }

    const uint32_t n_ctas = gridDim.x, b = blockIdx.x;
    const uint32_t lo = (uint32_t)(((uint64_t)total * b) / n_ctas);
    const uint32_t hi = (uint32_t)(((uint64_t)total * (b + 1)) / n_ctas);
    // The sequence holding cost offset x (< total): cost[s] <= x < cost[s + 1].  A warp looks at 32 table entries at
    // a time -- every 32nd first, then the 32 of the block found -- so the search is two shared-memory reads deep
    // whatever the batch (dependent steps cost their full latency here: the CTA has nothing else to issue yet).
    auto seq_of = [&](uint32_t x) -> int {
        const int i1 = (lane + 1) * 32 < n_seqs ? (lane + 1) * 32 : n_seqs;
        const int blk = __ffs(__ballot_sync(0xffffffffu, s_cost[i1] > x)) - 1;       // cost[n_seqs] = total > x: never empty
        const int i2 = 32 * blk + 1 + lane < n_seqs ? 32 * blk + 1 + lane : n_seqs;
        return 32 * blk + __ffs(__ballot_sync(0xffffffffu, s_cost[i2] > x)) - 1;
    };
    // cut_positions() of pask_layout.h, exactly, with the 64-bit division replaced by a double one and a correction step
    auto cut_at = [&](uint32_t x, uint32_t cs, uint32_t n) -> uint32_t {
        if (x >= cs) return n;
        const uint64_t prod = (uint64_t)x * n;                        // < 2^53: exact as a double
        uint64_t q = (uint64_t)__double2ll_rz((double)prod / (double)cs);
        if ((q + 1) * cs <= prod) q++; else if (q * cs > prod) q--;
        return (uint32_t)q;
    };
    const int s0 = seq_of(lo);   // first sequence of the span

    // the CTA's range of the page-order list, and this warp's pipeline over it
    auto position_of = [&](uint32_t x, int s) -> uint32_t {   // first position at or after cost offset x, which lies in sequence s
        return s_page[s] + cut_at(x - s_cost[s], s_cost[s + 1] - s_cost[s], s_page[s + 1] - s_page[s]);
    };
    Pipe<kLow> w;
    w.policy = l2_evict_first_policy();
    w.lane = lane;
    w.warp = warp;
    w.ring = smem_u32(s_ring + (size_t)warp * kStages * kStageBytes);
    w.bars = smem_u32(s_bar) + warp * kBarBytesPerWarp;      // three mbarriers, then the three entry words
    w.p_pos = position_of(lo, s0);
    w.p_end = hi >= total ? s_page[n_seqs] : position_of(hi, seq_of(hi));
    w.p_sub = 0; w.pw_base = 0x80000000u; w.pw_entry = 0;
    w.p_stage = 0; w.c_stage = 0; w.c_parity = 0; w.outstanding = 0; w.dead = false;
    const uint32_t scratch = smem_u32(s_scratch + (size_t)warp * kScratchBytes);
    if (lane == 0) {
        for (int i = 0; i < kStages; i++) mbar_init(w.bars + i * 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    // Wait-limit test only: the barrier of the warp's first job is told to expect more bytes than the copy brings.
    const bool had_job = w.p_pos != w.p_end;
    if (p.overpost && had_job) {
        if (lane == 0) mbar_expect_tx(w.bars, p.overpost);
        __syncwarp();
    }
    for (int i = 0; i < kStages; i++) w.produce(p);
    if (p.early) {
        pdl_wait();
        pdl_launch_dependents();   // (the append that runs beside this kernel must not start before this wait is over)
        if (p.span && tid == 0) atomicMin(p.span, globaltimer_ns());
    }

    const float kLog2Scale = 0.088388347648318440550f * 1.4426950408889634074f;  // log2(e) / sqrt(128)
    const float kSlack = 6.0f;               // log2 units a score may exceed the reference maximum by
    const int head_a = 2 * (t & 1);          // this lane's two score / output columns are heads a, a + 1
    const int qh0 = warp * 4;                // first query head of this KV head
    // selector that broadcasts the fp16 scale of this lane's column group (low or high half of a word)
    const uint32_t bsel = (t >> 1) ? 0x3232u : 0x1010u;

    for (int s = s0; s < n_seqs && s_cost[s] < hi; ++s) {
        if (s_cost[s + 1] == s_cost[s]) continue;
        const uint32_t c0 = s_cost[s], c1 = s_cost[s + 1], n_pos = s_page[s + 1] - s_page[s];
        // number of this sequence's pages that fall to this CTA (same cuts as position_of)
        const uint32_t n_pages = cut_at((hi < c1 ? hi : c1) - c0, c1 - c0, n_pos) - cut_at((lo > c0 ? lo : c0) - c0, c1 - c0, n_pos);
        const uint2 tk = __ldg(p.ws.tokens + s);
        const uint32_t seq_n_low = tk.y;

        // ---- query fragments: lane (g,t) holds dims 8(4j+t) .. +7 of head g & 3 for j = 0..3
        uint4 qf[4];
        {
            const uint4 *qrow = p.q + ((size_t)s * c.n_q + qh0 + (g & 3)) * 16;
#pragma unroll
            for (int j = 0; j < 4; j++) qf[j] = __ldg(qrow + 4 * j + t);
        }
        // P * (V scale) is formed in fp16 relative to the largest V scale the stream holds: everything
        // that feeds the output accumulators of this segment is multiplied by `down` = 2^k (the
        // scales of LOW tokens, P of HIGH tokens) and the partial is multiplied by `up` = 2^-k.
        uint32_t down = 0x3C003C00u;
        float down_f = 1.0f, up = 1.0f;
        if (kHasLow && seq_n_low > 0) {
            // fp16 copies of q for the LOW stream's MMAs.  Its A operands are 1024 + code (register
            // pairs x, z of a chunk) and 1024 + 16 code (pairs y, w), so q is stored as is for the
            // former and divided by 16 for the latter, and -(1032 b) resp. -(1152 b) summed over a
            // 32-dim group seeds the accumulator so that what comes out is sum q (code - 8).
            __syncwarp();
            bool too_big = false;
#pragma unroll
            for (int j = 0; j < 4; j++) {
                const uint32_t r[4] = {qf[j].x, qf[j].y, qf[j].z, qf[j].w};
                uint32_t h[4];
                float seed = 0.f;
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    const float f0 = bf_lo(r[i]), f1 = bf_hi(r[i]);
                    too_big |= fabsf(f0) > 65504.f || fabsf(f1) > 65504.f;
                    // (8-bit codes: every A operand is 1024 + code, so q is stored as is and the offset is 1152;
                    // 2-bit codes: pair i of a chunk comes out as 1024 + 4^i code, so q is divided by 4^i and the
                    // offset is 1024 + 2 * 4^i)
                    const float sc = kLow == 4 ? ((i & 1) ? 0.0625f : 1.0f)
                                   : kLow == 2 ? (i == 0 ? 1.0f : i == 1 ? 0.25f : i == 2 ? 0.0625f : 0.015625f) : 1.0f;
                    const float offs = kLow == 8 ? 1152.f : kLow == 4 ? ((i & 1) ? 1152.f : 1032.f)
                                     : (i == 0 ? 1026.f : i == 1 ? 1032.f : i == 2 ? 1056.f : 1152.f);
                    h[i] = pack_f16(f0 * sc, f1 * sc);
                    const float2 bq = unpack_f16(h[i]);
                    seed -= offs * (bq.x + bq.y);
                }
                seed += __shfl_xor_sync(0xffffffffu, seed, 1);
                seed += __shfl_xor_sync(0xffffffffu, seed, 2);
                // the seed of head a+1 sits one 4-lane row further on
                const float seed_b = __shfl_down_sync(0xffffffffu, seed, 4);
                if (kLow == 8) {
                    // B operands of the k-chunks of 16 dims: chunk c, head, lane t -> {dims 16c+2t,+1 | dims 16c+2t+8,+9};
                    // this lane holds dims 32j + 8t + 2i, +1, i.e. chunk 2j + t/2, slot i, half t & 1
                    if (g < 4) {
#pragma unroll
                        for (int i = 0; i < 4; i++) sts32(scratch + (2 * j + (t >> 1)) * 128 + g * 32 + i * 8 + (t & 1) * 4, h[i]);
                    }
                } else if (g < 4) {
                    sts128(scratch + j * 256 + g * 64 + t * 16, make_uint4(h[0], h[1], h[2], h[3]));
                }
                // accumulator quads {seed[a], seed[a+1], seed[a], seed[a+1]} of head pairs (0,1) and (2,3)
                if (t == 0 && (g == 0 || g == 2)) {
                    const uint32_t sa = __float_as_uint(seed), sb = __float_as_uint(seed_b);
                    sts128(scratch + 1024 + ((g >> 1) * 4 + j) * 16, make_uint4(sa, sb, sa, sb));
                }
            }
            if (__any_sync(0xffffffffu, too_big) && lane == 0) atomicOr(&c.ctrl[kCtrlStatus], PASK_DEV_RANGE);
            const uint32_t vmax = c.low_vmax[(size_t)p.seq_ids[s] * c.n_layers + p.layer];   // fp16 bits
            const int k = max(15 - (int)(vmax >> 10), -14);
            down = (uint32_t)(15 + k) << 10;
            down |= down << 16;
            down_f = __int_as_float((127 + k) << 23);
            up = __int_as_float((127 - k) << 23);
            __syncwarp();
        }

        float acc[8][4];
#pragma unroll
        for (int m = 0; m < 8; m++) acc[m][0] = acc[m][1] = acc[m][2] = acc[m][3] = 0.f;
        float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;

        // P.V over the four-bit V codes of the page in stage `stage`, weights p0..p3 (heads a, a+1 x tokens g, g+8); the
        // stage is handed back as soon as its V half is in registers
        auto pv_low4 = [&](uint32_t stage, uint32_t n_valid, float p0, float p1, float p2, float p3) {
            const uint32_t vb = stage + kLowHalfBytes;
            const uint4 v0 = lds128(vb + lane * 16);        // tokens 2t, 2t+1
            const uint4 v1 = lds128(vb + 512 + lane * 16);  // tokens 2t+8, 2t+9
            uint2 vs0 = lds64(vb + kLowCodesBytes + g * 8);
            uint2 vs1 = lds64(vb + kLowCodesBytes + (g + 8) * 8);
            w.release(p);   // everything of this stage is in registers now
            if (n_valid < 16u) {   // partial tail page: stale scales must not reach the MMA
                if ((uint32_t)g >= n_valid) vs0 = make_uint2(0, 0);
                if ((uint32_t)g + 8u >= n_valid) vs1 = make_uint2(0, 0);
            }
            const uint32_t c0[4] = {v0.x, v0.y, v0.z, v0.w}, c1[4] = {v1.x, v1.y, v1.z, v1.w};
            const uint32_t p01 = pack_f16(p0, p1), p23 = pack_f16(p2, p3);
#pragma unroll
            for (int v = 0; v < 2; v++) {
                // B columns 0-3: heads x group 2v, columns 4-7: heads x group 2v + 1
                const uint32_t s0b = hmul2(prmt(v ? vs0.y : vs0.x, 0u, bsel), down);
                const uint32_t s1b = hmul2(prmt(v ? vs1.y : vs1.x, 0u, bsel), down);
                const uint32_t b0 = movmatrix_trans(hmul2(p01, s0b)), b1 = movmatrix_trans(hmul2(p23, s1b));
#pragma unroll
                for (int qq = 0; qq < 2; qq++) {
                    const int q = 2 * v + qq;
                    const uint32_t e0 = c0[q] >> 8, e1 = c1[q] >> 8;
                    uint32_t a[2][4];
                    a[0][0] = hsub2(nib_even(c0[q]), 0x64086408u);               // (1024 + code) - 1032
                    a[0][1] = hfma2(nib_odd(c0[q]), 0x2C002C00u, 0xD480D480u);   // (1024 + 16 code) / 16 - 72
                    a[0][2] = hsub2(nib_even(e0), 0x64086408u);
                    a[0][3] = hfma2(nib_odd(e0), 0x2C002C00u, 0xD480D480u);
                    a[1][0] = hsub2(nib_even(c1[q]), 0x64086408u);
                    a[1][1] = hfma2(nib_odd(c1[q]), 0x2C002C00u, 0xD480D480u);
                    a[1][2] = hsub2(nib_even(e1), 0x64086408u);
                    a[1][3] = hfma2(nib_odd(e1), 0x2C002C00u, 0xD480D480u);
#pragma unroll
                    for (int r = 0; r < 2; r++)
                        mma_f16(acc[2 * q + r], a[0][2 * r], a[0][2 * r + 1], a[1][2 * r], a[1][2 * r + 1], b0, b1);
                }
            }
        };

        // the same for a page of two-bit codes, and its scores (QK^T: one word per 32-dim group holds both token rows of
        // this lane; byte 0: token g, byte 1: token g + 8)
        auto qk_low2 = [&](uint32_t stage, float (&sc)[4]) {
            const uint4 kq = lds128(stage + lane * 16);
            const uint2 ks0 = lds64(stage + kLow2CodesBytes + g * 8);
            const uint2 ks1 = lds64(stage + kLow2CodesBytes + (g + 8) * 8);
            const uint32_t kwd[4] = {kq.x, kq.y, kq.z, kq.w};
            const float2 f0[2] = {unpack_f16(ks0.x), unpack_f16(ks0.y)};
            const float2 f1[2] = {unpack_f16(ks1.x), unpack_f16(ks1.y)};
#pragma unroll
            for (int j = 0; j < 4; j++) {
                const uint4 qa = lds128(scratch + j * 256 + (g & 3) * 64 + t * 16);
                const uint4 seed = lds128(scratch + 1024 + ((t & 1) * 4 + j) * 16);
                float cj[4];
                const uint32_t x = kwd[j], y = x >> 8;
                mma_f16_seed(cj, two_bit(x, 0), two_bit(y, 0), two_bit(x, 1), two_bit(y, 1), qa.x, qa.y, seed);
                mma_f16(cj, two_bit(x, 2), two_bit(y, 2), two_bit(x, 3), two_bit(y, 3), qa.z, qa.w);
                const float s0f = (j & 1) ? f0[j >> 1].y : f0[j >> 1].x;
                const float s1f = (j & 1) ? f1[j >> 1].y : f1[j >> 1].x;
                sc[0] = fmaf(s0f, cj[0], sc[0]);
                sc[1] = fmaf(s0f, cj[1], sc[1]);
                sc[2] = fmaf(s1f, cj[2], sc[2]);
                sc[3] = fmaf(s1f, cj[3], sc[3]);
            }
        };
        // P.V over 2-bit V codes: fields 0, 1 of a byte are rows g, g+8 of tile 2q, fields 2, 3 of tile 2q+1
        auto pv_low2 = [&](uint32_t stage, uint32_t n_valid, float p0, float p1, float p2, float p3) {
            const uint32_t vb2 = stage + kLow2HalfBytes;
            const uint4 vq = lds128(vb2 + lane * 16);        // byte 0: tokens 2t, 2t+1; byte 1: tokens 2t+8, 2t+9
            uint2 vs0 = lds64(vb2 + kLow2CodesBytes + g * 8);
            uint2 vs1 = lds64(vb2 + kLow2CodesBytes + (g + 8) * 8);
            w.release(p);   // everything of this stage is in registers now
            if (n_valid < 16u) {   // partial tail page: stale scales must not reach the MMA
                if ((uint32_t)g >= n_valid) vs0 = make_uint2(0, 0);
                if ((uint32_t)g + 8u >= n_valid) vs1 = make_uint2(0, 0);
            }
            const uint32_t cw[4] = {vq.x, vq.y, vq.z, vq.w};
            const uint32_t p01 = pack_f16(p0, p1), p23 = pack_f16(p2, p3);
#pragma unroll
            for (int v = 0; v < 2; v++) {
                const uint32_t s0b = hmul2(prmt(v ? vs0.y : vs0.x, 0u, bsel), down);
                const uint32_t s1b = hmul2(prmt(v ? vs1.y : vs1.x, 0u, bsel), down);
                const uint32_t b0 = movmatrix_trans(hmul2(p01, s0b)), b1 = movmatrix_trans(hmul2(p23, s1b));
#pragma unroll
                for (int qq = 0; qq < 2; qq++) {
                    const int q = 2 * v + qq;
                    const uint32_t x = cw[q], y = x >> 8;
                    // (1024 + 4^i code) / 4^i - (1024 / 4^i + 2) = code - 2, exact in fp16
                    mma_f16(acc[2 * q], hsub2(two_bit(x, 0), 0x64026402u), hfma2(two_bit(x, 1), 0x34003400u, 0xDC08DC08u),
                            hsub2(two_bit(y, 0), 0x64026402u), hfma2(two_bit(y, 1), 0x34003400u, 0xDC08DC08u), b0, b1);
                    mma_f16(acc[2 * q + 1], hfma2(two_bit(x, 2), 0x2C002C00u, 0xD420D420u), hfma2(two_bit(x, 3), 0x24002400u, 0xCC80CC80u),
                            hfma2(two_bit(y, 2), 0x2C002C00u, 0xD420D420u), hfma2(two_bit(y, 3), 0x24002400u, 0xCC80CC80u), b0, b1);
                }
            }
        };

        for (uint32_t page = 0; page < n_pages; ++page) {
            uint32_t entry;
            uint32_t st = w.acquire(p, entry);
            if (w.dead) break;
            const bool is_high = entry & kOrderHigh;
            const uint32_t n_valid = (((entry >> kOrderValidShift) - 1u) & 15u) + 1u;   // 0 in the entry means all 16

            // ---- two full four-bit (or two-bit) pages in a row are taken together: two independent chains of loads, logic, MMAs
            // and exponentials for the four resident warps of a scheduler to interleave instead of one (the warp-level
            // MMA and the half-rate logic pipe leave an in-order warp waiting most of the time), one look at the running
            // maxima, and the query operands fetched once for both
            if ((kLow == 4 || kLow == 2) && !is_high && n_valid == 16u && page + 1 < n_pages) {
                uint32_t entry_b;
                const uint32_t st_b = w.acquire_next(p, entry_b);
                if (w.dead) break;
                if (!(entry_b & kOrderHigh) && ((entry_b >> kOrderValidShift) & 15u) == 0u) {
                    float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
                    if (kLow == 2) {
                        qk_low2(st, sa);
                        qk_low2(st_b, sb);
                    } else {
                        const uint4 ka0 = lds128(st + lane * 16), ka1 = lds128(st + 512 + lane * 16);
                        const uint4 kb0 = lds128(st_b + lane * 16), kb1 = lds128(st_b + 512 + lane * 16);
                        const uint2 sa0 = lds64(st + kLowCodesBytes + g * 8), sa1 = lds64(st + kLowCodesBytes + (g + 8) * 8);
                        const uint2 sb0 = lds64(st_b + kLowCodesBytes + g * 8), sb1 = lds64(st_b + kLowCodesBytes + (g + 8) * 8);
                        const uint32_t wa0[4] = {ka0.x, ka0.y, ka0.z, ka0.w}, wa1[4] = {ka1.x, ka1.y, ka1.z, ka1.w};
                        const uint32_t wb0[4] = {kb0.x, kb0.y, kb0.z, kb0.w}, wb1[4] = {kb1.x, kb1.y, kb1.z, kb1.w};
                        const float2 fa0[2] = {unpack_f16(sa0.x), unpack_f16(sa0.y)}, fa1[2] = {unpack_f16(sa1.x), unpack_f16(sa1.y)};
                        const float2 fb0[2] = {unpack_f16(sb0.x), unpack_f16(sb0.y)}, fb1[2] = {unpack_f16(sb1.x), unpack_f16(sb1.y)};
#pragma unroll
                        for (int j = 0; j < 4; j++) {
                            const uint4 qa = lds128(scratch + j * 256 + (g & 3) * 64 + t * 16);
                            const uint4 seed = lds128(scratch + 1024 + ((t & 1) * 4 + j) * 16);
                            float ca[4], cb[4];
                            const uint32_t ua0 = wa0[j] >> 8, ua1 = wa1[j] >> 8, ub0 = wb0[j] >> 8, ub1 = wb1[j] >> 8;
                            mma_f16_seed(ca, nib_even(wa0[j]), nib_even(wa1[j]), nib_odd(wa0[j]), nib_odd(wa1[j]), qa.x, qa.y, seed);
                            mma_f16_seed(cb, nib_even(wb0[j]), nib_even(wb1[j]), nib_odd(wb0[j]), nib_odd(wb1[j]), qa.x, qa.y, seed);
                            mma_f16(ca, nib_even(ua0), nib_even(ua1), nib_odd(ua0), nib_odd(ua1), qa.z, qa.w);
                            mma_f16(cb, nib_even(ub0), nib_even(ub1), nib_odd(ub0), nib_odd(ub1), qa.z, qa.w);
                            const float a0f = (j & 1) ? fa0[j >> 1].y : fa0[j >> 1].x, a1f = (j & 1) ? fa1[j >> 1].y : fa1[j >> 1].x;
                            const float b0f = (j & 1) ? fb0[j >> 1].y : fb0[j >> 1].x, b1f = (j & 1) ? fb1[j >> 1].y : fb1[j >> 1].x;
                            sa[0] = fmaf(a0f, ca[0], sa[0]); sa[1] = fmaf(a0f, ca[1], sa[1]);
                            sa[2] = fmaf(a1f, ca[2], sa[2]); sa[3] = fmaf(a1f, ca[3], sa[3]);
                            sb[0] = fmaf(b0f, cb[0], sb[0]); sb[1] = fmaf(b0f, cb[1], sb[1]);
                            sb[2] = fmaf(b1f, cb[2], sb[2]); sb[3] = fmaf(b1f, cb[3], sb[3]);
                        }
                    }
                    // online softmax over the 32 tokens of the two pages, as below for one
                    const float za0 = sa[0] * kLog2Scale, za1 = sa[1] * kLog2Scale, za2 = sa[2] * kLog2Scale, za3 = sa[3] * kLog2Scale;
                    const float zb0 = sb[0] * kLog2Scale, zb1 = sb[1] * kLog2Scale, zb2 = sb[2] * kLog2Scale, zb3 = sb[3] * kLog2Scale;
                    float ta = fmaxf(fmaxf(za0, za2), fmaxf(zb0, zb2)), tb = fmaxf(fmaxf(za1, za3), fmaxf(zb1, zb3));
                    if (__any_sync(0xffffffffu, ta > m_a + kSlack || tb > m_b + kSlack)) {
#pragma unroll
                        for (int d = 4; d < 32; d <<= 1) {
                            ta = fmaxf(ta, __shfl_xor_sync(0xffffffffu, ta, d));
                            tb = fmaxf(tb, __shfl_xor_sync(0xffffffffu, tb, d));
                        }
                        const float mna = fmaxf(m_a, ta), mnb = fmaxf(m_b, tb);
                        const float fa = mna == -INFINITY ? 1.f : ex2(m_a - mna), fb = mnb == -INFINITY ? 1.f : ex2(m_b - mnb);
#pragma unroll
                        for (int m = 0; m < 8; m++) { acc[m][0] *= fa; acc[m][2] *= fa; acc[m][1] *= fb; acc[m][3] *= fb; }
                        l_a *= fa; l_b *= fb;
                        m_a = mna; m_b = mnb;
                    }
                    const float pa0 = ex2(za0 - m_a), pa1 = ex2(za1 - m_b), pa2 = ex2(za2 - m_a), pa3 = ex2(za3 - m_b);
                    const float pb0 = ex2(zb0 - m_a), pb1 = ex2(zb1 - m_b), pb2 = ex2(zb2 - m_a), pb3 = ex2(zb3 - m_b);
                    l_a += (pa0 + pa2) + (pb0 + pb2);
                    l_b += (pa1 + pa3) + (pb1 + pb3);
                    if (kLow == 2) {
                        pv_low2(st, 16u, pa0, pa1, pa2, pa3);
                        pv_low2(st_b, 16u, pb0, pb1, pb2, pb3);
                    } else {
                        pv_low4(st, 16u, pa0, pa1, pa2, pa3);
                        pv_low4(st_b, 16u, pb0, pb1, pb2, pb3);
                    }
                    ++page;          // (the loop's own increment counts the second page)
                    continue;
                }
            }

            float sc[4] = {0.f, 0.f, 0.f, 0.f};
            if (is_high) {
                // ---- QK^T over a bf16 K tile: 8 MMAs, two independent accumulators
                float sc2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    const uint4 ka = lds128(st + (2 * j) * 512 + lane * 16);      // operand quad, dims 8c .. 8c+3
                    const uint4 kb = lds128(st + (2 * j + 1) * 512 + lane * 16);  // dims 8c+4 .. 8c+7
                    mma_bf16(sc, ka.x, ka.y, ka.z, ka.w, qf[j].x, qf[j].y);
                    mma_bf16(sc2, kb.x, kb.y, kb.z, kb.w, qf[j].z, qf[j].w);
                }
#pragma unroll
                for (int i = 0; i < 4; i++) sc[i] += sc2[i];
                w.release(p);
            } else if (kLow == 8) {
                // ---- QK^T over 8-bit K codes: per 32-dim group two k-chunks, A = 1024 + code by byte permutes
                const uint2 ks0 = lds64(st + kLow8CodesBytes + g * 8);
                const uint2 ks1 = lds64(st + kLow8CodesBytes + (g + 8) * 8);
                const float2 f0[2] = {unpack_f16(ks0.x), unpack_f16(ks0.y)};
                const float2 f1[2] = {unpack_f16(ks1.x), unpack_f16(ks1.y)};
                uint4 kw[4];
#pragma unroll
                for (int j = 0; j < 4; j++) kw[j] = lds128(st + j * 512 + lane * 16);
                w.release(p);
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    const uint2 qa = lds64(scratch + (2 * j) * 128 + (g & 3) * 32 + t * 8);
                    const uint2 qb = lds64(scratch + (2 * j + 1) * 128 + (g & 3) * 32 + t * 8);
                    const uint4 seed = lds128(scratch + 1024 + ((t & 1) * 4 + j) * 16);
                    float cj[4];
                    mma_f16_seed(cj, prmt(kw[j].x, 0x64646464u, 0x4140), prmt(kw[j].x, 0x64646464u, 0x4342),
                                 prmt(kw[j].y, 0x64646464u, 0x4140), prmt(kw[j].y, 0x64646464u, 0x4342), qa.x, qa.y, seed);
                    mma_f16(cj, prmt(kw[j].z, 0x64646464u, 0x4140), prmt(kw[j].z, 0x64646464u, 0x4342),
                            prmt(kw[j].w, 0x64646464u, 0x4140), prmt(kw[j].w, 0x64646464u, 0x4342), qb.x, qb.y);
                    const float s0f = (j & 1) ? f0[j >> 1].y : f0[j >> 1].x;
                    const float s1f = (j & 1) ? f1[j >> 1].y : f1[j >> 1].x;
                    sc[0] = fmaf(s0f, cj[0], sc[0]);
                    sc[1] = fmaf(s0f, cj[1], sc[1]);
                    sc[2] = fmaf(s1f, cj[2], sc[2]);
                    sc[3] = fmaf(s1f, cj[3], sc[3]);
                }
            } else if (kLow == 2) {
                qk_low2(st, sc);
            } else if (kHasLow) {
                const uint4 k0 = lds128(st + lane * 16);
                const uint4 k1 = lds128(st + 512 + lane * 16);
                const uint2 ks0 = lds64(st + kLowCodesBytes + g * 8);
                const uint2 ks1 = lds64(st + kLowCodesBytes + (g + 8) * 8);
                const uint32_t w0[4] = {k0.x, k0.y, k0.z, k0.w}, w1[4] = {k1.x, k1.y, k1.z, k1.w};
                const float2 f0[2] = {unpack_f16(ks0.x), unpack_f16(ks0.y)};
                const float2 f1[2] = {unpack_f16(ks1.x), unpack_f16(ks1.y)};
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    const uint4 qa = lds128(scratch + j * 256 + (g & 3) * 64 + t * 16);
                    const uint4 seed = lds128(scratch + 1024 + ((t & 1) * 4 + j) * 16);
                    float cj[4];
                    const uint32_t u0 = w0[j] >> 8, u1 = w1[j] >> 8;
                    mma_f16_seed(cj, nib_even(w0[j]), nib_even(w1[j]), nib_odd(w0[j]), nib_odd(w1[j]), qa.x, qa.y, seed);
                    mma_f16(cj, nib_even(u0), nib_even(u1), nib_odd(u0), nib_odd(u1), qa.z, qa.w);
                    const float s0f = (j & 1) ? f0[j >> 1].y : f0[j >> 1].x;
                    const float s1f = (j & 1) ? f1[j >> 1].y : f1[j >> 1].x;
                    sc[0] = fmaf(s0f, cj[0], sc[0]);
                    sc[1] = fmaf(s0f, cj[1], sc[1]);
                    sc[2] = fmaf(s1f, cj[2], sc[2]);
                    sc[3] = fmaf(s1f, cj[3], sc[3]);
                }
            }

            // ---- online softmax for heads a, a+1 over tokens g and g + 8 of the tile
            // The reference maxima m_a, m_b are only raised when some score of the tile exceeds them by
            // more than kSlack (then to the true running maximum): weights stay below 2^kSlack, and
            // the cross-lane reduction and the rescaling of the accumulators leave the common path.
            float z0 = sc[0] * kLog2Scale, z1 = sc[1] * kLog2Scale, z2 = sc[2] * kLog2Scale, z3 = sc[3] * kLog2Scale;
            if (n_valid < 16u) {
                if ((uint32_t)g >= n_valid) z0 = z1 = -INFINITY;
                if ((uint32_t)g + 8u >= n_valid) z2 = z3 = -INFINITY;
            }
            float ta = fmaxf(z0, z2), tb = fmaxf(z1, z3);
            if (__any_sync(0xffffffffu, ta > m_a + kSlack || tb > m_b + kSlack)) {
#pragma unroll
                for (int d = 4; d < 32; d <<= 1) {
                    ta = fmaxf(ta, __shfl_xor_sync(0xffffffffu, ta, d));
                    tb = fmaxf(tb, __shfl_xor_sync(0xffffffffu, tb, d));
                }
                const float mna = fmaxf(m_a, ta), mnb = fmaxf(m_b, tb);
                const float fa = mna == -INFINITY ? 1.f : ex2(m_a - mna), fb = mnb == -INFINITY ? 1.f : ex2(m_b - mnb);
#pragma unroll
                for (int m = 0; m < 8; m++) { acc[m][0] *= fa; acc[m][2] *= fa; acc[m][1] *= fb; acc[m][3] *= fb; }
                l_a *= fa; l_b *= fb;
                m_a = mna; m_b = mnb;
            }
            const float p0 = ex2(z0 - m_a), p1 = ex2(z1 - m_b), p2 = ex2(z2 - m_a), p3 = ex2(z3 - m_b);
            l_a += p0 + p2;
            l_b += p1 + p3;

            if (is_high) {
                // ---- P (hi + lo) as the B operand: transpose the score fragment's layout
                uint32_t h01, l01, h23, l23;
                split_pair(p0 * down_f, p1 * down_f, h01, l01);
                split_pair(p2 * down_f, p3 * down_f, h23, l23);
                const uint32_t bh0 = movmatrix_trans(h01), bh1 = movmatrix_trans(h23);
                const uint32_t bl0 = movmatrix_trans(l01), bl1 = movmatrix_trans(l23);
                st = w.acquire(p, entry);
                if (w.dead) break;
#pragma unroll
                for (int e = 0; e < 2; e++) {
                    uint4 x[4];
#pragma unroll
                    for (int k = 0; k < 4; k++) x[k] = lds128(st + (4 * e + k) * 512 + lane * 16);
                    if (n_valid < 16u) {  // partial tail page: stale slots must not reach the MMA
#pragma unroll
                        for (int k = 0; k < 4; k++)
                            if ((uint32_t)(2 * t + (k & 1) + 8 * (k >> 1)) >= n_valid) x[k] = make_uint4(0, 0, 0, 0);
                    }
                    const uint32_t x0[4] = {x[0].x, x[0].y, x[0].z, x[0].w}, x1[4] = {x[1].x, x[1].y, x[1].z, x[1].w};
                    const uint32_t x2[4] = {x[2].x, x[2].y, x[2].z, x[2].w}, x3[4] = {x[3].x, x[3].y, x[3].z, x[3].w};
#pragma unroll
                    for (int r = 0; r < 4; r++) {
                        const uint32_t a0 = prmt(x0[r], x1[r], 0x5410), a1 = prmt(x0[r], x1[r], 0x7632);
                        const uint32_t a2 = prmt(x2[r], x3[r], 0x5410), a3 = prmt(x2[r], x3[r], 0x7632);
                        mma_bf16(acc[4 * e + r], a0, a1, a2, a3, bh0, bh1);
                        mma_bf16(acc[4 * e + r], a0, a1, a2, a3, bl0, bl1);
                    }
                }
                w.release(p);
            } else if (kLow == 8) {
                // ---- P.V over 8-bit V codes: the V half is a job of its own
                const uint32_t p01 = pack_f16(p0, p1), p23 = pack_f16(p2, p3);
                st = w.acquire(p, entry);
                if (w.dead) break;
                uint4 vw[4];
#pragma unroll
                for (int q = 0; q < 4; q++) vw[q] = lds128(st + q * 512 + lane * 16);   // group q: tiles r = 0 (x, y) and 1 (z, w)
                uint2 vs0 = lds64(st + kLow8CodesBytes + g * 8);
                uint2 vs1 = lds64(st + kLow8CodesBytes + (g + 8) * 8);
                w.release(p);
                if (n_valid < 16u) {   // partial tail page: stale scales must not reach the MMA
                    if ((uint32_t)g >= n_valid) vs0 = make_uint2(0, 0);
                    if ((uint32_t)g + 8u >= n_valid) vs1 = make_uint2(0, 0);
                }
#pragma unroll
                for (int v = 0; v < 2; v++) {
                    const uint32_t s0b = hmul2(prmt(v ? vs0.y : vs0.x, 0u, bsel), down);
                    const uint32_t s1b = hmul2(prmt(v ? vs1.y : vs1.x, 0u, bsel), down);
                    const uint32_t b0 = movmatrix_trans(hmul2(p01, s0b)), b1 = movmatrix_trans(hmul2(p23, s1b));
#pragma unroll
                    for (int qq = 0; qq < 2; qq++) {
                        const int q = 2 * v + qq;
#pragma unroll
                        for (int r = 0; r < 2; r++) {
                            const uint32_t w0 = r ? vw[q].z : vw[q].x, w1 = r ? vw[q].w : vw[q].y;
                            // (1024 + code) - 1152 = code - 128, exact in fp16
                            mma_f16(acc[2 * q + r], hsub2(prmt(w0, 0x64646464u, 0x4140), 0x64806480u),
                                    hsub2(prmt(w0, 0x64646464u, 0x4342), 0x64806480u),
                                    hsub2(prmt(w1, 0x64646464u, 0x4140), 0x64806480u),
                                    hsub2(prmt(w1, 0x64646464u, 0x4342), 0x64806480u), b0, b1);
                        }
                    }
                }
            } else if (kLow == 2) {
                pv_low2(st, n_valid, p0, p1, p2, p3);
            } else if (kHasLow) {
                pv_low4(st, n_valid, p0, p1, p2, p3);
            }
        }
        // A wait ran out: the status word says so and the results of the call are void.  This warp's partials of
        // this and of the CTA's later sequences are written as empty ones, which the merge skips.
        if (w.dead) { m_a = m_b = -INFINITY; l_a = l_b = 0.f; }

        // ---- this segment's partial: (m, l) per head, unnormalised o
#pragma unroll
        for (int d = 4; d < 32; d <<= 1) {
            l_a += __shfl_xor_sync(0xffffffffu, l_a, d);
            l_b += __shfl_xor_sync(0xffffffffu, l_b, d);
        }
        const size_t slot = (size_t)b + s;
        const size_t hrow = slot * c.n_q + qh0 + head_a;
        if (g == 0 && t < 2) {
            p.ws.part_ml[hrow] = make_float2(m_a, l_a);
            p.ws.part_ml[hrow + 1] = make_float2(m_b, l_b);
        }
#pragma unroll
        for (int m = 0; m < 8; m++) {
            const int q = m >> 1, r = m & 1;
            if ((t >> 1) == (q & 1)) {   // even groups are valid in columns 0-3, odd groups in 4-7
                const int dim = 32 * q + 4 * g + 2 * r;
                *reinterpret_cast<float2 *>(p.ws.part_o + hrow * kHeadDim + dim) = make_float2(acc[m][0] * up, acc[m][2] * up);
                *reinterpret_cast<float2 *>(p.ws.part_o + (hrow + 1) * kHeadDim + dim) = make_float2(acc[m][1] * up, acc[m][3] * up);
            }
        }
    }

    if (p.span && lane == 0) atomicMax(p.span + 1, globaltimer_ns());
    // A wait gave up: copies may still be in flight towards this CTA's shared memory.  Give each
    // outstanding stage one more bounded wait before the CTA retires; the ring is not read again.
    if (w.dead) {
        if (p.overpost && had_job) {   // wait-limit test: bytes were announced that no copy brings; take them off, so that the
                        // barrier completes exactly when the real copy has landed
            if (lane == 0) mbar_complete_tx(w.bars, p.overpost);
            __syncwarp();
        }
        while (w.outstanding > 0) {
            const uint32_t bar = w.bars + w.c_stage * 8;
            if (!mbar_try_wait(bar, w.c_parity)) mbar_wait_slow(bar, w.c_parity, p.wait_cycles > 200000000LL ? p.wait_cycles : 200000000LL);
            if (++w.c_stage == kStages) { w.c_stage = 0; w.c_parity ^= 1u; }
            w.outstanding--;
        }
    }
}

// Merge the partials of each (sequence, query head): `split` adjacent warps a row, lane = 4 output dims.
__global__ void __launch_bounds__(kMergeThreads)
combine_kernel(const uint32_t *__restrict__ prefix, const float2 *__restrict__ part_ml, const float *__restrict__ part_o,
               float *__restrict__ out, float *__restrict__ lse, int n_seqs, int n_q, uint32_t n_ctas, uint32_t split) {
    const int wid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    pdl_launch_dependents();
    // The cost prefix is the plan's, written before the streaming kernel started (that kernel lets
    // its dependents go only after its own wait for the plan's writer): it can be fetched while the
    // streaming kernel's last CTAs are still running.
    const int row_id = wid / (int)split;
    const uint32_t sub = (uint32_t)wid % split;
    const int s = row_id / n_q, h = row_id % n_q;
    const bool mine = row_id < n_seqs * n_q;
    uint32_t p0 = 0, p1 = 0;
    uint64_t total = 0;
    if (mine) { p0 = __ldg(prefix + s); p1 = __ldg(prefix + s + 1); total = __ldg(prefix + n_seqs); }
    uint32_t b_first = 1, b_last = 0;       // the CTAs that hold partials of this sequence (two 64-bit divisions, ahead of the wait)
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
    const size_t orow = (size_t)s * n_q + h;
    if (L > 0.f) {
        const float inv = 1.0f / L;
        o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
    }
    *reinterpret_cast<float4 *>(out + orow * kHeadDim + lane * 4) = o;
    if (lse && lane == 0) lse[orow] = L > 0.f ? (M + log2f(L)) * 0.69314718055994530942f : -INFINITY;
}

// cu_tokens of a call with one token per sequence, and the list of sequences a stand-alone plan is for
__global__ void ahead_setup_kernel(int32_t *iota, int n_iota, int32_t *ids_out, const int32_t *__restrict__ seq_ids, int n_seqs) {
    pdl_launch_dependents();
    pdl_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_iota) iota[i] = i;
    if (i < n_seqs) ids_out[i] = seq_ids[i];
}

size_t attn_smem_bytes(int n_seqs, int n_warps) {
    size_t off = align_up((size_t)(2 * n_seqs + 2) * 4, 128) + 384;
    off = align_up(off, 1024);
    return off + (size_t)n_warps * (kStages * kStageBytes + kScratchBytes);
}

}  // namespace

// carve the caller's workspace
size_t carve_workspace(const pask_cache *c, int n_seqs, uint8_t *base, Workspace *ws) {
    const size_t slots = (size_t)c->attn_ctas + n_seqs;
    const size_t max_pages = (size_t)n_seqs * (2 * c->dev.max_pages + c->dev.window / kPageTokens);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes, 256); return at; };
    const size_t o_cost = take((size_t)(n_seqs + 1) * 4), o_page = take((size_t)(n_seqs + 1) * 4);
    const size_t o_tok = take((size_t)n_seqs * sizeof(uint2)), o_order = take(max_pages * 4);
    const size_t o_ml = take(slots * c->desc.n_q_heads * sizeof(float2));
    const size_t o_o = take(slots * c->desc.n_q_heads * kHeadDim * sizeof(float));
    if (ws) {
        ws->cost_prefix = reinterpret_cast<uint32_t *>(base + o_cost);
        ws->page_prefix = reinterpret_cast<uint32_t *>(base + o_page);
        ws->tokens = reinterpret_cast<uint2 *>(base + o_tok);
        ws->order = reinterpret_cast<uint32_t *>(base + o_order);
        ws->part_ml = reinterpret_cast<float2 *>(base + o_ml);
        ws->part_o = reinterpret_cast<float *>(base + o_o);
    }
    return off;
}


int attention_grid(const pask_cache *c) { return 2 * c->sm_count; }

size_t attention_workspace_bytes(const pask_cache *c, int n_seqs) { return carve_workspace(c, n_seqs, nullptr, nullptr); }

// The streaming kernel of one call: grid, shared memory, optional timing events around it.
static cudaError_t launch_stream_kernel(pask_cache *c, bool has_low, AttnParams &p, cudaStream_t stream) {
    const int n_warps = c->desc.n_kv_heads;
    p.c = c->dev;
    p.wait_cycles = c->wait_cycles;
    p.overpost = c->wait_test_surplus;
    const size_t smem = attn_smem_bytes(p.n_seqs, n_warps);
    auto kern = !has_low ? decode_attn_kernel<0> : c->dev.low_bits == 8 ? decode_attn_kernel<8>
              : c->dev.low_bits == 2 ? decode_attn_kernel<2> : decode_attn_kernel<4>;
    // The shared-memory opt-in is a property of (device, kernel): ask for it once, and again only for a larger size.
    {
        static size_t granted[64][4] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
        size_t &have = granted[dev][!has_low ? 0 : c->dev.low_bits == 8 ? 1 : c->dev.low_bits == 2 ? 2 : 3];
        if (smem > have) {
            const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            have = smem;
        }
    }
    p.span = c->span;
    if (c->ev_start) cudaEventRecord(c->ev_start, stream);
    const cudaError_t e = launch_pdl(kern, dim3(c->attn_ctas), dim3(32 * n_warps), smem, stream, p);
    if (c->ev_stop) cudaEventRecord(c->ev_stop, stream);
    c->ev_start = c->ev_stop = nullptr;
    c->span = nullptr;
    return e;
}

pask_status_t launch_attention(pask_cache *c, bool has_low, int layer, int n_seqs, const int32_t *seq_ids, const void *q,
                               float *out, float *lse, void *workspace, size_t, cudaStream_t stream, bool plan_done) {
    AttnParams p;
    p.layer = layer;
    p.n_seqs = n_seqs;
    p.seq_ids = seq_ids;
    p.q = static_cast<const uint4 *>(q);
    carve_workspace(c, n_seqs, static_cast<uint8_t *>(workspace), &p.ws);
    p.early = 0;
    cudaError_t e = cudaSuccess;
    if (!plan_done)   // (a fused append has already left the plan in the workspace)
        e = launch_pdl(attn_plan_kernel, dim3(c->sm_count), dim3(kPlanThreads), (size_t)(5 * n_seqs + 2) * 4, stream, c->dev,
                       layer, n_seqs, seq_ids, p.ws, has_low ? 1 : 0);
    if (e == cudaSuccess) e = launch_stream_kernel(c, has_low, p, stream);
    const int split = merge_split(n_seqs, c->attn_ctas), warps = n_seqs * c->desc.n_q_heads * split;
    if (e == cudaSuccess)
        e = launch_pdl(combine_kernel, dim3((warps + 7) / 8), dim3(kMergeThreads), 0, stream, (const uint32_t *)p.ws.cost_prefix,
                       (const float2 *)p.ws.part_ml, (const float *)p.ws.part_o, out, lse, n_seqs, (int)c->desc.n_q_heads,
                       (uint32_t)c->attn_ctas, (uint32_t)split);
    return e == cudaSuccess ? PASK_OK : PASK_ERR_CUDA;
}

// ---------------------------------------------------------------- planned-ahead decode steps

// Plan area of a batch of n_seqs sequences: cu_tokens = 0, 1, ..., 255 for the one-token-per-sequence append, then per
// layer two plan blocks (ids, cost prefix, page prefix, token counts, page-order list), used in turn.
size_t carve_plan_area(const pask_cache *c, int n_seqs, int layer, int parity, uint8_t *base, PlanBlock *pb) {
    const size_t max_pages = (size_t)n_seqs * (2 * c->dev.max_pages + c->dev.window / kPageTokens);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes, 256); return at; };
    take(257 * 4);                                         // cu_tokens
    const size_t head = off;
    const size_t o_ids = take((size_t)n_seqs * 4), o_cost = take((size_t)(n_seqs + 1) * 4), o_page = take((size_t)(n_seqs + 1) * 4);
    const size_t o_tok = take((size_t)n_seqs * sizeof(uint2)), o_order = take(max_pages * 4);
    const size_t block = off - head;
    if (pb) {
        uint8_t *b = base + (size_t)(2 * layer + parity) * block;
        pb->ids = reinterpret_cast<int32_t *>(b + o_ids);
        pb->cost_prefix = reinterpret_cast<uint32_t *>(b + o_cost);
        pb->page_prefix = reinterpret_cast<uint32_t *>(b + o_page);
        pb->tokens = reinterpret_cast<uint2 *>(b + o_tok);
        pb->order = reinterpret_cast<uint32_t *>(b + o_order);
    }
    return head + (size_t)2 * c->desc.n_layers * block;
}

static Workspace plan_view(const PlanBlock &pb, const Workspace &parts) {
    Workspace w = parts;
    w.cost_prefix = pb.cost_prefix;
    w.page_prefix = pb.page_prefix;
    w.tokens = pb.tokens;
    w.order = pb.order;
    return w;
}

pask_status_t launch_plan_ahead(pask_cache *c, int layer, int n_seqs, const int32_t *seq_ids, void *area, int parity,
                                cudaStream_t stream) {
    PlanBlock pb;
    carve_plan_area(c, n_seqs, layer, parity, static_cast<uint8_t *>(area), &pb);
    cudaError_t e = launch_pdl(ahead_setup_kernel, dim3(2), dim3(256), 0, stream, static_cast<int32_t *>(area), 257, pb.ids,
                               seq_ids, n_seqs);
    if (e == cudaSuccess)
        e = launch_pdl(attn_plan_kernel, dim3(c->sm_count), dim3(kPlanThreads), (size_t)(5 * n_seqs + 2) * 4, stream, c->dev,
                       layer, n_seqs, seq_ids, plan_view(pb, Workspace{}), 1);
    return e == cudaSuccess ? PASK_OK : PASK_ERR_CUDA;
}

// One layer of a planned-ahead decode step.  In stream order: the streaming kernel over the plan of the cache as
// it was before this call; then one kernel that ends the step: its first CTAs do the one-launch append, which does
// not wait for the streaming kernel (it needs nothing from it and writes nothing it reads: slots past the planned
// token counts, table entries and counters the plan has replaced, the other plan block) and so runs as that kernel's
// CTAs retire; all of its CTAs then wait for the streaming kernel and merge its partials with the new tokens.
pask_status_t launch_step_ahead(pask_cache *c, int layer, int n_seqs, const int32_t *seq_ids, const void *k, const void *v,
                                const uint8_t *tags, const uint8_t *decided, uint8_t *actions_out, const void *q, float *out,
                                float *lse, void *workspace, void *area, int cur, bool early, cudaStream_t stream) {
    PlanBlock pc, pn;
    carve_plan_area(c, n_seqs, layer, cur, static_cast<uint8_t *>(area), &pc);
    carve_plan_area(c, n_seqs, layer, cur ^ 1, static_cast<uint8_t *>(area), &pn);
    AttnParams p;
    p.layer = layer;
    p.n_seqs = n_seqs;
    p.seq_ids = seq_ids;
    p.q = static_cast<const uint4 *>(q);
    Workspace parts;
    carve_workspace(c, n_seqs, static_cast<uint8_t *>(workspace), &parts);
    p.ws = plan_view(pc, parts);
    p.early = early ? 1 : 0;
    cudaError_t e = launch_stream_kernel(c, true, p, stream);
    if (e != cudaSuccess) return PASK_ERR_CUDA;
    NewTokens nt;
    nt.k = static_cast<const uint2 *>(k);
    nt.v = static_cast<const uint2 *>(v);
    nt.q = static_cast<const uint2 *>(q);
    nt.tags = tags;
    nt.decided = decided;
    nt.seq_ids = seq_ids;
    nt.planned_ids = pc.ids;
    nt.status = c->dev.ctrl + kCtrlStatus;
    nt.group = c->layer_group[layer];
    nt.n_groups = c->dev.n_groups;
    nt.n_kv = c->desc.n_kv_heads;
    nt.low_bits = (int)c->dev.low_bits;
    return launch_step_tail(c, layer, n_seqs, seq_ids, static_cast<const int32_t *>(area), k, v, tags, decided, actions_out,
                            plan_view(pn, Workspace{}), pn.ids, pc.cost_prefix, parts.part_ml, parts.part_o, out, lse, nt, stream);
}

}  // namespace pask


// ---------------------------------------------------------------- decode attention without a caller workspace
//
// Scratch for pask_decode_attention_static: the split partials, prefix tables and page-order list of
// one call live in this array instead of a buffer the caller allocates.  It is part of the library
// image, so every GPU on which the library runs a kernel holds these bytes until the process exits.
// In host code the name `g_static_workspace` is only a handle for the runtime; the device address
// is asked for once per device (cudaGetSymbolAddress) and handed to the kernels.
namespace {
constexpr size_t kStaticWorkspaceBytes = PASK_STATIC_WORKSPACE_BYTES;
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];
constexpr int kMaxDevices = 64;
void *g_static_workspace_addr[kMaxDevices] = {};   // device address of the array, per device ordinal
}  // namespace

extern "C" pask_status_t pask_decode_attention_static(pask_cache_t *c, int32_t layer, int32_t n_seqs,
                                                      const int32_t *seq_ids, const void *q, float *out, float *lse,
                                                      pask_stream_t stream) {
    if (!c || !seq_ids || !q || !out) return PASK_ERR_INVALID_ARG;
    if (layer < 0 || layer >= c->desc.n_layers) return PASK_ERR_INVALID_ARG;
    if (n_seqs < 1 || n_seqs > PASK_MAX_SEQS_PER_CALL) return PASK_ERR_INVALID_ARG;
    if ((((uintptr_t)q | (uintptr_t)out) & 15) || ((uintptr_t)lse & 3)) return PASK_ERR_INVALID_ARG;
    // the built-in scratch has a fixed size: a batch (or a page-table bound) that needs more is refused
    if (pask::attention_workspace_bytes(c, n_seqs) > kStaticWorkspaceBytes) return PASK_ERR_WORKSPACE;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PASK_ERR_CUDA;
    if (!g_static_workspace_addr[dev]) {   // first call on this device: look the array's device address up
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess || !ptr) return PASK_ERR_CUDA;
        g_static_workspace_addr[dev] = ptr;
    }
    // Nothing in the scratch has to start at zero: the plan kernel writes the tables before anyone
    // reads them, and every partial slot that is merged was written earlier in the same call.
    return pask::launch_attention(c, true, layer, n_seqs, seq_ids, q, out, lse, g_static_workspace_addr[dev],
                                  kStaticWorkspaceBytes, static_cast<cudaStream_t>(stream));
}

