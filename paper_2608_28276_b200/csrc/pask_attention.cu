// pask_decode_attention: split GQA decode attention over the mixed-precision paged cache.
//
// out = softmax(q k^T / sqrt(128)) v over a sequence's retained tokens at one layer: the HIGH
// stream holds bf16 K/V, the LOW stream int4 codes with one fp16 scale per 32 dims, read back
// as (code - 8) * scale.  Released tokens were never stored.
//
// Shape of the kernel (B200, sm_100a)
//   * The work is HBM-bound streaming with a 4-wide GQA group, not a dense contraction, so the
//     design centres on keeping many bytes in flight: every warp owns a 3-stage shared-memory
//     ring fed by cp.async.bulk (TMA bulk copies completing on mbarriers) and is its own
//     producer and consumer -- no block-wide barrier in the streaming loop.
//   * A CTA is n_kv warps; warp w handles KV head w for the CTA's page range, so the four query
//     heads of a group share every K/V byte and no cross-warp reduction exists at all.
//   * Sequences are laid end to end in cost space and cut into gridDim.x equal spans
//     (pask_layout.h), each cut splitting a sequence's HIGH and LOW page lists at the same
//     fraction, so every CTA streams the same bytes and the same HIGH/LOW mix whatever the lengths;
//     a span may cover several sequences, each yields one partial (m, l, o) and the ring is not
//     drained in between.  A second small kernel merges the partials.
//   * Pages are stored fragment-major (pask_layout.h): a 128-bit shared load per lane is exactly
//     a tensor-core fragment.  QK^T runs as m16n8k16 bf16 MMAs with tokens on M and the four
//     query heads (duplicated to fill N = 8) on N; P.V with head dims on M and tokens on K.  All
//     MMA operands are exact (bf16 values, small integers), accumulation is fp32, and P is split
//     into bf16 hi + lo parts so that nothing is rounded to 8 bits.  int4 codes are expanded in
//     registers with one LOP3 per pair (0x4300 | code = 128 + code as bf16).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "pask_internal.h"

namespace pask {

namespace {

constexpr int kStages = 3;
constexpr int kStageBytes = 4096;
constexpr int kMaxWarps = 8;
constexpr long long kWaitCycles = 2000000000LL;  // about one second: give up instead of hanging

struct AttnParams {
    DevCache c;
    int layer, n_seqs;
    const int32_t *seq_ids;
    const uint4 *q;        // bf16 [n_seqs][n_q][128] viewed as 16-byte chunks
    uint32_t *prefix_out;  // [n_seqs + 1] cost prefix for the combine kernel
    float2 *part_ml;       // [slots][n_q] (running max in log2 units, sum)
    float *part_o;         // [slots][n_q][128] unnormalised outputs
};

// ---------------------------------------------------------------- PTX helpers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
// Bounded wait: false if the phase did not complete within kWaitCycles.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 256; i++)
            if (mbar_try_wait(bar, parity)) return true;
        if (clock64() - t0 > kWaitCycles) return false;
    }
}
// TMA bulk copy global -> this CTA's shared memory, completion counted on an mbarrier.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
    return v;
}
// D = A(16x16, row) * B(16x8, col) + D, bf16 operands, fp32 accumulate
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
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
// (x >> shift) & 0x000F000F | 0x43004300 : two nibbles -> two bf16 values 128 + code
__device__ __forceinline__ uint32_t nib2bf16(uint32_t x) {
    uint32_t d;
    asm("lop3.b32 %0, %1, 0x000F000F, 0x43004300, 0xEA;" : "=r"(d) : "r"(x));
    return d;
}
__device__ __forceinline__ uint32_t sub_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// two floats -> bf16x2 (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float h2f_lo(uint32_t w) { return __half2float(__ushort_as_half((unsigned short)(w & 0xffffu))); }
__device__ __forceinline__ float h2f_hi(uint32_t w) { return __half2float(__ushort_as_half((unsigned short)(w >> 16))); }
__device__ __forceinline__ float pick4(uint2 v, int i) {  // i-th fp16 of four
    const uint32_t w = (i & 2) ? v.y : v.x;
    return (i & 1) ? h2f_hi(w) : h2f_lo(w);
}

// split x into bf16 hi + bf16 lo (pairs), hi + lo carries 16 mantissa bits
__device__ __forceinline__ void split_pair(float x0, float x1, uint32_t &hi, uint32_t &lo) {
    hi = pack_bf16(x0, x1);
    const float r0 = x0 - __uint_as_float(hi << 16);
    const float r1 = x1 - __uint_as_float(hi & 0xffff0000u);
    lo = pack_bf16(r0, r1);
}

// ---------------------------------------------------------------- work partition

struct Segment {
    uint32_t high_begin, high_count;  // this CTA's run of the sequence's HIGH pages
    uint32_t low_begin, low_count;    // and of its LOW pages; jobs take the two runs interleaved (PageOrder)
    uint32_t n_high, n_low;           // tokens in the whole streams (for the ragged tail pages)
};

__device__ __forceinline__ Segment make_segment(int s, uint32_t lo, uint32_t hi, const uint32_t *s_prefix,
                                                const uint32_t *s_nh, const uint32_t *s_nl) {
    Segment g;
    g.n_high = s_nh[s];
    g.n_low = s_nl[s];
    const uint32_t pages_high = (g.n_high + kPageTokens - 1) / kPageTokens;
    const uint32_t pages_low = (g.n_low + kPageTokens - 1) / kPageTokens;
    const uint32_t p0 = s_prefix[s], p1 = s_prefix[s + 1], cs = p1 - p0;
    const uint32_t a = (lo > p0 ? lo : p0) - p0, e = (hi < p1 ? hi : p1) - p0;
    g.high_begin = cut_pages(a, cs, pages_high);
    g.high_count = cut_pages(e, cs, pages_high) - g.high_begin;
    g.low_begin = cut_pages(a, cs, pages_low);
    g.low_count = cut_pages(e, cs, pages_low) - g.low_begin;
    return g;
}

// Order in which a segment's pages are visited: its HIGH and LOW runs are interleaved evenly
// (page v is a HIGH page iff floor((v+1) nH / n) > floor(v nH / n), n = nH + nL).  HIGH pages are
// bandwidth-heavy and LOW pages instruction-heavy; taking them in turn lets the bulk copies of
// the former land while the latter are being decoded, instead of alternating between a
// memory-bound and an issue-bound phase.
struct PageOrder {
    uint32_t rem, hi_idx, lo_idx;
    __device__ __forceinline__ void reset() { rem = hi_idx = lo_idx = 0; }
    __device__ __forceinline__ bool is_high(const Segment &g) const { return rem + g.high_count >= g.high_count + g.low_count; }
    __device__ __forceinline__ void advance(const Segment &g) {
        if (is_high(g)) { rem -= g.low_count; hi_idx++; }
        else { rem += g.high_count; lo_idx++; }
    }
};

// Producer side of a warp's pipeline: walks the CTA's pages in order and issues one bulk copy
// per job (HIGH page: K tile, then V tile; LOW page: K and V halves together).
struct Producer {
    int s;                    // current sequence index in the call, n_seqs when exhausted
    Segment seg;
    PageOrder ord;
    uint32_t page;            // next job's page: position in the segment's interleaved order
    uint32_t sub;             // 0: K tile next, 1: V tile next (HIGH pages)
    uint32_t win_base, win_id;  // 32 page ids cached across the lanes, starting at win_base
    bool win_valid;
};

template <bool kHasLow>
struct Warp {
    const AttnParams &p;
    const uint32_t *s_prefix, *s_nh, *s_nl;
    uint32_t lo, hi;
    int lane, kv;
    uint32_t ring, bars;      // shared-space addresses of this warp's stages and mbarriers
    Producer pr;
    uint32_t issued, consumed;
    bool dead;

    __device__ __forceinline__ bool in_span(int s) const { return s < p.n_seqs && s_prefix[s] < hi; }

    __device__ __forceinline__ void producer_open(int s) {
        // advance to the next sequence of the span that has pages for this CTA
        for (; in_span(s); ++s) {
            if (s_prefix[s + 1] == s_prefix[s]) continue;
            pr.seg = make_segment(s, lo, hi, s_prefix, s_nh, s_nl);
            if (pr.seg.high_count + pr.seg.low_count > 0) break;
        }
        if (!in_span(s)) s = p.n_seqs;
        pr.s = s;
        pr.page = 0;
        pr.sub = 0;
        pr.ord.reset();
        pr.win_valid = false;
    }

    // Issue the next job into stage (issued % kStages).  Warp-uniform; lane 0 talks to the TMA.
    __device__ __forceinline__ void produce() {
        if (pr.s >= p.n_seqs) return;
        const DevCache &c = p.c;
        const bool is_high = pr.ord.is_high(pr.seg);
        const uint32_t n_pages = pr.seg.high_count + pr.seg.low_count;
        if (!pr.win_valid || pr.page - pr.win_base >= 32u) {
            // refill the page-id window: lane i holds the id of the page at position win_base + i
            pr.win_base = pr.page;
            pr.win_valid = true;
            const uint32_t pg = pr.page + lane;
            const size_t sl = ((size_t)p.seq_ids[pr.s] * c.n_layers + p.layer) * c.max_pages;
            uint32_t id = 0;
            if (pg < n_pages) {
                const uint32_t h0 = (uint32_t)(((uint64_t)pg * pr.seg.high_count) / n_pages);
                const uint32_t h1 = (uint32_t)(((uint64_t)(pg + 1) * pr.seg.high_count) / n_pages);
                id = h1 > h0 ? c.tbl_high[sl + pr.seg.high_begin + h0] : c.tbl_low[sl + pr.seg.low_begin + (pg - h0)];
            }
            pr.win_id = id;
        }
        const uint32_t id = __shfl_sync(0xffffffffu, pr.win_id, (int)(pr.page - pr.win_base));
        const uint32_t stage = issued % kStages;
        const uint8_t *src;
        uint32_t bytes;
        if (is_high) {
            src = c.pool_high + (size_t)id * c.high_page_bytes + (size_t)kv * kHighHeadBytes + pr.sub * kHighTileBytes;
            bytes = kHighTileBytes;
        } else {
            src = c.pool_low + (size_t)id * c.low_page_bytes + (size_t)kv * kLowHeadBytes;
            bytes = kLowHeadBytes;
        }
        if (lane == 0) {
            const uint32_t bar = bars + stage * 8;
            mbar_expect_tx(bar, bytes);
            bulk_g2s(ring + stage * kStageBytes, src, bytes, bar);
        }
        issued++;
        if (is_high && pr.sub == 0) {
            pr.sub = 1;
        } else {
            pr.sub = 0;
            pr.ord.advance(pr.seg);
            if (++pr.page == n_pages) producer_open(pr.s + 1);
        }
    }

    // Wait for the oldest outstanding job; returns the shared address of its stage.
    __device__ __forceinline__ uint32_t acquire() {
        const uint32_t stage = consumed % kStages, parity = (consumed / kStages) & 1u;
        if (!dead && !mbar_wait(bars + stage * 8, parity)) {
            dead = true;
            if (lane == 0) atomicOr(&p.c.ctrl[kCtrlStatus], PASK_DEV_TIMEOUT);
        }
        return ring + stage * kStageBytes;
    }
    // All lanes are done reading the oldest stage: hand it back to the producer.
    __device__ __forceinline__ void release() {
        __syncwarp();
        if (!dead) {
            consumed++;
            produce();
        }
    }
};

// ---------------------------------------------------------------- the kernel

template <bool kHasLow>
__global__ void __launch_bounds__(32 * kMaxWarps, 2) decode_attn_kernel(const __grid_constant__ AttnParams p) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const DevCache &c = p.c;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, n_warps = blockDim.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int n_seqs = p.n_seqs;

    uint32_t *s_prefix = reinterpret_cast<uint32_t *>(smem);
    uint32_t *s_nh = s_prefix + n_seqs + 1;
    uint32_t *s_nl = s_nh + n_seqs;
    size_t off = ((size_t)(3 * n_seqs + 1) * 4 + 127) & ~(size_t)127;
    uint64_t *s_bar = reinterpret_cast<uint64_t *>(smem + off);
    off += 256;                                             // kMaxWarps * kStages * 8 = 192 bytes of barriers
    off = (off + 1023) & ~(size_t)1023;
    uint8_t *s_ring = smem + off;

    // ---- per-sequence costs and their prefix sum (every CTA computes the same table)
    for (int s = tid; s < n_seqs; s += blockDim.x) {
        const int sid = p.seq_ids[s];
        uint32_t nh = 0, nl = 0;
        if (sid >= 0 && sid < c.max_seqs) {
            const size_t sl = (size_t)sid * c.n_layers + p.layer;
            nh = c.n_high[sl];
            if (kHasLow) nl = c.n_low[sl];
        }
        s_nh[s] = nh;
        s_nl[s] = nl;
        s_prefix[s + 1] = ((nh + kPageTokens - 1) / kPageTokens) * kCostHighPage +
                          ((nl + kPageTokens - 1) / kPageTokens) * kCostLowPage;
    }
    if (tid == 0) s_prefix[0] = 0;
    __syncthreads();
    if (warp == 0) {
        uint32_t carry = 0;
        for (int base = 0; base < n_seqs; base += 32) {
            const int idx = base + lane;
            uint32_t inc = idx < n_seqs ? s_prefix[idx + 1] : 0u;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t o = __shfl_up_sync(0xffffffffu, inc, d);
                if (lane >= d) inc += o;
            }
            if (idx < n_seqs) s_prefix[idx + 1] = carry + inc;
            carry += __shfl_sync(0xffffffffu, inc, 31);
        }
    }
    __syncthreads();
    const uint32_t total = s_prefix[n_seqs];
    if (blockIdx.x == 0)
        for (int s = tid; s <= n_seqs; s += blockDim.x) p.prefix_out[s] = s_prefix[s];
    if (total == 0) return;

    const uint32_t n_ctas = gridDim.x, b = blockIdx.x;
    const uint32_t lo = (uint32_t)(((uint64_t)total * b) / n_ctas);
    const uint32_t hi = (uint32_t)(((uint64_t)total * (b + 1)) / n_ctas);
    // first sequence of the span: prefix[s0] <= lo < prefix[s0 + 1]
    int s0;
    {
        int a = 1, e = n_seqs;  // smallest idx in [1, n_seqs] with prefix[idx] > lo
        while (a < e) {
            const int mid = (a + e) >> 1;
            if (s_prefix[mid] > lo) e = mid; else a = mid + 1;
        }
        s0 = a - 1;
    }

    Warp<kHasLow> w{p, s_prefix, s_nh, s_nl, lo, hi, lane, warp,
                    smem_u32(s_ring + (size_t)warp * kStages * kStageBytes), smem_u32(s_bar + warp * kStages),
                    {}, 0u, 0u, false};
    if (lane == 0) {
        for (int i = 0; i < kStages; i++) mbar_init(w.bars + i * 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    w.producer_open(s0);
    for (int i = 0; i < kStages; i++) w.produce();

    const float kLog2Scale = 0.088388347648318440550f * 1.4426950408889634074f;  // log2(e) / sqrt(128)
    const int head_a = 2 * (t & 1);          // this lane's two score / output columns are heads a, a + 1
    const int qh0 = warp * 4;                // first query head of this KV head
    const uint32_t slot_bias = b;

    for (int s = s0; w.in_span(s); ++s) {
        if (s_prefix[s + 1] == s_prefix[s]) continue;
        const Segment seg = make_segment(s, lo, hi, s_prefix, s_nh, s_nl);

        // ---- query fragments: lane (g,t) holds dims 8(4j+t) .. +7 of head g & 3 for j = 0..3
        uint4 qf[4];
        {
            const uint4 *qrow = p.q + ((size_t)s * c.n_q + qh0 + (g & 3)) * 16;
#pragma unroll
            for (int j = 0; j < 4; j++) qf[j] = __ldg(qrow + 4 * j + t);
        }
        // -136 * sum of q over each 32-dim group, for this lane's two heads (initial accumulator of
        // the LOW-stream QK^T, which multiplies q with 128 + code instead of code - 8)
        float nq[4][2];
        if (kHasLow) {
#pragma unroll
            for (int j = 0; j < 4; j++) {
                const uint32_t r[4] = {qf[j].x, qf[j].y, qf[j].z, qf[j].w};
                float sum = 0.f;
#pragma unroll
                for (int i = 0; i < 4; i++) sum += __uint_as_float(r[i] << 16) + __uint_as_float(r[i] & 0xffff0000u);
                sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                nq[j][0] = -136.f * __shfl_sync(0xffffffffu, sum, 4 * head_a);
                nq[j][1] = -136.f * __shfl_sync(0xffffffffu, sum, 4 * (head_a + 1));
            }
        }

        float acc[8][4];
#pragma unroll
        for (int m = 0; m < 8; m++) acc[m][0] = acc[m][1] = acc[m][2] = acc[m][3] = 0.f;
        float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;

        PageOrder ord;
        ord.reset();
        for (uint32_t page = 0; page < seg.high_count + seg.low_count; ++page, ord.advance(seg)) {
            const bool is_high = ord.is_high(seg);
            uint32_t n_valid;
            if (is_high) n_valid = min(16u, seg.n_high - (seg.high_begin + ord.hi_idx) * kPageTokens);
            else n_valid = min(16u, seg.n_low - (seg.low_begin + ord.lo_idx) * kPageTokens);

            float sc[4] = {0.f, 0.f, 0.f, 0.f};
            uint32_t st = w.acquire();
            if (w.dead) break;
            if (is_high) {
                // ---- QK^T over a bf16 K tile: 8 MMAs, two independent accumulators
                float sc2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    const uint4 k0 = lds128(st + (2 * j) * 512 + lane * 16);      // token g
                    const uint4 k1 = lds128(st + (2 * j + 1) * 512 + lane * 16);  // token g + 8
                    mma_bf16(sc, k0.x, k1.x, k0.y, k1.y, qf[j].x, qf[j].y);
                    mma_bf16(sc2, k0.z, k1.z, k0.w, k1.w, qf[j].z, qf[j].w);
                }
#pragma unroll
                for (int i = 0; i < 4; i++) sc[i] += sc2[i];
                w.release();
            } else if (kHasLow) {
                const uint4 k0 = lds128(st + lane * 16);
                const uint4 k1 = lds128(st + 512 + lane * 16);
                const uint2 ks0 = lds64(st + kLowCodesBytes + g * 8);
                const uint2 ks1 = lds64(st + kLowCodesBytes + (g + 8) * 8);
                const uint32_t w0[4] = {k0.x, k0.y, k0.z, k0.w}, w1[4] = {k1.x, k1.y, k1.z, k1.w};
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    float cj[4] = {nq[j][0], nq[j][1], nq[j][0], nq[j][1]};
                    mma_bf16(cj, nib2bf16(w0[j]), nib2bf16(w1[j]), nib2bf16(w0[j] >> 4), nib2bf16(w1[j] >> 4),
                             qf[j].x, qf[j].y);
                    mma_bf16(cj, nib2bf16(w0[j] >> 8), nib2bf16(w1[j] >> 8), nib2bf16(w0[j] >> 12),
                             nib2bf16(w1[j] >> 12), qf[j].z, qf[j].w);
                    const float f0 = pick4(ks0, j), f1 = pick4(ks1, j);
                    sc[0] = fmaf(f0, cj[0], sc[0]);
                    sc[1] = fmaf(f0, cj[1], sc[1]);
                    sc[2] = fmaf(f1, cj[2], sc[2]);
                    sc[3] = fmaf(f1, cj[3], sc[3]);
                }
            }

            // ---- online softmax for heads a, a+1 over tokens g and g + 8 of the tile
            float z0 = sc[0] * kLog2Scale, z1 = sc[1] * kLog2Scale, z2 = sc[2] * kLog2Scale, z3 = sc[3] * kLog2Scale;
            if ((uint32_t)g >= n_valid) z0 = z1 = -INFINITY;
            if ((uint32_t)g + 8u >= n_valid) z2 = z3 = -INFINITY;
            float ta = fmaxf(z0, z2), tb = fmaxf(z1, z3);
#pragma unroll
            for (int d = 4; d < 32; d <<= 1) {
                ta = fmaxf(ta, __shfl_xor_sync(0xffffffffu, ta, d));
                tb = fmaxf(tb, __shfl_xor_sync(0xffffffffu, tb, d));
            }
            const float mna = fmaxf(m_a, ta), mnb = fmaxf(m_b, tb);
            if (__any_sync(0xffffffffu, mna > m_a || mnb > m_b)) {
                const float fa = ex2(m_a - mna), fb = ex2(m_b - mnb);
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
                split_pair(p0, p1, h01, l01);
                split_pair(p2, p3, h23, l23);
                const uint32_t bh0 = movmatrix_trans(h01), bh1 = movmatrix_trans(h23);
                const uint32_t bl0 = movmatrix_trans(l01), bl1 = movmatrix_trans(l23);
                st = w.acquire();
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
                w.release();
            } else if (kHasLow) {
                const uint32_t vb = st + kLowHalfBytes;
                const uint4 v0 = lds128(vb + lane * 16);        // tokens 2t, 2t+1
                const uint4 v1 = lds128(vb + 512 + lane * 16);  // tokens 2t+8, 2t+9
                uint2 vs0 = lds64(vb + kLowCodesBytes + g * 8);
                uint2 vs1 = lds64(vb + kLowCodesBytes + (g + 8) * 8);
                w.release();   // everything of this stage is in registers now
                if ((uint32_t)g >= n_valid) vs0 = make_uint2(0, 0);
                if ((uint32_t)g + 8u >= n_valid) vs1 = make_uint2(0, 0);
                const uint32_t c0[4] = {v0.x, v0.y, v0.z, v0.w}, c1[4] = {v1.x, v1.y, v1.z, v1.w};
#pragma unroll
                for (int v = 0; v < 2; v++) {
                    // B columns 0-3: heads x group 2v, columns 4-7: heads x group 2v + 1
                    const int grp = 2 * v + (t >> 1);
                    const float f0 = pick4(vs0, grp), f1 = pick4(vs1, grp);
                    uint32_t h01, l01, h23, l23;
                    split_pair(p0 * f0, p1 * f0, h01, l01);
                    split_pair(p2 * f1, p3 * f1, h23, l23);
                    const uint32_t bh0 = movmatrix_trans(h01), bh1 = movmatrix_trans(h23);
                    const uint32_t bl0 = movmatrix_trans(l01), bl1 = movmatrix_trans(l23);
#pragma unroll
                    for (int qq = 0; qq < 2; qq++) {
                        const int q = 2 * v + qq;
                        uint32_t a[2][4];
#pragma unroll
                        for (int i = 0; i < 4; i++) {
                            a[0][i] = sub_bf16x2(nib2bf16(c0[q] >> (4 * i)), 0x43084308u);  // (128 + code) - 136
                            a[1][i] = sub_bf16x2(nib2bf16(c1[q] >> (4 * i)), 0x43084308u);
                        }
#pragma unroll
                        for (int r = 0; r < 2; r++) {
                            mma_bf16(acc[2 * q + r], a[0][2 * r], a[0][2 * r + 1], a[1][2 * r], a[1][2 * r + 1], bh0, bh1);
                            mma_bf16(acc[2 * q + r], a[0][2 * r], a[0][2 * r + 1], a[1][2 * r], a[1][2 * r + 1], bl0, bl1);
                        }
                    }
                }
            }
        }

        if (w.dead) break;   // a wait ran out: results are void, the status word says so

        // ---- this segment's partial: (m, l) per head, unnormalised o
#pragma unroll
        for (int d = 4; d < 32; d <<= 1) {
            l_a += __shfl_xor_sync(0xffffffffu, l_a, d);
            l_b += __shfl_xor_sync(0xffffffffu, l_b, d);
        }
        const size_t slot = (size_t)slot_bias + s;
        const size_t hrow = slot * c.n_q + qh0 + head_a;
        if (g == 0 && t < 2) {
            p.part_ml[hrow] = make_float2(m_a, l_a);
            p.part_ml[hrow + 1] = make_float2(m_b, l_b);
        }
#pragma unroll
        for (int m = 0; m < 8; m++) {
            const int q = m >> 1, r = m & 1;
            if ((t >> 1) == (q & 1)) {   // even groups are valid in columns 0-3, odd groups in 4-7
                const int dim = 32 * q + 4 * g + 2 * r;
                *reinterpret_cast<float2 *>(p.part_o + hrow * kHeadDim + dim) = make_float2(acc[m][0], acc[m][2]);
                *reinterpret_cast<float2 *>(p.part_o + (hrow + 1) * kHeadDim + dim) = make_float2(acc[m][1], acc[m][3]);
            }
        }
    }

    // A wait gave up: copies may still be in flight towards this CTA's shared memory.  Give each
    // outstanding stage one more bounded wait before the CTA retires.
    if (w.dead) {
        while (w.consumed < w.issued) {
            const uint32_t stage = w.consumed % kStages, parity = (w.consumed / kStages) & 1u;
            mbar_wait(w.bars + stage * 8, parity);
            w.consumed++;
        }
    }
}

// Merge the partials of each (sequence, query head): one warp each, lane = 4 output dims.
__global__ void __launch_bounds__(256)
combine_kernel(const uint32_t *__restrict__ prefix, const float2 *__restrict__ part_ml, const float *__restrict__ part_o,
               float *__restrict__ out, float *__restrict__ lse, int n_seqs, int n_q, uint32_t n_ctas) {
    const int wid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (wid >= n_seqs * n_q) return;
    const int s = wid / n_q, h = wid % n_q;
    const uint32_t p0 = prefix[s], p1 = prefix[s + 1];
    const uint64_t total = prefix[n_seqs];
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    float M = -INFINITY, L = 0.f;
    if (p1 > p0) {
        const uint32_t b_first = (uint32_t)((((uint64_t)p0 + 1) * n_ctas - 1) / total);
        const uint32_t b_last = (uint32_t)(((uint64_t)p1 * n_ctas - 1) / total);
        for (uint32_t b = b_first; b <= b_last; b++) M = fmaxf(M, part_ml[((size_t)b + s) * n_q + h].x);
        if (M > -INFINITY) {
            for (uint32_t b = b_first; b <= b_last; b++) {
                const size_t row = ((size_t)b + s) * n_q + h;
                const float2 ml = part_ml[row];
                if (ml.x == -INFINITY) continue;      // a CTA whose share of this sequence was empty
                const float wgt = exp2f(ml.x - M);
                const float4 v = *reinterpret_cast<const float4 *>(part_o + row * kHeadDim + lane * 4);
                o.x = fmaf(wgt, v.x, o.x); o.y = fmaf(wgt, v.y, o.y); o.z = fmaf(wgt, v.z, o.z); o.w = fmaf(wgt, v.w, o.w);
                L = fmaf(wgt, ml.y, L);
            }
        }
    }
    const size_t orow = (size_t)s * n_q + h;
    if (L > 0.f) {
        const float inv = 1.0f / L;
        o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
    }
    *reinterpret_cast<float4 *>(out + orow * kHeadDim + lane * 4) = o;
    if (lse && lane == 0) lse[orow] = L > 0.f ? (M + log2f(L)) * 0.69314718055994530942f : -INFINITY;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

size_t attn_smem_bytes(int n_seqs, int n_warps) {
    size_t off = align_up((size_t)(3 * n_seqs + 1) * 4, 128) + 256;
    off = align_up(off, 1024);
    return off + (size_t)n_warps * kStages * kStageBytes;
}

}  // namespace

int attention_grid(const pask_cache *c) { return 2 * c->sm_count; }

size_t attention_workspace_bytes(const pask_cache *c, int n_seqs) {
    const size_t slots = (size_t)c->attn_ctas + n_seqs;
    return align_up((size_t)(n_seqs + 1) * 4, 256) + align_up(slots * c->desc.n_q_heads * sizeof(float2), 256) +
           slots * c->desc.n_q_heads * kHeadDim * sizeof(float);
}

pask_status_t launch_attention(pask_cache *c, bool has_low, int layer, int n_seqs, const int32_t *seq_ids, const void *q,
                               float *out, float *lse, void *workspace, size_t, cudaStream_t stream) {
    const int n_warps = c->desc.n_kv_heads;
    const size_t slots = (size_t)c->attn_ctas + n_seqs;
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    AttnParams p;
    p.c = c->dev;
    p.layer = layer;
    p.n_seqs = n_seqs;
    p.seq_ids = seq_ids;
    p.q = static_cast<const uint4 *>(q);
    p.prefix_out = reinterpret_cast<uint32_t *>(ws);
    ws += align_up((size_t)(n_seqs + 1) * 4, 256);
    p.part_ml = reinterpret_cast<float2 *>(ws);
    ws += align_up(slots * c->desc.n_q_heads * sizeof(float2), 256);
    p.part_o = reinterpret_cast<float *>(ws);
    const size_t smem = attn_smem_bytes(n_seqs, n_warps);
    auto kern = has_low ? decode_attn_kernel<true> : decode_attn_kernel<false>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return PASK_ERR_CUDA;
    if (c->ev_start) cudaEventRecord(c->ev_start, stream);
    kern<<<c->attn_ctas, 32 * n_warps, smem, stream>>>(p);
    if (c->ev_stop) cudaEventRecord(c->ev_stop, stream);
    c->ev_start = c->ev_stop = nullptr;
    const int warps = n_seqs * c->desc.n_q_heads;
    combine_kernel<<<(warps + 7) / 8, 256, 0, stream>>>(p.prefix_out, p.part_ml, p.part_o, out, lse, n_seqs,
                                                        c->desc.n_q_heads, (uint32_t)c->attn_ctas);
    return cudaGetLastError() == cudaSuccess ? PASK_OK : PASK_ERR_CUDA;
}

}  // namespace pask
