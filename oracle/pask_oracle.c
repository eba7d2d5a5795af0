/*
 * PASK online hot path -- plain CPU oracle.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, sequential, obviously-correct statement of what the CUDA library must
 * compute.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may call it; the
 * product never does, and it shares no source, header, table or helper with the CUDA path.
 *
 * What it follows (the paper's section / equation / algorithm):
 *   - actions R < L < H with costs m(R)=0 < m(L) < m(H); release removes a KV state from future
 *     attention (Section 3.1, "Setup and Objective");
 *   - buckets q = (tag, layer group), so one token may get different actions at different depths
 *     (Eq. 3 and the paragraph after it);
 *   - the frozen table stores selected action, floor and upgrade scores per bucket (end of
 *     Section 3.3); online, a = max(a0, a_floor) (Eq. 10, Algorithm 2 steps 1-2);
 *   - Persist(a) (Algorithm 2 step 7) and the budget recurrence R' = R - sum m(a) (step 8);
 *   - the dynamic adjustment between them (Algorithm 2 steps 3-6, Eq. 10 and the paragraph after
 *     it): B = [R - Gamma(s)]+, demotions above the floors in ascending upgrade score while the
 *     token's cost exceeds B, promotions in descending score in critical states while they fit,
 *     floors first when budget and protection conflict (orc_decide);
 *   - the protected recent window (Section 3.1): release and the low format take effect on a state
 *     only after it has left the window, so the last W tokens are attended at full precision;
 *   - normalised cost C_KV = sum m(a) / sum m(H) (Eq. 1);
 *   - the reference policy is full high precision (Section 3.1), whose attention outputs are the
 *     ones Eq. 4 compares against: plain softmax(q k^T / sqrt(d)) v over the retained history.
 *
 * Readings where the paper is silent (the low-precision format, paging, budget units, unknown
 * tags) are the library's documented ones: RETAIN-LOW is symmetric int4 per token, per KV head,
 * per group of 32 consecutive head dimensions with one fp16 scale (amax/7, round to nearest
 * even, codes stored offset by 8) -- or, policy low_bits = 8, symmetric int8 in the same grouping
 * (amax/127, codes offset by 128), or, low_bits = 2, the three levels -s, 0, +s with s = amax
 * (codes offset by 2); RETAIN-HIGH keeps the bf16 bits; pages hold 16 tokens and
 * are handed out in call order from a per-pool free stack, else a bump counter; costs are
 * payload bytes.  Parity unpinned by the paper for: the low-bit format itself, the size of the
 * recent window (a policy parameter here, 0 by default; the paper gives no number) and that a
 * token is charged m(a) when it arrives rather than when it leaves the window, the initial
 * budget, and the treatment of prompt tags -- those are pinned only
 * by this library's own documentation.  The paper gives Demote, Promote and Crit in one sentence
 * each and R's starting value not at all: the reading written out above decide_token (budget
 * accrued per token seen, one step at a time, ties to the first group, "eligible" = fits in B)
 * is this library's, pinned by hand-worked cases and invariants, not by values the paper prints.
 *
 * Arithmetic: decisions, codes, scales, page ids and counters are integer / IEEE fp32 with no
 * contraction (build with -ffp-contract=off); attention is fp64 over the dequantised values.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_ERR_ARG (-1)
#define ORC_ERR_POLICY (-2)
#define ORC_ERR_POOL (-4)
#define ORC_ERR_SEQ (-5)

#define HEAD_DIM 128
#define PAGE_TOKENS 16
#define QGROUP 32
#define GROUPS_PER_HEAD (HEAD_DIM / QGROUP)
#define MAX_GROUPS 8
#define MAX_WINDOW 256
#define TAG_PROTECTED 0xFF

enum { ACT_R = 0, ACT_L = 1, ACT_H = 2 };

typedef struct {
    uint32_t n_tags, n_groups, n_layers, n_states;
    uint32_t budget_q16, recent_window, low_bits, group_size;
    uint8_t *layer_group;   /* [n_layers] */
    uint8_t *a0, *a_floor;  /* [n_tags * n_groups] */
    uint8_t *eff;           /* max(a0, a_floor) */
    float *rho_rl, *rho_lh;
    uint32_t *gamma;        /* [n_states] reserve, in units of 2^gamma_shift bytes */
    uint8_t *crit;          /* [n_states] 1 = critical or lookahead-critical state */
    uint32_t gamma_shift;
} orc_policy;

typedef struct {
    uint64_t n_seen[MAX_GROUPS], n_high[MAX_GROUPS], n_low[MAX_GROUPS], n_drop[MAX_GROUPS];
    uint64_t retained_bytes, full_bytes;
    int64_t remaining_bytes;
    uint64_t bad_tags;
    uint32_t pages_high, pages_low;
    /* Algorithm 2's own running budget, advanced by orc_decide (one step per token, all groups) */
    uint64_t decided_full_bytes, decided_retained_bytes;
    uint64_t n_demoted, n_promoted, n_floor_conflicts;
} orc_budget;

typedef struct {          /* one (sequence, layer) pair: two compacted streams */
    uint32_t n_high, n_low;
    uint32_t cap_high, cap_low;
    uint16_t *hk, *hv;    /* [n_high][n_kv][128] bf16 bit patterns */
    uint8_t *lk, *lv;     /* [n_low][n_kv][128] codes 1..15 */
    uint16_t *lks, *lvs;  /* [n_low][n_kv][4] fp16 scale bit patterns */
    uint32_t *pg_high, *pg_low; /* page ids, one per started 16-token page */
    uint32_t npg_high, npg_low, cap_pg_high, cap_pg_low;
    /* protected recent window (W = policy recent_window > 0): the last W tokens of this
     * (sequence, layer), whatever their action, as bf16 bits; token t sits in slot t mod W */
    uint32_t n_tok;       /* tokens appended so far, released ones included */
    uint16_t *wk, *wv;    /* [W][n_kv][128] */
    uint8_t *wact;        /* [W] the action each of them took */
} orc_stream;

typedef struct {
    uint32_t cap, next, n_free;
    uint32_t *free_stack;
} orc_pool;

typedef struct {
    const orc_policy *pol;
    int n_q, n_kv, max_seqs;
    uint32_t n_layers;    /* copy of pol->n_layers, so that tearing down needs no policy */
    orc_stream *streams;  /* [max_seqs][n_layers] */
    orc_budget *budget;   /* [max_seqs] */
    orc_pool pool_high, pool_low;
} orc_cache;

/* ------------------------------------------------------------------ number formats */

static float bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* fp32 -> fp16 bit pattern, round to nearest even, done by hand on the bit fields.
 * Finite values too large for fp16 saturate to 65504 (0x7BFF) instead of becoming infinite. */
uint16_t orc_f32_to_f16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    uint32_t ex = (u >> 23) & 0xFFu;
    uint32_t man = u & 0x7FFFFFu;
    if (ex == 0xFF) return (uint16_t)(sign | (man ? 0x7E00u : 0x7C00u));
    int e = (int)ex - 127;                       /* unbiased exponent of 1.man */
    if (e > 15) return (uint16_t)(sign | 0x7BFFu);
    if (e >= -14) {                              /* normal fp16: keep 10 mantissa bits */
        uint32_t keep = man >> 13, rest = man & 0x1FFFu;
        uint32_t h = ((uint32_t)(e + 15) << 10) | keep;
        if (rest > 0x1000u || (rest == 0x1000u && (keep & 1u))) h += 1; /* may carry into exponent */
        if (h >= 0x7C00u) h = 0x7BFFu;
        return (uint16_t)(sign | h);
    }
    if (e < -25) return sign;                    /* below half of the smallest subnormal */
    /* subnormal: value = full * 2^(e-23), unit = 2^-24 -> shift right by (-e-1) in [14,24] */
    uint32_t full = man | 0x800000u;
    int sh = -e - 1;
    uint32_t keep = full >> sh;
    uint32_t rest = full & ((1u << sh) - 1u);
    uint32_t half = 1u << (sh - 1);
    if (rest > half || (rest == half && (keep & 1u))) keep += 1;
    return (uint16_t)(sign | keep);
}

float orc_f16_to_f32(uint16_t h) {
    uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    uint32_t ex = (h >> 10) & 0x1Fu, man = h & 0x3FFu;
    float mag;
    if (ex == 0) mag = ldexpf((float)man, -24);
    else if (ex == 31) mag = man ? NAN : INFINITY;
    else mag = ldexpf((float)(man | 0x400u), (int)ex - 25);
    uint32_t u;
    memcpy(&u, &mag, 4);
    u |= sign;
    memcpy(&mag, &u, 4);
    return mag;
}

/* RETAIN-LOW of one group of 32 values (bf16 bit patterns in): one fp16 scale, 32 codes.
 * bits = 4: codes clamp(rint(x / s), -7, 7) + 8 with s = fp16(amax / 7);
 * bits = 8: codes clamp(rint(x / s), -127, 127) + 128 with s = fp16(amax / 127);
 * bits = 2: codes clamp(rint(x / s), -1, 1) + 2 with s = fp16(amax) (three levels: -s, 0, +s).
 * In general the largest level is 2^(bits-1) - 1 and the code of zero 2^(bits-1). */
void orc_quantize_group_bits(const uint16_t *x_bits, uint16_t *scale_bits, uint8_t *codes, int bits) {
    const float qmax = (float)((1 << (bits - 1)) - 1);
    const int zero = 1 << (bits - 1);
    float amax = 0.0f;
    for (int i = 0; i < QGROUP; i++) {
        float a = fabsf(bf16_to_f32(x_bits[i]));
        if (a > amax) amax = a;
    }
    float s32 = amax / qmax;
    uint16_t sh = orc_f32_to_f16_rne(s32);
    float s = orc_f16_to_f32(sh);
    *scale_bits = sh;
    if (s == 0.0f) {
        for (int i = 0; i < QGROUP; i++) codes[i] = (uint8_t)zero;
        return;
    }
    float inv = 1.0f / s;
    for (int i = 0; i < QGROUP; i++) {
        float r = rintf(bf16_to_f32(x_bits[i]) * inv); /* ties to even in the default mode */
        if (r > qmax) r = qmax;
        if (r < -qmax) r = -qmax;
        codes[i] = (uint8_t)((int)r + zero);
    }
}

void orc_quantize_group(const uint16_t *x_bits, uint16_t *scale_bits, uint8_t *codes) {
    orc_quantize_group_bits(x_bits, scale_bits, codes, 4);
}

/* ------------------------------------------------------------------ policy */

int orc_lut_fold(int a0, int a_floor) { return a0 > a_floor ? a0 : a_floor; } /* Eq. 10 */

static uint32_t rd32(const uint8_t *p) {
    return (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24);
}

void orc_policy_free(orc_policy *p) {
    if (!p) return;
    free(p->layer_group); free(p->a0); free(p->a_floor); free(p->eff);
    free(p->rho_rl); free(p->rho_lh); free(p->gamma); free(p->crit);
    free(p);
}

orc_policy *orc_policy_load(const uint8_t *blob, size_t len, int *err) {
    *err = ORC_ERR_POLICY;
    if (!blob || len < 40 || memcmp(blob, "PASK", 4) != 0) return NULL;
    const uint32_t version = rd32(blob + 4);
    if (version != 1 && version != 2) return NULL;
    orc_policy *p = (orc_policy *)calloc(1, sizeof(*p));
    p->n_tags = rd32(blob + 8); p->n_groups = rd32(blob + 12); p->n_layers = rd32(blob + 16);
    p->n_states = rd32(blob + 20); p->budget_q16 = rd32(blob + 24); p->recent_window = rd32(blob + 28);
    p->low_bits = rd32(blob + 32); p->group_size = rd32(blob + 36);
    if (p->n_tags == 0 || p->n_tags > 255 || p->n_groups == 0 || p->n_groups > MAX_GROUPS ||
        p->n_layers == 0 || p->n_layers > 4096 || p->n_states > (1u << 20) || p->recent_window % PAGE_TOKENS != 0 || p->recent_window > MAX_WINDOW ||
        (p->low_bits != 4 && p->low_bits != 8 && p->low_bits != 2) || p->group_size != QGROUP) { free(p); return NULL; }
    size_t lg_pad = (p->n_layers + 3u) & ~(size_t)3u;
    size_t n_ent = (size_t)p->n_tags * p->n_groups;
    size_t need = 40 + lg_pad + n_ent * 12 + (size_t)p->n_states * 4;
    if (version == 2) need += 4 + (((size_t)p->n_states + 3u) & ~(size_t)3u);
    if (len != need) { free(p); return NULL; }
    p->layer_group = (uint8_t *)malloc(p->n_layers);
    memcpy(p->layer_group, blob + 40, p->n_layers);
    p->a0 = (uint8_t *)malloc(n_ent); p->a_floor = (uint8_t *)malloc(n_ent); p->eff = (uint8_t *)malloc(n_ent);
    p->rho_rl = (float *)malloc(n_ent * 4); p->rho_lh = (float *)malloc(n_ent * 4);
    p->gamma = (uint32_t *)malloc((size_t)p->n_states * 4 + 4);
    p->crit = (uint8_t *)calloc((size_t)p->n_states + 4, 1);
    int bad = 0;
    for (uint32_t l = 0; l < p->n_layers; l++) if (p->layer_group[l] >= p->n_groups) bad = 1;
    const uint8_t *e = blob + 40 + lg_pad;
    for (size_t i = 0; i < n_ent; i++, e += 12) {
        p->a0[i] = e[0]; p->a_floor[i] = e[1];
        if (e[0] > ACT_H || e[1] > ACT_H || e[2] || e[3]) bad = 1;
        memcpy(&p->rho_rl[i], e + 4, 4); memcpy(&p->rho_lh[i], e + 8, 4);
        if (isnan(p->rho_rl[i]) || isnan(p->rho_lh[i])) bad = 1;   /* scores must be comparable */
        p->eff[i] = (uint8_t)orc_lut_fold(e[0], e[1]);
    }
    for (uint32_t s = 0; s < p->n_states; s++, e += 4) p->gamma[s] = rd32(e);
    if (version == 2) {
        p->gamma_shift = rd32(e); e += 4;
        if (p->gamma_shift > 16) bad = 1;
        for (uint32_t s = 0; s < p->n_states; s++) { p->crit[s] = e[s]; if (e[s] > 1) bad = 1; }
    }
    if (bad) { orc_policy_free(p); return NULL; }
    *err = ORC_OK;
    return p;
}

int orc_policy_action(const orc_policy *p, int tag, int group) { return p->eff[(size_t)tag * p->n_groups + group]; }

/* ------------------------------------------------------------------ cache */

static uint64_t bytes_high(const orc_cache *c) { return 2ull * c->n_kv * HEAD_DIM * 2; }
static uint64_t bytes_low(const orc_cache *c) {   /* codes at low_bits each, one fp16 scale per group */
    return 2ull * c->n_kv * (HEAD_DIM * c->pol->low_bits / 8 + GROUPS_PER_HEAD * 2);
}

static void pool_init(orc_pool *p, uint32_t cap) {
    p->cap = cap; p->next = 0; p->n_free = 0;
    p->free_stack = (uint32_t *)malloc((size_t)(cap ? cap : 1) * 4);
}
static uint32_t pool_available(const orc_pool *p) { return p->n_free + (p->cap - p->next); }
static uint32_t pool_alloc(orc_pool *p) { return p->n_free ? p->free_stack[--p->n_free] : p->next++; }

orc_cache *orc_cache_create(const orc_policy *pol, int n_q, int n_kv, int max_seqs,
                            uint32_t pool_high_pages, uint32_t pool_low_pages) {
    if (!pol || n_kv <= 0 || n_q != 4 * n_kv || max_seqs <= 0) return NULL;
    orc_cache *c = (orc_cache *)calloc(1, sizeof(*c));
    c->pol = pol; c->n_q = n_q; c->n_kv = n_kv; c->max_seqs = max_seqs; c->n_layers = pol->n_layers;
    c->streams = (orc_stream *)calloc((size_t)max_seqs * pol->n_layers, sizeof(orc_stream));
    c->budget = (orc_budget *)calloc((size_t)max_seqs, sizeof(orc_budget));
    pool_init(&c->pool_high, pool_high_pages);
    pool_init(&c->pool_low, pool_low_pages);
    return c;
}

static void stream_free(orc_stream *s) {
    free(s->hk); free(s->hv); free(s->lk); free(s->lv); free(s->lks); free(s->lvs);
    free(s->pg_high); free(s->pg_low); free(s->wk); free(s->wv); free(s->wact);
    memset(s, 0, sizeof(*s));
}

void orc_cache_destroy(orc_cache *c) {
    if (!c) return;
    for (size_t i = 0; i < (size_t)c->max_seqs * c->n_layers; i++) stream_free(&c->streams[i]);
    free(c->streams); free(c->budget); free(c->pool_high.free_stack); free(c->pool_low.free_stack);
    free(c);
}

static orc_stream *stream_of(orc_cache *c, int seq, int layer) { return &c->streams[(size_t)seq * c->pol->n_layers + layer]; }

/* Release every page of a sequence: layers ascending, within a layer the HIGH table then the LOW
 * table, each in table order; a page pushed later is handed out earlier (LIFO). */
int orc_seq_reset(orc_cache *c, int seq) {
    if (seq < 0 || seq >= c->max_seqs) return ORC_ERR_SEQ;
    for (uint32_t l = 0; l < c->pol->n_layers; l++) {
        orc_stream *s = stream_of(c, seq, (int)l);
        for (uint32_t i = 0; i < s->npg_high; i++) c->pool_high.free_stack[c->pool_high.n_free++] = s->pg_high[i];
        for (uint32_t i = 0; i < s->npg_low; i++) c->pool_low.free_stack[c->pool_low.n_free++] = s->pg_low[i];
        stream_free(s);
    }
    memset(&c->budget[seq], 0, sizeof(orc_budget));
    return ORC_OK;
}

static int decide(const orc_policy *p, int group, uint8_t tag, int *bad) {
    *bad = 0;
    if (tag == TAG_PROTECTED) return ACT_H;
    if (tag >= p->n_tags) { *bad = 1; return ACT_H; }
    return p->eff[(size_t)tag * p->n_groups + group];
}

#define GROW(ptr, cap, need, elem)                                             \
    do { if ((need) > (cap)) { uint32_t nc = (cap) ? (cap) * 2 : 64;            \
         while (nc < (need)) nc *= 2;                                          \
         (ptr) = realloc((ptr), (size_t)nc * (elem)); (cap) = nc; } } while (0)

/* The action of token t at layer group `group`: the table's (Algorithm 2 steps 1-2), or, when
 * `decided` is given, the one orc_decide chose for it (steps 3-6), row t of [total][n_groups]. */
static int action_of(const orc_policy *p, int group, const uint8_t *tags, const uint8_t *decided, int t, int *bad) {
    int a = decide(p, group, tags[t], bad);
    if (decided) a = decided[(size_t)t * p->n_groups + group];
    return a;
}

/* Algorithm 2 steps 1, 2, 7, 8 for one layer call.  Sequences in call order, tokens in order.
 * If the call needs more pages than a pool can supply nothing changes at all.
 * With `decided` (may be NULL) step 7 persists the actions chosen by orc_decide instead. */
int orc_append_decided(orc_cache *c, int layer, int n_seqs, const int32_t *seq_ids, const int32_t *cu_tokens,
                       const uint16_t *k_bits, const uint16_t *v_bits, const uint8_t *tags, const uint8_t *decided,
                       uint8_t *actions_out) {
    const orc_policy *p = c->pol;
    if (layer < 0 || (uint32_t)layer >= p->n_layers || n_seqs < 0) return ORC_ERR_ARG;
    int group = p->layer_group[layer];
    if (decided)
        for (int t = 0; t < cu_tokens[n_seqs]; t++)
            if (decided[(size_t)t * p->n_groups + group] > ACT_H) return ORC_ERR_ARG;
    /* pass 1: how many new pages does the whole call need? */
    uint64_t need_high = 0, need_low = 0;
    for (int i = 0; i < n_seqs; i++) {
        int seq = seq_ids[i];
        if (seq < 0 || seq >= c->max_seqs) return ORC_ERR_SEQ;
        for (int j = 0; j < i; j++) if (seq_ids[j] == seq) return ORC_ERR_SEQ;
        orc_stream *s = stream_of(c, seq, layer);
        uint32_t nh = s->n_high, nl = s->n_low;
        for (int t = cu_tokens[i]; t < cu_tokens[i + 1]; t++) {
            int bad, a = action_of(p, group, tags, decided, t, &bad);
            if (a == ACT_H) { if (nh % PAGE_TOKENS == 0) need_high++; nh++; }
            else if (a == ACT_L) { if (nl % PAGE_TOKENS == 0) need_low++; nl++; }
        }
    }
    if (need_high > pool_available(&c->pool_high) || need_low > pool_available(&c->pool_low)) return ORC_ERR_POOL;
    /* pass 2: persist */
    const size_t row = (size_t)c->n_kv * HEAD_DIM, srow = (size_t)c->n_kv * GROUPS_PER_HEAD;
    for (int i = 0; i < n_seqs; i++) {
        int seq = seq_ids[i];
        orc_stream *s = stream_of(c, seq, layer);
        orc_budget *b = &c->budget[seq];
        for (int t = cu_tokens[i]; t < cu_tokens[i + 1]; t++) {
            int bad, a = action_of(p, group, tags, decided, t, &bad);
            if (actions_out) actions_out[t] = (uint8_t)a;
            b->bad_tags += (uint64_t)bad;
            b->n_seen[group]++;
            b->full_bytes += bytes_high(c);
            if (p->recent_window) {   /* every token, released ones too, enters the recent window */
                const uint32_t W = p->recent_window, slot = s->n_tok % W;
                if (!s->wk) {
                    s->wk = (uint16_t *)malloc((size_t)W * row * 2); s->wv = (uint16_t *)malloc((size_t)W * row * 2);
                    s->wact = (uint8_t *)malloc(W);
                }
                memcpy(s->wk + (size_t)slot * row, k_bits + (size_t)t * row, row * 2);
                memcpy(s->wv + (size_t)slot * row, v_bits + (size_t)t * row, row * 2);
                s->wact[slot] = (uint8_t)a;
            }
            s->n_tok++;
            if (a == ACT_R) { b->n_drop[group]++; continue; }
            if (a == ACT_H) {
                uint32_t pos = s->n_high;
                if (pos % PAGE_TOKENS == 0) {
                    GROW(s->pg_high, s->cap_pg_high, s->npg_high + 1, 4);
                    s->pg_high[s->npg_high++] = pool_alloc(&c->pool_high);
                    b->pages_high++;
                }
                if (pos + 1 > s->cap_high) {
                    uint32_t cap = s->cap_high;
                    GROW(s->hk, cap, pos + 1, row * 2);
                    GROW(s->hv, s->cap_high, pos + 1, row * 2);
                }
                memcpy(s->hk + (size_t)pos * row, k_bits + (size_t)t * row, row * 2);
                memcpy(s->hv + (size_t)pos * row, v_bits + (size_t)t * row, row * 2);
                s->n_high++;
                b->n_high[group]++;
                b->retained_bytes += bytes_high(c);
            } else {
                uint32_t pos = s->n_low;
                if (pos % PAGE_TOKENS == 0) {
                    GROW(s->pg_low, s->cap_pg_low, s->npg_low + 1, 4);
                    s->pg_low[s->npg_low++] = pool_alloc(&c->pool_low);
                    b->pages_low++;
                }
                if (pos + 1 > s->cap_low) {
                    uint32_t c1 = s->cap_low, c2 = s->cap_low, c3 = s->cap_low;
                    GROW(s->lk, c1, pos + 1, row);
                    GROW(s->lv, c2, pos + 1, row);
                    GROW(s->lks, c3, pos + 1, srow * 2);
                    GROW(s->lvs, s->cap_low, pos + 1, srow * 2);
                }
                for (size_t g = 0; g < srow; g++) {
                    orc_quantize_group_bits(k_bits + (size_t)t * row + g * QGROUP, s->lks + (size_t)pos * srow + g,
                                            s->lk + (size_t)pos * row + g * QGROUP, (int)p->low_bits);
                    orc_quantize_group_bits(v_bits + (size_t)t * row + g * QGROUP, s->lvs + (size_t)pos * srow + g,
                                            s->lv + (size_t)pos * row + g * QGROUP, (int)p->low_bits);
                }
                s->n_low++;
                b->n_low[group]++;
                b->retained_bytes += bytes_low(c);
            }
        }
        /* floor(B * full) - retained with B in Q16; full_bytes < 2^47 here so the product fits */
        b->remaining_bytes = (int64_t)(((uint64_t)p->budget_q16 * b->full_bytes) >> 16) - (int64_t)b->retained_bytes;
    }
    return ORC_OK;
}

int orc_append(orc_cache *c, int layer, int n_seqs, const int32_t *seq_ids, const int32_t *cu_tokens,
               const uint16_t *k_bits, const uint16_t *v_bits, const uint8_t *tags, uint8_t *actions_out) {
    return orc_append_decided(c, layer, n_seqs, seq_ids, cu_tokens, k_bits, v_bits, tags, NULL, actions_out);
}

/* ------------------------------------------------------------------ dynamic budget adjustment */

/* m(a, c): what action a costs for one token over all the layers of group c (Section 3.1's
 * m(R) = 0 < m(L) < m(H), summed over the group's layers). */
static uint64_t group_cost(const orc_cache *c, int a, uint32_t layers_in_group) {
    if (a == ACT_H) return layers_in_group * bytes_high(c);
    if (a == ACT_L) return layers_in_group * bytes_low(c);
    return 0;
}

/* The adjacent upgrade score of bucket (tag, group) for the step (a-1 -> a). */
static float rho_of(const orc_policy *p, int tag, int group, int a) {
    size_t i = (size_t)tag * p->n_groups + group;
    return a == ACT_H ? p->rho_lh[i] : p->rho_rl[i];
}

/* Algorithm 2 for one token, all layer groups at once (steps 1-6 and 8; step 7, Persist, is
 * orc_append_decided, layer by layer).  a_out [n_groups].
 *   R_t   = floor(target * (full cost of every token seen so far, this one included))
 *           - (cost of everything decided so far)          -- the remaining target budget
 *   B_t   = max(0, R_t - Gamma(s_t))                                           (Eq. 10)
 *   Demote: while the token's cost exceeds B_t and some group sits above its floor, lower by
 *           one step the group whose step (a-1 -> a) has the smallest upgrade score: that is
 *           the smallest distortion loss per saved cost (first such group on ties).  Floors are
 *           never crossed, even if the cost still exceeds B_t.
 *   Promote (critical states only): while some group below H can take one step up and the
 *           token's cost stays within B_t, raise the one with the largest upgrade score (first
 *           such group on ties).
 * Groups that own no layer cost nothing and are left alone.  Protected and unknown tags are
 * high precision with a high-precision floor.  A state id outside the reserve table has
 * Gamma = 0 and is not critical. */
static void decide_token(const orc_cache *c, orc_budget *b, const uint32_t *layers_in_group, uint8_t tag,
                         int has_state, uint32_t state, uint8_t *a_out) {
    const orc_policy *p = c->pol;
    const int G = (int)p->n_groups;
    int a[MAX_GROUPS], fl[MAX_GROUPS];
    const int table_tag = tag != TAG_PROTECTED && tag < p->n_tags;
    uint64_t token_full = 0;
    for (int g = 0; g < G; g++) {                                      /* steps 1-2 */
        if (table_tag) {
            fl[g] = p->a_floor[(size_t)tag * G + g];
            a[g] = orc_lut_fold(p->a0[(size_t)tag * G + g], fl[g]);
        } else {
            fl[g] = a[g] = ACT_H;
        }
        token_full += group_cost(c, ACT_H, layers_in_group[g]);
    }
    uint64_t gamma = 0;
    int crit = 0;
    if (has_state && state < p->n_states) {
        gamma = (uint64_t)p->gamma[state] << p->gamma_shift;
        crit = p->crit[state];
    }
    const uint64_t full_now = b->decided_full_bytes + token_full;
    const int64_t R = (int64_t)(((uint64_t)p->budget_q16 * full_now) >> 16) - (int64_t)b->decided_retained_bytes;
    const int64_t B = R - (int64_t)gamma > 0 ? R - (int64_t)gamma : 0;   /* step 3 */

    uint64_t cost = 0;
    for (int g = 0; g < G; g++) cost += group_cost(c, a[g], layers_in_group[g]);

    while ((int64_t)cost > B) {                                        /* step 4: Demote */
        int pick = -1;
        for (int g = 0; g < G; g++) {
            if (a[g] <= fl[g] || layers_in_group[g] == 0) continue;
            if (pick < 0 || rho_of(p, tag, g, a[g]) < rho_of(p, tag, pick, a[pick])) pick = g;
        }
        if (pick < 0) break;                                           /* only floors left */
        cost -= group_cost(c, a[pick], layers_in_group[pick]) - group_cost(c, a[pick] - 1, layers_in_group[pick]);
        a[pick]--;
        b->n_demoted++;
    }
    if ((int64_t)cost > B) b->n_floor_conflicts++;

    if (crit) {                                                        /* steps 5-6: Promote */
        for (;;) {
            int pick = -1;
            for (int g = 0; g < G; g++) {
                if (a[g] >= ACT_H || layers_in_group[g] == 0) continue;
                uint64_t up = group_cost(c, a[g] + 1, layers_in_group[g]) - group_cost(c, a[g], layers_in_group[g]);
                if ((int64_t)(cost + up) > B) continue;                /* not eligible: does not fit */
                if (pick < 0 || rho_of(p, tag, g, a[g] + 1) > rho_of(p, tag, pick, a[pick] + 1)) pick = g;
            }
            if (pick < 0) break;
            cost += group_cost(c, a[pick] + 1, layers_in_group[pick]) - group_cost(c, a[pick], layers_in_group[pick]);
            a[pick]++;
            b->n_promoted++;
        }
    }
    b->decided_full_bytes = full_now;                                  /* step 8 */
    b->decided_retained_bytes += cost;
    for (int g = 0; g < G; g++) a_out[g] = (uint8_t)a[g];
}

/* Algorithm 2 steps 1-6 and 8 for a ragged batch: each sequence's tokens in order, one budget
 * state per sequence.  states may be NULL (no reserve, nothing critical).
 * actions_out [total_tokens][n_groups].  A bad sequence id or a sequence named twice refuses the
 * whole call and changes nothing. */
int orc_decide(orc_cache *c, int n_seqs, const int32_t *seq_ids, const int32_t *cu_tokens, const uint8_t *tags,
               const uint16_t *states, uint8_t *actions_out) {
    const orc_policy *p = c->pol;
    if (n_seqs < 0) return ORC_ERR_ARG;
    for (int i = 0; i < n_seqs; i++) {
        if (seq_ids[i] < 0 || seq_ids[i] >= c->max_seqs) return ORC_ERR_SEQ;
        for (int j = 0; j < i; j++) if (seq_ids[j] == seq_ids[i]) return ORC_ERR_SEQ;
        if (cu_tokens[i + 1] < cu_tokens[i]) return ORC_ERR_ARG;
    }
    uint32_t layers_in_group[MAX_GROUPS] = {0};
    for (uint32_t l = 0; l < p->n_layers; l++) layers_in_group[p->layer_group[l]]++;
    for (int i = 0; i < n_seqs; i++)
        for (int t = cu_tokens[i]; t < cu_tokens[i + 1]; t++)
            decide_token(c, &c->budget[seq_ids[i]], layers_in_group, tags[t], states != NULL,
                         states ? states[t] : 0u, actions_out + (size_t)t * p->n_groups);
    return ORC_OK;
}

int orc_stream_len(orc_cache *c, int layer, int seq, uint32_t *n_high, uint32_t *n_low) {
    if (seq < 0 || seq >= c->max_seqs || layer < 0 || (uint32_t)layer >= c->pol->n_layers) return ORC_ERR_ARG;
    orc_stream *s = stream_of(c, seq, layer);
    *n_high = s->n_high; *n_low = s->n_low;
    return ORC_OK;
}

/* Canonical dump of the HIGH stream in arrival order. */
int orc_dump_high(orc_cache *c, int layer, int seq, uint16_t *k_out, uint16_t *v_out, uint32_t *pages_out) {
    orc_stream *s = stream_of(c, seq, layer);
    size_t row = (size_t)c->n_kv * HEAD_DIM;
    if (s->n_high) { memcpy(k_out, s->hk, s->n_high * row * 2); memcpy(v_out, s->hv, s->n_high * row * 2); }
    if (s->npg_high) memcpy(pages_out, s->pg_high, (size_t)s->npg_high * 4);
    return (int)s->npg_high;
}

/* Canonical dump of the LOW stream in arrival order. */
int orc_dump_low(orc_cache *c, int layer, int seq, uint8_t *kc, uint16_t *ks, uint8_t *vc, uint16_t *vs,
                 uint32_t *pages_out) {
    orc_stream *s = stream_of(c, seq, layer);
    size_t row = (size_t)c->n_kv * HEAD_DIM, srow = (size_t)c->n_kv * GROUPS_PER_HEAD;
    if (s->n_low) {
        memcpy(kc, s->lk, s->n_low * row); memcpy(vc, s->lv, s->n_low * row);
        memcpy(ks, s->lks, s->n_low * srow * 2); memcpy(vs, s->lvs, s->n_low * srow * 2);
    }
    if (s->npg_low) memcpy(pages_out, s->pg_low, (size_t)s->npg_low * 4);
    return (int)s->npg_low;
}

int orc_budget_state(orc_cache *c, int seq, orc_budget *out) {
    if (seq < 0 || seq >= c->max_seqs) return ORC_ERR_SEQ;
    *out = c->budget[seq];
    return ORC_OK;
}

void orc_pool_state(orc_cache *c, uint32_t *high_next, uint32_t *high_free, uint32_t *low_next, uint32_t *low_free) {
    *high_next = c->pool_high.next; *high_free = c->pool_high.n_free;
    *low_next = c->pool_low.next; *low_free = c->pool_low.n_free;
}

/* ------------------------------------------------------------------ attention */

/* One query head: softmax(q k^T / sqrt(d)) v over every retained token of (seq, layer), fp64.
 * q_bits [128] bf16 bit patterns of head h; out [128]; *lse natural log of the softmax denominator
 * (times e^max).  Nothing retained: out = 0, lse = -inf.
 * With a protected recent window W > 0 (Section 3.1: release and the low format apply to a state
 * only once it has left the window) the last min(W, tokens seen) tokens are attended with their
 * original bf16 values whatever their action; only older tokens are attended as stored.  Both
 * streams are in arrival order, so the window's high- and low-precision members are exactly the
 * last entries of the HIGH and of the LOW stream: those are skipped there. */
static void attention_head(orc_cache *c, int layer, int seq, int h, const uint16_t *q_bits, double *out, double *lse) {
    orc_stream *s = stream_of(c, seq, layer);
    const int kv = h / (c->n_q / c->n_kv);
    const size_t row = (size_t)c->n_kv * HEAD_DIM, srow = (size_t)c->n_kv * GROUPS_PER_HEAD;
    const int zero = 1 << (c->pol->low_bits - 1);                     /* the code that stands for 0 */
    const uint32_t W = c->pol->recent_window;
    const size_t nw = W ? (s->n_tok < W ? s->n_tok : W) : 0;          /* tokens in the window */
    size_t win_h = 0, win_l = 0;
    for (size_t i = 0; i < nw; i++) { win_h += s->wact[i] == ACT_H; win_l += s->wact[i] == ACT_L; }
    const size_t nh = s->n_high - win_h, nl = s->n_low - win_l;        /* older than the window */
    const size_t n = nh + nl + nw;
    const double inv_sqrt_d = 1.0 / sqrt((double)HEAD_DIM);
    double *score = (double *)malloc((n ? n : 1) * sizeof(double));
    double q[HEAD_DIM];
    for (int i = 0; i < HEAD_DIM; i++) q[i] = (double)bf16_to_f32(q_bits[i]);
    double m = -INFINITY;
    for (size_t j = 0; j < n; j++) {
        double dot = 0.0;
        if (j < nh) {
            const uint16_t *k = s->hk + j * row + (size_t)kv * HEAD_DIM;
            for (int i = 0; i < HEAD_DIM; i++) dot += q[i] * (double)bf16_to_f32(k[i]);
        } else if (j >= nh + nl) {
            const uint16_t *k = s->wk + (j - nh - nl) * row + (size_t)kv * HEAD_DIM;
            for (int i = 0; i < HEAD_DIM; i++) dot += q[i] * (double)bf16_to_f32(k[i]);
        } else {
            size_t jl = j - nh;
            const uint8_t *kc = s->lk + jl * row + (size_t)kv * HEAD_DIM;
            const uint16_t *ks = s->lks + jl * srow + (size_t)kv * GROUPS_PER_HEAD;
            for (int i = 0; i < HEAD_DIM; i++)
                dot += q[i] * ((double)((int)kc[i] - zero) * (double)orc_f16_to_f32(ks[i / QGROUP]));
        }
        score[j] = dot * inv_sqrt_d;
        if (score[j] > m) m = score[j];
    }
    double acc[HEAD_DIM];
    for (int i = 0; i < HEAD_DIM; i++) acc[i] = 0.0;
    double denom = 0.0;
    for (size_t j = 0; j < n; j++) {
        double pj = exp(score[j] - m);
        denom += pj;
        if (j < nh) {
            const uint16_t *v = s->hv + j * row + (size_t)kv * HEAD_DIM;
            for (int i = 0; i < HEAD_DIM; i++) acc[i] += pj * (double)bf16_to_f32(v[i]);
        } else if (j >= nh + nl) {
            const uint16_t *v = s->wv + (j - nh - nl) * row + (size_t)kv * HEAD_DIM;
            for (int i = 0; i < HEAD_DIM; i++) acc[i] += pj * (double)bf16_to_f32(v[i]);
        } else {
            size_t jl = j - nh;
            const uint8_t *vc = s->lv + jl * row + (size_t)kv * HEAD_DIM;
            const uint16_t *vs = s->lvs + jl * srow + (size_t)kv * GROUPS_PER_HEAD;
            for (int i = 0; i < HEAD_DIM; i++)
                acc[i] += pj * ((double)((int)vc[i] - zero) * (double)orc_f16_to_f32(vs[i / QGROUP]));
        }
    }
    for (int i = 0; i < HEAD_DIM; i++) out[i] = n ? acc[i] / denom : 0.0;
    *lse = n ? m + log(denom) : -INFINITY;
    free(score);
}

/* All query heads of one sequence.  q_bits [n_q][128]; out [n_q][128]; lse [n_q]. */
int orc_attention(orc_cache *c, int layer, int seq, const uint16_t *q_bits, double *out, double *lse) {
    if (seq < 0 || seq >= c->max_seqs || layer < 0 || (uint32_t)layer >= c->pol->n_layers) return ORC_ERR_ARG;
    for (int h = 0; h < c->n_q; h++)
        attention_head(c, layer, seq, h, q_bits + (size_t)h * HEAD_DIM, out + (size_t)h * HEAD_DIM, lse + h);
    return ORC_OK;
}

/* A batch of sequences, host threads over (sequence, query head).
 * q [n_seqs][n_q][128], out [n_seqs][n_q][128], lse [n_seqs][n_q]. */
int orc_attention_batch(orc_cache *c, int layer, int n_seqs, const int32_t *seq_ids, const uint16_t *q_bits,
                        double *out, double *lse) {
    if (layer < 0 || (uint32_t)layer >= c->pol->n_layers) return ORC_ERR_ARG;
    for (int i = 0; i < n_seqs; i++) if (seq_ids[i] < 0 || seq_ids[i] >= c->max_seqs) return ORC_ERR_SEQ;
    const int n_q = c->n_q;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int i = 0; i < n_seqs; i++)
        for (int h = 0; h < n_q; h++) {
            size_t o = ((size_t)i * n_q + h);
            attention_head(c, layer, seq_ids[i], h, q_bits + o * HEAD_DIM, out + o * HEAD_DIM, lse + o);
        }
    return ORC_OK;
}

/* Eq. 4's inner term for each row: max over heads of the squared Euclidean distance between two
 * attention outputs.  o_ref, o_test fp32 [n_rows][n_q][128]; per_row fp64 [n_rows]; returns their sum. */
double orc_distortion(int n_rows, int n_q, const float *o_ref, const float *o_test, double *per_row) {
    double total = 0.0;
    for (int r = 0; r < n_rows; r++) {
        double worst = 0.0;
        for (int h = 0; h < n_q; h++) {
            double d2 = 0.0;
            for (int i = 0; i < HEAD_DIM; i++) {
                size_t at = ((size_t)r * n_q + h) * HEAD_DIM + i;
                double d = (double)o_ref[at] - (double)o_test[at];
                d2 += d * d;
            }
            if (d2 > worst) worst = d2;
        }
        if (per_row) per_row[r] = worst;
        total += worst;
    }
    return total;
}

int orc_max_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Threads of the parallel loops (a launcher may have pinned OMP_NUM_THREADS to 1 for every rank). */
void orc_set_threads(int n) {
#ifdef _OPENMP
    extern void omp_set_num_threads(int);
    if (n >= 1) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

int orc_sizeof_budget(void) { return (int)sizeof(orc_budget); }
