/*
 * libpask -- the online hot path of PASK (parser-aware structural KV persistence) for B200.
 *
 * Each token arrives with a parser-derived structural tag.  A frozen, offline-calibrated table
 * maps (tag, layer group) to RELEASE (drop), RETAIN-LOW or RETAIN-HIGH; that decision is applied
 * to the token's K/V at every layer, the result is compacted into a paged mixed-precision
 * cache with a constant-size budget state per sequence, and decode attention runs over what was
 * retained.  This header is the whole boundary: plain C, plain pointers and sizes.
 *
 * Conventions
 *   - "dev" pointers are CUDA device memory, "host" pointers ordinary host memory.
 *   - The caller owns every device buffer and the stream.  The library allocates no device
 *     memory and owns only its small host-side handles.
 *   - Kernels are enqueued on the given stream and calls return without waiting unless stated
 *     otherwise.  Errors that the host can see (bad arguments, shapes, sizes) are returned at
 *     once and enqueue nothing.  Conditions only the device can see (pool exhaustion, unknown
 *     tags, page-table overflow, a wait that ran out) set sticky bits in a device status word
 *     that pask_budget_state reports; an append that cannot get all its pages writes nothing
 *     and changes no counter.
 *   - Every dev pointer must be 16-byte aligned; the pools and meta 256-byte aligned.
 *   - One host thread drives a cache at a time; ordering between calls is stream order.
 *   - Calls that only enqueue work (append, decide, attention, pask_append_attend) may be recorded by
 *     a stream capture and replayed as a CUDA graph: nothing that changes from call to call is passed
 *     by value, a replay works on whatever the recorded device buffers hold then.  Not for capture:
 *     calls that wait for the stream (pask_budget_state, pask_debug_*), the host-buffer steps, and the
 *     first pask_decode_attention_static call on a device.
 *   - Supported shapes: head_dim 128, 16-token pages, n_q_heads = 4 * n_kv_heads with
 *     n_kv_heads in {1, 2, 4, 8}.  Anything else: PASK_ERR_UNSUPPORTED_SHAPE.
 *   - No function throws or aborts.
 *
 * Formats (the paper leaves them open; these are the library's documented readings)
 *   RETAIN-HIGH keeps the token's bf16 K and V bits (any finite bf16 value).  RETAIN-LOW stores, per token, per KV head
 *   and per group of 32 consecutive head dimensions, one fp16 scale s = fp16(amax / 7) (IEEE
 *   fp32 division, round to nearest even, saturating at 65504) and 32 four-bit codes
 *   clamp(rint(x * (1 / s)), -7, 7) + 8; the value read back is (code - 8) * s.  s == 0 gives
 *   codes 8.  Costs are payload bytes per token per layer: m(R) = 0,
 *   m(L) = 2 * n_kv * (64 + 8), m(H) = 2 * n_kv * 256.
 *   A policy with low_bits = 8 keeps RETAIN-LOW at eight bits instead: s = fp16(amax / 127), codes
 *   clamp(rint(x * (1 / s)), -127, 127) + 128, value (code - 128) * s, m(L) = 2 * n_kv * (128 + 8).
 *   A policy with low_bits = 2 keeps three levels: s = fp16(amax), codes clamp(rint(x * (1 / s)), -1, 1) + 2,
 *   value (code - 2) * s, m(L) = 2 * n_kv * (32 + 8).
 */
#ifndef PASK_H_
#define PASK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t pask_status_t;
#define PASK_OK 0
#define PASK_ERR_INVALID_ARG (-1)
#define PASK_ERR_BAD_POLICY (-2)
#define PASK_ERR_UNSUPPORTED_SHAPE (-3)
#define PASK_ERR_POOL_EXHAUSTED (-4)
#define PASK_ERR_BAD_SEQ (-5)
#define PASK_ERR_CUDA (-6)
#define PASK_ERR_TIMEOUT (-7)
#define PASK_ERR_WORKSPACE (-8)
#define PASK_ERR_NO_MEMORY (-9)   /* host memory for a handle or a staging copy could not be had */
#define PASK_ERR_STALE_PLAN (-10) /* pask_decode_step_ahead without a valid plan for this layer and batch */

/* Sticky bits of the device status word (pask_budget_state_t.device_status). */
#define PASK_DEV_POOL_EXHAUSTED 0x1u  /* an append needed more pages than a pool had: nothing written */
#define PASK_DEV_BAD_SEQ 0x2u         /* sequence id out of range or repeated within one call */
#define PASK_DEV_SEQ_OVERFLOW 0x4u    /* a stream would exceed max_tokens_per_seq: nothing written */
#define PASK_DEV_BAD_RAGGED 0x8u      /* cu_tokens not ascending or not ending at total_tokens */
#define PASK_DEV_TIMEOUT 0x10u        /* a bounded wait inside a kernel ran out: the call's out / lse are void
                                         (contributions of the pages behind the wait are missing) */
#define PASK_DEV_RANGE 0x20u          /* a query element had |q| > 65504, outside what the low-precision path
                                         computes in; results for that sequence may be infinite or NaN */

#define PASK_DEV_INTERNAL 0x40u       /* an internal bounds check refused an access (a page id out of range) */
#define PASK_DEV_BAD_ACTION 0x80u     /* pask_append_kv_decided was given an action outside R, L, H; call refused */
#define PASK_DEV_STALE_PLAN 0x100u    /* pask_decode_step_ahead: the sequences named are not those the plan was made for */

#define PASK_ACTION_RELEASE 0
#define PASK_ACTION_RETAIN_LOW 1
#define PASK_ACTION_RETAIN_HIGH 2
#define PASK_TAG_PROTECTED 0xFF /* always RETAIN-HIGH, not counted as unknown */
#define PASK_MAX_GROUPS 8
#define PASK_MAX_SEQS_PER_CALL 1024
#define PASK_MAX_WINDOW 256

typedef struct pask_policy pask_policy_t;
typedef struct pask_cache pask_cache_t;
typedef void *pask_stream_t; /* a cudaStream_t */
typedef void *pask_event_t;  /* a cudaEvent_t */

typedef struct {
    int32_t n_layers;
    int32_t n_q_heads;
    int32_t n_kv_heads;
    int32_t head_dim;           /* 128 */
    int32_t page_tokens;        /* 16 */
    int32_t max_seqs;           /* sequence ids are 0 .. max_seqs-1 */
    int32_t max_tokens_per_seq; /* bound on each stream's length (sizes the page tables) */
    int32_t max_append_tokens;  /* largest total_tokens of one pask_append_kv call */
    uint32_t pool_high_pages;   /* capacity of the bf16 page pool, shared by all layers */
    uint32_t pool_low_pages;    /* capacity of the int4 page pool */
    int32_t recent_window;      /* the policy's protected recent window W (0, or a multiple of 16 up to
                                   PASK_MAX_WINDOW); sizes W/16 bf16 pages per (sequence, layer) behind the bf16 pool */
    int32_t low_bits;           /* the policy's low_bits: 4 (0 means 4), 8 or 2; sizes the pages of the low pool */
} pask_cache_desc_t;

typedef struct {
    size_t pool_high_bytes; /* (pool_high_pages + max_seqs * n_layers * recent_window / 16) * high_page_bytes */
    size_t pool_low_bytes;
    size_t meta_bytes;      /* counters, page tables, budget states, free stacks, append scratch */
    size_t high_page_bytes; /* n_kv * 8192: per KV head a 16x128 bf16 K tile then V tile */
    size_t low_page_bytes;  /* n_kv * 2304 (4-bit codes), n_kv * 4352 (8-bit) or n_kv * 1280 (2-bit): per KV head K codes, K scales, V codes, V scales */
} pask_cache_sizes_t;

/* Constant-size per-sequence budget state (Algorithm 2's R_t with the counts it is made of).
 * Counts are token-layer events: one per token per layer call, binned by the layer's group. */
typedef struct {
    uint64_t n_seen[PASK_MAX_GROUPS];
    uint64_t n_high[PASK_MAX_GROUPS];
    uint64_t n_low[PASK_MAX_GROUPS];
    uint64_t n_drop[PASK_MAX_GROUPS];
    uint64_t retained_bytes;  /* sum of m(a) over everything persisted so far */
    uint64_t full_bytes;      /* sum of m(H): what full high precision would have cost */
    int64_t remaining_bytes;  /* floor(budget_target * full_bytes) - retained_bytes */
    uint64_t bad_tags;        /* tags >= n_tags (kept at high precision) */
    uint32_t pages_high;      /* pages this sequence holds in each pool */
    uint32_t pages_low;
    uint32_t device_status;   /* PASK_DEV_* bits, cache-wide, sticky until pask_cache_reset */
    uint32_t reserved;
    /* Algorithm 2's own running budget, advanced by pask_decide once per token for all groups:
     * R_t = floor(budget_target * decided_full_bytes, this token included) - decided_retained_bytes.
     * Once every layer of the decided tokens has been appended with pask_append_kv_decided these
     * two equal full_bytes and retained_bytes. */
    uint64_t decided_full_bytes;
    uint64_t decided_retained_bytes;
    uint64_t n_demoted;         /* single steps H->L or L->R taken by Demote */
    uint64_t n_promoted;        /* single steps R->L or L->H taken by Promote */
    uint64_t n_floor_conflicts; /* tokens whose floors alone exceeded B_t (floors were kept) */
} pask_budget_state_t;

/* ---------------------------------------------------------------------------------------------
 * pask_load_policy -- load the frozen table Lambda and the reserve Gamma.
 * Follows: the table stores, per bucket q = (tag, layer group), the selected action, the
 * calibrated floor and the adjacent upgrade scores (end of Section 3.3); online the action is
 * a = max(a0, a_floor) under R < L < H (Eq. 10, Algorithm 2 steps 1-2).  Gamma is Eq. 9's
 * per-state reserve; the upgrade scores, Gamma and the critical-state flags are read by
 * pask_decide only.
 *   blob (host, len bytes), little endian:
 *     "PASK", u32 version (1 or 2), u32 n_tags (1..255), u32 n_groups (1..8), u32 n_layers,
 *     u32 n_states, u32 budget_target_q16, u32 recent_window (0, or a multiple of 16 up to
 *     PASK_MAX_WINDOW: the protected recent window in tokens, see pask_decode_attention), u32 low_bits (4, 8 or 2),
 *     u32 group_size (32),
 *     u8 layer_group[n_layers] zero-padded to 4 bytes,
 *     n_tags*n_groups entries, tag-major: u8 a0, u8 a_floor, u16 0, f32 rho_RL, f32 rho_LH
 *       (scores of the adjacent upgrades R->L and L->H; any value but NaN),
 *     u32 gamma[n_states],
 *     version 2 only: u32 gamma_shift (0..16; the reserve of state s is gamma[s] << gamma_shift
 *       bytes), u8 crit[n_states] (1 = critical or lookahead-critical) zero-padded to 4 bytes.
 *       Version 1 means gamma_shift = 0 and no critical state.
 * The blob is copied; *out is a host handle to free with pask_free_policy.  Needs no GPU.
 * Errors: PASK_ERR_INVALID_ARG (null), PASK_ERR_BAD_POLICY (magic, version, sizes, ranges, length).
 */
pask_status_t pask_load_policy(const void *blob, size_t len, pask_policy_t **out);
void pask_free_policy(pask_policy_t *policy);
/* Effective action max(a0, a_floor) for a bucket, or -1 if out of range.  Host only. */
int32_t pask_policy_action(const pask_policy_t *policy, int32_t tag, int32_t group);

/* Bytes the caller must allocate for a cache of this shape.  Host only, needs no GPU. */
pask_status_t pask_cache_sizes(const pask_cache_desc_t *desc, pask_cache_sizes_t *out);

/* Bind caller-owned device memory (sizes from pask_cache_sizes) to a new cache and initialise
 * it on `stream` (copies the folded table into meta, zeroes counters).  The policy's n_layers
 * and recent_window must equal desc's.  The handle is host memory; destroy frees only that. */
pask_status_t pask_cache_create(const pask_cache_desc_t *desc, const pask_policy_t *policy, void *pool_high_dev,
                                void *pool_low_dev, void *meta_dev, pask_stream_t stream, pask_cache_t **out);
void pask_cache_destroy(pask_cache_t *cache);
/* Forget every sequence, return all pages, clear the device status word. */
pask_status_t pask_cache_reset(pask_cache_t *cache, pask_stream_t stream);
/* Forget one sequence.  Its pages go back on the free stacks in a fixed order (layers
 * ascending; per layer the HIGH table then the LOW table, each in table order) and are handed
 * out again last-in first-out. */
pask_status_t pask_seq_reset(pask_cache_t *cache, int32_t seq, pask_stream_t stream);

/* ---------------------------------------------------------------------------------------------
 * pask_append_kv -- Algorithm 2 steps 1, 2, 7 and 8 for one layer and a ragged batch of tokens:
 * look up each token's bucket (its tag, this layer's group), take a = max(a0, a_floor), persist
 * the token's K/V accordingly (nothing, int4 + scales, or the bf16 bits) at the end of the
 * sequence's LOW or HIGH stream, and charge m(a) to the sequence's budget state.  The call
 * takes no query and no attention statistics: the online path may use only the tag, the layer
 * group and the constant-size budget state (Section 3.1, Section 3.4).
 *   layer          0 .. n_layers-1
 *   n_seqs         sequences in this call (1 .. PASK_MAX_SEQS_PER_CALL), each id at most once
 *   total_tokens   sum of the per-sequence token counts (<= max_append_tokens)
 *   seq_ids        dev int32 [n_seqs]
 *   cu_tokens      dev int32 [n_seqs+1], ascending, cu_tokens[0] = 0, last = total_tokens
 *                  (one token per sequence in decode, many in prefill)
 *   k, v           dev bf16 [total_tokens][n_kv][128], post-RoPE, tokens of a sequence in order.
 *                  Values must be finite.  An infinity saturates its group's scale; what a NaN
 *                  leaves in the low-precision codes of its 32-dim group is undefined and may
 *                  differ between a small and a large call (the high-precision copy keeps its bits)
 *   tags           dev uint8 [total_tokens]; PASK_TAG_PROTECTED = always high; >= n_tags = high
 *                  and counted in bad_tags
 *   states         dev uint16 [total_tokens] or NULL; not read: this call applies the frozen table
 *                  as it stands, the budget-dependent adjustment is pask_decide
 *   actions_out    dev uint8 [total_tokens] or NULL: the action taken for each token
 * New pages are numbered in call order (sequence-major, position ascending) from each pool's
 * free stack, else its bump counter.  If either pool cannot supply the whole call, or a stream
 * would outgrow its page table, nothing is written and no counter changes; the condition is a
 * sticky PASK_DEV_* bit.
 */
pask_status_t pask_append_kv(pask_cache_t *cache, int32_t layer, int32_t n_seqs, int32_t total_tokens,
                             const int32_t *seq_ids, const int32_t *cu_tokens, const void *k, const void *v,
                             const uint8_t *tags, const uint16_t *states, uint8_t *actions_out,
                             pask_stream_t stream);

/* ---------------------------------------------------------------------------------------------
 * pask_decide -- Algorithm 2 steps 1-6 and 8 for a ragged batch of tokens, all layer groups at
 * once: the budget-dependent adjustment of the table's actions (Eq. 10 and the paragraph after
 * it).  For each token, in sequence order, with the sequence's own running budget:
 *   a_c  = max(a0, a_floor) per group c (protected and unknown tags: H with floor H);
 *   R_t  = floor(budget_target * decided_full_bytes, this token's full cost included)
 *          - decided_retained_bytes;         B_t = max(0, R_t - Gamma(s_t));
 *   cost = sum over groups of (layers in the group) * m(a_c);
 *   Demote: while cost > B_t and some group is above its floor, lower by one step (H->L or L->R)
 *     the group whose step has the smallest upgrade score rho (the least distortion lost per
 *     byte saved; the first such group on ties).  Floors are never crossed: if they alone exceed
 *     B_t they stay and n_floor_conflicts counts the token;
 *   Promote, only if crit[s_t]: while some group below H can go up one step with cost still
 *     <= B_t, raise the one with the largest rho (first group on ties);
 *   decided_full_bytes += the token's full cost; decided_retained_bytes += cost.
 * Groups that own no layer are left alone.  A state id >= n_states (or states == NULL) has no
 * reserve and is not critical.
 *   seq_ids, cu_tokens, tags, states (may be NULL)   as for pask_append_kv, device memory
 *   actions_out    dev uint8 [total_tokens][n_groups]: feed it to pask_append_kv_decided for
 *                  every layer (in any order) before the next pask_decide of these sequences
 * The call takes no query and no statistics of K or V: constant work and constant state per token
 * (Section 3.4).  A bad sequence id, a sequence named twice or a malformed cu_tokens refuses the
 * whole call (sticky PASK_DEV_* bit): no budget state changes and actions_out is undefined.
 */
pask_status_t pask_decide(pask_cache_t *cache, int32_t n_seqs, int32_t total_tokens, const int32_t *seq_ids,
                          const int32_t *cu_tokens, const uint8_t *tags, const uint16_t *states,
                          uint8_t *actions_out, pask_stream_t stream);
/* pask_append_kv with Algorithm 2 step 7 applied to decided actions: token t takes
 * actions[t * n_groups + group of `layer`] instead of the table's entry (tags still count
 * bad_tags).  An action > 2 refuses the call with PASK_DEV_BAD_ACTION.  Everything else --
 * arguments, page numbering, all-or-nothing refusal, accounting -- is pask_append_kv's. */
pask_status_t pask_append_kv_decided(pask_cache_t *cache, int32_t layer, int32_t n_seqs, int32_t total_tokens,
                                     const int32_t *seq_ids, const int32_t *cu_tokens, const void *k, const void *v,
                                     const uint8_t *tags, const uint8_t *actions, uint8_t *actions_out,
                                     pask_stream_t stream);

/* ---------------------------------------------------------------------------------------------
 * pask_decode_attention -- attention of one new query per sequence over that sequence's
 * retained history at `layer`, at stored precision: out = softmax(q k^T / sqrt(128)) v over
 * the HIGH stream (bf16 values) and the LOW stream ((code - 8) * scale); released tokens take no
 * part (Section 3.1: release removes a KV state from future attention; these are the attention
 * outputs o of Eq. 4).  Query head h reads KV head h / 4.
 * Protected recent window (Section 3.1: release and the low format apply to a state only after it
 * has left the window): with recent_window = W > 0 the last min(W, tokens appended) tokens of the
 * sequence at this layer are attended with their original bf16 K/V whatever their action; only
 * older tokens are attended as stored.  Appends then also keep a bf16 copy of every token,
 * released ones included, in a ring of W slots per (sequence, layer); streams, page ids and the
 * budget state are the same as with W = 0 (a token is charged m(a) when it arrives).
 *   seq_ids   dev int32 [n_seqs]
 *   q         dev bf16 [n_seqs][n_q][128]
 *   out       dev fp32 [n_seqs][n_q][128]
 *   lse       dev fp32 [n_seqs][n_q] or NULL: natural-log sum of exp of the scaled scores
 *   workspace dev, at least pask_workspace_bytes(cache, n_seqs) bytes, 256-byte aligned; holds
 *             split partials between the two kernels of the call, contents undefined afterwards
 * A sequence with nothing retained gets out = 0 and lse = -inf.
 * Errors: PASK_ERR_INVALID_ARG, PASK_ERR_WORKSPACE (too small), PASK_ERR_CUDA (launch failed).
 */
pask_status_t pask_decode_attention(pask_cache_t *cache, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                                    const void *q, float *out, float *lse, void *workspace,
                                    size_t workspace_bytes, pask_stream_t stream);
/* pask_append_attend -- one layer of a decode step in one call: pask_append_kv (or, with `actions`
 * != NULL, pask_append_kv_decided) for a ragged batch, then pask_decode_attention with one query
 * per sequence of the same batch.  Results are those of the two calls made one after the other.
 * For small batches (<= 255 sequences and tokens) the append's single launch also
 * writes the attention's work plan, which saves a launch per layer; otherwise the two calls are
 * simply issued in turn.  If the append is refused (sticky PASK_DEV_* bit) out and lse are
 * undefined.  Arguments as for the two calls. */
pask_status_t pask_append_attend(pask_cache_t *cache, int32_t layer, int32_t n_seqs, int32_t total_tokens,
                                 const int32_t *seq_ids, const int32_t *cu_tokens, const void *k, const void *v,
                                 const uint8_t *tags, const uint8_t *actions, uint8_t *actions_out, const void *q,
                                 float *out, float *lse, void *workspace, size_t workspace_bytes,
                                 pask_stream_t stream);

/* ---------------------------------------------------------------------------------------------
 * Planned-ahead decode steps: the append taken off the layer's critical path.
 *
 * In a decode loop the same batch comes back step after step, and what the attention of step t+1
 * streams at a layer is known as soon as step t has appended there.  pask_decode_step_ahead uses
 * that: the streaming kernel of a call starts at once from a work plan that describes the cache
 * BEFORE this call's append (written by the call of the step before, or by pask_plan_ahead); the
 * append of the new tokens (Algorithm 2 step 7) runs in the shadow of the streaming kernel's tail
 * and writes the plan of the next step; the merge kernel attends each new token straight from the
 * call's k / v -- at its stored precision: as given when its action is RETAIN-HIGH, quantised on
 * the fly exactly as the append quantises it when RETAIN-LOW, not at all when released -- and adds
 * that one partial to those of the history.  Cache state after the call is bit-identical to
 * pask_append_attend's; out / lse are the same attention (Section 3.1) summed in another order.
 *
 *   plan_area   dev, >= pask_plan_area_bytes(cache, n_seqs), 256-byte aligned, owned by the caller
 *               and left alone by it from pask_plan_ahead on: it holds, per layer, two plans used in
 *               turn.  One area serves one batch (a fixed list of sequences in a fixed order).
 *   pask_plan_ahead(layer)      writes the layer's plan from the cache as it stands.  Call it for
 *               every layer once the batch is formed (after prefill) and again after anything else
 *               touched the cache at that layer: pask_append_kv*, pask_append_attend,
 *               pask_decode_step_*, pask_seq_reset, pask_cache_reset.  The handle remembers which
 *               layers have a plan; those calls forget it.
 *   pask_decode_step_ahead(layer)   exactly one new token per sequence: k, v [n_seqs][n_kv][128],
 *               tags [n_seqs], actions NULL or [n_seqs][n_groups] (from pask_decide), q, out, lse,
 *               workspace as for pask_append_attend.  seq_ids must be the list the plan was made for.
 * Errors: PASK_ERR_STALE_PLAN if the handle holds no plan of this layer for n_seqs sequences in
 * this plan_area (nothing is enqueued); a different list of the same length is only seen on the
 * device: sticky PASK_DEV_STALE_PLAN, results void.  PASK_ERR_UNSUPPORTED_SHAPE with a protected
 * recent window (the token that leaves the window changes what the history holds) or more than
 * 255 sequences: use pask_append_attend there.  A refused append (sticky PASK_DEV_* bit) leaves
 * out / lse undefined and an empty plan behind.  k, v, tags, actions, q must stay untouched
 * until the call's kernels have run, as for every call.  The calls only enqueue work and may be
 * recorded by a stream capture; which of a layer's two plan blocks a call reads is fixed when it is
 * recorded, so a graph that is replayed repeatedly must hold an even number of calls per layer. */
size_t pask_plan_area_bytes(const pask_cache_t *cache, int32_t n_seqs);
pask_status_t pask_plan_ahead(pask_cache_t *cache, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                              void *plan_area, size_t plan_area_bytes, pask_stream_t stream);
pask_status_t pask_decode_step_ahead(pask_cache_t *cache, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                                     const void *k, const void *v, const uint8_t *tags, const uint8_t *actions,
                                     uint8_t *actions_out, const void *q, float *out, float *lse,
                                     void *workspace, size_t workspace_bytes, void *plan_area,
                                     size_t plan_area_bytes, pask_stream_t stream);

/* The full high-precision reference (the paper's "Full KV", C_KV = 1): same arguments, for a
 * cache whose policy keeps everything at high precision; the LOW stream is not read at all
 * (its code path is compiled out), so any LOW tokens present would be ignored. */
pask_status_t pask_decode_attention_full(pask_cache_t *cache, int32_t layer, int32_t n_seqs,
                                         const int32_t *seq_ids, const void *q, float *out, float *lse,
                                         void *workspace, size_t workspace_bytes, pask_stream_t stream);
size_t pask_workspace_bytes(const pask_cache_t *cache, int32_t n_seqs);

/* pask_decode_attention_static -- pask_decode_attention for callers that cannot provide a workspace.
 * (The paper has no counterpart; this is a deployment convenience of the library.)
 * Some integrations cannot allocate device memory where they call the library: a serving engine that
 * gave all free HBM to its own block pool at start-up (a later cudaMalloc fails or fragments the
 * pool), a plugin that runs inside a region where allocation is forbidden, or a real-time loop that
 * must not risk the device-wide synchronisation an allocation brings.  For them the library carries
 * its own scratch: a fixed array of PASK_STATIC_WORKSPACE_BYTES inside the library image, resident on
 * every GPU the library is used on for the life of the process.  The call allocates and frees
 * nothing, on the host side too.
 *   Same arguments and results as pask_decode_attention, minus workspace / workspace_bytes.
 *   PASK_ERR_WORKSPACE if pask_workspace_bytes(cache, n_seqs) exceeds PASK_STATIC_WORKSPACE_BYTES (a
 *   large batch or a large max_tokens_per_seq); use pask_decode_attention with a workspace then.
 *   The first call on a device looks up the scratch's device address (a one-off set-up step); make
 *   that first call outside of any stream capture.
 *   All calls, from every cache and stream of the process, share the one scratch per GPU: two calls
 *   that overlap on the GPU (different streams) race on it and both results are garbage.  Calls
 *   on one stream are fine.  The scratch keeps whatever the last call left; the kernels rewrite what
 *   they read, nothing needs clearing. */
#define PASK_STATIC_WORKSPACE_BYTES (8u << 20)
pask_status_t pask_decode_attention_static(pask_cache_t *cache, int32_t layer, int32_t n_seqs,
                                           const int32_t *seq_ids, const void *q, float *out, float *lse,
                                           pask_stream_t stream);

/* One decode step of one layer from HOST buffers: copies seq_ids, the new token's k, v, tag and
 * the query to the device (into `staging`), appends one token per sequence, runs decode
 * attention and copies `out` back -- all enqueued on `stream`; the host buffers must stay valid
 * (and should be pinned) until the stream has drained.
 *   seq_ids_host int32 [n_seqs]; k_host, v_host bf16 [n_seqs][n_kv][128]; tags_host u8 [n_seqs];
 *   q_host bf16 [n_seqs][n_q][128]; out_host fp32 [n_seqs][n_q][128];
 *   staging dev, >= pask_step_staging_bytes(cache, n_seqs), 256-byte aligned. */
pask_status_t pask_decode_step_host(pask_cache_t *cache, int32_t layer, int32_t n_seqs, const int32_t *seq_ids_host,
                                    const void *k_host, const void *v_host, const uint8_t *tags_host,
                                    const void *q_host, float *out_host, void *staging, size_t staging_bytes,
                                    void *workspace, size_t workspace_bytes, pask_stream_t stream);
size_t pask_step_staging_bytes(const pask_cache_t *cache, int32_t n_seqs);
/* The same step from ONE host block (one host-to-device copy instead of five): the caller lays the
 * step's inputs out in a pinned block at the byte offsets pask_step_packed_layout returns --
 * offsets[0..5] = seq_ids (int32 [n]), cu_tokens (int32 [n+1] = 0, 1, ..., n), k, v (bf16
 * [n][n_kv][128]), tags (u8 [n]), q (bf16 [n][n_q][128]); *in_bytes is the size of the block.
 * staging and workspace as for pask_decode_step_host. */
pask_status_t pask_step_packed_layout(const pask_cache_t *cache, int32_t n_seqs, size_t offsets[6], size_t *in_bytes);
pask_status_t pask_decode_step_packed(pask_cache_t *cache, int32_t layer, int32_t n_seqs, const void *packed_host,
                                      float *out_host, void *staging, size_t staging_bytes, void *workspace,
                                      size_t workspace_bytes, pask_stream_t stream);

/* Pipelined form of pask_decode_step_packed for a caller that issues layer after layer from host
 * blocks: the host-to-device copy of a call runs on a copy stream of its own and so overlaps the
 * kernels of the call before, and the device-to-host copy of the output runs on a second copy
 * stream and overlaps the call after.  The two streams and six events are created for the cache at
 * the first call (host-side handles; no device memory) and destroyed with it; kernels still run
 * on `stream`, in call order.
 *   staging        dev, 256-byte aligned: its two halves (the second starts at staging_bytes / 2
 *                  rounded down to 256) are used in turn, whatever n_seqs is, and each must hold
 *                  pask_step_staging_bytes(cache, n_seqs), else PASK_ERR_WORKSPACE.  n_seqs may
 *                  change from call to call.  Pass the same buffer and size until the next drain;
 *                  a call that brings another one first waits for the earlier calls' use of theirs.
 *                  A call that fails after it was given its slot still uses the slot up: the
 *                  next call takes the other half.
 *   packed_host    must stay valid, and out_host is not valid, until pask_decode_step_drain returns
 *                  (synchronising `stream` alone is not enough: the output copy is not on it)
 * pask_decode_step_drain blocks the host until every pipelined call issued so far has finished. */
pask_status_t pask_decode_step_pipelined(pask_cache_t *cache, int32_t layer, int32_t n_seqs, const void *packed_host,
                                         float *out_host, void *staging, size_t staging_bytes, void *workspace,
                                         size_t workspace_bytes, pask_stream_t stream);
/* The same with the layer's step issued as pask_decode_step_ahead (plan made a step ahead; plan_area as
 * there, pask_plan_ahead for the layer first; the block's cu_tokens field is not read).  Errors as for the two. */
pask_status_t pask_decode_step_pipelined_ahead(pask_cache_t *cache, int32_t layer, int32_t n_seqs,
                                               const void *packed_host, float *out_host, void *staging,
                                               size_t staging_bytes, void *workspace, size_t workspace_bytes,
                                               void *plan_area, size_t plan_area_bytes, pask_stream_t stream);
pask_status_t pask_decode_step_drain(pask_cache_t *cache);

/* ---------------------------------------------------------------------------------------------
 * pask_distortion -- the inner term of the attention-output distortion (Eq. 4): for each row r
 * (one decode position of one sequence at one layer) max over query heads h of
 * || o_ref[r][h][:] - o_test[r][h][:] ||_2^2, where o_ref is the output of pask_decode_attention_full
 * on the full high-precision cache and o_test the output under the policy being probed.  Summing it
 * over the layers of a group and averaging over positions, as Eq. 4 does, is left to the caller:
 * sum_inout accumulates over calls.
 *   o_ref, o_test  dev fp32 [n_rows][n_q_heads][128], 16-byte aligned; n_q_heads <= 32
 *   per_row_out    dev fp32 [n_rows] or NULL
 *   sum_inout      dev fp64 or NULL: the sum over rows is ADDED to it (clear it before the first call;
 *                  the order of the additions, hence the last bits, is not fixed)
 */
pask_status_t pask_distortion(int32_t n_rows, int32_t n_q_heads, const float *o_ref, const float *o_test,
                              float *per_row_out, double *sum_inout, pask_stream_t stream);

/* ---------------------------------------------------------------------------------------------
 * pask_budget_state -- the constant-size budget state of one sequence (Algorithm 2 step 8:
 * R' = R - sum_c m(a_c, c); normalised cost of Eq. 1 is retained_bytes / full_bytes) plus the
 * cache-wide device status word.  Copies to host memory and WAITS for `stream`. */
pask_status_t pask_budget_state(pask_cache_t *cache, int32_t seq, pask_budget_state_t *host_out,
                                pask_stream_t stream);

/* Optional timing hook: the next pask_decode_attention[_full] call records `start` just before
 * and `stop` just after its main (page-streaming) kernel on the call's stream, then forgets
 * them.  Pass NULLs to clear. */
pask_status_t pask_cache_set_timing_events(pask_cache_t *cache, pask_event_t start, pask_event_t stop);
/* The same from inside the kernel: the streaming kernel of the next decode-attention call on this
 * cache (any flavour) leaves in span_dev[0] the earliest time at which one of its CTAs was free to
 * start its work (its dependency wait over) and in span_dev[1] the latest time at which one had
 * finished, both in nanoseconds of the GPU's global timer (atomicMin / atomicMax: the caller sets
 * the two 64-bit words to all ones and to zero beforehand; dev memory, 8-byte aligned).  Unlike the
 * pair of events this does not keep the kernel from overlapping its launch with its neighbours,
 * and it leaves out the launch and completion latency that a pair of events includes.  NULL
 * cancels.  One launch only, like the events. */
pask_status_t pask_cache_set_timing_span(pask_cache_t *cache, void *span_dev);

/* ---------------------------------------------------------------------------------------------
 * Debug / test access to the cache in canonical form (the physical packing inside pages is
 * private).  All of these wait for `stream` and write HOST memory.
 */
pask_status_t pask_debug_stream_len(pask_cache_t *cache, int32_t layer, int32_t seq, uint32_t *n_high,
                                    uint32_t *n_low, pask_stream_t stream);
/* HIGH stream in arrival order: k_out, v_out bf16 bits [n_high][n_kv][128]; pages_out [ceil(n_high/16)]. */
pask_status_t pask_debug_dump_high(pask_cache_t *cache, int32_t layer, int32_t seq, uint16_t *k_out,
                                   uint16_t *v_out, uint32_t *pages_out, pask_stream_t stream);
/* LOW stream in arrival order: codes u8 [n_low][n_kv][128] (values 1..15), fp16 scale bits
 * [n_low][n_kv][4]; pages_out [ceil(n_low/16)]. */
pask_status_t pask_debug_dump_low(pask_cache_t *cache, int32_t layer, int32_t seq, uint8_t *k_codes,
                                  uint16_t *k_scales, uint8_t *v_codes, uint16_t *v_scales, uint32_t *pages_out,
                                  pask_stream_t stream);
/* Page ids only (no page contents): high_out [ceil(n_high/16)], low_out [ceil(n_low/16)]; either may be NULL. */
pask_status_t pask_debug_page_ids(pask_cache_t *cache, int32_t layer, int32_t seq, uint32_t *high_out, uint32_t *low_out,
                                  pask_stream_t stream);
/* out[4] = { high bump counter, high free-stack depth, low bump counter, low free-stack depth }. */
pask_status_t pask_debug_pool_state(pask_cache_t *cache, uint32_t *out4, pask_stream_t stream);
/* The cache's first `count` (<= 64) control words: [0] device status, [2..5] pool state. */
pask_status_t pask_debug_ctrl_words(pask_cache_t *cache, uint32_t *out, int32_t count, pask_stream_t stream);
/* How the decode-attention kernel splits work.  Each sequence's pages are visited in a fixed order
 * that interleaves its HIGH and LOW pages evenly; pask_debug_page_order writes that order for a
 * sequence with the given page counts: order[v] = page index within its stream, with bit 31 set
 * for a HIGH page.  For a batch whose sequences hold the given page counts and a grid of `n_ctas`,
 * pask_debug_partition writes for each CTA b and sequence index s the half-open range of positions
 * of that order which b processes, as ranges[(b * n_seqs + s) * 2 + {0,1}] (empty: begin == end).
 * A batch of at most n_ctas / 16 sequences is cut so that every non-empty sequence has whole CTAs
 * of its own (its share of the cost, rounded, at least one; inside it equal numbers of positions):
 * no CTA then works on two sequences.  Host only, no GPU. */
pask_status_t pask_debug_page_order(uint32_t pages_high, uint32_t pages_low, uint32_t *order);
pask_status_t pask_debug_partition(int32_t n_seqs, const uint32_t *pages_high, const uint32_t *pages_low,
                                   int32_t n_ctas, uint32_t *ranges);
/* Override the number of CTAs the decode-attention main kernel is launched with (default: two per
 * SM).  Any value >= 1 gives the same result up to summation order; tests use it to check that.
 * Workspaces must be sized (pask_workspace_bytes) after the change. */
pask_status_t pask_debug_set_attention_ctas(pask_cache_t *cache, int32_t n_ctas);
/* The device-side waits of the library are those of the decode-attention kernel for its bulk copies
 * into shared memory (and one of the same kind, with a fixed bound of about a second, in the bulk
 * append's write kernel for a page's source rows).  Each is bounded: after `limit_cycles` SM clock cycles (default 2e9,
 * about a second) the warp gives up, sets PASK_DEV_TIMEOUT, writes empty partials for the rest of
 * its range, waits (bounded again) until every copy it had issued has landed, and returns; the
 * context stays usable and pask_cache_reset clears the bit.  pask_debug_set_wait sets the limit
 * (>= 1000) and, for testing that path without anything going wrong on the GPU, a number of bytes
 * (multiple of 16, <= 65536; 0 = normal operation) that the first copy of every warp announces to its
 * barrier on top of what it brings: the copy completes as always, the barrier does not, the wait
 * runs out.  Host-side settings of the handle, used by the calls issued after it. */
pask_status_t pask_debug_set_wait(pask_cache_t *cache, int64_t limit_cycles, uint32_t surplus_bytes);
/* Where, inside a plan area for n_seqs sequences, the page-order list of (layer, parity) lies: byte
 * offset and length.  For tests of the streaming kernel's own bounds check: a page id beyond what
 * the pools hold (a plan somebody overwrote) is never dereferenced -- the kernel reads page 0
 * instead and sets PASK_DEV_INTERNAL.  Host only. */
pask_status_t pask_debug_plan_order_span(const pask_cache_t *cache, int32_t n_seqs, int32_t layer, int32_t parity,
                                         size_t *offset, size_t *bytes);

const char *pask_status_string(pask_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* PASK_H_ */
