// Internal types shared by the host API and the kernels of libpask.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/pask.h"
#include "pask_layout.h"

namespace pask {

// control words at the start of meta
enum CtrlWord : int {
    kCtrlStatus = 0,    // sticky PASK_DEV_* bits
    kCtrlTicket = 1,    // arrival counter of the append plan kernel (self-resetting)
    kCtrlHighNext = 2,  // bump counter of the HIGH pool
    kCtrlHighFree = 3,  // depth of the HIGH free stack
    kCtrlLowNext = 4,
    kCtrlLowFree = 5,
    kCtrlPlanOk = 6,    // 1 if the last append plan was committed, 0 if it was refused
    kCtrlItems = 7,     // work items (stream pages touched) of the last committed bulk append
    kCtrlSerial = 8,    // serial of the last launch that marks sequences (duplicate detection); kept on the device so
                        // that a launch recorded in a CUDA graph gets a fresh one at every replay
    kCtrlWords = 64
};

// one record per sequence of an append call, written by the plan kernel
struct AppendPlan {
    int32_t seq;
    uint32_t old_high, old_low;    // stream lengths before the call
    uint32_t cnt_high, cnt_low;    // tokens this call adds to each stream
    uint32_t cnt_drop, bad_tags;
    uint32_t new_pages_high, new_pages_low;
    int32_t tok0, tok1;            // the sequence's token range in the call
    uint32_t old_tok;              // tokens the (sequence, layer) had seen before the call
    uint32_t pad[4];
};
static_assert(sizeof(AppendPlan) == 64, "plan record");

// pask_decide reuses the plan records (calls on one cache are ordered by their stream): what one
// sequence's tokens add to its running budget, committed by the CTA that arrives last
struct DecidePlan {
    int32_t seq;                   // -1: this entry of the call is invalid
    uint32_t pad0;
    uint64_t full, retained;       // bytes added to decided_full_bytes / decided_retained_bytes
    uint64_t demoted, promoted, conflicts;
    uint64_t pad1[2];
};
static_assert(sizeof(DecidePlan) == sizeof(AppendPlan), "plan record");
constexpr uint32_t kMaxStatesDev = 65536;   // state ids are 16-bit

// Device view of a cache, passed to kernels by value.
struct DevCache {
    uint8_t *pool_high, *pool_low;
    uint32_t *ctrl;
    uint32_t *free_high, *free_low;
    uint32_t *n_high, *n_low;        // [max_seqs][n_layers] stream lengths in tokens
    uint32_t *tbl_high, *tbl_low;    // [max_seqs][n_layers][max_pages] page ids
    pask_budget_state_t *budget;     // [max_seqs]
    uint32_t *seq_mark;              // [max_seqs] serial of the last append call that named the sequence
    uint32_t *low_vmax;              // [max_seqs][n_layers] largest V scale (fp16 bits) in the LOW stream
    uint32_t *n_tok;                 // [max_seqs][n_layers] tokens appended so far, released ones included
    uint8_t *win_act;                // [max_seqs][n_layers][window] action of the token in each slot of the recent window
    uint32_t window;                 // protected recent window W in tokens (0: none); its W/16 bf16 pages per (sequence,
                                     // layer) are pages cap_high + (seq * n_layers + layer) * W/16 .. of the HIGH pool
    AppendPlan *plan;                // [PASK_MAX_SEQS_PER_CALL]
    uint32_t *tok_list;              // [max_append_tokens] bulk appends: each sequence's retained tokens in stream order
                                     // (HIGH from the front of its token range, LOW from the back)
    uint32_t *item_base;             // [PASK_MAX_SEQS_PER_CALL + 1] prefix over sequences of the pages a bulk append touches
    uint8_t *lut;                    // [n_tags][n_groups] effective action max(a0, floor)
    uint8_t *layer_group;            // [n_layers]
    // tables of the budget-dependent adjustment (pask_decide)
    uint2 *dec_row;                  // [256] per tag byte: x = actions (2 bits per group) | floors << 16, y = cost of the actions
    float2 *dec_rho;                 // [n_tags][n_groups] upgrade scores {R->L, L->H}
    uint32_t *gamma;                 // [n_states_dev] reserve in units of 2^gamma_shift bytes
    uint8_t *crit;                   // [n_states_dev] critical-state flags
    uint32_t n_states_dev, gamma_shift;
    uint32_t group_layers[PASK_MAX_GROUPS];   // layers per group
    int32_t n_layers, n_q, n_kv, max_seqs, max_pages, max_append_tokens;
    int32_t n_tags, n_groups;
    uint32_t cap_high, cap_low;
    uint32_t high_limit;             // cap_high plus the pages of the recent-window rings
    uint32_t budget_q16;
    uint32_t high_page_bytes, low_page_bytes;
    uint32_t bytes_h, bytes_l;       // m(H), m(L) per token per layer
    uint32_t low_bits;               // 2, 4 or 8: width of the RETAIN-LOW codes
    uint32_t low_head_bytes;         // one KV head of a LOW page (2304 or 4352)
    uint32_t cost_low_page;          // cost of a LOW page in units of n_kv * 256 bytes (9 or 17)
    uint32_t attn_ctas;              // grid of the decode-attention main kernel (the plans are cut for it)
};

// workspace of one decode-attention call
struct Workspace {
    uint32_t *cost_prefix;  // [n_seqs + 1] cost of the sequences before s
    uint32_t *page_prefix;  // [n_seqs + 1] pages of the sequences before s
    uint2 *tokens;          // [n_seqs] (n_high, n_low) tokens attended from the two streams
    uint32_t *order;        // [page_prefix[n_seqs]] pages in visiting order: kOrderHigh | tokens to attend << 27 | page id
    float2 *part_ml;        // [slots][n_q] (reference maximum in log2 units, sum)
    float *part_o;          // [slots][n_q][128] unnormalised outputs
};

// One layer's work plan of a planned-ahead decode step, inside the caller's plan area: what Workspace holds of a
// plan, plus the list of sequences it was made for.
struct PlanBlock {
    int32_t *ids;           // [n_seqs] the sequences the plan describes, in call order
    uint32_t *cost_prefix, *page_prefix;
    uint2 *tokens;
    uint32_t *order;
};

struct MetaOffsets {
    size_t ctrl, free_high, free_low, n_high, n_low, tbl_high, tbl_low, budget, seq_mark, low_vmax, n_tok, win_act, plan, tok_list, item_base, lut,
        layer_group, dec_row, dec_rho, gamma, crit, total;
    size_t zero_begin, zero_end;     // the span cleared by a reset (counters, tables, budgets, marks)
};

}  // namespace pask

struct pask_policy {
    uint32_t n_tags, n_groups, n_layers, n_states, budget_q16, window, low_bits;
    std::vector<uint8_t> layer_group, a0, a_floor, eff;
    std::vector<float> rho_rl, rho_lh;
    std::vector<uint32_t> gamma;
    std::vector<uint8_t> crit;
    uint32_t gamma_shift;
};

struct pask_cache {
    pask_cache_desc_t desc;
    pask::DevCache dev;
    pask::MetaOffsets off;
    void *meta;
    std::vector<uint8_t> lut, layer_group;   // host copies of the folded table [n_tags][n_groups] and the layer map
    int sm_count;
    int attn_ctas;                // grid of the decode-attention main kernel
    cudaEvent_t ev_start, ev_stop;
    unsigned long long *span;     // pask_cache_set_timing_span: where the next streaming kernel leaves its start and end
    // planned-ahead decode steps: which layers hold a plan, for how many sequences, in which area, and which of the
    // layer's two plan blocks is the current one
    struct Ahead {
        bool valid = false;
        int n_seqs = 0, parity = 0;
        const void *area = nullptr;
        uint64_t early_from = 0;  // first planned-ahead call (by number) that may read the plan before its dependency wait
    };
    std::vector<Ahead> ahead;     // [n_layers]
    uint64_t ahead_calls = 0;     // planned-ahead step calls issued so far
    long long wait_cycles;        // bound of a device-side wait for a bulk copy, in SM clock cycles (about a second)
    uint32_t wait_test_surplus;   // pask_debug_set_wait: bytes a warp's first copy announces but does not bring
    // pask_decode_step_pipelined: two copy streams and the events that order them against the caller's stream
    struct StepPipe {
        bool ready = false;
        cudaStream_t in = nullptr, out = nullptr;
        cudaEvent_t ev_in[2] = {}, ev_done[2] = {}, ev_out[2] = {};
        uint64_t calls = 0;
        int recorded[2] = {0, 0};         // per slot: bit 0 = ev_done has been recorded, bit 1 = ev_out
        const void *staging = nullptr;    // the staging buffer of the call before
        size_t staging_bytes = 0;
    } pipe;
};

namespace pask {

// Programmatic dependent launch: the kernels of the hot path are launched so that a kernel's CTAs
// may be scheduled while its predecessor in the stream is still draining.  Each of them executes
// pdl_launch_dependents() on entry and pdl_wait() before it touches global memory, and pdl_wait()
// returns only when the predecessor has completed and its writes are visible -- so ordering is
// what plain stream order gives, minus the launch latency between the kernels.
#if defined(__CUDACC__)
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

// launchers implemented next to their kernels
// fuse_ws != nullptr: if the call goes down the one-launch path, that launch also writes the decode-attention plan for
// the same sequences into *fuse_ws and *fused is set
pask_status_t launch_append(pask_cache *c, int layer, int n_seqs, int total_tokens, const int32_t *seq_ids,
                            const int32_t *cu_tokens, const void *k, const void *v, const uint8_t *tags,
                            const uint8_t *decided, uint8_t *actions_out, cudaStream_t stream,
                            const Workspace *fuse_ws = nullptr, bool *fused = nullptr);
pask_status_t launch_decide(pask_cache *c, int n_seqs, int total_tokens, const int32_t *seq_ids, const int32_t *cu_tokens,
                            const uint8_t *tags, const uint16_t *states, uint8_t *actions_out, cudaStream_t stream);
pask_status_t launch_seq_reset(pask_cache *c, int seq, cudaStream_t stream);
pask_status_t launch_attention(pask_cache *c, bool has_low, int layer, int n_seqs, const int32_t *seq_ids,
                               const void *q, float *out, float *lse, void *workspace, size_t workspace_bytes,
                               cudaStream_t stream, bool plan_done = false);
size_t carve_workspace(const pask_cache *c, int n_seqs, uint8_t *base, Workspace *ws);
// the plan block of (layer, parity) inside a plan area for n_seqs sequences; returns the size of the whole area
size_t carve_plan_area(const pask_cache *c, int n_seqs, int layer, int parity, uint8_t *base, PlanBlock *pb);
pask_status_t launch_plan_ahead(pask_cache *c, int layer, int n_seqs, const int32_t *seq_ids, void *area, int parity,
                                cudaStream_t stream);
// streaming kernel over the plan block `cur`, then the append that writes the other block, then the merge with the new tokens
pask_status_t launch_step_ahead(pask_cache *c, int layer, int n_seqs, const int32_t *seq_ids, const void *k, const void *v,
                                const uint8_t *tags, const uint8_t *decided, uint8_t *actions_out, const void *q, float *out,
                                float *lse, void *workspace, void *area, int cur, bool early, cudaStream_t stream);
// the kernel that ends a planned-ahead step: the one-launch append (its first n_seqs CTAs; it writes the plan `plan_ws`
// and the sequence list `ids_out`), then, behind the dependency wait, the merge of the streaming kernel's partials
// with the new tokens
struct NewTokens;
pask_status_t launch_step_tail(pask_cache *c, int layer, int n_seqs, const int32_t *seq_ids, const int32_t *cu_tokens,
                               const void *k, const void *v, const uint8_t *tags, const uint8_t *decided, uint8_t *actions_out,
                               const Workspace &plan_ws, int32_t *ids_out, const uint32_t *prefix, const float2 *part_ml,
                               const float *part_o, float *out, float *lse, const NewTokens &nt, cudaStream_t stream);
struct SmallLut { uint8_t action[256]; };
void fill_small_lut(const pask_cache *c, int layer, SmallLut *lut);
size_t attention_workspace_bytes(const pask_cache *c, int n_seqs);
int attention_grid(const pask_cache *c);
}  // namespace pask
