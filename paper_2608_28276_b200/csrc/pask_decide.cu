// pask_decide: the budget-dependent adjustment of the table's actions -- Algorithm 2 of the paper,
// steps 1-6 and the recurrence of step 8, for a ragged batch of tokens and all layer groups at once.
//
// The work per token is constant and tiny (at most eight groups, two steps each); what orders it is
// the running budget R, which every token of a sequence reads and changes.  One warp owns one
// sequence: its lanes fetch 32 tokens' tags, states and table rows side by side, then walk those
// tokens in order with all lanes holding the same R.  A token whose table actions fit B and whose
// state is not critical -- the common case -- costs a handful of integer instructions; only the
// others enter the Demote / Promote loops and read the upgrade scores.  Decisions use integers and
// comparisons of the stored fp32 scores only, so they are bit-exact against any other
// implementation of the same rule.
//
// The call is all-or-nothing like an append: every warp writes what its sequence adds to the
// budget state into a per-call record, and the CTA that arrives last commits all records, or none
// if any entry of the call was invalid.
#include "pask_internal.h"

namespace pask {

namespace {

constexpr int kDecideThreads = 256;
constexpr int kDecideWarps = kDecideThreads / 32;

__device__ __forceinline__ uint32_t act_of(uint32_t packed, int g) { return (packed >> (2 * g)) & 3u; }

__global__ void __launch_bounds__(kDecideThreads)
decide_kernel(DevCache c, int n_seqs, int total_tokens, const int32_t *__restrict__ seq_ids,
              const int32_t *__restrict__ cu_tokens, const uint8_t *__restrict__ tags,
              const uint16_t *__restrict__ states, uint8_t *__restrict__ actions_out) {
    __shared__ uint2 s_row[256];
    __shared__ float2 s_rho[255 * PASK_MAX_GROUPS];   // upgrade scores: read inside the Demote / Promote loops
    __shared__ uint32_t s_layers[PASK_MAX_GROUPS];
    __shared__ int s_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = c.n_groups;
    // this launch's serial (for spotting a sequence named twice): read by every CTA before its arrival
    // ticket, stored back by the CTA that arrives last
    uint32_t serial = c.ctrl[kCtrlSerial] + 1u;
    if (serial == 0) serial = 1;
    s_row[tid] = c.dec_row[tid];
    for (int x = tid; x < c.n_tags * G; x += kDecideThreads) s_rho[x] = c.dec_rho[x];
    if (tid < PASK_MAX_GROUPS) s_layers[tid] = c.group_layers[tid];
    __syncthreads();
    uint32_t token_full = 0;                       // full cost of one token over all layers
    for (int g = 0; g < G; g++) token_full += s_layers[g] * c.bytes_h;
    const uint32_t step_hl = c.bytes_h - c.bytes_l, step_lr = c.bytes_l;   // bytes saved by H->L and L->R per layer

    const int i = blockIdx.x * kDecideWarps + warp;
    if (i < n_seqs) {
        const int seq = seq_ids[i];
        const int t0 = cu_tokens[i], t1 = cu_tokens[i + 1];
        uint32_t err = 0;
        if (t0 < 0 || t1 < t0 || t1 > total_tokens || (i == 0 && t0 != 0) || (i == n_seqs - 1 && t1 != total_tokens))
            err |= PASK_DEV_BAD_RAGGED;
        if (seq < 0 || seq >= c.max_seqs) err |= PASK_DEV_BAD_SEQ;
        if (!err) {                                // a sequence named twice in one call
            uint32_t prev = 0;
            if (lane == 0) prev = atomicExch(&c.seq_mark[seq], serial);
            if (__shfl_sync(0xffffffffu, prev, 0) == serial) err |= PASK_DEV_BAD_SEQ;
        }
        DecidePlan plan{};
        plan.seq = -1;
        if (!err) {
            const uint64_t full0 = c.budget[seq].decided_full_bytes, ret0 = c.budget[seq].decided_retained_bytes;
            uint64_t full = full0, ret = ret0, n_dem = 0, n_pro = 0, n_conf = 0;
            for (int base = t0; base < t1; base += 32) {
                const int t = base + lane;
                const bool valid = t < t1;
                const uint32_t my_tag = valid ? tags[t] : (uint32_t)PASK_TAG_PROTECTED;
                const uint2 my_row = s_row[my_tag];
                uint32_t my_gamma = 0, my_crit = 0;
                if (valid && states) {
                    const uint32_t st = states[t];
                    if (st < c.n_states_dev) { my_gamma = c.gamma[st]; my_crit = c.crit[st]; }
                }
                uint32_t my_actions = 0;
                const int cnt = t1 - base < 32 ? t1 - base : 32;
                for (int j = 0; j < cnt; j++) {    // the sequence's tokens in order; every lane holds the same values
                    const uint32_t packed = __shfl_sync(0xffffffffu, my_row.x, j);
                    uint64_t cost = __shfl_sync(0xffffffffu, my_row.y, j);
                    const uint64_t gamma = (uint64_t)__shfl_sync(0xffffffffu, my_gamma, j) << c.gamma_shift;
                    const uint32_t crit = __shfl_sync(0xffffffffu, my_crit, j);
                    const uint32_t tag = __shfl_sync(0xffffffffu, my_tag, j);
                    uint32_t a = packed & 0xffffu;
                    const uint32_t fl = packed >> 16;
                    full += token_full;
                    // R = floor(target * full) - retained; B = [R - Gamma]+   (Eq. 10)
                    const int64_t R = (int64_t)(((uint64_t)c.budget_q16 * full) >> 16) - (int64_t)ret;
                    int64_t B = R - (int64_t)gamma;
                    if (B < 0) B = 0;
                    // Protected and unknown tags sit at H with floor H in every group and have no row of upgrade
                    // scores (s_rho holds n_tags rows): neither loop may run for them.
                    const bool scored = tag < (uint32_t)c.n_tags;
                    if (scored && (int64_t)cost > B) {
                        // Demote: one adjacent step at a time, smallest upgrade score first, never below a floor
                        while ((int64_t)cost > B) {
                            int pick = -1;
                            float best = 0.f;
                            for (int g = 0; g < G; g++) {
                                const uint32_t ag = act_of(a, g);
                                if (ag <= act_of(fl, g) || s_layers[g] == 0) continue;
                                const float2 rho = s_rho[tag * G + g];
                                const float score = ag == PASK_ACTION_RETAIN_HIGH ? rho.y : rho.x;
                                if (pick < 0 || score < best) { pick = g; best = score; }
                            }
                            if (pick < 0) break;
                            cost -= (uint64_t)s_layers[pick] * (act_of(a, pick) == PASK_ACTION_RETAIN_HIGH ? step_hl : step_lr);
                            a -= 1u << (2 * pick);
                            n_dem++;
                        }
                        if ((int64_t)cost > B) n_conf++;   // floors first
                    } else if ((int64_t)cost > B) {
                        n_conf++;                          // a protected / unknown tag over budget: its floors stay
                    }
                    if (crit && scored) {
                        // Promote: while an adjacent step up still fits in B, take the one with the largest score
                        for (;;) {
                            int pick = -1;
                            float best = 0.f;
                            for (int g = 0; g < G; g++) {
                                const uint32_t ag = act_of(a, g);
                                if (ag >= PASK_ACTION_RETAIN_HIGH || s_layers[g] == 0) continue;
                                const uint64_t up = (uint64_t)s_layers[g] * (ag == PASK_ACTION_RETAIN_LOW ? step_hl : step_lr);
                                if ((int64_t)(cost + up) > B) continue;
                                const float2 rho = s_rho[tag * G + g];
                                const float score = ag == PASK_ACTION_RETAIN_LOW ? rho.y : rho.x;
                                if (pick < 0 || score > best) { pick = g; best = score; }
                            }
                            if (pick < 0) break;
                            cost += (uint64_t)s_layers[pick] * (act_of(a, pick) == PASK_ACTION_RETAIN_LOW ? step_hl : step_lr);
                            a += 1u << (2 * pick);
                            n_pro++;
                        }
                    }
                    ret += cost;                   // step 8
                    if (lane == j) my_actions = a;
                }
                if (valid)
                    for (int g = 0; g < G; g++) actions_out[(size_t)t * G + g] = (uint8_t)act_of(my_actions, g);
            }
            plan.seq = seq;
            plan.full = full - full0;
            plan.retained = ret - ret0;
            plan.demoted = n_dem;
            plan.promoted = n_pro;
            plan.conflicts = n_conf;
        }
        if (lane == 0) {
            if (err) atomicOr(&c.ctrl[kCtrlStatus], err);
            reinterpret_cast<DecidePlan *>(c.plan)[i] = plan;
        }
    }

    // ---- the CTA that arrives last commits every sequence's record, or none of them
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        s_last = atomicAdd(&c.ctrl[kCtrlTicket], 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const DecidePlan *plans = reinterpret_cast<const DecidePlan *>(c.plan);
    int any_bad = 0;
    for (int j = tid; j < n_seqs; j += kDecideThreads) any_bad |= __ldcg(&plans[j].seq) < 0;
    any_bad = __syncthreads_or(any_bad);
    if (!any_bad) {
        for (int j = tid; j < n_seqs; j += kDecideThreads) {
            const uint4 *src = reinterpret_cast<const uint4 *>(&plans[j]);
            union { DecidePlan p; uint4 q[4]; } u;
#pragma unroll
            for (int x = 0; x < 4; x++) u.q[x] = __ldcg(src + x);
            pask_budget_state_t &b = c.budget[u.p.seq];
            b.decided_full_bytes += u.p.full;
            b.decided_retained_bytes += u.p.retained;
            b.n_demoted += u.p.demoted;
            b.n_promoted += u.p.promoted;
            b.n_floor_conflicts += u.p.conflicts;
        }
    }
    if (tid == 0) { c.ctrl[kCtrlSerial] = serial; c.ctrl[kCtrlTicket] = 0; }
}

}  // namespace

pask_status_t launch_decide(pask_cache *c, int n_seqs, int total_tokens, const int32_t *seq_ids, const int32_t *cu_tokens,
                            const uint8_t *tags, const uint16_t *states, uint8_t *actions_out, cudaStream_t stream) {
    const int ctas = (n_seqs + kDecideWarps - 1) / kDecideWarps;
    decide_kernel<<<ctas, kDecideThreads, 0, stream>>>(c->dev, n_seqs, total_tokens, seq_ids, cu_tokens, tags, states,
                                                      actions_out);
    return cudaGetLastError() == cudaSuccess ? PASK_OK : PASK_ERR_CUDA;
}

}  // namespace pask
