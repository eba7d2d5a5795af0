// Host side of libpask: policy blobs, cache set-up, budget state, canonical dumps.
#include <cstring>
#include <memory>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "pask_internal.h"

using namespace pask;

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// NVTX range around the host side of an entry point (header-only NVTX: a no-op unless a profiler is attached)
struct NvtxRange {
    explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
};

uint32_t rd32(const uint8_t *p) {
    return (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24);
}

bool shape_ok(const pask_cache_desc_t *d) {
    if (d->head_dim != kHeadDim || d->page_tokens != kPageTokens) return false;
    const int kv = d->n_kv_heads;
    if (!(kv == 1 || kv == 2 || kv == 4 || kv == 8)) return false;
    return d->n_q_heads == 4 * kv;
}

MetaOffsets meta_offsets(const pask_cache_desc_t *d, int n_tags, int n_groups) {
    MetaOffsets o{};
    const size_t max_pages = (size_t)(d->max_tokens_per_seq + kPageTokens - 1) / kPageTokens;
    const size_t sl = (size_t)d->max_seqs * d->n_layers;
    size_t p = 0;
    auto take = [&](size_t bytes) { size_t at = p; p = align_up(p + bytes, 256); return at; };
    o.ctrl = take(kCtrlWords * 4);
    o.free_high = take((size_t)d->pool_high_pages * 4);
    o.free_low = take((size_t)d->pool_low_pages * 4);
    o.zero_begin = p;
    o.n_high = take(sl * 4);
    o.n_low = take(sl * 4);
    o.tbl_high = take(sl * max_pages * 4);
    o.tbl_low = take(sl * max_pages * 4);
    o.budget = take((size_t)d->max_seqs * sizeof(pask_budget_state_t));
    o.seq_mark = take((size_t)d->max_seqs * 4);
    o.low_vmax = take(sl * 4);
    o.n_tok = take(sl * 4);
    o.zero_end = p;
    o.win_act = take(sl * (size_t)d->recent_window);
    o.plan = take((size_t)PASK_MAX_SEQS_PER_CALL * sizeof(AppendPlan));
    o.tok_list = take((size_t)d->max_append_tokens * 4);
    o.item_base = take((size_t)(PASK_MAX_SEQS_PER_CALL + 1) * 4);
    o.lut = take((size_t)n_tags * n_groups);
    o.layer_group = take((size_t)d->n_layers);
    o.dec_row = take(256 * sizeof(uint2));
    o.dec_rho = take((size_t)n_tags * n_groups * sizeof(float2));
    o.gamma = take((size_t)kMaxStatesDev * 4);
    o.crit = take((size_t)kMaxStatesDev);
    o.total = p;
    return o;
}

// pages of the recent-window rings, which sit behind the HIGH pool's own pages
size_t window_pages(const pask_cache_desc_t *d) {
    return (size_t)d->max_seqs * d->n_layers * (size_t)(d->recent_window / kPageTokens);
}

bool desc_ok(const pask_cache_desc_t *d) {
    return d->n_layers > 0 && d->n_layers <= 4096 && d->max_seqs > 0 && d->max_tokens_per_seq > 0 &&
           d->max_append_tokens > 0 && d->recent_window >= 0 && d->recent_window <= PASK_MAX_WINDOW &&
           d->recent_window % kPageTokens == 0 && (d->low_bits == 0 || d->low_bits == 4 || d->low_bits == 8 || d->low_bits == 2);
}

pask_status_t cuda_rc(cudaError_t e) { return e == cudaSuccess ? PASK_OK : PASK_ERR_CUDA; }

// read n_high / n_low of (seq, layer) after draining the stream
pask_status_t read_lens(pask_cache *c, int layer, int seq, uint32_t *nh, uint32_t *nl, cudaStream_t s) {
    if (cudaStreamSynchronize(s) != cudaSuccess) return PASK_ERR_CUDA;
    const size_t i = (size_t)seq * c->desc.n_layers + layer;
    if (cudaMemcpy(nh, c->dev.n_high + i, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return PASK_ERR_CUDA;
    if (cudaMemcpy(nl, c->dev.n_low + i, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return PASK_ERR_CUDA;
    return PASK_OK;
}

bool seq_layer_ok(const pask_cache *c, int layer, int seq) {
    return layer >= 0 && layer < c->desc.n_layers && seq >= 0 && seq < c->desc.max_seqs;
}

}  // namespace

extern "C" {

const char *pask_status_string(pask_status_t s) {
    switch (s) {
        case PASK_OK: return "ok";
        case PASK_ERR_INVALID_ARG: return "invalid argument";
        case PASK_ERR_BAD_POLICY: return "malformed policy blob";
        case PASK_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case PASK_ERR_POOL_EXHAUSTED: return "page pool exhausted";
        case PASK_ERR_BAD_SEQ: return "bad sequence id";
        case PASK_ERR_CUDA: return "CUDA runtime error";
        case PASK_ERR_TIMEOUT: return "device wait timed out";
        case PASK_ERR_WORKSPACE: return "workspace too small";
        case PASK_ERR_NO_MEMORY: return "out of host memory";
        case PASK_ERR_STALE_PLAN: return "no valid plan made ahead for this layer and batch";
        default: return "unknown status";
    }
}

pask_status_t pask_load_policy(const void *blob_v, size_t len, pask_policy_t **out) try {
    if (!blob_v || !out) return PASK_ERR_INVALID_ARG;
    *out = nullptr;
    const uint8_t *blob = static_cast<const uint8_t *>(blob_v);
    if (len < 40 || std::memcmp(blob, "PASK", 4) != 0) return PASK_ERR_BAD_POLICY;
    const uint32_t version = rd32(blob + 4);
    if (version != 1 && version != 2) return PASK_ERR_BAD_POLICY;
    std::unique_ptr<pask_policy> p(new (std::nothrow) pask_policy());
    if (!p) return PASK_ERR_NO_MEMORY;
    p->n_tags = rd32(blob + 8);
    p->n_groups = rd32(blob + 12);
    p->n_layers = rd32(blob + 16);
    p->n_states = rd32(blob + 20);
    p->budget_q16 = rd32(blob + 24);
    p->window = rd32(blob + 28);
    p->low_bits = rd32(blob + 32);
    const uint32_t window = p->window, low_bits = rd32(blob + 32), group_size = rd32(blob + 36);
    bool ok = p->n_tags >= 1 && p->n_tags <= 255 && p->n_groups >= 1 && p->n_groups <= PASK_MAX_GROUPS &&
              p->n_layers >= 1 && p->n_layers <= 4096 && p->n_states <= (1u << 20) && window <= PASK_MAX_WINDOW && window % kPageTokens == 0 && (low_bits == 4 || low_bits == 8 || low_bits == 2) &&
              group_size == (uint32_t)kQGroup;
    const size_t lg_pad = ok ? align_up(p->n_layers, 4) : 0;
    const size_t n_ent = ok ? (size_t)p->n_tags * p->n_groups : 0;
    const size_t tail = ok && version == 2 ? 4 + align_up(p->n_states, 4) : 0;
    ok = ok && len == 40 + lg_pad + n_ent * 12 + (size_t)p->n_states * 4 + tail;
    p->gamma_shift = 0;
    if (ok) {
        p->layer_group.assign(blob + 40, blob + 40 + p->n_layers);
        for (uint8_t g : p->layer_group) ok = ok && g < p->n_groups;
        const uint8_t *e = blob + 40 + lg_pad;
        p->a0.resize(n_ent); p->a_floor.resize(n_ent); p->eff.resize(n_ent);
        p->rho_rl.resize(n_ent); p->rho_lh.resize(n_ent);
        for (size_t i = 0; i < n_ent; i++, e += 12) {
            p->a0[i] = e[0];
            p->a_floor[i] = e[1];
            ok = ok && e[0] <= PASK_ACTION_RETAIN_HIGH && e[1] <= PASK_ACTION_RETAIN_HIGH && e[2] == 0 && e[3] == 0;
            std::memcpy(&p->rho_rl[i], e + 4, 4);
            std::memcpy(&p->rho_lh[i], e + 8, 4);
            ok = ok && p->rho_rl[i] == p->rho_rl[i] && p->rho_lh[i] == p->rho_lh[i];   // scores are compared: no NaN
            p->eff[i] = e[0] > e[1] ? e[0] : e[1];  // floors take priority: a = max(a0, a_floor)
        }
        p->gamma.resize(p->n_states);
        for (uint32_t s = 0; s < p->n_states; s++, e += 4) p->gamma[s] = rd32(e);
        p->crit.assign(p->n_states, 0);
        if (version == 2) {
            p->gamma_shift = rd32(e);
            e += 4;
            ok = ok && p->gamma_shift <= 16;
            for (uint32_t s = 0; s < p->n_states; s++) { p->crit[s] = e[s]; ok = ok && e[s] <= 1; }
        }
    }
    if (!ok) return PASK_ERR_BAD_POLICY;
    *out = p.release();
    return PASK_OK;
} catch (...) {   // the tables could not be allocated
    return PASK_ERR_NO_MEMORY;
}

void pask_free_policy(pask_policy_t *p) { delete p; }

int32_t pask_policy_action(const pask_policy_t *p, int32_t tag, int32_t group) {
    if (!p || tag < 0 || (uint32_t)tag >= p->n_tags || group < 0 || (uint32_t)group >= p->n_groups) return -1;
    return p->eff[(size_t)tag * p->n_groups + group];
}

pask_status_t pask_cache_sizes(const pask_cache_desc_t *d, pask_cache_sizes_t *out) {
    if (!d || !out) return PASK_ERR_INVALID_ARG;
    if (!shape_ok(d)) return PASK_ERR_UNSUPPORTED_SHAPE;
    if (!desc_ok(d)) return PASK_ERR_INVALID_ARG;
    out->high_page_bytes = (size_t)d->n_kv_heads * kHighHeadBytes;
    out->low_page_bytes = (size_t)d->n_kv_heads * (d->low_bits == 8 ? kLow8HeadBytes : d->low_bits == 2 ? kLow2HeadBytes : kLowHeadBytes);
    out->pool_high_bytes = out->high_page_bytes * ((size_t)d->pool_high_pages + window_pages(d));
    out->pool_low_bytes = out->low_page_bytes * d->pool_low_pages;
    out->meta_bytes = meta_offsets(d, 255, PASK_MAX_GROUPS).total;  // independent of the policy loaded later
    return PASK_OK;
}

pask_status_t pask_cache_create(const pask_cache_desc_t *d, const pask_policy_t *pol, void *pool_high, void *pool_low,
                                void *meta, pask_stream_t stream_v, pask_cache_t **out) try {
    if (!d || !pol || !meta || !out) return PASK_ERR_INVALID_ARG;
    *out = nullptr;
    if (!shape_ok(d)) return PASK_ERR_UNSUPPORTED_SHAPE;
    if (!desc_ok(d) || (uint32_t)d->n_layers != pol->n_layers || (uint32_t)d->recent_window != pol->window ||
        (uint32_t)(d->low_bits ? d->low_bits : 4) != pol->low_bits)
        return PASK_ERR_INVALID_ARG;
    if (((d->pool_high_pages || d->recent_window) && !pool_high) || (d->pool_low_pages && !pool_low)) return PASK_ERR_INVALID_ARG;
    if (((uintptr_t)pool_high | (uintptr_t)pool_low | (uintptr_t)meta) & 255) return PASK_ERR_INVALID_ARG;
    if ((size_t)d->pool_high_pages + window_pages(d) > kOrderIdMask || d->pool_low_pages > kOrderIdMask)
        return PASK_ERR_INVALID_ARG;   // page ids travel in the low bits of the page-order entries
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int dev_id = 0, sms = 0;
    if (cudaGetDevice(&dev_id) != cudaSuccess) return PASK_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev_id) != cudaSuccess) return PASK_ERR_CUDA;
    std::unique_ptr<pask_cache> holder(new (std::nothrow) pask_cache());
    if (!holder) return PASK_ERR_NO_MEMORY;
    pask_cache *c = holder.get();
    c->desc = *d;
    c->meta = meta;
    c->sm_count = sms;
    c->ev_start = c->ev_stop = nullptr;
    c->span = nullptr;
    c->ahead.resize((size_t)d->n_layers);
    c->wait_cycles = 2000000000LL;   // about one second: give up instead of hanging
    c->wait_test_surplus = 0;
    c->off = meta_offsets(d, 255, PASK_MAX_GROUPS);
    uint8_t *m = static_cast<uint8_t *>(meta);
    DevCache &v = c->dev;
    v.pool_high = static_cast<uint8_t *>(pool_high);
    v.pool_low = static_cast<uint8_t *>(pool_low);
    v.ctrl = reinterpret_cast<uint32_t *>(m + c->off.ctrl);
    v.free_high = reinterpret_cast<uint32_t *>(m + c->off.free_high);
    v.free_low = reinterpret_cast<uint32_t *>(m + c->off.free_low);
    v.n_high = reinterpret_cast<uint32_t *>(m + c->off.n_high);
    v.n_low = reinterpret_cast<uint32_t *>(m + c->off.n_low);
    v.tbl_high = reinterpret_cast<uint32_t *>(m + c->off.tbl_high);
    v.tbl_low = reinterpret_cast<uint32_t *>(m + c->off.tbl_low);
    v.budget = reinterpret_cast<pask_budget_state_t *>(m + c->off.budget);
    v.seq_mark = reinterpret_cast<uint32_t *>(m + c->off.seq_mark);
    v.low_vmax = reinterpret_cast<uint32_t *>(m + c->off.low_vmax);
    v.n_tok = reinterpret_cast<uint32_t *>(m + c->off.n_tok);
    v.win_act = m + c->off.win_act;
    v.window = (uint32_t)d->recent_window;
    v.plan = reinterpret_cast<AppendPlan *>(m + c->off.plan);
    v.tok_list = reinterpret_cast<uint32_t *>(m + c->off.tok_list);
    v.item_base = reinterpret_cast<uint32_t *>(m + c->off.item_base);
    v.lut = m + c->off.lut;
    v.layer_group = m + c->off.layer_group;
    v.dec_row = reinterpret_cast<uint2 *>(m + c->off.dec_row);
    v.dec_rho = reinterpret_cast<float2 *>(m + c->off.dec_rho);
    v.gamma = reinterpret_cast<uint32_t *>(m + c->off.gamma);
    v.crit = m + c->off.crit;
    v.n_states_dev = pol->n_states < kMaxStatesDev ? pol->n_states : kMaxStatesDev;
    v.gamma_shift = pol->gamma_shift;
    for (int g = 0; g < PASK_MAX_GROUPS; g++) v.group_layers[g] = 0;
    for (uint8_t g : pol->layer_group) v.group_layers[g]++;
    v.n_layers = d->n_layers;
    v.n_q = d->n_q_heads;
    v.n_kv = d->n_kv_heads;
    v.max_seqs = d->max_seqs;
    v.max_pages = (d->max_tokens_per_seq + kPageTokens - 1) / kPageTokens;
    v.max_append_tokens = d->max_append_tokens;
    v.n_tags = (int32_t)pol->n_tags;
    v.n_groups = (int32_t)pol->n_groups;
    v.cap_high = d->pool_high_pages;
    v.cap_low = d->pool_low_pages;
    v.high_limit = d->pool_high_pages + (uint32_t)window_pages(d);
    v.budget_q16 = pol->budget_q16;
    v.high_page_bytes = (uint32_t)d->n_kv_heads * kHighHeadBytes;
    v.low_bits = pol->low_bits;
    v.low_head_bytes = pol->low_bits == 8 ? kLow8HeadBytes : pol->low_bits == 2 ? kLow2HeadBytes : kLowHeadBytes;
    v.cost_low_page = pol->low_bits == 8 ? kCostLow8Page : pol->low_bits == 2 ? kCostLow2Page : kCostLowPage;
    v.low_page_bytes = (uint32_t)d->n_kv_heads * v.low_head_bytes;
    v.bytes_h = 2u * d->n_kv_heads * kHeadDim * 2u;
    v.bytes_l = 2u * d->n_kv_heads * (kHeadDim * pol->low_bits / 8 + kGroupsPerHead * 2);
    c->attn_ctas = attention_grid(c);
    c->dev.attn_ctas = (uint32_t)c->attn_ctas;
    c->lut = pol->eff;
    c->layer_group = pol->layer_group;
    // per tag byte: the table's actions and floors packed two bits per group, and what the actions cost
    std::vector<uint2> dec_row(256);
    std::vector<float2> dec_rho((size_t)pol->n_tags * pol->n_groups);
    for (uint32_t z = 0; z < 256; z++) {
        uint32_t acts = 0, floors = 0, cost = 0;
        for (uint32_t g = 0; g < pol->n_groups; g++) {
            uint32_t a = PASK_ACTION_RETAIN_HIGH, f = PASK_ACTION_RETAIN_HIGH;   // protected and unknown tags
            if (z < pol->n_tags) {
                a = pol->eff[(size_t)z * pol->n_groups + g];
                f = pol->a_floor[(size_t)z * pol->n_groups + g];
                dec_rho[(size_t)z * pol->n_groups + g] = make_float2(pol->rho_rl[(size_t)z * pol->n_groups + g],
                                                                     pol->rho_lh[(size_t)z * pol->n_groups + g]);
            }
            acts |= a << (2 * g);
            floors |= f << (2 * g);
            cost += v.group_layers[g] * (a == PASK_ACTION_RETAIN_HIGH ? v.bytes_h : a == PASK_ACTION_RETAIN_LOW ? v.bytes_l : 0u);
        }
        dec_row[z] = make_uint2(acts | (floors << 16), cost);
    }
    // pageable host sources: the runtime stages these copies, so the vectors may die afterwards
    cudaError_t e = cudaMemcpyAsync(v.lut, pol->eff.data(), pol->eff.size(), cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(v.layer_group, pol->layer_group.data(), pol->layer_group.size(), cudaMemcpyHostToDevice,
                            stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(v.dec_row, dec_row.data(), dec_row.size() * sizeof(uint2), cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(v.dec_rho, dec_rho.data(), dec_rho.size() * sizeof(float2), cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess && v.n_states_dev)
        e = cudaMemcpyAsync(v.gamma, pol->gamma.data(), (size_t)v.n_states_dev * 4, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess && v.n_states_dev)
        e = cudaMemcpyAsync(v.crit, pol->crit.data(), (size_t)v.n_states_dev, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return PASK_ERR_CUDA;
    pask_status_t rc = pask_cache_reset(c, stream_v);
    if (rc != PASK_OK) return rc;
    *out = holder.release();
    return PASK_OK;
} catch (...) {   // a host-side table could not be allocated
    return PASK_ERR_NO_MEMORY;
}

void pask_cache_destroy(pask_cache_t *c) {
    if (!c) return;
    if (c->pipe.ready) {
        cudaStreamSynchronize(c->pipe.in);
        cudaStreamSynchronize(c->pipe.out);
        for (int i = 0; i < 2; i++) {
            cudaEventDestroy(c->pipe.ev_in[i]);
            cudaEventDestroy(c->pipe.ev_done[i]);
            cudaEventDestroy(c->pipe.ev_out[i]);
        }
        cudaStreamDestroy(c->pipe.in);
        cudaStreamDestroy(c->pipe.out);
    }
    delete c;
}

pask_status_t pask_cache_reset(pask_cache_t *c, pask_stream_t stream_v) {
    if (!c) return PASK_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    uint8_t *m = static_cast<uint8_t *>(c->meta);
    for (auto &a : c->ahead) a.valid = false;
    cudaError_t e = cudaMemsetAsync(m + c->off.ctrl, 0, kCtrlWords * 4, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(m + c->off.zero_begin, 0, c->off.zero_end - c->off.zero_begin, stream);
    return cuda_rc(e);
}

pask_status_t pask_seq_reset(pask_cache_t *c, int32_t seq, pask_stream_t stream) {
    if (!c) return PASK_ERR_INVALID_ARG;
    if (seq < 0 || seq >= c->desc.max_seqs) return PASK_ERR_BAD_SEQ;
    for (auto &a : c->ahead) a.valid = false;
    return launch_seq_reset(c, seq, static_cast<cudaStream_t>(stream));
}

static pask_status_t append_common(pask_cache_t *c, int32_t layer, int32_t n_seqs, int32_t total_tokens,
                                   const int32_t *seq_ids, const int32_t *cu_tokens, const void *k, const void *v,
                                   const uint8_t *tags, const uint8_t *decided, uint8_t *actions_out,
                                   pask_stream_t stream, const Workspace *fuse_ws = nullptr, bool *fused = nullptr) {
    if (!c || !seq_ids || !cu_tokens || !tags) return PASK_ERR_INVALID_ARG;
    if (layer < 0 || layer >= c->desc.n_layers) return PASK_ERR_INVALID_ARG;
    if (n_seqs < 1 || n_seqs > PASK_MAX_SEQS_PER_CALL || n_seqs > c->desc.max_seqs) return PASK_ERR_INVALID_ARG;
    if (total_tokens < 0 || total_tokens > c->desc.max_append_tokens) return PASK_ERR_INVALID_ARG;
    if (total_tokens > 0 && (!k || !v)) return PASK_ERR_INVALID_ARG;
    if (((uintptr_t)k | (uintptr_t)v) & 15) return PASK_ERR_INVALID_ARG;
    if (((uintptr_t)seq_ids | (uintptr_t)cu_tokens) & 3) return PASK_ERR_INVALID_ARG;
    NvtxRange range("pask_append_kv");
    c->ahead[layer].valid = false;       // a plan made ahead for this layer no longer describes it
    return launch_append(c, layer, n_seqs, total_tokens, seq_ids, cu_tokens, k, v, tags, decided, actions_out,
                         static_cast<cudaStream_t>(stream), fuse_ws, fused);
}

pask_status_t pask_append_kv(pask_cache_t *c, int32_t layer, int32_t n_seqs, int32_t total_tokens,
                             const int32_t *seq_ids, const int32_t *cu_tokens, const void *k, const void *v,
                             const uint8_t *tags, const uint16_t *states, uint8_t *actions_out, pask_stream_t stream) {
    (void)states;  // the frozen table as it stands; the budget-dependent adjustment is pask_decide
    return append_common(c, layer, n_seqs, total_tokens, seq_ids, cu_tokens, k, v, tags, nullptr, actions_out, stream);
}

pask_status_t pask_append_kv_decided(pask_cache_t *c, int32_t layer, int32_t n_seqs, int32_t total_tokens,
                                     const int32_t *seq_ids, const int32_t *cu_tokens, const void *k, const void *v,
                                     const uint8_t *tags, const uint8_t *actions, uint8_t *actions_out,
                                     pask_stream_t stream) {
    if (!actions) return PASK_ERR_INVALID_ARG;
    return append_common(c, layer, n_seqs, total_tokens, seq_ids, cu_tokens, k, v, tags, actions, actions_out, stream);
}

pask_status_t pask_decide(pask_cache_t *c, int32_t n_seqs, int32_t total_tokens, const int32_t *seq_ids,
                          const int32_t *cu_tokens, const uint8_t *tags, const uint16_t *states, uint8_t *actions_out,
                          pask_stream_t stream) {
    if (!c || !seq_ids || !cu_tokens || !tags || !actions_out) return PASK_ERR_INVALID_ARG;
    if (n_seqs < 1 || n_seqs > PASK_MAX_SEQS_PER_CALL || n_seqs > c->desc.max_seqs) return PASK_ERR_INVALID_ARG;
    if (total_tokens < 0) return PASK_ERR_INVALID_ARG;
    if (((uintptr_t)seq_ids | (uintptr_t)cu_tokens) & 3 || ((uintptr_t)states & 1)) return PASK_ERR_INVALID_ARG;
    NvtxRange range("pask_decide");
    return launch_decide(c, n_seqs, total_tokens, seq_ids, cu_tokens, tags, states, actions_out,
                         static_cast<cudaStream_t>(stream));
}

static pask_status_t attention_common(pask_cache_t *c, bool has_low, int32_t layer, int32_t n_seqs,
                                      const int32_t *seq_ids, const void *q, float *out, float *lse, void *ws,
                                      size_t ws_bytes, pask_stream_t stream, bool plan_done = false, bool check_only = false) {
    if (!c || !seq_ids || !q || !out || !ws) return PASK_ERR_INVALID_ARG;
    if (layer < 0 || layer >= c->desc.n_layers) return PASK_ERR_INVALID_ARG;
    if (n_seqs < 1 || n_seqs > PASK_MAX_SEQS_PER_CALL) return PASK_ERR_INVALID_ARG;
    if (((uintptr_t)q | (uintptr_t)out) & 15 || ((uintptr_t)ws & 255) || ((uintptr_t)lse & 3)) return PASK_ERR_INVALID_ARG;
    if (ws_bytes < attention_workspace_bytes(c, n_seqs)) return PASK_ERR_WORKSPACE;
    if (check_only) return PASK_OK;
    NvtxRange range(has_low ? "pask_decode_attention" : "pask_decode_attention_full");
    return launch_attention(c, has_low, layer, n_seqs, seq_ids, q, out, lse, ws, ws_bytes,
                            static_cast<cudaStream_t>(stream), plan_done);
}

pask_status_t pask_append_attend(pask_cache_t *c, int32_t layer, int32_t n_seqs, int32_t total_tokens,
                                 const int32_t *seq_ids, const int32_t *cu_tokens, const void *k, const void *v,
                                 const uint8_t *tags, const uint8_t *actions, uint8_t *actions_out, const void *q,
                                 float *out, float *lse, void *ws, size_t ws_bytes, pask_stream_t stream) {
    // every argument of the second call is checked before the first one is issued
    pask_status_t rc = attention_common(c, true, layer, n_seqs, seq_ids, q, out, lse, ws, ws_bytes, stream, false, true);
    if (rc != PASK_OK) return rc;
    Workspace plan;
    carve_workspace(c, n_seqs, static_cast<uint8_t *>(ws), &plan);
    bool fused = false;
    rc = append_common(c, layer, n_seqs, total_tokens, seq_ids, cu_tokens, k, v, tags, actions, actions_out, stream, &plan,
                       &fused);
    if (rc != PASK_OK) return rc;
    return attention_common(c, true, layer, n_seqs, seq_ids, q, out, lse, ws, ws_bytes, stream, fused);
}

pask_status_t pask_decode_attention(pask_cache_t *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                                    const void *q, float *out, float *lse, void *ws, size_t ws_bytes,
                                    pask_stream_t stream) {
    return attention_common(c, true, layer, n_seqs, seq_ids, q, out, lse, ws, ws_bytes, stream);
}

pask_status_t pask_decode_attention_full(pask_cache_t *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids,
                                         const void *q, float *out, float *lse, void *ws, size_t ws_bytes,
                                         pask_stream_t stream) {
    return attention_common(c, false, layer, n_seqs, seq_ids, q, out, lse, ws, ws_bytes, stream);
}

size_t pask_workspace_bytes(const pask_cache_t *c, int32_t n_seqs) {
    if (!c || n_seqs < 1) return 0;
    return attention_workspace_bytes(c, n_seqs);
}

size_t pask_plan_area_bytes(const pask_cache_t *c, int32_t n_seqs) {
    if (!c || n_seqs < 1 || n_seqs > 255) return 0;
    return carve_plan_area(c, n_seqs, 0, 0, nullptr, nullptr);
}

static pask_status_t ahead_args_ok(pask_cache_t *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids, void *area,
                                   size_t area_bytes) {
    if (!c || !seq_ids || !area) return PASK_ERR_INVALID_ARG;
    if (layer < 0 || layer >= c->desc.n_layers || n_seqs < 1 || n_seqs > c->desc.max_seqs) return PASK_ERR_INVALID_ARG;
    if (n_seqs > 255 || c->dev.window) return PASK_ERR_UNSUPPORTED_SHAPE;
    if (((uintptr_t)seq_ids & 3) || ((uintptr_t)area & 255)) return PASK_ERR_INVALID_ARG;
    if (area_bytes < pask_plan_area_bytes(c, n_seqs)) return PASK_ERR_WORKSPACE;
    return PASK_OK;
}

pask_status_t pask_plan_ahead(pask_cache_t *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids, void *area,
                              size_t area_bytes, pask_stream_t stream) {
    const pask_status_t ok = ahead_args_ok(c, layer, n_seqs, seq_ids, area, area_bytes);
    if (ok != PASK_OK) return ok;
    NvtxRange range("pask_plan_ahead");
    auto &a = c->ahead[layer];
    a.valid = false;
    const pask_status_t rc = launch_plan_ahead(c, layer, n_seqs, seq_ids, area, 0, static_cast<cudaStream_t>(stream));
    if (rc != PASK_OK) return rc;
    a.valid = true;
    a.n_seqs = n_seqs;
    a.parity = 0;
    a.area = area;
    a.early_from = c->ahead_calls + 2;
    return PASK_OK;
}

pask_status_t pask_decode_step_ahead(pask_cache_t *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids, const void *k,
                                     const void *v, const uint8_t *tags, const uint8_t *actions, uint8_t *actions_out,
                                     const void *q, float *out, float *lse, void *ws, size_t ws_bytes, void *area,
                                     size_t area_bytes, pask_stream_t stream) {
    pask_status_t rc = ahead_args_ok(c, layer, n_seqs, seq_ids, area, area_bytes);
    if (rc != PASK_OK) return rc;
    if (!k || !v || !tags) return PASK_ERR_INVALID_ARG;
    if (((uintptr_t)k | (uintptr_t)v) & 15) return PASK_ERR_INVALID_ARG;
    rc = attention_common(c, true, layer, n_seqs, seq_ids, q, out, lse, ws, ws_bytes, stream, false, true);
    if (rc != PASK_OK) return rc;
    auto &a = c->ahead[layer];
    if (!a.valid || a.n_seqs != n_seqs || a.area != area) return PASK_ERR_STALE_PLAN;
    NvtxRange range("pask_decode_step_ahead");
    // The streaming kernel may look its range up and start its first copies before its dependency wait only if the
    // plan's writer is surely complete by then: that holds once another planned-ahead call lies between the two in
    // the stream (its streaming kernel lets later kernels start only after it has waited for everything before it).
    const uint64_t call = ++c->ahead_calls;
    rc = launch_step_ahead(c, layer, n_seqs, seq_ids, k, v, tags, actions, actions_out, q, out, lse, ws, area, a.parity,
                           call >= a.early_from, static_cast<cudaStream_t>(stream));
    if (rc != PASK_OK) { a.valid = false; return rc; }
    a.parity ^= 1;                      // the append has left the next step's plan in the other block
    a.early_from = call + 2;
    return PASK_OK;
}

size_t pask_step_staging_bytes(const pask_cache_t *c, int32_t n_seqs) {
    if (!c || n_seqs < 1) return 0;
    const size_t n = (size_t)n_seqs;
    size_t p = 0;
    p += align_up(n * 4, 256);                                    // seq_ids
    p += align_up((n + 1) * 4, 256);                              // cu_tokens
    p += 2 * align_up(n * c->desc.n_kv_heads * kHeadDim * 2, 256);  // k, v
    p += align_up(n, 256);                                        // tags
    p += align_up(n * c->desc.n_q_heads * kHeadDim * 2, 256);     // q
    p += align_up(n * c->desc.n_q_heads * kHeadDim * 4, 256);     // out
    return p;
}

// fills cu_tokens = 0, 1, ..., n on the device (one token per sequence)
__global__ void iota_kernel(int32_t *p, int n) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) p[i] = i;
}

pask_status_t pask_decode_step_host(pask_cache_t *c, int32_t layer, int32_t n_seqs, const int32_t *seq_ids_host,
                                    const void *k_host, const void *v_host, const uint8_t *tags_host,
                                    const void *q_host, float *out_host, void *staging, size_t staging_bytes,
                                    void *ws, size_t ws_bytes, pask_stream_t stream_v) {
    if (!c || !seq_ids_host || !k_host || !v_host || !tags_host || !q_host || !out_host || !staging)
        return PASK_ERR_INVALID_ARG;
    if (n_seqs < 1 || n_seqs > PASK_MAX_SEQS_PER_CALL) return PASK_ERR_INVALID_ARG;
    if (((uintptr_t)staging & 255) || staging_bytes < pask_step_staging_bytes(c, n_seqs)) return PASK_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const size_t n = (size_t)n_seqs;
    const size_t kv_bytes = n * c->desc.n_kv_heads * kHeadDim * 2, q_bytes = n * c->desc.n_q_heads * kHeadDim * 2;
    uint8_t *p = static_cast<uint8_t *>(staging);
    int32_t *d_ids = reinterpret_cast<int32_t *>(p); p += align_up(n * 4, 256);
    int32_t *d_cu = reinterpret_cast<int32_t *>(p); p += align_up((n + 1) * 4, 256);
    void *d_k = p; p += align_up(kv_bytes, 256);
    void *d_v = p; p += align_up(kv_bytes, 256);
    uint8_t *d_tags = p; p += align_up(n, 256);
    void *d_q = p; p += align_up(q_bytes, 256);
    float *d_out = reinterpret_cast<float *>(p);
    cudaError_t e = cudaMemcpyAsync(d_ids, seq_ids_host, n * 4, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_k, k_host, kv_bytes, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_v, v_host, kv_bytes, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_tags, tags_host, n, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_q, q_host, q_bytes, cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) return PASK_ERR_CUDA;
    iota_kernel<<<(n_seqs + 1 + 255) / 256, 256, 0, stream>>>(d_cu, n_seqs + 1);
    if (cudaPeekAtLastError() != cudaSuccess) return PASK_ERR_CUDA;
    pask_status_t rc = pask_append_attend(c, layer, n_seqs, n_seqs, d_ids, d_cu, d_k, d_v, d_tags, nullptr, nullptr, d_q, d_out,
                                          nullptr, ws, ws_bytes, stream_v);
    if (rc != PASK_OK) return rc;
    e = cudaMemcpyAsync(out_host, d_out, n * c->desc.n_q_heads * kHeadDim * 4, cudaMemcpyDeviceToHost, stream);
    return cuda_rc(e);
}

pask_status_t pask_step_packed_layout(const pask_cache_t *c, int32_t n_seqs, size_t offsets[6], size_t *in_bytes) {
    if (!c || n_seqs < 1 || !offsets || !in_bytes) return PASK_ERR_INVALID_ARG;
    const size_t n = (size_t)n_seqs;
    const size_t kv_bytes = n * c->desc.n_kv_heads * kHeadDim * 2, q_bytes = n * c->desc.n_q_heads * kHeadDim * 2;
    size_t p = 0;
    offsets[0] = p; p += align_up(n * 4, 256);          // seq_ids
    offsets[1] = p; p += align_up((n + 1) * 4, 256);    // cu_tokens
    offsets[2] = p; p += align_up(kv_bytes, 256);       // k
    offsets[3] = p; p += align_up(kv_bytes, 256);       // v
    offsets[4] = p; p += align_up(n, 256);              // tags
    offsets[5] = p; p += align_up(q_bytes, 256);        // q
    *in_bytes = p;
    return PASK_OK;
}

pask_status_t pask_decode_step_packed(pask_cache_t *c, int32_t layer, int32_t n_seqs, const void *packed_host,
                                      float *out_host, void *staging, size_t staging_bytes, void *ws, size_t ws_bytes,
                                      pask_stream_t stream_v) {
    if (!c || !packed_host || !out_host || !staging) return PASK_ERR_INVALID_ARG;
    if (n_seqs < 1 || n_seqs > PASK_MAX_SEQS_PER_CALL) return PASK_ERR_INVALID_ARG;
    if (((uintptr_t)staging & 255) || staging_bytes < pask_step_staging_bytes(c, n_seqs)) return PASK_ERR_WORKSPACE;
    size_t off[6], in_bytes = 0;
    pask_step_packed_layout(c, n_seqs, off, &in_bytes);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    uint8_t *p = static_cast<uint8_t *>(staging);
    if (cudaMemcpyAsync(p, packed_host, in_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) return PASK_ERR_CUDA;
    float *d_out = reinterpret_cast<float *>(p + in_bytes);
    pask_status_t rc = pask_append_attend(c, layer, n_seqs, n_seqs, reinterpret_cast<const int32_t *>(p + off[0]),
                                          reinterpret_cast<const int32_t *>(p + off[1]), p + off[2], p + off[3], p + off[4],
                                          nullptr, nullptr, p + off[5], d_out, nullptr, ws, ws_bytes, stream_v);
    if (rc != PASK_OK) return rc;
    return cuda_rc(cudaMemcpyAsync(out_host, d_out, (size_t)n_seqs * c->desc.n_q_heads * kHeadDim * 4, cudaMemcpyDeviceToHost,
                                   stream));
}

static pask_status_t step_pipelined(pask_cache_t *c, int32_t layer, int32_t n_seqs, const void *packed_host,
                                    float *out_host, void *staging, size_t staging_bytes, void *ws, size_t ws_bytes,
                                    void *plan_area, size_t plan_area_bytes, pask_stream_t stream_v) {
    if (!c || !packed_host || !out_host || !staging) return PASK_ERR_INVALID_ARG;
    if (n_seqs < 1 || n_seqs > PASK_MAX_SEQS_PER_CALL) return PASK_ERR_INVALID_ARG;
    const size_t slot_bytes = pask_step_staging_bytes(c, n_seqs);
    // The two slots are the two halves of the staging buffer, whatever the batch: a call's slot never overlaps the
    // other slot of an earlier call with a different n_seqs.
    const size_t slot_stride = (staging_bytes / 2) & ~(size_t)255;
    if (((uintptr_t)staging & 255) || slot_stride < slot_bytes) return PASK_ERR_WORKSPACE;
    auto &pp = c->pipe;
    if (!pp.ready) {   // host-side handles only; no device memory
        bool ok = cudaStreamCreateWithFlags(&pp.in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&pp.out, cudaStreamNonBlocking) == cudaSuccess;
        for (int i = 0; i < 2 && ok; i++)
            ok = cudaEventCreateWithFlags(&pp.ev_in[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&pp.ev_done[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&pp.ev_out[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return PASK_ERR_CUDA;
        pp.ready = true;
        pp.calls = 0;
    }
    size_t off[6], in_bytes = 0;
    pask_step_packed_layout(c, n_seqs, off, &in_bytes);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const int slot = (int)(pp.calls & 1);
    uint8_t *p = static_cast<uint8_t *>(staging) + (size_t)slot * slot_stride;
    float *d_out = reinterpret_cast<float *>(p + in_bytes);
    cudaError_t e = cudaSuccess;
    // A different staging buffer (or size: the halves move) than the call before: the new slot may overlap either of
    // the old ones, so the input copy waits for everything the earlier calls still read or write there.
    const bool moved = pp.calls > 0 && (staging != pp.staging || staging_bytes != pp.staging_bytes);
    pp.staging = staging;
    pp.staging_bytes = staging_bytes;
    // from here on the slot counts as used, whatever happens: the next call takes the other one
    const uint64_t call = pp.calls++;
    if (moved) {
        for (int i = 0; i < 2 && e == cudaSuccess; i++) {
            if (pp.recorded[i] & 1) e = cudaStreamWaitEvent(pp.in, pp.ev_done[i], 0);
            if (e == cudaSuccess && (pp.recorded[i] & 2)) e = cudaStreamWaitEvent(pp.in, pp.ev_out[i], 0);
        }
    }
    // this slot's inputs were last read by the kernels of two calls ago, its output by that call's copy-out
    if (e == cudaSuccess && (pp.recorded[slot] & 1)) e = cudaStreamWaitEvent(pp.in, pp.ev_done[slot], 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(p, packed_host, in_bytes, cudaMemcpyHostToDevice, pp.in);
    if (e == cudaSuccess) e = cudaEventRecord(pp.ev_in[slot], pp.in);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, pp.ev_in[slot], 0);
    if (e == cudaSuccess && (pp.recorded[slot] & 2)) e = cudaStreamWaitEvent(stream, pp.ev_out[slot], 0);
    if (e == cudaSuccess && moved && (pp.recorded[slot ^ 1] & 2)) e = cudaStreamWaitEvent(stream, pp.ev_out[slot ^ 1], 0);
    if (e != cudaSuccess) return PASK_ERR_CUDA;
    (void)call;
    pask_status_t rc = plan_area
        ? pask_decode_step_ahead(c, layer, n_seqs, reinterpret_cast<const int32_t *>(p + off[0]), p + off[2], p + off[3], p + off[4],
                                 nullptr, nullptr, p + off[5], d_out, nullptr, ws, ws_bytes, plan_area, plan_area_bytes, stream_v)
        : pask_append_attend(c, layer, n_seqs, n_seqs, reinterpret_cast<const int32_t *>(p + off[0]),
                             reinterpret_cast<const int32_t *>(p + off[1]), p + off[2], p + off[3], p + off[4],
                             nullptr, nullptr, p + off[5], d_out, nullptr, ws, ws_bytes, stream_v);
    // whatever was enqueued reads this slot: mark its end on the caller's stream even if the step was refused
    e = cudaEventRecord(pp.ev_done[slot], stream);
    if (e == cudaSuccess) pp.recorded[slot] |= 1;
    if (rc != PASK_OK) return rc;
    if (e == cudaSuccess) e = cudaStreamWaitEvent(pp.out, pp.ev_done[slot], 0);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(out_host, d_out, (size_t)n_seqs * c->desc.n_q_heads * kHeadDim * 4, cudaMemcpyDeviceToHost, pp.out);
    if (e == cudaSuccess) e = cudaEventRecord(pp.ev_out[slot], pp.out);
    if (e == cudaSuccess) pp.recorded[slot] |= 2;
    return cuda_rc(e);
}

pask_status_t pask_decode_step_pipelined(pask_cache_t *c, int32_t layer, int32_t n_seqs, const void *packed_host,
                                         float *out_host, void *staging, size_t staging_bytes, void *ws, size_t ws_bytes,
                                         pask_stream_t stream) {
    return step_pipelined(c, layer, n_seqs, packed_host, out_host, staging, staging_bytes, ws, ws_bytes, nullptr, 0, stream);
}

pask_status_t pask_decode_step_pipelined_ahead(pask_cache_t *c, int32_t layer, int32_t n_seqs, const void *packed_host,
                                               float *out_host, void *staging, size_t staging_bytes, void *ws, size_t ws_bytes,
                                               void *plan_area, size_t plan_area_bytes, pask_stream_t stream) {
    if (!plan_area) return PASK_ERR_INVALID_ARG;
    return step_pipelined(c, layer, n_seqs, packed_host, out_host, staging, staging_bytes, ws, ws_bytes, plan_area,
                          plan_area_bytes, stream);
}

pask_status_t pask_decode_step_drain(pask_cache_t *c) {
    if (!c) return PASK_ERR_INVALID_ARG;
    if (!c->pipe.ready) return PASK_OK;
    cudaError_t e = cudaStreamSynchronize(c->pipe.in);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->pipe.out);
    return cuda_rc(e);
}

pask_status_t pask_budget_state(pask_cache_t *c, int32_t seq, pask_budget_state_t *host_out, pask_stream_t stream_v) {
    if (!c || !host_out) return PASK_ERR_INVALID_ARG;
    if (seq < 0 || seq >= c->desc.max_seqs) return PASK_ERR_BAD_SEQ;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    uint32_t status = 0;
    cudaError_t e = cudaMemcpyAsync(host_out, c->dev.budget + seq, sizeof(*host_out), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(&status, c->dev.ctrl + kCtrlStatus, 4, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return PASK_ERR_CUDA;
    host_out->remaining_bytes =
        (int64_t)(((uint64_t)c->dev.budget_q16 * host_out->full_bytes) >> 16) - (int64_t)host_out->retained_bytes;
    host_out->device_status = status;
    host_out->reserved = 0;
    return PASK_OK;
}

pask_status_t pask_cache_set_timing_events(pask_cache_t *c, pask_event_t start, pask_event_t stop) {
    if (!c) return PASK_ERR_INVALID_ARG;
    c->ev_start = static_cast<cudaEvent_t>(start);
    c->ev_stop = static_cast<cudaEvent_t>(stop);
    return PASK_OK;
}

pask_status_t pask_cache_set_timing_span(pask_cache_t *c, void *span_dev) {
    if (!c || ((uintptr_t)span_dev & 7)) return PASK_ERR_INVALID_ARG;
    c->span = static_cast<unsigned long long *>(span_dev);
    return PASK_OK;
}

pask_status_t pask_debug_stream_len(pask_cache_t *c, int32_t layer, int32_t seq, uint32_t *n_high, uint32_t *n_low,
                                    pask_stream_t stream) {
    if (!c || !n_high || !n_low) return PASK_ERR_INVALID_ARG;
    if (!seq_layer_ok(c, layer, seq)) return PASK_ERR_INVALID_ARG;
    return read_lens(c, layer, seq, n_high, n_low, static_cast<cudaStream_t>(stream));
}

pask_status_t pask_debug_pool_state(pask_cache_t *c, uint32_t *out4, pask_stream_t stream) {
    if (!c || !out4) return PASK_ERR_INVALID_ARG;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return PASK_ERR_CUDA;
    return cuda_rc(cudaMemcpy(out4, c->dev.ctrl + kCtrlHighNext, 16, cudaMemcpyDeviceToHost));
}

pask_status_t pask_debug_ctrl_words(pask_cache_t *c, uint32_t *out, int32_t count, pask_stream_t stream) {
    if (!c || !out || count < 1 || count > kCtrlWords) return PASK_ERR_INVALID_ARG;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return PASK_ERR_CUDA;
    return cuda_rc(cudaMemcpy(out, c->dev.ctrl, (size_t)count * 4, cudaMemcpyDeviceToHost));
}

pask_status_t pask_debug_page_ids(pask_cache_t *c, int32_t layer, int32_t seq, uint32_t *high_out, uint32_t *low_out,
                                  pask_stream_t stream) {
    if (!c || !seq_layer_ok(c, layer, seq)) return PASK_ERR_INVALID_ARG;
    uint32_t nh = 0, nl = 0;
    pask_status_t rc = read_lens(c, layer, seq, &nh, &nl, static_cast<cudaStream_t>(stream));
    if (rc != PASK_OK) return rc;
    const size_t tbl = ((size_t)seq * c->desc.n_layers + layer) * c->dev.max_pages;
    const uint32_t ph = (nh + kPageTokens - 1) / kPageTokens, pl = (nl + kPageTokens - 1) / kPageTokens;
    if (high_out && ph && cudaMemcpy(high_out, c->dev.tbl_high + tbl, (size_t)ph * 4, cudaMemcpyDeviceToHost) != cudaSuccess)
        return PASK_ERR_CUDA;
    if (low_out && pl && cudaMemcpy(low_out, c->dev.tbl_low + tbl, (size_t)pl * 4, cudaMemcpyDeviceToHost) != cudaSuccess)
        return PASK_ERR_CUDA;
    return PASK_OK;
}

pask_status_t pask_debug_dump_high(pask_cache_t *c, int32_t layer, int32_t seq, uint16_t *k_out, uint16_t *v_out,
                                   uint32_t *pages_out, pask_stream_t stream) try {
    if (!c || !seq_layer_ok(c, layer, seq)) return PASK_ERR_INVALID_ARG;
    uint32_t nh = 0, nl = 0;
    pask_status_t rc = read_lens(c, layer, seq, &nh, &nl, static_cast<cudaStream_t>(stream));
    if (rc != PASK_OK) return rc;
    const uint32_t n_pages = (nh + kPageTokens - 1) / kPageTokens;
    if (n_pages == 0) return PASK_OK;
    if (!k_out || !v_out || !pages_out) return PASK_ERR_INVALID_ARG;
    const size_t tbl = ((size_t)seq * c->desc.n_layers + layer) * c->dev.max_pages;
    if (cudaMemcpy(pages_out, c->dev.tbl_high + tbl, (size_t)n_pages * 4, cudaMemcpyDeviceToHost) != cudaSuccess)
        return PASK_ERR_CUDA;
    const int n_kv = c->desc.n_kv_heads;
    std::vector<uint8_t> page(c->dev.high_page_bytes);
    for (uint32_t p = 0; p < n_pages; p++) {
        if (pages_out[p] >= c->dev.cap_high) return PASK_ERR_CUDA;
        if (cudaMemcpy(page.data(), c->dev.pool_high + (size_t)pages_out[p] * c->dev.high_page_bytes, page.size(),
                       cudaMemcpyDeviceToHost) != cudaSuccess)
            return PASK_ERR_CUDA;
        for (uint32_t tau = 0; tau < (uint32_t)kPageTokens && p * kPageTokens + tau < nh; tau++) {
            const size_t tok = (size_t)p * kPageTokens + tau;
            for (int h = 0; h < n_kv; h++) {
                const uint8_t *kt = page.data() + (size_t)h * kHighHeadBytes;
                const uint8_t *vt = kt + kHighTileBytes;
                uint16_t *kd = k_out + (tok * n_kv + h) * kHeadDim, *vd = v_out + (tok * n_kv + h) * kHeadDim;
                for (int pr = 0; pr < 64; pr++) std::memcpy(kd + 2 * pr, kt + high_k_pair_off((int)tau, pr), 4);
                for (int q = 0; q < 4; q++)
                    for (int g = 0; g < 8; g++)
                        std::memcpy(vd + 32 * q + 4 * g, vt + high_v_piece_off((int)tau, q, g), 8);
            }
        }
    }
    return PASK_OK;
} catch (...) {   // the staging copy could not be allocated
    return PASK_ERR_NO_MEMORY;
}

pask_status_t pask_debug_dump_low(pask_cache_t *c, int32_t layer, int32_t seq, uint8_t *k_codes, uint16_t *k_scales,
                                  uint8_t *v_codes, uint16_t *v_scales, uint32_t *pages_out, pask_stream_t stream) try {
    if (!c || !seq_layer_ok(c, layer, seq)) return PASK_ERR_INVALID_ARG;
    uint32_t nh = 0, nl = 0;
    pask_status_t rc = read_lens(c, layer, seq, &nh, &nl, static_cast<cudaStream_t>(stream));
    if (rc != PASK_OK) return rc;
    const uint32_t n_pages = (nl + kPageTokens - 1) / kPageTokens;
    if (n_pages == 0) return PASK_OK;
    if (!k_codes || !k_scales || !v_codes || !v_scales || !pages_out) return PASK_ERR_INVALID_ARG;
    const size_t tbl = ((size_t)seq * c->desc.n_layers + layer) * c->dev.max_pages;
    if (cudaMemcpy(pages_out, c->dev.tbl_low + tbl, (size_t)n_pages * 4, cudaMemcpyDeviceToHost) != cudaSuccess)
        return PASK_ERR_CUDA;
    const int n_kv = c->desc.n_kv_heads;
    std::vector<uint8_t> page(c->dev.low_page_bytes);
    for (uint32_t p = 0; p < n_pages; p++) {
        if (pages_out[p] >= c->dev.cap_low) return PASK_ERR_CUDA;
        if (cudaMemcpy(page.data(), c->dev.pool_low + (size_t)pages_out[p] * c->dev.low_page_bytes, page.size(),
                       cudaMemcpyDeviceToHost) != cudaSuccess)
            return PASK_ERR_CUDA;
        for (uint32_t tau = 0; tau < (uint32_t)kPageTokens && p * kPageTokens + tau < nl; tau++) {
            const size_t tok = (size_t)p * kPageTokens + tau;
            for (int h = 0; h < n_kv; h++) {
                const uint8_t *kh = page.data() + (size_t)h * c->dev.low_head_bytes;
                uint8_t *kc = k_codes + (tok * n_kv + h) * kHeadDim, *vc = v_codes + (tok * n_kv + h) * kHeadDim;
                uint16_t *ks = k_scales + (tok * n_kv + h) * kGroupsPerHead;
                uint16_t *vs = v_scales + (tok * n_kv + h) * kGroupsPerHead;
                if (c->dev.low_bits == 8) {
                    const uint8_t *v8 = kh + kLow8HalfBytes;
                    for (int w = 0; w < 4; w++) {
                        std::memcpy(ks + w, kh + low8_scale_off((int)tau, w), 2);
                        std::memcpy(vs + w, v8 + low8_scale_off((int)tau, w), 2);
                    }
                    for (int dd = 0; dd < kHeadDim; dd++) {
                        kc[dd] = kh[low8_k_off((int)tau, dd)];
                        vc[dd] = v8[low8_v_off((int)tau, dd)];
                    }
                    continue;
                }
                if (c->dev.low_bits == 2) {
                    const uint8_t *v2 = kh + kLow2HalfBytes;
                    for (int w = 0; w < 4; w++) {
                        std::memcpy(ks + w, kh + low2_scale_off((int)tau, w), 2);
                        std::memcpy(vs + w, v2 + low2_scale_off((int)tau, w), 2);
                    }
                    for (int dd = 0; dd < kHeadDim; dd++) {
                        kc[dd] = (kh[low2_k_byte_off((int)tau, dd >> 3, dd & 1)] >> (2 * ((dd >> 1) & 3))) & 3;
                        vc[dd] = (v2[low2_v_byte_off((int)tau, dd >> 2)] >> (2 * (dd & 3))) & 3;
                    }
                    continue;
                }
                const uint8_t *vh = kh + kLowHalfBytes;
                for (int w = 0; w < 4; w++) {
                    std::memcpy(ks + w, kh + low_scale_off((int)tau, w), 2);
                    std::memcpy(vs + w, vh + low_scale_off((int)tau, w), 2);
                    for (int t = 0; t < 4; t++) {
                        uint32_t word;
                        std::memcpy(&word, kh + low_k_word_off((int)tau, w, t), 4);
                        for (int e = 0; e < 8; e++) kc[32 * w + 8 * t + e] = (word >> (4 * low_k_nibble(e))) & 0xF;
                    }
                    for (int g = 0; g < 8; g++) {
                        uint16_t half;
                        std::memcpy(&half, vh + low_v_half_off((int)tau, w, g), 2);
                        for (int i = 0; i < 4; i++) vc[32 * w + 4 * g + i] = (half >> (4 * i)) & 0xF;
                    }
                }
            }
        }
    }
    return PASK_OK;
} catch (...) {   // the staging copy could not be allocated
    return PASK_ERR_NO_MEMORY;
}

pask_status_t pask_debug_set_attention_ctas(pask_cache_t *c, int32_t n_ctas) {
    if (!c || n_ctas < 1 || n_ctas > 65536) return PASK_ERR_INVALID_ARG;
    c->attn_ctas = n_ctas;
    c->dev.attn_ctas = (uint32_t)n_ctas;
    return PASK_OK;
}

pask_status_t pask_debug_plan_order_span(const pask_cache_t *c, int32_t n_seqs, int32_t layer, int32_t parity, size_t *offset,
                                         size_t *bytes) {
    if (!c || !offset || !bytes || n_seqs < 1 || n_seqs > 255 || layer < 0 || layer >= c->desc.n_layers || (parity & ~1))
        return PASK_ERR_INVALID_ARG;
    PlanBlock pb;
    uint8_t origin = 0;                                             // any base will do: only the distance from it is used
    carve_plan_area(c, n_seqs, layer, parity, &origin, &pb);
    *offset = (size_t)(reinterpret_cast<const uint8_t *>(pb.order) - &origin);
    *bytes = (size_t)n_seqs * (2 * (size_t)c->dev.max_pages + c->dev.window / kPageTokens) * 4;
    return PASK_OK;
}

pask_status_t pask_debug_set_wait(pask_cache_t *c, int64_t limit_cycles, uint32_t surplus_bytes) {
    if (!c || limit_cycles < 1000 || surplus_bytes > 65536u || (surplus_bytes & 15u)) return PASK_ERR_INVALID_ARG;
    c->wait_cycles = limit_cycles;
    c->wait_test_surplus = surplus_bytes;
    return PASK_OK;
}

pask_status_t pask_debug_partition(int32_t n_seqs, const uint32_t *pages_high, const uint32_t *pages_low,
                                   int32_t n_ctas, uint32_t *ranges) try {
    if (n_seqs < 1 || n_ctas < 1 || !pages_high || !pages_low || !ranges) return PASK_ERR_INVALID_ARG;
    std::vector<uint64_t> prefix((size_t)n_seqs + 1, 0);
    for (int s = 0; s < n_seqs; s++)
        prefix[s + 1] = prefix[s] + (uint64_t)pages_high[s] * kCostHighPage + (uint64_t)pages_low[s] * kCostLowPage;
    if (prefix[n_seqs] <= 0xffffffffull) {      // a small batch: whole CTAs per sequence, as the plan kernels cut it
        std::vector<uint32_t> snapped(prefix.begin(), prefix.end());
        snap_cost_prefix(snapped.data(), n_seqs, (uint32_t)n_ctas);
        for (int s = 0; s <= n_seqs; s++) prefix[s] = snapped[s];
    }
    const uint64_t total = prefix[n_seqs];
    for (int b = 0; b < n_ctas; b++) {
        const uint64_t lo = total * b / n_ctas, hi = total * (b + 1) / n_ctas;
        for (int s = 0; s < n_seqs; s++) {
            uint32_t *r = ranges + ((size_t)b * n_seqs + s) * 2;
            r[0] = r[1] = 0;
            if (prefix[s + 1] <= lo || prefix[s] >= hi || prefix[s + 1] == prefix[s]) continue;
            const uint32_t cs = (uint32_t)(prefix[s + 1] - prefix[s]), n = pages_high[s] + pages_low[s];
            const uint32_t a = (uint32_t)((lo > prefix[s] ? lo : prefix[s]) - prefix[s]);
            const uint32_t e = (uint32_t)((hi < prefix[s + 1] ? hi : prefix[s + 1]) - prefix[s]);
            r[0] = cut_positions(a, cs, n);
            r[1] = cut_positions(e, cs, n);
        }
    }
    return PASK_OK;
} catch (...) {   // the staging copy could not be allocated
    return PASK_ERR_NO_MEMORY;
}

pask_status_t pask_debug_page_order(uint32_t pages_high, uint32_t pages_low, uint32_t *order) {
    if (!order && pages_high + pages_low > 0) return PASK_ERR_INVALID_ARG;
    for (uint32_t v = 0; v < pages_high + pages_low; v++) {
        uint32_t idx;
        order[v] = page_at(v, pages_high, pages_low, idx) ? (idx | kOrderHigh) : idx;
    }
    return PASK_OK;
}

}  // extern "C"
