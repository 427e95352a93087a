// Host side of the C ABI: context, workspace carve-up, per-request state machine, slot allocation and
// kernel dispatch.  No device memory is allocated here; every launch goes to the caller's stream.
#include <algorithm>
#include <cstdint>
#include <new>
#include <vector>

#include "onela_internal.h"

using namespace onela;

namespace {

constexpr size_t kAlign = 1024;
size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct ReqState {
    int32_t depth = 0;  // decode calls opened so far (reorder_beams calls since the last restart)
    int32_t W = 0;      // beam width of the current call
    std::vector<uint8_t> has_state;      // per layer: S_0 stored
    std::vector<int32_t> appended_depth; // per layer: depth at which records were last appended
    std::vector<int32_t> step_base;      // per decode call: first slot
    std::vector<int32_t> step_width;     // per decode call: beam width
};

bool config_sane(const onela_config* c) {
    if (!c) return false;
    if (c->num_requests < 1 || c->num_layers < 1 || c->num_heads < 1) return false;
    if (c->dk < 1 || c->dv < 1 || c->max_beam < 1 || c->max_steps < 1) return false;
    if ((c->rec_dtype != ONELA_DTYPE_F32 && c->rec_dtype != ONELA_DTYPE_BF16) ||
        (c->out_dtype != ONELA_DTYPE_F32 && c->out_dtype != ONELA_DTYPE_BF16))
        return false;
    if (c->arena_slots < 1 || c->arena_slots > 0x7fffffffLL - c->max_beam) return false;
    if (c->num_v_heads < 0 || (c->num_v_heads > 0 && c->num_v_heads % c->num_heads != 0)) return false;
    const int es = c->rec_dtype == ONELA_DTYPE_BF16 ? 2 : 4;
    if ((c->dk * es) % 16 != 0 || (c->dv * es) % 16 != 0) return false;  // 16-byte vector rows
    return true;
}

// Whether decode_step of this configuration runs the tiled tcgen05 kernel (the other shapes from 64 x 64 up).
bool uses_tiled_kernel(const onela_config& c) {
    const bool forced = c.flags & ONELA_FLAG_FORCE_GENERIC;
    if (forced || decode_sm100_supported(c.dk, c.dv, c.rec_dtype)) return false;
    return decode_tiled_supported(c.dk, c.dv) && (!(c.flags & ONELA_FLAG_GTR_DELTA) || c.dk == c.dv);   // delta records: square heads
}

// Carve the workspace.  `base` may be null (size query only).
Layout carve(const onela_config& c, char* base) {
    const size_t es = c.rec_dtype == ONELA_DTYPE_BF16 ? 2 : 4;
    const size_t Hv = c.num_v_heads > 0 ? c.num_v_heads : c.num_heads;   // value heads
    size_t off = 0;
    Layout l{};
    auto take = [&](size_t bytes) {
        char* p = base ? base + off : nullptr;
        off += align_up(bytes);
        return p;
    };
    l.status = reinterpret_cast<int32_t*>(take(4 * sizeof(int32_t)));
    l.tables = reinterpret_cast<int32_t*>(take((size_t)c.num_requests * 2 * c.max_steps * c.max_beam * sizeof(int32_t)));
    l.sidx = reinterpret_cast<int32_t*>(take((size_t)c.num_requests * c.max_steps * c.max_beam * sizeof(int32_t)));
    l.ulist = reinterpret_cast<int32_t*>(take((size_t)c.num_requests * c.max_steps * c.max_beam * sizeof(int32_t)));
    l.uoff = reinterpret_cast<int32_t*>(take((size_t)c.num_requests * (c.max_steps + 1) * sizeof(int32_t)));
    l.s0 = reinterpret_cast<float*>(take((size_t)c.num_requests * c.num_layers * Hv * c.dv * c.dk * sizeof(float)));
    l.gates = reinterpret_cast<float2*>(take((size_t)c.num_layers * Hv * (size_t)c.arena_slots * sizeof(float2)));
    if (Hv == (size_t)c.num_heads) {
        l.kv = take((size_t)c.num_layers * c.num_heads * (size_t)c.arena_slots * (c.dk + c.dv) * es);
    } else {   // grouped value heads: keys per key head, values per value head
        l.kv = take((size_t)c.num_layers * c.num_heads * (size_t)c.arena_slots * c.dk * es);
        l.vv = take((size_t)c.num_layers * Hv * (size_t)c.arena_slots * c.dv * es);
    }
    l.select_scratch = reinterpret_cast<unsigned long long*>(
        take((size_t)c.num_requests * ONELA_SELECT_PARTS * ONELA_SELECT_CAP * sizeof(unsigned long long)));
    l.s0_scale = reinterpret_cast<float*>(take((size_t)c.num_requests * c.num_layers * Hv * sizeof(float)));
    l.urep = reinterpret_cast<int32_t*>(take((size_t)c.num_requests * c.max_steps * c.max_beam * sizeof(int32_t)));
    l.sg8 = reinterpret_cast<uint8_t*>(take((size_t)c.num_requests * c.max_steps * sg_row_stride(c.max_beam)));
    l.unode = reinterpret_cast<uint8_t*>(take((size_t)c.num_requests * ONELA_UNODE_CAP * 16));
    if (uses_tiled_kernel(c))
        l.s0_f16 = reinterpret_cast<uint16_t*>(take((size_t)c.num_requests * c.num_layers * Hv * s0_f16_head_bytes(c.dk, c.dv)));
    l.total_bytes = off;
    return l;
}

}  // namespace

struct onela_ctx {
    onela_config cfg;
    Layout lay;
    std::vector<ReqState> req;
    int64_t cursor = 0;        // next free arena slot
    int64_t launches = 0;
    int64_t decode_mark = -1;  // value of `launches` right after the last decode launch
    bool status_cleared = false;
    bool tensor_core = false;  // decode_step runs the warp-specialised tcgen05 kernel
    bool tiled_tc = false;     // decode_step runs the tiled tcgen05 kernel (the other shapes from 64 x 64 up)
    int32_t elem_bytes = 4;

    bool dry() const { return cfg.flags & ONELA_FLAG_DRY_RUN; }
    bool gtr() const { return cfg.flags & ONELA_FLAG_GTR_DELTA; }   // (alpha, delta, k) records, forward replay
    int32_t Hv() const { return cfg.num_v_heads > 0 ? cfg.num_v_heads : cfg.num_heads; }   // value heads
    bool grouped() const { return Hv() != cfg.num_heads; }
    char* k_plane(int l) const { return lay.kv + (size_t)l * cfg.num_heads * (size_t)cfg.arena_slots * cfg.dk * elem_bytes; }
    char* v_plane(int l) const { return lay.vv + (size_t)l * Hv() * (size_t)cfg.arena_slots * cfg.dv * elem_bytes; }
    long long table_req_stride() const { return 2LL * cfg.max_steps * cfg.max_beam; }
    long long s0_layer_floats() const { return (long long)Hv() * cfg.dv * cfg.dk; }
    float* s0_slot(int r, int l) const { return lay.s0 + ((long long)r * cfg.num_layers + l) * s0_layer_floats(); }
    float* s0_scale_slot(int r, int l) const { return lay.s0_scale + ((long long)r * cfg.num_layers + l) * Hv(); }
    uint16_t* s0_f16_slot(int r, int l) const {       // tiled kernel's operand copy of (request, layer, head 0)
        return lay.s0_f16 + ((long long)r * cfg.num_layers + l) * Hv() * (long long)(s0_f16_head_bytes(cfg.dk, cfg.dv) / 2);
    }
    // after a state write: the tiled kernel's operand copy of the n_heads states from (r, l) on
    cudaError_t pack_states(int r, int l, long long n_heads, cudaStream_t s) {
        if (!tiled_tc) return cudaSuccess;
        launches++;
        return launch_pack_state(s0_slot(r, l), s0_scale_slot(r, l), s0_f16_slot(r, l), n_heads, cfg.dk, cfg.dv, s);
    }
    int32_t* table_cur(int r) const {
        const int d = req[r].depth;
        return lay.tables + r * table_req_stride() + (long long)((d - 1) & 1) * cfg.max_steps * cfg.max_beam;
    }
    long long sidx_req_stride() const { return (long long)cfg.max_steps * cfg.max_beam; }
    long long uoff_req_stride() const { return cfg.max_steps + 1; }
    long long sg8_req_stride() const { return (long long)cfg.max_steps * sg_row_stride(cfg.max_beam); }
    size_t plane_rows() const { return (size_t)cfg.num_heads * (size_t)cfg.arena_slots; }
    char* kv_plane(int l) const { return lay.kv + (size_t)l * plane_rows() * (cfg.dk + cfg.dv) * elem_bytes; }
    float2* gate_plane(int l) const { return lay.gates + (size_t)l * Hv() * (size_t)cfg.arena_slots; }

    onela_status prepare(cudaStream_t s) {
        if (dry() || status_cleared) return ONELA_OK;
        if (cudaMemsetAsync(lay.status, 0, 4 * sizeof(int32_t), s) != cudaSuccess) return ONELA_E_CUDA;
        status_cleared = true;
        return ONELA_OK;
    }
    // Slots given back by onela_release_request: (first slot, count), ascending, neighbours merged; a range that
    // ends at the cursor lowers the cursor instead.  Allocation takes the lowest range that fits, else the cursor.
    std::vector<std::pair<int64_t, int64_t>> free_ranges;
    int64_t free_slots() const {
        int64_t n = 0;
        for (const auto& f : free_ranges) n += f.second;
        return n;
    }
    static int64_t take_slots(std::vector<std::pair<int64_t, int64_t>>& ranges, int64_t& cur, int64_t limit, int64_t n) {
        for (size_t i = 0; i < ranges.size(); ++i) {
            if (ranges[i].second >= n) {
                const int64_t at = ranges[i].first;
                ranges[i].first += n;
                ranges[i].second -= n;
                if (ranges[i].second == 0) ranges.erase(ranges.begin() + (long)i);
                return at;
            }
        }
        if (cur + n > limit) return -1;
        const int64_t at = cur;
        cur += n;
        return at;
    }
    void give_back(int64_t first, int64_t n) {
        if (n <= 0) return;
        auto it = free_ranges.begin();
        while (it != free_ranges.end() && it->first < first) ++it;
        it = free_ranges.insert(it, {first, n});
        if (it + 1 != free_ranges.end() && it->first + it->second == (it + 1)->first) {   // merge with the next range
            it->second += (it + 1)->second;
            free_ranges.erase(it + 1);
        }
        if (it != free_ranges.begin() && (it - 1)->first + (it - 1)->second == it->first) {   // and with the one before
            (it - 1)->second += it->second;
            it = free_ranges.erase(it) - 1;
        }
        if (!free_ranges.empty() && free_ranges.back().first + free_ranges.back().second == cursor) {
            cursor = free_ranges.back().first;
            free_ranges.pop_back();
        }
    }
    void restart(ReqState& r) {
        r.depth = 0;
        r.W = 0;
        std::fill(r.appended_depth.begin(), r.appended_depth.end(), -1);
        r.step_base.clear();
        r.step_width.clear();
    }
};

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// Requests of a batched call must exist and share beam width and depth.
onela_status check_batch(const onela_ctx* ctx, int32_t req_begin, int32_t req_count) {
    if (!ctx) return ONELA_E_INVAL;
    if (req_count < 1 || req_count > ONELA_MAX_BATCH || req_begin < 0 ||
        (int64_t)req_begin + req_count > ctx->cfg.num_requests)
        return ONELA_E_INVAL;
    const ReqState& r0 = ctx->req[req_begin];
    for (int i = 1; i < req_count; ++i) {
        const ReqState& r = ctx->req[req_begin + i];
        if (r.depth != r0.depth || r.W != r0.W) return ONELA_E_INVAL;
    }
    return ONELA_OK;
}

onela_status begin_state_write(onela_ctx* ctx, int32_t request, int32_t layer) {
    if (!ctx || request < 0 || request >= ctx->cfg.num_requests || layer < 0 || layer >= ctx->cfg.num_layers)
        return ONELA_E_INVAL;
    return ONELA_OK;
}

void finish_state_write(onela_ctx* ctx, int32_t request, int32_t layer) {
    ReqState& r = ctx->req[request];
    if (r.depth > 0) {  // a new prompt in this request slot: forget the old beams and every layer's state
        ctx->restart(r);
        std::fill(r.has_state.begin(), r.has_state.end(), 0);
    }
    r.has_state[layer] = 1;
}

}  // namespace

extern "C" {

size_t onela_workspace_bytes(const onela_config* cfg) {
    if (!config_sane(cfg)) return 0;
    return carve(*cfg, nullptr).total_bytes;
}

onela_status onela_create(const onela_config* cfg, void* workspace_dev, size_t workspace_bytes, onela_ctx** out) {
    if (!out) return ONELA_E_INVAL;
    *out = nullptr;
    if (!config_sane(cfg) || !workspace_dev) return ONELA_E_INVAL;
    if (reinterpret_cast<uintptr_t>(workspace_dev) % kAlign != 0) return ONELA_E_INVAL;
    if (!decode_generic_supported(cfg->dk, cfg->dv, cfg->rec_dtype)) return ONELA_E_UNSUPPORTED;
    if ((cfg->flags & ONELA_FLAG_GTR_DELTA) && !(cfg->dk == cfg->dv && (cfg->dk == 32 || cfg->dk == 64 || cfg->dk == 128)))
        return ONELA_E_UNSUPPORTED;
    const bool grouped_cfg = cfg->num_v_heads > 0 && cfg->num_v_heads != cfg->num_heads;
    if (grouped_cfg && (!decode_grouped_supported(cfg->dk, cfg->dv) || (cfg->flags & ONELA_FLAG_GTR_DELTA)))
        return ONELA_E_UNSUPPORTED;
    const Layout lay = carve(*cfg, static_cast<char*>(workspace_dev));
    if (workspace_bytes < lay.total_bytes) return ONELA_E_CAPACITY;
    onela_ctx* ctx = new (std::nothrow) onela_ctx();
    if (!ctx) return ONELA_E_INVAL;
    ctx->cfg = *cfg;
    ctx->lay = lay;
    ctx->elem_bytes = cfg->rec_dtype == ONELA_DTYPE_BF16 ? 2 : 4;
    ctx->req.resize(cfg->num_requests);
    for (auto& r : ctx->req) {
        r.has_state.assign(cfg->num_layers, 0);
        r.appended_depth.assign(cfg->num_layers, -1);
    }
    ctx->tensor_core = decode_sm100_supported(cfg->dk, cfg->dv, cfg->rec_dtype) && !(cfg->flags & ONELA_FLAG_FORCE_GENERIC);
    ctx->tiled_tc = uses_tiled_kernel(*cfg);
    *out = ctx;
    return ONELA_OK;
}

onela_status onela_destroy(onela_ctx* ctx) {
    delete ctx;
    return ONELA_OK;
}

onela_status onela_reset(onela_ctx* ctx, void* stream) {
    if (!ctx) return ONELA_E_INVAL;
    for (auto& r : ctx->req) {
        ctx->restart(r);
        std::fill(r.has_state.begin(), r.has_state.end(), 0);
    }
    ctx->cursor = 0;
    ctx->free_ranges.clear();
    ctx->status_cleared = false;
    return ctx->prepare(static_cast<cudaStream_t>(stream));
}

onela_status onela_init_shared_state(onela_ctx* ctx, int32_t request, int32_t layer, const float* S0_dev,
                                     void* stream) {
    onela_status st = begin_state_write(ctx, request, layer);
    if (st != ONELA_OK) return st;
    if (!S0_dev || !aligned16(S0_dev)) return ONELA_E_INVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if ((st = ctx->prepare(s)) != ONELA_OK) return st;
    if (!ctx->dry()) {
        if (launch_store_state(S0_dev, ctx->s0_slot(request, layer), ctx->s0_scale_slot(request, layer), ctx->Hv(),
                               ctx->cfg.dk, ctx->cfg.dv, s) != cudaSuccess)
            return ONELA_E_CUDA;
        ctx->launches++;
        if (ctx->pack_states(request, layer, ctx->Hv(), s) != cudaSuccess) return ONELA_E_CUDA;
    }
    finish_state_write(ctx, request, layer);
    return ONELA_OK;
}

onela_status onela_init_shared_states(onela_ctx* ctx, int32_t req_begin, int32_t req_count, const float* S0_dev,
                                      void* stream) {
    if (!ctx || req_begin < 0 || req_count <= 0 || req_begin > ctx->cfg.num_requests - req_count) return ONELA_E_INVAL;
    if (!S0_dev || !aligned16(S0_dev)) return ONELA_E_INVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    onela_status st = ctx->prepare(s);
    if (st != ONELA_OK) return st;
    if (!ctx->dry()) {
        // the store keeps a request's layers next to each other and the requests in order: one contiguous range
        if (launch_store_state(S0_dev, ctx->s0_slot(req_begin, 0), ctx->s0_scale_slot(req_begin, 0),
                               (long long)req_count * ctx->cfg.num_layers * ctx->Hv(), ctx->cfg.dk, ctx->cfg.dv,
                               s) != cudaSuccess)
            return ONELA_E_CUDA;
        ctx->launches++;
        if (ctx->pack_states(req_begin, 0, (long long)req_count * ctx->cfg.num_layers * ctx->Hv(), s) != cudaSuccess) return ONELA_E_CUDA;
    }
    for (int32_t r = req_begin; r < req_begin + req_count; ++r)
        for (int32_t l = 0; l < ctx->cfg.num_layers; ++l) finish_state_write(ctx, r, l);
    return ONELA_OK;
}

onela_status onela_prefill_shared_state(onela_ctx* ctx, int32_t request, int32_t layer, const void* k_dev,
                                        const void* v_dev, const float* alpha_dev, const float* beta_dev,
                                        int32_t n_tokens, void* stream) {
    onela_status st = begin_state_write(ctx, request, layer);
    if (st != ONELA_OK) return st;
    if (ctx->grouped()) return ONELA_E_UNSUPPORTED;   // grouped value heads: the state comes through init_shared_state
    if (n_tokens < 0) return ONELA_E_INVAL;
    if (n_tokens > 0 && (!k_dev || !v_dev || !alpha_dev || !beta_dev || !aligned16(k_dev) || !aligned16(v_dev)))
        return ONELA_E_INVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if ((st = ctx->prepare(s)) != ONELA_OK) return st;
    if (!ctx->dry()) {
        bool supported = true;
        const cudaError_t e = launch_prefill(k_dev, v_dev, alpha_dev, beta_dev, ctx->s0_slot(request, layer),
                                             ctx->s0_scale_slot(request, layer), n_tokens, ctx->cfg.num_heads, ctx->cfg.dk,
                                             ctx->cfg.dv, ctx->cfg.rec_dtype, &supported, s);
        if (!supported) return ONELA_E_UNSUPPORTED;
        if (e != cudaSuccess) return ONELA_E_CUDA;
        ctx->launches++;
        if (ctx->pack_states(request, layer, ctx->Hv(), s) != cudaSuccess) return ONELA_E_CUDA;
    }
    finish_state_write(ctx, request, layer);
    return ONELA_OK;
}

onela_status onela_export_shared_state(onela_ctx* ctx, int32_t request, int32_t layer, float* S0_out_dev,
                                       void* stream) {
    onela_status st = begin_state_write(ctx, request, layer);
    if (st != ONELA_OK) return st;
    if (!S0_out_dev || !aligned16(S0_out_dev)) return ONELA_E_INVAL;
    if (!ctx->req[request].has_state[layer]) return ONELA_E_ORDER;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if ((st = ctx->prepare(s)) != ONELA_OK) return st;
    if (ctx->dry()) return ONELA_OK;
    if (launch_export_state(ctx->s0_slot(request, layer), S0_out_dev, ctx->Hv(), ctx->cfg.dk, ctx->cfg.dv,
                            s) != cudaSuccess)
        return ONELA_E_CUDA;
    ctx->launches++;
    return ONELA_OK;
}

onela_status onela_reorder_beams(onela_ctx* ctx, int32_t req_begin, int32_t req_count, const int32_t* parents_dev,
                                 int32_t W_new, void* stream) {
    onela_status st = check_batch(ctx, req_begin, req_count);
    if (st != ONELA_OK) return st;
    const onela_config& c = ctx->cfg;
    if (W_new < 1) return ONELA_E_INVAL;
    if (W_new > c.max_beam) return ONELA_E_CAPACITY;
    const int32_t depth_old = ctx->req[req_begin].depth, W_prev = ctx->req[req_begin].W;
    if ((depth_old == 0) != (parents_dev == nullptr)) return ONELA_E_ORDER;
    for (int i = 0; i < req_count; ++i) {
        const ReqState& r = ctx->req[req_begin + i];
        bool any_state = false;
        for (uint8_t hs : r.has_state) any_state |= hs != 0;
        if (!any_state) return ONELA_E_ORDER;  // no shared state stored for this request yet
        // the previous call must have appended its records in every layer that holds a state
        if (depth_old > 0)
            for (int l = 0; l < c.num_layers; ++l)
                if (r.has_state[l] && r.appended_depth[l] != depth_old) return ONELA_E_ORDER;
    }
    if (depth_old >= c.max_steps) return ONELA_E_CAPACITY;
    // slots of this call's records, request by request: the lowest released range that fits, else the bump cursor
    // (with nothing released this is base(req, t) = cursor, cursor += W_new in request order)
    auto ranges = ctx->free_ranges;
    int64_t cur = ctx->cursor;
    BatchBases bases{};
    for (int i = 0; i < req_count; ++i) {
        const int64_t at = onela_ctx::take_slots(ranges, cur, c.arena_slots, W_new);
        if (at < 0) return ONELA_E_CAPACITY;          // nothing has been changed yet
        bases.base[i] = (int32_t)at;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if ((st = ctx->prepare(s)) != ONELA_OK) return st;
    if (!ctx->dry()) {
        if (launch_reorder(ctx->lay.tables + req_begin * ctx->table_req_stride(), ctx->table_req_stride(), req_count,
                           parents_dev, W_new, W_prev, depth_old, c.max_beam, c.max_steps, bases, ctx->lay.status,
                           s) != cudaSuccess)
            return ONELA_E_CUDA;
        ctx->launches++;
    }
    if (!ctx->dry() && ctx->tensor_core && depth_old >= 1) {
        // distinct-record index of the table just written (buffer depth_old & 1), for the decode kernel's
        // shared-ancestor staging
        const int32_t* cur = ctx->lay.tables + req_begin * ctx->table_req_stride() +
                             (long long)(depth_old & 1) * c.max_steps * c.max_beam;
        if (launch_dedupe(cur, ctx->table_req_stride(), ctx->lay.sidx + req_begin * ctx->sidx_req_stride(),
                          ctx->sidx_req_stride(), ctx->lay.ulist + req_begin * ctx->sidx_req_stride(),
                          ctx->sidx_req_stride(), ctx->lay.urep + req_begin * ctx->sidx_req_stride(),
                          ctx->lay.uoff + req_begin * ctx->uoff_req_stride(),
                          ctx->uoff_req_stride(), ctx->lay.sg8 + req_begin * ctx->sg8_req_stride(), ctx->sg8_req_stride(),
                          sg_row_stride(c.max_beam), ctx->lay.unode + (size_t)req_begin * ONELA_UNODE_CAP * 16, req_count, W_new,
                          depth_old + 1, c.max_beam, s) != cudaSuccess)
            return ONELA_E_CUDA;
        ctx->launches++;
    }
    for (int i = 0; i < req_count; ++i) {
        ReqState& r = ctx->req[req_begin + i];
        r.depth = depth_old + 1;
        r.W = W_new;
        r.step_base.push_back(bases.base[i]);
        r.step_width.push_back(W_new);
    }
    ctx->free_ranges.swap(ranges);
    ctx->cursor = cur;
    return ONELA_OK;
}

onela_status onela_release_request(onela_ctx* ctx, int32_t request) {
    if (!ctx || request < 0 || request >= ctx->cfg.num_requests) return ONELA_E_INVAL;
    ReqState& r = ctx->req[request];
    for (size_t t = 0; t < r.step_base.size(); ++t) ctx->give_back(r.step_base[t], r.step_width[t]);
    ctx->restart(r);
    std::fill(r.has_state.begin(), r.has_state.end(), 0);
    return ONELA_OK;
}

onela_status onela_select_beams(onela_ctx* ctx, int32_t req_begin, int32_t req_count, const float* beam_scores_dev,
                                const float* cand_logp_dev, int32_t C, int32_t W_new, int32_t* parents_out_dev,
                                int32_t* codes_out_dev, float* scores_out_dev, void* stream) {
    onela_status st = check_batch(ctx, req_begin, req_count);
    if (st != ONELA_OK) return st;
    if (!beam_scores_dev || !cand_logp_dev || !parents_out_dev || !codes_out_dev || !scores_out_dev || C < 1 || W_new < 1)
        return ONELA_E_INVAL;
    const ReqState& r0 = ctx->req[req_begin];
    const int64_t W_prev = r0.depth >= 1 ? r0.W : 1;
    if (W_prev * C > (int64_t)ONELA_SELECT_PARTS * 4096) return ONELA_E_CAPACITY;
    if (W_new > ONELA_SELECT_CAP || W_new > W_prev * C) return ONELA_E_CAPACITY;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if ((st = ctx->prepare(s)) != ONELA_OK) return st;
    if (ctx->dry()) return ONELA_OK;
    if (launch_select(beam_scores_dev, cand_logp_dev, req_count, (int32_t)W_prev, C, W_new,
                      ctx->lay.select_scratch + (size_t)req_begin * ONELA_SELECT_PARTS * ONELA_SELECT_CAP, parents_out_dev,
                      codes_out_dev, scores_out_dev, s) != cudaSuccess)
        return ONELA_E_CUDA;
    ctx->launches += (W_prev * C > 4096) ? 2 : 1;
    return ONELA_OK;
}

onela_status onela_append_records(onela_ctx* ctx, int32_t req_begin, int32_t req_count, int32_t layer,
                                  const void* k_dev, const void* v_dev, const float* alpha_dev,
                                  const float* beta_dev, void* stream) {
    onela_status st = check_batch(ctx, req_begin, req_count);
    if (st != ONELA_OK) return st;
    if (ctx->gtr()) return ONELA_E_UNSUPPORTED;   // delta records are produced by append_decode_step only
    const onela_config& c = ctx->cfg;
    if (layer < 0 || layer >= c.num_layers) return ONELA_E_INVAL;
    if (!k_dev || !v_dev || !alpha_dev || !beta_dev || !aligned16(k_dev) || !aligned16(v_dev)) return ONELA_E_INVAL;
    const int32_t depth = ctx->req[req_begin].depth, W = ctx->req[req_begin].W;
    if (depth < 1) return ONELA_E_ORDER;
    for (int i = 0; i < req_count; ++i) {
        const ReqState& r = ctx->req[req_begin + i];
        if (!r.has_state[layer] || r.appended_depth[layer] == depth) return ONELA_E_ORDER;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if ((st = ctx->prepare(s)) != ONELA_OK) return st;
    BatchBases bases{};
    for (int i = 0; i < req_count; ++i) bases.base[i] = ctx->req[req_begin + i].step_base.back();
    if (!ctx->dry()) {
        const cudaError_t e =
            ctx->grouped() ? launch_append_grouped(k_dev, v_dev, alpha_dev, beta_dev, ctx->k_plane(layer), ctx->v_plane(layer),
                                                   ctx->gate_plane(layer), c.arena_slots, req_count, W, c.num_heads,
                                                   ctx->Hv() / c.num_heads, c.dk, c.dv, ctx->elem_bytes, bases, s)
                           : launch_append(k_dev, v_dev, alpha_dev, beta_dev, ctx->kv_plane(layer), ctx->gate_plane(layer),
                                           c.arena_slots, req_count, W, c.num_heads, c.dk, c.dv, ctx->elem_bytes, bases, s);
        if (e != cudaSuccess) return ONELA_E_CUDA;
        ctx->launches++;
    }
    for (int i = 0; i < req_count; ++i) ctx->req[req_begin + i].appended_depth[layer] = depth;
    return ONELA_OK;
}

}  // extern "C"

namespace {

// Shared by decode_step and append_decode_step: fill the kernel arguments and launch.
onela_status launch_decode(onela_ctx* ctx, int32_t req_begin, int32_t req_count, int32_t layer, const void* q_dev,
                           void* out_dev, const void* k_dev, const void* v_dev, const float* alpha_dev,
                           const float* beta_dev, cudaStream_t s) {
    const onela_config& c = ctx->cfg;
    const int32_t depth = ctx->req[req_begin].depth, W = ctx->req[req_begin].W;
    if (ctx->tiled_tc) {
        TiledArgs ta{};
        ta.q = q_dev;
        ta.out = out_dev;
        ta.k_in = k_dev;
        ta.v_in = v_dev;
        ta.alpha_in = alpha_dev;
        ta.beta_in = beta_dev;
        ta.s0 = ctx->s0_slot(req_begin, layer);
        ta.s0_scale = ctx->s0_scale_slot(req_begin, layer);
        ta.s0_f16 = reinterpret_cast<const char*>(ctx->s0_f16_slot(req_begin, layer));
        ta.s0_f16_req_stride = (long long)c.num_layers * ctx->Hv() * (long long)s0_f16_head_bytes(c.dk, c.dv);
        if (ctx->grouped()) {
            ta.kplane = ctx->k_plane(layer);
            ta.vplane = ctx->v_plane(layer);
            ta.k_stride = c.dk;
            ta.v_stride = c.dv;
        } else {      // one plane of k | v rows
            ta.kplane = ctx->kv_plane(layer);
            ta.vplane = ctx->kv_plane(layer) + (size_t)c.dk * ctx->elem_bytes;
            ta.k_stride = ta.v_stride = c.dk + c.dv;
        }
        ta.gates = ctx->gate_plane(layer);
        ta.table = ctx->table_cur(req_begin);
        ta.status = ctx->lay.status;
        ta.s0_req_stride = (long long)c.num_layers * ctx->s0_layer_floats();
        ta.s0_scale_req_stride = (long long)c.num_layers * ctx->Hv();
        ta.table_req_stride = ctx->table_req_stride();
        ta.arena_slots = c.arena_slots;
        ta.req_count = req_count;
        ta.W = W;
        ta.Hk = c.num_heads;
        ta.g = ctx->Hv() / c.num_heads;
        ta.depth = depth;
        ta.max_beam = c.max_beam;
        ta.delta = ctx->gtr() ? 1 : 0;
        for (int i = 0; i < req_count; ++i) ta.bases.base[i] = ctx->req[req_begin + i].step_base.back();
        if (launch_decode_tiled(ta, c.dk, c.dv, c.rec_dtype, c.out_dtype, s) != cudaSuccess) return ONELA_E_CUDA;
        ctx->launches++;
        return ONELA_OK;
    }
    if (ctx->grouped() && !ctx->tensor_core) {
        GroupedArgs ga{};
        ga.q = q_dev;
        ga.out = out_dev;
        ga.s0 = ctx->s0_slot(req_begin, layer);
        ga.kplane = ctx->k_plane(layer);
        ga.vplane = ctx->v_plane(layer);
        ga.gates = ctx->gate_plane(layer);
        ga.table = ctx->table_cur(req_begin);
        ga.s0_req_stride = (long long)c.num_layers * ctx->s0_layer_floats();
        ga.table_req_stride = ctx->table_req_stride();
        ga.arena_slots = c.arena_slots;
        ga.req_count = req_count;
        ga.W = W;
        ga.Hk = c.num_heads;
        ga.g = ctx->Hv() / c.num_heads;
        ga.depth = depth;
        ga.max_beam = c.max_beam;
        for (int i = 0; i < req_count; ++i) ga.bases.base[i] = ctx->req[req_begin + i].step_base.back();
        if (launch_decode_grouped(ga, c.dk, c.dv, c.rec_dtype, c.out_dtype, s) != cudaSuccess) return ONELA_E_CUDA;
        ctx->launches++;
        return ONELA_OK;
    }
    DecodeArgs a{};
    a.q = q_dev;
    a.out = out_dev;
    a.k_in = k_dev;
    a.v_in = v_dev;
    a.alpha_in = alpha_dev;
    a.beta_in = beta_dev;
    // The tensor-core kernel works on value heads of 128 outputs: a wider value head is cut into tiles = dv / 128 of
    // them (its instantiation for grouped value heads serves both), addressed through per-slot strides.
    const int tiles = ctx->tensor_core ? c.dv / 128 : 1;
    a.kv_out = ctx->grouped() ? ctx->k_plane(layer) : ctx->kv_plane(layer);
    a.vv_out = ctx->grouped() ? ctx->v_plane(layer) : (tiles > 1 ? a.kv_out + (size_t)c.dk * ctx->elem_bytes : nullptr);
    a.gates_out = ctx->gate_plane(layer);
    a.s0 = ctx->s0_slot(req_begin, layer);
    a.kv = a.kv_out;
    a.vv = a.vv_out;
    a.Hk = c.num_heads;
    a.g = ctx->Hv() / c.num_heads * tiles;
    a.tiles = tiles;
    a.k_stride = (long long)(ctx->grouped() ? c.dk : c.dk + c.dv) * ctx->elem_bytes;
    a.v_stride = (long long)(ctx->grouped() ? c.dv : c.dk + c.dv) * ctx->elem_bytes;
    a.gates = ctx->gate_plane(layer);
    a.table = ctx->table_cur(req_begin);
    a.status = ctx->lay.status;
    a.s0_req_stride = (long long)c.num_layers * ctx->s0_layer_floats();
    a.s0_scale = ctx->s0_scale_slot(req_begin, layer);
    a.s0_scale_req_stride = (long long)c.num_layers * ctx->Hv();
    a.table_req_stride = ctx->table_req_stride();
    a.arena_slots = c.arena_slots;
    a.sidx = ctx->lay.sidx + req_begin * ctx->sidx_req_stride();
    a.ulist = ctx->lay.ulist + req_begin * ctx->sidx_req_stride();
    a.uoff = ctx->lay.uoff + req_begin * ctx->uoff_req_stride();
    a.urep = ctx->lay.urep + req_begin * ctx->sidx_req_stride();
    a.sg8 = ctx->lay.sg8 + req_begin * ctx->sg8_req_stride();
    a.unode = ctx->lay.unode + (size_t)req_begin * ONELA_UNODE_CAP * 16;
    a.sg8_req_stride = ctx->sg8_req_stride();
    a.sg_stride = sg_row_stride(c.max_beam);
    a.sidx_req_stride = ctx->sidx_req_stride();
    a.ulist_req_stride = ctx->sidx_req_stride();
    a.uoff_req_stride = ctx->uoff_req_stride();
    a.req_count = req_count;
    a.W = W;
    a.H = ctx->Hv() * tiles;
    a.depth = depth;
    a.max_beam = c.max_beam;
    for (int i = 0; i < req_count; ++i) a.bases.base[i] = ctx->req[req_begin + i].step_base.back();
    a.early_ok = ctx->launches == ctx->decode_mark ? 1 : 0;
    bool supported = true;
    const bool wy = ctx->tensor_core && !ctx->gtr() && (c.flags & ONELA_FLAG_SHARED_CHAINS) && !ctx->grouped() && tiles == 1 && depth >= 2 &&
                    depth <= WY_MAX_LEVELS + 1;
    const cudaError_t e = ctx->gtr() && !ctx->tensor_core ? launch_decode_gtr(a, c.dk, c.dv, c.rec_dtype, c.out_dtype, &supported, s)
                          : wy               ? launch_decode_wy(a, c.out_dtype, s)
                          : ctx->tensor_core ? launch_decode_sm100_ws(a, c.out_dtype, ctx->grouped() || tiles > 1, ctx->gtr(), s)
                                             : launch_decode_generic(a, c.dk, c.dv, c.rec_dtype, c.out_dtype, &supported, s);
    if (!supported) return ONELA_E_UNSUPPORTED;
    if (e != cudaSuccess) return ONELA_E_CUDA;
    ctx->launches++;
    ctx->decode_mark = ctx->launches;
    return ONELA_OK;
}

}  // namespace

extern "C" {

onela_status onela_decode_step(onela_ctx* ctx, int32_t req_begin, int32_t req_count, int32_t layer,
                               const void* q_dev, void* out_dev, void* stream) {
    onela_status st = check_batch(ctx, req_begin, req_count);
    if (st != ONELA_OK) return st;
    if (ctx->gtr()) return ONELA_E_UNSUPPORTED;   // the forward replay needs the call's token: append_decode_step
    const onela_config& c = ctx->cfg;
    if (layer < 0 || layer >= c.num_layers) return ONELA_E_INVAL;
    if (!q_dev || !out_dev || !aligned16(q_dev) || !aligned16(out_dev)) return ONELA_E_INVAL;
    const int32_t depth = ctx->req[req_begin].depth;
    if (depth < 1) return ONELA_E_ORDER;
    for (int i = 0; i < req_count; ++i) {
        const ReqState& r = ctx->req[req_begin + i];
        if (!r.has_state[layer] || r.appended_depth[layer] != depth) return ONELA_E_ORDER;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if ((st = ctx->prepare(s)) != ONELA_OK) return st;
    if (ctx->dry()) return ONELA_OK;
    return launch_decode(ctx, req_begin, req_count, layer, q_dev, out_dev, nullptr, nullptr, nullptr, nullptr, s);
}

onela_status onela_append_decode_step(onela_ctx* ctx, int32_t req_begin, int32_t req_count, int32_t layer,
                                      const void* k_dev, const void* v_dev, const float* alpha_dev,
                                      const float* beta_dev, const void* q_dev, void* out_dev, void* stream) {
    onela_status st = check_batch(ctx, req_begin, req_count);
    if (st != ONELA_OK) return st;
    const onela_config& c = ctx->cfg;
    if (layer < 0 || layer >= c.num_layers) return ONELA_E_INVAL;
    if (!k_dev || !v_dev || !alpha_dev || !beta_dev || !aligned16(k_dev) || !aligned16(v_dev)) return ONELA_E_INVAL;
    if (!q_dev || !out_dev || !aligned16(q_dev) || !aligned16(out_dev)) return ONELA_E_INVAL;
    const int32_t depth = ctx->req[req_begin].depth, W = ctx->req[req_begin].W;
    if (depth < 1) return ONELA_E_ORDER;
    for (int i = 0; i < req_count; ++i) {
        const ReqState& r = ctx->req[req_begin + i];
        if (!r.has_state[layer] || r.appended_depth[layer] == depth) return ONELA_E_ORDER;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if ((st = ctx->prepare(s)) != ONELA_OK) return st;
    if (!ctx->dry()) {
        if (ctx->tensor_core || ctx->tiled_tc || ctx->gtr()) {
            st = launch_decode(ctx, req_begin, req_count, layer, q_dev, out_dev, k_dev, v_dev, alpha_dev, beta_dev, s);
            if (st != ONELA_OK) return st;
        } else {   // shapes without the fused kernel: the copy kernel, then the decode kernel
            BatchBases bases{};
            for (int i = 0; i < req_count; ++i) bases.base[i] = ctx->req[req_begin + i].step_base.back();
            const cudaError_t e =
                ctx->grouped() ? launch_append_grouped(k_dev, v_dev, alpha_dev, beta_dev, ctx->k_plane(layer), ctx->v_plane(layer),
                                                       ctx->gate_plane(layer), c.arena_slots, req_count, W, c.num_heads,
                                                       ctx->Hv() / c.num_heads, c.dk, c.dv, ctx->elem_bytes, bases, s)
                               : launch_append(k_dev, v_dev, alpha_dev, beta_dev, ctx->kv_plane(layer), ctx->gate_plane(layer),
                                               c.arena_slots, req_count, W, c.num_heads, c.dk, c.dv, ctx->elem_bytes, bases, s);
            if (e != cudaSuccess) return ONELA_E_CUDA;
            ctx->launches++;
            st = launch_decode(ctx, req_begin, req_count, layer, q_dev, out_dev, nullptr, nullptr, nullptr, nullptr, s);
            if (st != ONELA_OK) return st;
        }
    }
    for (int i = 0; i < req_count; ++i) ctx->req[req_begin + i].appended_depth[layer] = depth;
    return ONELA_OK;
}

onela_status onela_export_chains(onela_ctx* ctx, int32_t request, int32_t* slots_dev, int32_t* depth_host,
                                 int32_t* width_host, void* stream) {
    if (!ctx || request < 0 || request >= ctx->cfg.num_requests) return ONELA_E_INVAL;
    const ReqState& r = ctx->req[request];
    if (depth_host) *depth_host = r.depth;
    if (width_host) *width_host = r.W;
    if (r.depth < 1) return ONELA_E_ORDER;
    if (!slots_dev) return ONELA_E_INVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    onela_status st = ctx->prepare(s);
    if (st != ONELA_OK) return st;
    if (ctx->dry()) return ONELA_OK;
    if (launch_export_chains(ctx->table_cur(request), r.W, r.depth, ctx->cfg.max_beam, slots_dev, s) != cudaSuccess)
        return ONELA_E_CUDA;
    ctx->launches++;
    return ONELA_OK;
}

onela_status onela_poll_device_status(onela_ctx* ctx, int32_t* code_host, int32_t* detail_host) {
    if (!ctx) return ONELA_E_INVAL;
    int32_t w[4] = {0, 0, 0, 0};
    if (!ctx->dry() && ctx->status_cleared) {
        if (cudaDeviceSynchronize() != cudaSuccess) return ONELA_E_CUDA;
        if (cudaMemcpy(w, ctx->lay.status, sizeof(w), cudaMemcpyDeviceToHost) != cudaSuccess) return ONELA_E_CUDA;
        if (w[0] != ONELA_OK && cudaMemset(ctx->lay.status, 0, sizeof(w)) != cudaSuccess) return ONELA_E_CUDA;
    }
    if (code_host) *code_host = w[0];
    if (detail_host) *detail_host = w[1];
    return ONELA_OK;
}

onela_status onela_get_stats(const onela_ctx* ctx, int64_t* s0_bytes_host, int64_t* arena_bytes_used_host,
                             int64_t* index_bytes_host) {
    if (!ctx) return ONELA_E_INVAL;
    const onela_config& c = ctx->cfg;
    int64_t states = 0, index = 0;
    for (const auto& r : ctx->req) {
        for (uint8_t hs : r.has_state) states += hs;
        index += (int64_t)r.W * r.depth * (int64_t)sizeof(int32_t);
    }
    // bytes one slot holds across the heads of a layer: k per key head, v and the two gates per value head
    const int64_t slot_bytes = (int64_t)c.num_heads * c.dk * ctx->elem_bytes +
                               (int64_t)ctx->Hv() * (c.dv * ctx->elem_bytes + 2 * (int64_t)sizeof(float));
    if (s0_bytes_host) *s0_bytes_host = states * ctx->s0_layer_floats() * (int64_t)sizeof(float);
    if (arena_bytes_used_host)
        *arena_bytes_used_host = (ctx->cursor - ctx->free_slots()) * slot_bytes * c.num_layers;
    if (index_bytes_host) *index_bytes_host = index;
    return ONELA_OK;
}

onela_status onela_get_step_base(const onela_ctx* ctx, int32_t request, int32_t step, int32_t* base_host) {
    if (!ctx || !base_host || request < 0 || request >= ctx->cfg.num_requests) return ONELA_E_INVAL;
    const ReqState& r = ctx->req[request];
    if (step < 0 || step >= (int32_t)r.step_base.size()) return ONELA_E_INVAL;
    *base_host = r.step_base[step];
    return ONELA_OK;
}

int64_t onela_launch_count(const onela_ctx* ctx) { return ctx ? ctx->launches : 0; }

int32_t onela_uses_tensor_core_path(const onela_ctx* ctx) { return !ctx ? 0 : ctx->tensor_core ? 1 : ctx->tiled_tc ? 2 : 0; }

const char* onela_status_string(onela_status s) {
    switch (s) {
        case ONELA_OK: return "ok";
        case ONELA_E_INVAL: return "invalid argument";
        case ONELA_E_CAPACITY: return "capacity exhausted";
        case ONELA_E_ORDER: return "call order violated";
        case ONELA_E_CUDA: return "CUDA runtime error";
        case ONELA_E_UNSUPPORTED: return "unsupported head dimensions or dtype";
        case ONELA_E_DEVICE_CHECK: return "device found an out-of-range parent index";
        case ONELA_E_TIMEOUT: return "bounded device-side wait expired";
        default: return "unknown status";
    }
}

}  // extern "C"
