// Host side of the C ABI: argument validation, the static gather schedule, workspace layout and launches.
#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "cb_internal.cuh"

namespace cb {

static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

static constexpr uint32_t CTX_MAGIC = 0xCB0C7A11u;
static constexpr int MAX_SPLITS = 64;

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Layout {
    size_t slots_off, slots_bytes, tab_off, status_off, total;
};

static Layout workspace_layout(int Lt, int Ht, int d, int n_splits)
{
    Layout L;
    const size_t n_maps = 2 * (size_t)Lt * Ht;
    L.slots_off = 0;
    L.slots_bytes = (size_t)n_splits * n_maps * slot_floats(d) * sizeof(float);
    L.tab_off = align_up(L.slots_bytes, 256);
    L.status_off = align_up(L.tab_off + sizeof(int) * ((size_t)Lt + Ht), 256);
    L.total = L.status_off + 256;
    return L;
}

cb_status check_problem(const cb_problem *p)
{
    if (!p || !p->src_layer || !p->src_head) return CB_ERR_INVALID_ARG;
    if (p->Ls <= 0 || p->Hs <= 0 || p->Lt <= 0 || p->Ht <= 0 || p->ds <= 0 || p->dt <= 0) return CB_ERR_INVALID_ARG;
    if (p->n_splits < 0 || p->n_splits > MAX_SPLITS) return CB_ERR_INVALID_ARG;
    for (int l = 0; l < p->Lt; ++l)
        if (p->src_layer[l] < 0 || p->src_layer[l] >= p->Ls) return CB_ERR_INVALID_ARG;
    for (int h = 0; h < p->Ht; ++h)
        if (p->src_head[h] < 0 || p->src_head[h] >= p->Hs) return CB_ERR_INVALID_ARG;
    if (p->ds != p->dt || (p->ds != 64 && p->ds != 128)) return CB_ERR_UNSUPPORTED;
    if ((long long)p->Lt * p->Ht > (1 << 20)) return CB_ERR_UNSUPPORTED;
    return CB_OK;
}

// Token splits per map.  The statistics kernel runs one persistent block per SM over the units (map, split) in
// round-robin order, so the launch ends when the SMs with ceil(units / SMs) units finish; every further split costs
// one more read-modify-write of all partial slots per call (~0.4 % of a 51,200-token call each).  When the caller
// leaves the choice open, take the count in 1..8 that minimises the product of the two (1,024 maps: 1 split;
// 640 maps: 3; 8 maps: 8).  The count depends on the problem only, so workspace sizes are reproducible.
static int splits_of(const cb_problem *p)
{
    if (p->n_splits > 0) return p->n_splits;
    const long long n_maps = 2ll * p->Lt * p->Ht, sms = device_sm_count();
    int best = 1;
    double best_cost = 0.0;
    for (int s = 1; s <= 8; ++s) {
        const long long units = n_maps * s, rounds = (units + sms - 1) / sms;
        const double cost = (double)(rounds * sms) / (double)units * (1.0 + 0.004 * s);
        if (s == 1 || cost < best_cost - 1e-12) { best = s; best_cost = cost; }
    }
    return best;
}

cb_status check_view(const cb_kv_view *v, int L, int H, int d)
{
    if (!v) return CB_ERR_INVALID_ARG;
    if (v->n_layers != L || v->n_heads != H || v->head_dim != d) return CB_ERR_INVALID_ARG;
    if (v->n_tokens < 0) return CB_ERR_INVALID_ARG;
    if (v->n_tokens >= (1ll << 31)) return CB_ERR_UNSUPPORTED;
    if (v->n_tokens == 0) return CB_OK;
    if (!v->k || !v->v) return CB_ERR_INVALID_ARG;
    if (((uintptr_t)v->k | (uintptr_t)v->v) & 15) return CB_ERR_INVALID_ARG;
    if (v->stride_layer < 0 || v->stride_token <= 0 || v->stride_head < 0) return CB_ERR_INVALID_ARG;
    if ((v->stride_layer | v->stride_token | v->stride_head) & 7) return CB_ERR_INVALID_ARG;
    // a broadcast (stride 0) over more than one layer or head cannot be described to the tile copies
    if ((L > 1 && v->stride_layer == 0) || (H > 1 && v->stride_head == 0)) return CB_ERR_UNSUPPORTED;
    return CB_OK;
}

// Output strides of the apply calls: same rules as a view's.
cb_status check_out_strides(int Lt, int Ht, int64_t sl, int64_t st, int64_t sh)
{
    if (sl < 0 || st <= 0 || sh < 0) return CB_ERR_INVALID_ARG;
    if ((sl | st | sh) & 7) return CB_ERR_INVALID_ARG;
    if ((Lt > 1 && sl == 0) || (Ht > 1 && sh == 0)) return CB_ERR_UNSUPPORTED;
    return CB_OK;
}

// Status word, poll limit and test hooks of a launch.
template <class Args>
static void fill_launch_state(Args &a)
{
    if (!a.status) a.status = library_status_word();
    const TestHooks h = test_hooks();
    a.poll_limit = h.poll_limit;
    a.starve = h.starve;
}

}  // namespace cb

using namespace cb;

struct cb_ctx {
    uint32_t magic;
    cb_problem prob;
    std::vector<int32_t> src_layer, src_head;
    int d, n_maps, n_splits;
    char *ws;
    Layout lay;
    long long n_tokens;
    bool k_operands_centred;   // centred accumulation with the rotary boundary since the last reset (see cb_stats_reduce_centered)
};

extern "C" {

const char *cb_status_string(cb_status s)
{
    switch (s) {
        case CB_OK: return "ok";
        case CB_ERR_INVALID_ARG: return "invalid argument";
        case CB_ERR_UNSUPPORTED: return "unsupported shape";
        case CB_ERR_STATE: return "invalid context or call order";
        case CB_ERR_WORKSPACE: return "workspace too small or misaligned";
        case CB_ERR_CUDA: return "CUDA call failed";
        case CB_ERR_NOT_PD: return "ridge system not positive definite";
        case CB_ERR_TIMEOUT: return "device-side wait timed out";
        case CB_ERR_STATIC_LIMIT: return "problem exceeds the built-in scratch buffer of cb_stats_build_static";
    }
    return "unknown status";
}

int64_t cb_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

cb_status cb_head_map_nearest(int32_t Ls, int32_t Hs, int32_t Lt, int32_t Ht, int32_t *src_layer, int32_t *src_head)
{
    if (Ls <= 0 || Hs <= 0 || Lt <= 0 || Ht <= 0 || !src_layer || !src_head) return CB_ERR_INVALID_ARG;
    for (int32_t l = 0; l < Lt; ++l) {
        if (Lt == 1) { src_layer[l] = 0; continue; }
        const int64_t num = (int64_t)2 * l * (Ls - 1) + (Lt - 1);
        src_layer[l] = (int32_t)(num / ((int64_t)2 * (Lt - 1)));
    }
    for (int32_t h = 0; h < Ht; ++h) src_head[h] = (int32_t)(((int64_t)h * Hs) / Ht);
    return CB_OK;
}

cb_status cb_work_list(const cb_problem *prob, int32_t *n_items, int32_t *item_comp, int32_t *item_layer,
                       int32_t *item_head, int32_t *item_begin, int32_t *item_maps)
{
    cb_status s = check_problem(prob);
    if (s != CB_OK && s != CB_ERR_UNSUPPORTED) return s;   // the schedule itself does not depend on d
    if (!n_items || !item_comp || !item_layer || !item_head || !item_begin || !item_maps) return CB_ERR_INVALID_ARG;
    const int Ls = prob->Ls, Hs = prob->Hs, Lt = prob->Lt, Ht = prob->Ht;
    // bucket every map by its source head with a counting sort: key = (comp*Ls + j)*Hs + g
    const int n_keys = 2 * Ls * Hs, n_maps = 2 * Lt * Ht;
    std::vector<int32_t> count(n_keys + 1, 0);
    auto key_of = [&](int m) {
        const int comp = m / (Lt * Ht), l = (m / Ht) % Lt, h = m % Ht;
        return (comp * Ls + prob->src_layer[l]) * Hs + prob->src_head[h];
    };
    for (int m = 0; m < n_maps; ++m) ++count[key_of(m) + 1];
    for (int k = 0; k < n_keys; ++k) count[k + 1] += count[k];
    std::vector<int32_t> fill(count.begin(), count.end() - 1);
    for (int m = 0; m < n_maps; ++m) item_maps[fill[key_of(m)]++] = m;   // ascending m inside a bucket
    int n = 0;
    for (int k = 0; k < n_keys; ++k) {
        if (count[k + 1] == count[k]) continue;
        item_comp[n] = k / (Ls * Hs);
        item_layer[n] = (k / Hs) % Ls;
        item_head[n] = k % Hs;
        item_begin[n] = count[k];
        ++n;
    }
    item_begin[n] = n_maps;
    *n_items = n;
    return CB_OK;
}

cb_status cb_token_splits(const cb_problem *prob, int32_t *n_splits)
{
    cb_status s = check_problem(prob);
    if (s != CB_OK) return s;
    if (!n_splits) return CB_ERR_INVALID_ARG;
    *n_splits = splits_of(prob);
    return CB_OK;
}

cb_status cb_workspace_bytes(const cb_problem *prob, size_t *bytes)
{
    cb_status s = check_problem(prob);
    if (s != CB_OK) return s;
    if (!bytes) return CB_ERR_INVALID_ARG;
    *bytes = workspace_layout(prob->Lt, prob->Ht, prob->ds, splits_of(prob)).total;
    return CB_OK;
}

cb_status cb_create(const cb_problem *prob, void *workspace, size_t workspace_bytes, cb_ctx **out)
{
    if (!out) return CB_ERR_INVALID_ARG;
    *out = nullptr;
    cb_status s = check_problem(prob);
    if (s != CB_OK) return s;
    const int n_splits = splits_of(prob);
    const Layout lay = workspace_layout(prob->Lt, prob->Ht, prob->ds, n_splits);
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < lay.total) return CB_ERR_WORKSPACE;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { return cuda_failed(); }

    cb_ctx *c = new (std::nothrow) cb_ctx();
    if (!c) return CB_ERR_INVALID_ARG;
    c->magic = CTX_MAGIC;
    c->prob = *prob;
    c->src_layer.assign(prob->src_layer, prob->src_layer + prob->Lt);
    c->src_head.assign(prob->src_head, prob->src_head + prob->Ht);
    c->prob.src_layer = c->src_layer.data();
    c->prob.src_head = c->src_head.data();
    c->d = prob->ds;
    c->n_maps = 2 * prob->Lt * prob->Ht;
    c->n_splits = n_splits;
    c->ws = static_cast<char *>(workspace);
    c->lay = lay;
    c->n_tokens = 0;
    c->k_operands_centred = false;

    std::vector<int32_t> tab(c->src_layer);
    tab.insert(tab.end(), c->src_head.begin(), c->src_head.end());
    cudaError_t e = cudaMemcpy(c->ws + lay.tab_off, tab.data(), tab.size() * sizeof(int32_t), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + lay.slots_off, 0, lay.slots_bytes, 0);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + lay.status_off, 0, 256, 0);
    if (e == cudaSuccess) e = cudaStreamSynchronize(0);
    if (e != cudaSuccess) {
        const cb_status cf = cuda_failed(e);
        delete c;
        return cf;
    }
    *out = c;
    return CB_OK;
}

void cb_destroy(cb_ctx *ctx)
{
    if (!ctx || ctx->magic != CTX_MAGIC) return;
    ctx->magic = 0;
    delete ctx;
}

cb_status cb_stats_reset(cb_ctx *ctx, void *stream)
{
    if (!ctx || ctx->magic != CTX_MAGIC) return CB_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(ctx->ws + ctx->lay.slots_off, 0, ctx->lay.slots_bytes, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->ws + ctx->lay.status_off, 0, 256, st);
    if (e != cudaSuccess) return cuda_failed(e);
    ctx->n_tokens = 0;
    ctx->k_operands_centred = false;
    return CB_OK;
}

struct RopeOpt { const int32_t *pos; double base_src, base_tgt; };

static bool rope_base_ok(double b) { return b > 1.0 && b <= 1e12; }

static cb_status accumulate_impl(cb_ctx *ctx, const cb_kv_view *src, const cb_kv_view *tgt,
                                 const float *w_k, const float *w_v,
                                 int64_t w_stride_layer, int64_t w_stride_head, const float *mu, bool centred, void *stream,
                                 const RopeOpt *rope = nullptr)
{
    if (rope) {
        if (!ctx || ctx->magic != CTX_MAGIC) return CB_ERR_STATE;
        if (!rope_base_ok(rope->base_src) || !rope_base_ok(rope->base_tgt)) return CB_ERR_INVALID_ARG;
        if (ctx->prob.flags & CB_FLAG_SIMT) return CB_ERR_UNSUPPORTED;
        if (src && src->n_tokens > 0 && (!rope->pos || ((uintptr_t)rope->pos & 3))) return CB_ERR_INVALID_ARG;
    }
    if (!ctx || ctx->magic != CTX_MAGIC) return CB_ERR_STATE;
    if (centred && !mu) return CB_ERR_INVALID_ARG;
    if (centred && (ctx->prob.flags & CB_FLAG_SIMT)) return CB_ERR_UNSUPPORTED;
    const cb_problem &P = ctx->prob;
    cb_status s = check_view(src, P.Ls, P.Hs, P.ds);
    if (s != CB_OK) return s;
    s = check_view(tgt, P.Lt, P.Ht, P.dt);
    if (s != CB_OK) return s;
    if (src->n_tokens != tgt->n_tokens) return CB_ERR_INVALID_ARG;
    if (src->n_tokens == 0) return CB_OK;
    if (!w_k || !w_v || w_stride_layer < 0 || w_stride_head < 0) return CB_ERR_INVALID_ARG;
    if (((uintptr_t)w_k | (uintptr_t)w_v) & 3) return CB_ERR_INVALID_ARG;

    AccumArgs a;
    a.src = KVPtr{static_cast<const __nv_bfloat16 *>(src->k), static_cast<const __nv_bfloat16 *>(src->v),
                  src->stride_layer, src->stride_token, src->stride_head};
    a.tgt = KVPtr{static_cast<const __nv_bfloat16 *>(tgt->k), static_cast<const __nv_bfloat16 *>(tgt->v),
                  tgt->stride_layer, tgt->stride_token, tgt->stride_head};
    a.w_k = w_k; a.w_v = w_v; a.w_sl = w_stride_layer; a.w_sh = w_stride_head;
    a.n_tokens = (int)src->n_tokens;
    a.Lt = P.Lt; a.Ht = P.Ht; a.n_splits = ctx->n_splits;
    a.src_layer = reinterpret_cast<const int *>(ctx->ws + ctx->lay.tab_off);
    a.src_head = a.src_layer + P.Lt;
    a.slots = reinterpret_cast<float *>(ctx->ws + ctx->lay.slots_off);
    a.status = reinterpret_cast<int *>(ctx->ws + ctx->lay.status_off);
    a.compensated = (P.flags & CB_FLAG_COMPENSATED) ? 1 : 0;
    a.mu = centred ? mu : nullptr;
    if (rope) { a.rope_pos = rope->pos; a.rope_base_src = rope->base_src; a.rope_base_tgt = rope->base_tgt; }
    fill_launch_state(a);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = (P.flags & CB_FLAG_SIMT) ? launch_accum_simt(a, ctx->d, st)
                                             : launch_accum_tc(a, ctx->d, src, tgt, st);
    if (e != cudaSuccess) return cuda_failed(e);
    ctx->n_tokens += src->n_tokens;
    if (centred && rope) ctx->k_operands_centred = true;
    return CB_OK;
}

cb_status cb_stats_accumulate(cb_ctx *ctx, const cb_kv_view *src, const cb_kv_view *tgt,
                              const float *w_k, const float *w_v,
                              int64_t w_stride_layer, int64_t w_stride_head, void *stream)
{
    return accumulate_impl(ctx, src, tgt, w_k, w_v, w_stride_layer, w_stride_head, nullptr, false, stream);
}

// ---------------------------------------------------------------------------------------------------------------------
// Rotary embedding at the boundary
// ---------------------------------------------------------------------------------------------------------------------
cb_status cb_stats_accumulate_rope(cb_ctx *ctx, const cb_kv_view *src, const cb_kv_view *tgt,
                                   const float *w_k, const float *w_v, int64_t w_stride_layer, int64_t w_stride_head,
                                   const int32_t *positions, double rope_base_src, double rope_base_tgt, void *stream)
{
    const RopeOpt r{positions, rope_base_src, rope_base_tgt};
    return accumulate_impl(ctx, src, tgt, w_k, w_v, w_stride_layer, w_stride_head, nullptr, false, stream, &r);
}

cb_status cb_rope_rotate(void *k, int32_t n_layers, int32_t n_heads, int32_t head_dim, int64_t n_tokens,
                         int64_t stride_layer, int64_t stride_token, int64_t stride_head,
                         const int32_t *positions, double rope_base, int32_t inverse, void *stream)
{
    if (n_layers <= 0 || n_heads <= 0 || n_tokens < 0) return CB_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return CB_ERR_UNSUPPORTED;
    if (n_tokens >= (1ll << 31) || (long long)n_layers * n_heads > 65535) return CB_ERR_UNSUPPORTED;
    if (!rope_base_ok(rope_base)) return CB_ERR_INVALID_ARG;
    if (n_tokens == 0) return CB_OK;
    if (!k || ((uintptr_t)k & 15) || !positions || ((uintptr_t)positions & 3)) return CB_ERR_INVALID_ARG;
    if (stride_layer < 0 || stride_token <= 0 || stride_head < 0) return CB_ERR_INVALID_ARG;
    if ((stride_layer | stride_token | stride_head) & 7) return CB_ERR_INVALID_ARG;
    cudaError_t e = launch_rope_rotate(k, n_layers, n_heads, head_dim, n_tokens, stride_layer, stride_token, stride_head,
                                       positions, rope_base, inverse ? 1 : 0, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e);
    return CB_OK;
}

// ---------------------------------------------------------------------------------------------------------------------
// Two-pass centred construction
// ---------------------------------------------------------------------------------------------------------------------
static size_t means_bytes(const cb_ctx *ctx)
{
    return (size_t)MEANS_SPLITS * ctx->n_maps * means_stride(ctx->d) * sizeof(double);
}

cb_status cb_means_workspace_bytes(const cb_problem *prob, size_t *bytes)
{
    cb_status s = check_problem(prob);
    if (s != CB_OK) return s;
    if (!bytes) return CB_ERR_INVALID_ARG;
    *bytes = (size_t)MEANS_SPLITS * 2 * prob->Lt * prob->Ht * means_stride(prob->ds) * sizeof(double);
    return CB_OK;
}

cb_status cb_means_reset(cb_ctx *ctx, void *means_ws, size_t means_ws_bytes, void *stream)
{
    if (!ctx || ctx->magic != CTX_MAGIC) return CB_ERR_STATE;
    if (!means_ws || ((uintptr_t)means_ws & 255) || means_ws_bytes < means_bytes(ctx)) return CB_ERR_WORKSPACE;
    cudaError_t e = cudaMemsetAsync(means_ws, 0, means_bytes(ctx), static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e);
    return CB_OK;
}

static cb_status means_accumulate_impl(cb_ctx *ctx, const cb_kv_view *src, const cb_kv_view *tgt,
                                       const float *w_k, const float *w_v, int64_t w_stride_layer, int64_t w_stride_head,
                                       void *means_ws, size_t means_ws_bytes, void *stream, const RopeOpt *rope)
{
    if (!ctx || ctx->magic != CTX_MAGIC) return CB_ERR_STATE;
    if (rope) {
        if (!rope_base_ok(rope->base_src) || !rope_base_ok(rope->base_tgt)) return CB_ERR_INVALID_ARG;
        if (src && src->n_tokens > 0 && (!rope->pos || ((uintptr_t)rope->pos & 3))) return CB_ERR_INVALID_ARG;
    }
    const cb_problem &P = ctx->prob;
    cb_status s = check_view(src, P.Ls, P.Hs, P.ds);
    if (s != CB_OK) return s;
    s = check_view(tgt, P.Lt, P.Ht, P.dt);
    if (s != CB_OK) return s;
    if (src->n_tokens != tgt->n_tokens) return CB_ERR_INVALID_ARG;
    if (!means_ws || ((uintptr_t)means_ws & 255) || means_ws_bytes < means_bytes(ctx)) return CB_ERR_WORKSPACE;
    if (src->n_tokens == 0) return CB_OK;
    if (!w_k || !w_v || w_stride_layer < 0 || w_stride_head < 0) return CB_ERR_INVALID_ARG;
    if (((uintptr_t)w_k | (uintptr_t)w_v) & 3) return CB_ERR_INVALID_ARG;
    MeansArgs a;
    a.src = KVPtr{static_cast<const __nv_bfloat16 *>(src->k), static_cast<const __nv_bfloat16 *>(src->v),
                  src->stride_layer, src->stride_token, src->stride_head};
    a.tgt = KVPtr{static_cast<const __nv_bfloat16 *>(tgt->k), static_cast<const __nv_bfloat16 *>(tgt->v),
                  tgt->stride_layer, tgt->stride_token, tgt->stride_head};
    a.w_k = w_k; a.w_v = w_v; a.w_sl = w_stride_layer; a.w_sh = w_stride_head;
    a.n_tokens = (int)src->n_tokens;
    a.Lt = P.Lt; a.Ht = P.Ht;
    a.src_layer = reinterpret_cast<const int *>(ctx->ws + ctx->lay.tab_off);
    a.src_head = a.src_layer + P.Lt;
    a.msum = static_cast<double *>(means_ws);
    if (rope) { a.rope_pos = rope->pos; a.rope_base_src = rope->base_src; a.rope_base_tgt = rope->base_tgt; }
    cudaError_t e = launch_means(a, ctx->d, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e);
    return CB_OK;
}

cb_status cb_means_accumulate(cb_ctx *ctx, const cb_kv_view *src, const cb_kv_view *tgt,
                              const float *w_k, const float *w_v, int64_t w_stride_layer, int64_t w_stride_head,
                              void *means_ws, size_t means_ws_bytes, void *stream)
{
    return means_accumulate_impl(ctx, src, tgt, w_k, w_v, w_stride_layer, w_stride_head, means_ws, means_ws_bytes, stream, nullptr);
}

cb_status cb_means_accumulate_rope(cb_ctx *ctx, const cb_kv_view *src, const cb_kv_view *tgt,
                                   const float *w_k, const float *w_v, int64_t w_stride_layer, int64_t w_stride_head,
                                   void *means_ws, size_t means_ws_bytes,
                                   const int32_t *positions, double rope_base_src, double rope_base_tgt, void *stream)
{
    const RopeOpt r{positions, rope_base_src, rope_base_tgt};
    return means_accumulate_impl(ctx, src, tgt, w_k, w_v, w_stride_layer, w_stride_head, means_ws, means_ws_bytes, stream, &r);
}

cb_status cb_means_finalize(cb_ctx *ctx, const void *means_ws, size_t means_ws_bytes, float *mu, void *stream)
{
    if (!ctx || ctx->magic != CTX_MAGIC) return CB_ERR_STATE;
    if (!means_ws || ((uintptr_t)means_ws & 255) || means_ws_bytes < means_bytes(ctx)) return CB_ERR_WORKSPACE;
    if (!mu) return CB_ERR_INVALID_ARG;
    cudaError_t e = launch_means_finalize(static_cast<const double *>(means_ws), ctx->n_maps, ctx->d, mu,
                                          static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e);
    return CB_OK;
}

cb_status cb_means_energy(cb_ctx *ctx, const void *means_ws, size_t means_ws_bytes, float *syy, void *stream)
{
    if (!ctx || ctx->magic != CTX_MAGIC) return CB_ERR_STATE;
    if (!means_ws || ((uintptr_t)means_ws & 255) || means_ws_bytes < means_bytes(ctx)) return CB_ERR_WORKSPACE;
    if (!syy) return CB_ERR_INVALID_ARG;
    cudaError_t e = launch_means_energy(static_cast<const double *>(means_ws), ctx->n_maps, ctx->d, syy,
                                        static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e);
    return CB_OK;
}

// ---------------------------------------------------------------------------------------------------------------------
// Layer selector
// ---------------------------------------------------------------------------------------------------------------------
cb_status cb_probe_r2(const float *G, const float *C, const float *Wb, const float *syy, int32_t n_maps, int32_t d,
                      int64_t n_tokens, float lambda, uint32_t flags, float *r2, void *stream)
{
    if (!G || !C || !Wb || !syy || !r2) return CB_ERR_INVALID_ARG;
    if (n_maps < 0 || n_tokens < 0 || !(lambda >= 0.f)) return CB_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return CB_ERR_UNSUPPORTED;
    if (n_maps == 0) return CB_OK;
    cudaError_t e = launch_probe_r2(G, C, Wb, syy, n_maps, d, (double)lambda, n_tokens > 0 ? 1.0 / (double)n_tokens : 0.0,
                                    (flags & CB_FLAG_RAW_LAMBDA) ? 1 : 0, r2, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e);
    return CB_OK;
}

cb_status cb_probe_scores(const float *r2, int32_t Lt, int32_t Ht, const int32_t *src_layer, int32_t Ls, float *scores,
                          void *stream)
{
    if (!r2 || !src_layer || !scores || Lt <= 0 || Ht <= 0 || Ls <= 0) return CB_ERR_INVALID_ARG;
    if (Lt > 128) return CB_ERR_UNSUPPORTED;
    for (int l = 0; l < Lt; ++l)
        if (src_layer[l] < 0 || src_layer[l] >= Ls) return CB_ERR_INVALID_ARG;
    cudaError_t e = launch_probe_scores(r2, Lt, Ht, src_layer, Ls, scores, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e);
    return CB_OK;
}

cb_status cb_rank_layers(const float *scores, int32_t Lt, int32_t Ls, int32_t k, int32_t *layer_sets)
{
    if (!scores || !layer_sets || Lt <= 0 || Ls <= 0 || k <= 0 || k > Ls) return CB_ERR_INVALID_ARG;
    std::vector<char> taken((size_t)Ls);
    for (int l = 0; l < Lt; ++l) {
        std::fill(taken.begin(), taken.end(), 0);
        for (int q = 0; q < k; ++q) {
            int best = -1;
            for (int j = 0; j < Ls; ++j)
                if (!taken[j] && (best < 0 || scores[(size_t)l * Ls + j] > scores[(size_t)l * Ls + best])) best = j;
            taken[best] = 1;
        }
        int q = 0;
        for (int j = 0; j < Ls; ++j)
            if (taken[j]) layer_sets[(size_t)l * k + q++] = j;
    }
    return CB_OK;
}

cb_status cb_stats_accumulate_centered(cb_ctx *ctx, const cb_kv_view *src, const cb_kv_view *tgt,
                                       const float *w_k, const float *w_v,
                                       int64_t w_stride_layer, int64_t w_stride_head, const float *mu, void *stream)
{
    return accumulate_impl(ctx, src, tgt, w_k, w_v, w_stride_layer, w_stride_head, mu, true, stream);
}

cb_status cb_stats_accumulate_centered_rope(cb_ctx *ctx, const cb_kv_view *src, const cb_kv_view *tgt,
                                            const float *w_k, const float *w_v,
                                            int64_t w_stride_layer, int64_t w_stride_head, const float *mu,
                                            const int32_t *positions, double rope_base_src, double rope_base_tgt, void *stream)
{
    const RopeOpt r{positions, rope_base_src, rope_base_tgt};
    return accumulate_impl(ctx, src, tgt, w_k, w_v, w_stride_layer, w_stride_head, mu, true, stream, &r);
}

cb_status cb_stats_reduce_centered(cb_ctx *ctx, const float *mu, float *A, float *B, int64_t *n_tokens_out, void *stream)
{
    if (!ctx || ctx->magic != CTX_MAGIC) return CB_ERR_STATE;
    if (!mu || !A || !B) return CB_ERR_INVALID_ARG;
    cudaError_t e = launch_reduce_centered(reinterpret_cast<const float *>(ctx->ws + ctx->lay.slots_off), ctx->n_splits,
                                           ctx->n_maps, ctx->d, mu, A, B, ctx->k_operands_centred ? 1 : 0,
                                           static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e);
    if (n_tokens_out) *n_tokens_out = ctx->n_tokens;
    return CB_OK;
}

cb_status cb_ridge_solve_centered(const float *A, const float *B, const float *mu, int32_t n_maps, int32_t d,
                                  int64_t n_tokens, const float *lambdas, int32_t n_lambda, uint32_t flags,
                                  float *Wb, int32_t *info, void *stream)
{
    if (!A || !B || !mu || !lambdas || !Wb || !info) return CB_ERR_INVALID_ARG;
    if (n_maps < 0 || n_lambda <= 0 || n_lambda > 16 || n_tokens < 0) return CB_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return CB_ERR_UNSUPPORTED;
    if (n_maps > 65535 * 16) return CB_ERR_UNSUPPORTED;
    for (int i = 0; i < n_lambda; ++i)
        if (!(lambdas[i] >= 0.f)) return CB_ERR_INVALID_ARG;
    if (n_maps == 0) return CB_OK;
    cudaError_t e = launch_solve_centered(A, B, mu, n_maps, d, n_tokens, lambdas, n_lambda, flags, Wb, info,
                                          static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e);
    return CB_OK;
}

static bool dense_view(const cb_kv_view *v)
{
    return v->stride_head == v->head_dim && v->stride_token == (int64_t)v->n_heads * v->head_dim &&
           v->stride_layer == v->n_tokens * v->n_heads * v->head_dim;
}

struct StagingLayout { size_t src_k, src_v, tgt_k, tgt_v, w_k, w_v, total; };

static StagingLayout staging_layout(const cb_problem *p, int64_t T)
{
    StagingLayout L;
    const size_t sb = (size_t)p->Ls * T * p->Hs * p->ds * 2, tb = (size_t)p->Lt * T * p->Ht * p->dt * 2;
    const size_t wb = (size_t)p->Lt * p->Ht * T * 4;
    size_t o = 0;
    L.src_k = o; o = align_up(o + sb, 256);
    L.src_v = o; o = align_up(o + sb, 256);
    L.tgt_k = o; o = align_up(o + tb, 256);
    L.tgt_v = o; o = align_up(o + tb, 256);
    L.w_k = o; o = align_up(o + wb, 256);
    L.w_v = o; o = align_up(o + wb, 256);
    L.total = o;
    return L;
}

cb_status cb_staging_bytes(const cb_problem *prob, int64_t n_tokens, size_t *bytes)
{
    cb_status s = check_problem(prob);
    if (s != CB_OK) return s;
    if (!bytes || n_tokens < 0) return CB_ERR_INVALID_ARG;
    *bytes = staging_layout(prob, n_tokens).total;
    return CB_OK;
}

cb_status cb_stats_accumulate_host(cb_ctx *ctx, const cb_kv_view *src_host, const cb_kv_view *tgt_host,
                                   const float *w_k_host, const float *w_v_host,
                                   void *staging, size_t staging_bytes, void *stream)
{
    if (!ctx || ctx->magic != CTX_MAGIC) return CB_ERR_STATE;
    const cb_problem &P = ctx->prob;
    if (!src_host || !tgt_host) return CB_ERR_INVALID_ARG;
    if (src_host->n_layers != P.Ls || src_host->n_heads != P.Hs || src_host->head_dim != P.ds) return CB_ERR_INVALID_ARG;
    if (tgt_host->n_layers != P.Lt || tgt_host->n_heads != P.Ht || tgt_host->head_dim != P.dt) return CB_ERR_INVALID_ARG;
    const int64_t T = src_host->n_tokens;
    if (T < 0 || T != tgt_host->n_tokens) return CB_ERR_INVALID_ARG;
    if (T == 0) return CB_OK;
    if (!src_host->k || !src_host->v || !tgt_host->k || !tgt_host->v || !w_k_host || !w_v_host) return CB_ERR_INVALID_ARG;
    if (!dense_view(src_host) || !dense_view(tgt_host)) return CB_ERR_INVALID_ARG;
    const StagingLayout L = staging_layout(&P, T);
    if (!staging || ((uintptr_t)staging & 255) || staging_bytes < L.total) return CB_ERR_WORKSPACE;
    char *dv = static_cast<char *>(staging);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t sb = (size_t)P.Ls * T * P.Hs * P.ds * 2, tb = (size_t)P.Lt * T * P.Ht * P.dt * 2;
    const size_t wb = (size_t)P.Lt * P.Ht * T * 4;
    cudaError_t e = cudaMemcpyAsync(dv + L.src_k, src_host->k, sb, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dv + L.src_v, src_host->v, sb, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dv + L.tgt_k, tgt_host->k, tb, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dv + L.tgt_v, tgt_host->v, tb, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dv + L.w_k, w_k_host, wb, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && w_v_host != w_k_host) e = cudaMemcpyAsync(dv + L.w_v, w_v_host, wb, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_failed(e);
    cb_kv_view s = *src_host, t = *tgt_host;
    s.k = dv + L.src_k; s.v = dv + L.src_v;
    t.k = dv + L.tgt_k; t.v = dv + L.tgt_v;
    const float *wk = reinterpret_cast<const float *>(dv + L.w_k);
    const float *wv = (w_v_host != w_k_host) ? reinterpret_cast<const float *>(dv + L.w_v) : wk;
    return cb_stats_accumulate(ctx, &s, &t, wk, wv, (int64_t)P.Ht * T, T, stream);
}

cb_status cb_stats_state_bytes(cb_ctx *ctx, size_t *bytes)
{
    if (!ctx || ctx->magic != CTX_MAGIC) return CB_ERR_STATE;
    if (!bytes) return CB_ERR_INVALID_ARG;
    *bytes = ctx->lay.slots_bytes;
    return CB_OK;
}

cb_status cb_stats_export(cb_ctx *ctx, void *dst, size_t dst_bytes, int64_t *n_tokens_out, void *stream)
{
    if (!ctx || ctx->magic != CTX_MAGIC) return CB_ERR_STATE;
    if (!dst || !n_tokens_out) return CB_ERR_INVALID_ARG;
    if (dst_bytes < ctx->lay.slots_bytes) return CB_ERR_WORKSPACE;
    cudaError_t e = cudaMemcpyAsync(dst, ctx->ws + ctx->lay.slots_off, ctx->lay.slots_bytes, cudaMemcpyDefault,
                                    static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e);
    *n_tokens_out = ctx->n_tokens;
    return CB_OK;
}

cb_status cb_stats_import(cb_ctx *ctx, const void *src, size_t src_bytes, int64_t n_tokens, void *stream)
{
    if (!ctx || ctx->magic != CTX_MAGIC) return CB_ERR_STATE;
    if (!src || n_tokens < 0) return CB_ERR_INVALID_ARG;
    if (src_bytes != ctx->lay.slots_bytes) return CB_ERR_INVALID_ARG;      // a state of another problem or split count
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(ctx->ws + ctx->lay.slots_off, src, ctx->lay.slots_bytes, cudaMemcpyDefault, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->ws + ctx->lay.status_off, 0, 256, st);
    if (e != cudaSuccess) return cuda_failed(e);
    ctx->n_tokens = n_tokens;
    ctx->k_operands_centred = false;
    return CB_OK;
}

cb_status cb_stats_reduce(cb_ctx *ctx, float *G, float *C, int64_t *n_tokens_out, void *stream)
{
    if (!ctx || ctx->magic != CTX_MAGIC) return CB_ERR_STATE;
    if (!G || !C) return CB_ERR_INVALID_ARG;
    cudaError_t e = launch_reduce(reinterpret_cast<const float *>(ctx->ws + ctx->lay.slots_off), ctx->n_splits,
                                  ctx->n_maps, ctx->d, G, C, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e);
    if (n_tokens_out) *n_tokens_out = ctx->n_tokens;
    return CB_OK;
}

cb_status cb_ridge_solve(const float *G, const float *C, int32_t n_maps, int32_t d, int64_t n_tokens,
                         const float *lambdas, int32_t n_lambda, uint32_t flags,
                         float *Wb, int32_t *info, void *stream)
{
    if (!G || !C || !lambdas || !Wb || !info) return CB_ERR_INVALID_ARG;
    if (n_maps < 0 || n_lambda <= 0 || n_lambda > 16 || n_tokens < 0) return CB_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return CB_ERR_UNSUPPORTED;
    if (n_maps > 65535 * 16) return CB_ERR_UNSUPPORTED;
    for (int i = 0; i < n_lambda; ++i)
        if (!(lambdas[i] >= 0.f)) return CB_ERR_INVALID_ARG;
    if (n_maps == 0) return CB_OK;
    cudaError_t e = launch_solve(G, C, n_maps, d, n_tokens, lambdas, n_lambda, flags, Wb, info,
                                 static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e);
    return CB_OK;
}

cb_status cb_ridge_solve_large_workspace_bytes(int32_t P, int32_t d, int64_t n_systems, size_t *bytes)
{
    if (P < 2 || (d != 64 && d != 128) || n_systems < 1 || !bytes) return CB_ERR_INVALID_ARG;
    *bytes = solve_large_bytes_per_system(P, d) * (size_t)n_systems;
    return CB_OK;
}

cb_status cb_ridge_solve_large(const float *G, const float *C, int32_t n_maps, int32_t P, int32_t d, int64_t n_tokens,
                               const float *lambdas, int32_t n_lambda, uint32_t flags,
                               float *Wb, int32_t *info, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!G || !C || !lambdas || !Wb || !info) return CB_ERR_INVALID_ARG;
    if (n_maps < 0 || n_lambda <= 0 || n_lambda > 16 || n_tokens < 0 || P < 2) return CB_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return CB_ERR_UNSUPPORTED;
    if (P > 8193) return CB_ERR_UNSUPPORTED;
    for (int i = 0; i < n_lambda; ++i)
        if (!(lambdas[i] >= 0.f)) return CB_ERR_INVALID_ARG;
    if (n_maps == 0) return CB_OK;
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < solve_large_bytes_per_system(P, d)) return CB_ERR_WORKSPACE;
    cudaError_t e = launch_solve_large(G, C, n_maps, P, d, n_tokens, lambdas, n_lambda, flags, Wb, info, workspace,
                                       workspace_bytes, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e);
    return CB_OK;
}

cb_status cb_check_info(const int32_t *info, int64_t n, void *stream, int64_t *first_bad)
{
    if (!info || n < 0) return CB_ERR_INVALID_ARG;
    std::vector<int32_t> h((size_t)n);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(h.data(), info, sizeof(int32_t) * (size_t)n, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_failed(e);
    for (int64_t i = 0; i < n; ++i)
        if (h[(size_t)i] != 0) {
            if (first_bad) *first_bad = i;
            return CB_ERR_NOT_PD;
        }
    return CB_OK;
}

static cb_status apply_impl(const cb_problem *prob, const float *Wb, const cb_kv_view *src_cache,
                            void *tgt_k, void *tgt_v, int64_t t_stride_layer, int64_t t_stride_token,
                            int64_t t_stride_head, int32_t out_dtype, void *stream, const RopeOpt *rope)
{
    cb_status s = check_problem(prob);
    if (s != CB_OK) return s;
    if (prob->Lt > 128 || prob->Ht > 64) return CB_ERR_UNSUPPORTED;
    if (rope) {
        if (!rope_base_ok(rope->base_src) || !rope_base_ok(rope->base_tgt)) return CB_ERR_INVALID_ARG;
        if (prob->flags & CB_FLAG_SIMT) return CB_ERR_UNSUPPORTED;
        if (src_cache && src_cache->n_tokens > 0 && (!rope->pos || ((uintptr_t)rope->pos & 3))) return CB_ERR_INVALID_ARG;
    }
    s = check_view(src_cache, prob->Ls, prob->Hs, prob->ds);
    if (s != CB_OK) return s;
    if (out_dtype != CB_DTYPE_BF16 && out_dtype != CB_DTYPE_F32) return CB_ERR_INVALID_ARG;
    if (src_cache->n_tokens == 0) return CB_OK;
    if (!Wb || !tgt_k || !tgt_v) return CB_ERR_INVALID_ARG;
    if ((((uintptr_t)tgt_k | (uintptr_t)tgt_v | (uintptr_t)Wb) & 15)) return CB_ERR_INVALID_ARG;
    s = check_out_strides(prob->Lt, prob->Ht, t_stride_layer, t_stride_token, t_stride_head);
    if (s != CB_OK) return s;

    ApplyArgs a;
    a.src = KVPtr{static_cast<const __nv_bfloat16 *>(src_cache->k), static_cast<const __nv_bfloat16 *>(src_cache->v),
                  src_cache->stride_layer, src_cache->stride_token, src_cache->stride_head};
    a.Wb = Wb; a.out_k = tgt_k; a.out_v = tgt_v;
    a.o_sl = t_stride_layer; a.o_st = t_stride_token; a.o_sh = t_stride_head;
    a.out_dtype = out_dtype;
    a.n_tokens = (int)src_cache->n_tokens;
    a.Lt = prob->Lt; a.Ht = prob->Ht;
    std::memset(a.src_layer, 0, sizeof a.src_layer);
    std::memset(a.src_head, 0, sizeof a.src_head);
    for (int l = 0; l < prob->Lt; ++l) a.src_layer[l] = prob->src_layer[l];
    for (int h = 0; h < prob->Ht; ++h) a.src_head[h] = prob->src_head[h];
    if (rope) { a.rope_pos = rope->pos; a.rope_base_src = rope->base_src; a.rope_base_tgt = rope->base_tgt; }
    fill_launch_state(a);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = (prob->flags & CB_FLAG_SIMT) ? launch_apply_simt(a, prob->ds, st)
                                                 : launch_apply_tc(a, prob->ds, src_cache, st);
    if (e != cudaSuccess) return cuda_failed(e);
    return CB_OK;
}

cb_status cb_apply(const cb_problem *prob, const float *Wb, const cb_kv_view *src_cache,
                   void *tgt_k, void *tgt_v, int64_t t_stride_layer, int64_t t_stride_token,
                   int64_t t_stride_head, int32_t out_dtype, void *stream)
{
    return apply_impl(prob, Wb, src_cache, tgt_k, tgt_v, t_stride_layer, t_stride_token, t_stride_head, out_dtype, stream,
                      nullptr);
}

cb_status cb_apply_rope(const cb_problem *prob, const float *Wb, const cb_kv_view *src_cache,
                        void *tgt_k, void *tgt_v, int64_t t_stride_layer, int64_t t_stride_token,
                        int64_t t_stride_head, int32_t out_dtype,
                        const int32_t *positions, double rope_base_src, double rope_base_tgt, void *stream)
{
    const RopeOpt r{positions, rope_base_src, rope_base_tgt};
    return apply_impl(prob, Wb, src_cache, tgt_k, tgt_v, t_stride_layer, t_stride_token, t_stride_head, out_dtype, stream, &r);
}

cb_status cb_fullhead_layer_sets(int32_t Ls, int32_t Lt, int32_t k, int32_t *layer_sets)
{
    if (Ls <= 0 || Lt <= 0 || k <= 0 || k > Ls || !layer_sets) return CB_ERR_INVALID_ARG;
    for (int32_t l = 0; l < Lt; ++l) {
        int32_t c = 0;
        if (Lt > 1) c = (int32_t)(((int64_t)2 * l * (Ls - 1) + (Lt - 1)) / ((int64_t)2 * (Lt - 1)));
        int32_t lo = c - 1;
        if (lo + k > Ls) lo = Ls - k;
        if (lo < 0) lo = 0;
        for (int32_t q = 0; q < k; ++q) layer_sets[l * k + q] = lo + q;
    }
    return CB_OK;
}

static cb_status check_fullhead(const cb_fullhead_problem *p)
{
    if (!p || !p->layer_sets) return CB_ERR_INVALID_ARG;
    if (p->Ls <= 0 || p->Hs <= 0 || p->Lt <= 0 || p->Ht <= 0 || p->k <= 0 || p->k > p->Ls) return CB_ERR_INVALID_ARG;
    if (p->ds != p->dt || (p->ds != 64 && p->ds != 128)) return CB_ERR_UNSUPPORTED;
    const int F = p->k * p->Hs;
    if (F > 64) return CB_ERR_UNSUPPORTED;
    for (int i = 0; i < p->Lt * p->k; ++i)
        if (p->layer_sets[i] < 0 || p->layer_sets[i] >= p->Ls) return CB_ERR_INVALID_ARG;
    return CB_OK;
}

static int fullhead_ng(int F) { int n = 0; for (int i = 0; i < F; ++i) n += i / 2 + 1; return n; }

cb_status cb_fullhead_workspace_bytes(const cb_fullhead_problem *prob, size_t *bytes)
{
    cb_status s = check_fullhead(prob);
    if (s != CB_OK) return s;
    if (!bytes) return CB_ERR_INVALID_ARG;
    const int F = prob->k * prob->Hs;
    *bytes = align_up(sizeof(int) * ((size_t)prob->Lt * prob->k + 2 * (size_t)fullhead_ng(F)), 256);
    return CB_OK;
}

cb_status cb_fullhead_stats_accumulate(const cb_fullhead_problem *prob, const cb_kv_view *src, const cb_kv_view *tgt,
                                       const float *w_k, const float *w_v, int64_t w_stride_layer,
                                       float *G, float *C, void *workspace, size_t workspace_bytes, void *stream)
{
    cb_status s = check_fullhead(prob);
    if (s != CB_OK) return s;
    s = check_view(src, prob->Ls, prob->Hs, prob->ds);
    if (s != CB_OK) return s;
    s = check_view(tgt, prob->Lt, prob->Ht, prob->dt);
    if (s != CB_OK) return s;
    if (src->n_tokens != tgt->n_tokens) return CB_ERR_INVALID_ARG;
    if (src->n_tokens == 0) return CB_OK;
    if (!w_k || !w_v || w_stride_layer < 0 || !G || !C) return CB_ERR_INVALID_ARG;
    const int F = prob->k * prob->Hs, NG = fullhead_ng(F);
    size_t need = 0;
    cb_fullhead_workspace_bytes(prob, &need);
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return CB_ERR_WORKSPACE;

    std::vector<int32_t> tab(prob->layer_sets, prob->layer_sets + (size_t)prob->Lt * prob->k);
    std::vector<int32_t> gi, gq;
    for (int i = 0; i < F; ++i)
        for (int q = 0; 2 * q <= i; ++q) { gi.push_back(i); gq.push_back(q); }
    tab.insert(tab.end(), gi.begin(), gi.end());
    tab.insert(tab.end(), gq.begin(), gq.end());
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (const cudaError_t ce = cudaMemcpyAsync(workspace, tab.data(), tab.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st); ce != cudaSuccess) return cuda_failed(ce);
    AccumArgs a;
    a.src = KVPtr{static_cast<const __nv_bfloat16 *>(src->k), static_cast<const __nv_bfloat16 *>(src->v),
                  src->stride_layer, src->stride_token, src->stride_head};
    a.tgt = KVPtr{static_cast<const __nv_bfloat16 *>(tgt->k), static_cast<const __nv_bfloat16 *>(tgt->v),
                  tgt->stride_layer, tgt->stride_token, tgt->stride_head};
    a.w_k = w_k; a.w_v = w_v; a.w_sl = w_stride_layer; a.w_sh = 0;
    a.n_tokens = (int)src->n_tokens;
    a.Lt = prob->Lt; a.Ht = prob->Ht; a.n_splits = 1;
    a.src_layer = nullptr; a.src_head = nullptr; a.slots = nullptr; a.status = nullptr; a.compensated = 0;
    fill_launch_state(a);
    FullHeadArgs f;
    f.G = G; f.C = C;
    f.layer_sets = static_cast<const int *>(workspace);
    f.gi = f.layer_sets + (size_t)prob->Lt * prob->k;
    f.gq = f.gi + NG;
    f.src_head = nullptr; f.per_head = 0;
    f.F = F; f.k = prob->k; f.Hs = prob->Hs; f.PF = F * prob->ds + 1; f.NG = NG; f.NC = F * prob->Ht;
    const cudaError_t e = ((prob->flags & CB_FLAG_ONE_ROW_HEAD) || prob->ds != 128) ? launch_fullhead_tc(a, f, prob->ds, src, tgt, st)
                                                               : launch_gram2_tc(a, f, prob->ds, src, tgt, st);
    if (e != cudaSuccess) return cuda_failed(e);
    return CB_OK;
}

cb_status cb_multilayer_workspace_bytes(const cb_fullhead_problem *prob, size_t *bytes)
{
    if (!prob || !bytes || prob->k <= 0 || prob->k > 64 || prob->Lt <= 0 || prob->Ht <= 0) return CB_ERR_INVALID_ARG;
    *bytes = align_up(sizeof(int) * ((size_t)prob->Lt * prob->k + 2 * (size_t)fullhead_ng(prob->k) + (size_t)prob->Ht), 256);
    return CB_OK;
}

cb_status cb_multilayer_stats_accumulate(const cb_fullhead_problem *prob, const int32_t *src_head,
                                         const cb_kv_view *src, const cb_kv_view *tgt,
                                         const float *w_k, const float *w_v, int64_t w_stride_layer, int64_t w_stride_head,
                                         float *G, float *C, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!prob || !prob->layer_sets || !src_head) return CB_ERR_INVALID_ARG;
    if (prob->Ls <= 0 || prob->Hs <= 0 || prob->Lt <= 0 || prob->Ht <= 0 || prob->k <= 0 || prob->k > prob->Ls || prob->k > 64)
        return CB_ERR_INVALID_ARG;
    if (prob->ds != prob->dt || (prob->ds != 64 && prob->ds != 128)) return CB_ERR_UNSUPPORTED;
    for (int i = 0; i < prob->Lt * prob->k; ++i)
        if (prob->layer_sets[i] < 0 || prob->layer_sets[i] >= prob->Ls) return CB_ERR_INVALID_ARG;
    for (int h = 0; h < prob->Ht; ++h)
        if (src_head[h] < 0 || src_head[h] >= prob->Hs) return CB_ERR_INVALID_ARG;
    cb_status s = check_view(src, prob->Ls, prob->Hs, prob->ds);
    if (s != CB_OK) return s;
    s = check_view(tgt, prob->Lt, prob->Ht, prob->dt);
    if (s != CB_OK) return s;
    if (src->n_tokens != tgt->n_tokens) return CB_ERR_INVALID_ARG;
    if (src->n_tokens == 0) return CB_OK;
    if (!w_k || !w_v || w_stride_layer < 0 || w_stride_head < 0 || !G || !C) return CB_ERR_INVALID_ARG;
    const int F = prob->k, NG = fullhead_ng(F);
    size_t need = 0;
    cb_multilayer_workspace_bytes(prob, &need);
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return CB_ERR_WORKSPACE;
    std::vector<int32_t> tab(prob->layer_sets, prob->layer_sets + (size_t)prob->Lt * prob->k);
    for (int i = 0; i < F; ++i)
        for (int q = 0; 2 * q <= i; ++q) tab.push_back(i);
    for (int i = 0; i < F; ++i)
        for (int q = 0; 2 * q <= i; ++q) tab.push_back(q);
    tab.insert(tab.end(), src_head, src_head + prob->Ht);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (const cudaError_t ce = cudaMemcpyAsync(workspace, tab.data(), tab.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st); ce != cudaSuccess) return cuda_failed(ce);
    AccumArgs a;
    a.src = KVPtr{static_cast<const __nv_bfloat16 *>(src->k), static_cast<const __nv_bfloat16 *>(src->v),
                  src->stride_layer, src->stride_token, src->stride_head};
    a.tgt = KVPtr{static_cast<const __nv_bfloat16 *>(tgt->k), static_cast<const __nv_bfloat16 *>(tgt->v),
                  tgt->stride_layer, tgt->stride_token, tgt->stride_head};
    a.w_k = w_k; a.w_v = w_v; a.w_sl = w_stride_layer; a.w_sh = w_stride_head;
    a.n_tokens = (int)src->n_tokens;
    a.Lt = prob->Lt; a.Ht = prob->Ht; a.n_splits = 1;
    a.src_layer = nullptr; a.src_head = nullptr; a.slots = nullptr; a.status = nullptr; a.compensated = 0;
    fill_launch_state(a);
    FullHeadArgs f;
    f.G = G; f.C = C;
    f.layer_sets = static_cast<const int *>(workspace);
    f.gi = f.layer_sets + (size_t)prob->Lt * prob->k;
    f.gq = f.gi + NG;
    f.src_head = f.gq + NG;
    f.per_head = 1;
    f.F = F; f.k = prob->k; f.Hs = prob->Hs; f.PF = F * prob->ds + 1; f.NG = NG; f.NC = F;
    const cudaError_t e = ((prob->flags & CB_FLAG_ONE_ROW_HEAD) || prob->ds != 128) ? launch_fullhead_tc(a, f, prob->ds, src, tgt, st)
                                                               : launch_gram2_tc(a, f, prob->ds, src, tgt, st);
    if (e != cudaSuccess) return cuda_failed(e);
    return CB_OK;
}

cb_status cb_apply_multilayer_workspace_bytes(const cb_fullhead_problem *prob, size_t *bytes)
{
    if (!prob || !bytes || prob->k <= 0 || prob->Lt <= 0 || prob->Ht <= 0 || (prob->ds != 64 && prob->ds != 128)) return CB_ERR_INVALID_ARG;
    *bytes = apply_ml_workspace_bytes(2 * prob->Lt * prob->Ht, prob->k, prob->ds, prob->Lt);
    return CB_OK;
}

cb_status cb_apply_multilayer(const cb_fullhead_problem *prob, const int32_t *src_head, const float *Wb,
                              const cb_kv_view *src_cache, void *tgt_k, void *tgt_v,
                              int64_t t_stride_layer, int64_t t_stride_token, int64_t t_stride_head, int32_t out_dtype,
                              void *workspace, size_t workspace_bytes, void *stream)
{
    if (!prob || !prob->layer_sets || !src_head) return CB_ERR_INVALID_ARG;
    if (prob->Ls <= 0 || prob->Hs <= 0 || prob->Lt <= 0 || prob->Ht <= 0 || prob->k <= 0 || prob->k > prob->Ls) return CB_ERR_INVALID_ARG;
    if (prob->ds != prob->dt || (prob->ds != 64 && prob->ds != 128)) return CB_ERR_UNSUPPORTED;
    if (prob->Lt > 128 || prob->Ht > 64) return CB_ERR_UNSUPPORTED;
    for (int i = 0; i < prob->Lt * prob->k; ++i)
        if (prob->layer_sets[i] < 0 || prob->layer_sets[i] >= prob->Ls) return CB_ERR_INVALID_ARG;
    for (int h = 0; h < prob->Ht; ++h)
        if (src_head[h] < 0 || src_head[h] >= prob->Hs) return CB_ERR_INVALID_ARG;
    cb_status s = check_view(src_cache, prob->Ls, prob->Hs, prob->ds);
    if (s != CB_OK) return s;
    if (out_dtype != CB_DTYPE_BF16 && out_dtype != CB_DTYPE_F32) return CB_ERR_INVALID_ARG;
    if (src_cache->n_tokens == 0) return CB_OK;
    if (!Wb || !tgt_k || !tgt_v) return CB_ERR_INVALID_ARG;
    if ((((uintptr_t)tgt_k | (uintptr_t)tgt_v | (uintptr_t)Wb) & 15)) return CB_ERR_INVALID_ARG;
    s = check_out_strides(prob->Lt, prob->Ht, t_stride_layer, t_stride_token, t_stride_head);
    if (s != CB_OK) return s;
    size_t need = 0;
    cb_apply_multilayer_workspace_bytes(prob, &need);
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return CB_ERR_WORKSPACE;
    ApplyArgs a;
    a.src = KVPtr{static_cast<const __nv_bfloat16 *>(src_cache->k), static_cast<const __nv_bfloat16 *>(src_cache->v),
                  src_cache->stride_layer, src_cache->stride_token, src_cache->stride_head};
    a.Wb = Wb; a.out_k = tgt_k; a.out_v = tgt_v;
    a.o_sl = t_stride_layer; a.o_st = t_stride_token; a.o_sh = t_stride_head;
    a.out_dtype = out_dtype;
    a.n_tokens = (int)src_cache->n_tokens;
    a.Lt = prob->Lt; a.Ht = prob->Ht;
    std::memset(a.src_layer, 0, sizeof a.src_layer);
    std::memset(a.src_head, 0, sizeof a.src_head);
    for (int h = 0; h < prob->Ht; ++h) a.src_head[h] = src_head[h];
    fill_launch_state(a);
    if (const cudaError_t ce = launch_apply_ml_tc(a, prob->ds, prob->k, prob->layer_sets, src_cache, workspace, static_cast<cudaStream_t>(stream)); ce != cudaSuccess) return cuda_failed(ce);
    return CB_OK;
}

cb_status cb_device_status(cb_ctx *ctx, void *stream)
{
    if (!ctx || ctx->magic != CTX_MAGIC) return CB_ERR_STATE;
    int h = 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(&h, ctx->ws + ctx->lay.status_off, sizeof h, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_failed(e);
    return h == DEV_OK ? CB_OK : CB_ERR_TIMEOUT;
}

}  // extern "C"
