// Host runtime and C ABI of the KV-CAR decode path: configuration, reuse-map
// resolution, page allocator, weight packing, per-layer device tables and the
// launch logic.  See include/kvcar.h for the contract of every entry point.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "kvcar_internal.h"
#include "kvcar_tc.h"

using namespace kvcar;

namespace {

struct AEHost {
    bool set = false;
    int in_dim = 0, hidden = 0, latent = 0;
    float slope = 0.f, eps = 0.f;
    std::vector<float> enc_w1, enc_b1, enc_bn, enc_w2, enc_b2, dec_w1, dec_b1, dec_bn, dec_w2, dec_b2;
};

struct Resolved {
    int root_layer, root_head, slot;
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// A named range around each call that enqueues work, for timeline tools that read NVTX; without such a tool
// attached the two calls return at once.
struct Range {
    explicit Range(const char *name) { nvtxRangePushA(name); }
    ~Range() { nvtxRangePop(); }
};

constexpr size_t GUARD_BYTES = 256;        // behind every region of the pool buffer; no kernel writes there
constexpr unsigned char GUARD_FILL = 0xA5;

}  // namespace

struct kvcar_ctx {
    kvcar_config cfg{};
    int elem = 4;  // bytes per storage element
    std::vector<int32_t> src[2];
    std::vector<AEHost> ae;  // [layer*2 + which]
    bool bound = false;
    int kernel = KVCAR_KERNEL_AUTO;
    // kvcar_step_layer runs the tile kernel beside the encoder: a stream and two events of the library's own
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    // kvcar_step_layer_host: pinned host slots in which a call's k, v and q are laid out as on the device, so that they
    // cross in one copy; a slot is reused once the copy that read it last has completed (its event)
    static constexpr int H_SLOTS = 8;
    char *hstage = nullptr;
    size_t hslot_bytes = 0;
    cudaEvent_t ev_h[H_SLOTS] = {};
    bool ev_h_used[H_SLOTS] = {};
    unsigned hslot = 0;

    // pages
    std::vector<int32_t> free_pages;
    std::vector<std::vector<int32_t>> table;
    std::vector<int32_t> len;
    std::vector<char> open;
    std::vector<int4> pending;  // device table updates not yet enqueued
    bool table_dirty_all = false;
    std::vector<size_t> guard_off;  // offsets (pool buffer) of the GUARD_BYTES-byte guard regions, filled at bind

    // device buffers and layout
    char *pool = nullptr, *weights = nullptr, *ws = nullptr;
    std::vector<size_t> pool_off, cur_off;  // [layer*2+which]
    std::vector<int> width;                 // elements per row
    std::vector<size_t> qparam_off;         // int8 latent rows: offset of the (scale, zero-point) array, else 0
    std::vector<char> quant;                // [layer*2+which]: rows are int8 codes
    size_t pool_bytes = 0, weights_bytes = 0, ws_bytes = 0;
    size_t plan_off = 0, enc_off = 0, tmap_off = 0, tcpart_off = 0;  // inside weights
    size_t bt_off = 0, len_off = 0, status_off = 0, part_off = 0, stage_off = 0, enchid_off = 0, kvsplit_off = 0, pfhid_off = 0, abs_off = 0;  // inside workspace
    int max_k_sources = 0;  // most distinct source layers any layer's K heads resolve to
    bool raw_maps = false;  // every raw bf16 pool has its TMA descriptor (raw-row kernel stages with tensor loads)
    std::vector<EncPlan> enc_host;  // the device's EncPlan table, host copy (tensor-core prefill builds tensor maps from it)
    int max_chunks = 0, chunk_tokens = 128;
    int max_d = 0, max_m = 0, max_in = 0;
    std::vector<LayerPlan> plans_host;
    TcState tc;
    float *static_scratch = nullptr;  // device address of the built-in scratch array, looked up at bind time

    int64_t launches = 0;
    std::string err;
};

namespace {

kvcar_status fail(kvcar_ctx *c, kvcar_status s, const std::string &msg) {
    if (c) c->err = msg;
    return s;
}
kvcar_status cuda_fail(kvcar_ctx *c, cudaError_t e, const char *what) {
    return fail(c, KVCAR_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

std::vector<int> stored_heads(const kvcar_ctx *c, int layer, int which) {
    std::vector<int> h;
    for (int i = 0; i < c->cfg.n_kv_heads; ++i)
        if (c->src[which][layer * c->cfg.n_kv_heads + i] < 0) h.push_back(i);
    return h;
}

Resolved resolve(const kvcar_ctx *c, int layer, int head, int which) {
    const int hkv = c->cfg.n_kv_heads;
    int l = layer, h = head;
    while (c->src[which][l * hkv + h] >= 0) {
        h = c->src[which][l * hkv + h];
        --l;
    }
    int slot = 0;
    for (int i = 0; i < h; ++i)
        if (c->src[which][l * hkv + i] < 0) ++slot;
    return {l, h, slot};
}

int stored_width(const kvcar_ctx *c, int layer, int which) {
    const AEHost &a = c->ae[layer * 2 + which];
    if (a.set) return a.latent;
    return (int)stored_heads(c, layer, which).size() * c->cfg.head_dim;
}

void compute_layout(kvcar_ctx *c) {
    const kvcar_config &g = c->cfg;
    const int nl = g.n_layers;
    const size_t rows = (size_t)g.max_pages * g.page_tokens;
    const int W = g.n_kv_heads * g.head_dim;
    c->pool_off.assign(nl * 2, 0);
    c->cur_off.assign(nl * 2, 0);
    c->width.assign(nl * 2, 0);
    c->qparam_off.assign(nl * 2, 0);
    c->quant.assign(nl * 2, 0);
    size_t off = 0;
    c->guard_off.clear();
    c->max_d = c->max_m = c->max_in = 0;
    for (int i = 0; i < nl * 2; ++i) {
        c->width[i] = stored_width(c, i / 2, i % 2);
        c->pool_off[i] = off;
        const AEHost &a = c->ae[i];
        if (g.latent_quant && a.set) {  // Eq. 4: one byte per element, then (scale, zero-point) per row
            c->quant[i] = 1;
            off = align_up(off + rows * c->width[i], 256);
            c->guard_off.push_back(off);
            off += GUARD_BYTES;
            c->qparam_off[i] = off;
            off = align_up(off + rows * 2 * sizeof(float), 256);
        } else {
            off = align_up(off + rows * c->width[i] * c->elem, 256);
        }
        c->guard_off.push_back(off);  // 256 guard bytes behind every pool region
        off += GUARD_BYTES;
        if (a.set) {
            c->max_d = std::max(c->max_d, a.latent);
            c->max_m = std::max(c->max_m, a.hidden);
            c->max_in = std::max(c->max_in, a.in_dim);
        } else {
            c->max_in = std::max(c->max_in, c->width[i]);
        }
    }
    for (int i = 0; i < nl * 2; ++i) {
        c->cur_off[i] = off;
        off = align_up(off + (size_t)g.max_seqs * W * c->elem, 256);
        c->guard_off.push_back(off);
        off += GUARD_BYTES;
    }
    c->pool_bytes = off;

    // weights: per (layer, which) packed arrays, then LayerPlan[nl], EncPlan[nl*2]
    size_t w = 0;
    for (int i = 0; i < nl * 2; ++i) {
        const AEHost &a = c->ae[i];
        if (!a.set) continue;
        size_t mats = (size_t)a.in_dim * a.hidden + (size_t)a.hidden * a.latent;  // one half (enc or dec)
        w = align_up(w + 2 * mats * c->elem, 256);                                 // transposed enc + dec
        w = align_up(w + (size_t)(4 * a.hidden + a.latent + a.in_dim) * sizeof(float), 256);  // s,t x2, b2 x2
        if (g.storage == KVCAR_BF16) w = align_up(w + mats * 2, 256);             // K-major decoder copies
        w = align_up(w + mats * c->elem, 256);                                     // row-major encoder copies
    }
    c->plan_off = w;
    w = align_up(w + (size_t)nl * sizeof(LayerPlan), 256);
    c->enc_off = w;
    w = align_up(w + (size_t)nl * 2 * sizeof(EncPlan), 256);
    c->tmap_off = w;  // TMA descriptors of the tensor-core kernel: pool, decoder FC1, decoder FC2 per (layer, which)
    w = align_up(w + (size_t)nl * 2 * 3 * 128 + 128, 256);  // + the descriptor of the absorbed-score operands
    c->tcpart_off = w;  // per-layer job tables of the tensor-core kernel
    w = align_up(w + tc_part_bytes(nl), 256);
    c->weights_bytes = w;

    // workspace
    c->chunk_tokens = 128;
    const int cap = g.max_pages_per_seq * g.page_tokens;
    c->max_chunks = (cap + c->chunk_tokens - 1) / c->chunk_tokens;
    size_t s = 0;
    c->bt_off = s;
    s = align_up(s + (size_t)g.max_seqs * g.max_pages_per_seq * 4, 256);
    c->len_off = s;
    s = align_up(s + (size_t)g.max_seqs * 4, 256);
    c->status_off = s;
    s = align_up(s + 256, 256);
    c->part_off = s;
    const int nb = std::min(g.max_seqs, KVCAR_MAX_BATCH);
    s = align_up(s + (size_t)nb * c->max_chunks * g.n_q_heads * (g.head_dim + 2) * sizeof(float), 256);
    c->stage_off = s;
    s = align_up(s + (size_t)nb * (2 * W + 2 * g.n_q_heads * g.head_dim) * c->elem + 4 * 256, 256);
    c->enchid_off = s;  // hidden activations between the two decode-time encoder launches
    s = align_up(s + (size_t)2 * nb * c->max_m * sizeof(float), 256);
    c->kvsplit_off = s;  // probabilities handed from K clusters to V clusters (tensor-core kernel, small grids)
    s = align_up(s + tc_split_bytes(g), 256);
    c->pfhid_off = s;  // bf16 hidden activations between the two launches of the tensor-core prefill
    if (g.storage == KVCAR_BF16 && c->max_m > 0) s = align_up(s + prefill_tc_scratch_bytes(c->max_m), 256);
    c->max_k_sources = 0;
    for (int l = 0; l < nl; ++l) {
        std::vector<char> seen(nl, 0);
        int n = 0;
        for (int h = 0; h < g.n_kv_heads; ++h) {
            const int r = resolve(c, l, h, 0).root_layer;
            if (!seen[r]) {
                seen[r] = 1;
                ++n;
            }
        }
        c->max_k_sources = std::max(c->max_k_sources, n);
    }
    c->abs_off = s;  // operands of the absorbed K scores (tensor-core kernel, KVCAR_ABSORBED)
    s = align_up(s + tc_absorb_bytes(g, c->max_k_sources, c->max_m, nb, c->max_chunks), 256);
    c->ws_bytes = s;
}

void put_elems(char *dst, const float *src, size_t n, int dtype) {
    if (dtype == KVCAR_F32) {
        memcpy(dst, src, n * 4);
    } else {
        __nv_bfloat16 *d = reinterpret_cast<__nv_bfloat16 *>(dst);
        for (size_t i = 0; i < n; ++i) d[i] = __float2bfloat16_rn(src[i]);
    }
}

// transposed copy: src [rows][cols] -> dst [cols][rows]
void put_transposed(char *dst, const float *src, int rows, int cols, int dtype) {
    std::vector<float> t((size_t)rows * cols);
    for (int r = 0; r < rows; ++r)
        for (int cc = 0; cc < cols; ++cc) t[(size_t)cc * rows + r] = src[(size_t)r * cols + cc];
    put_elems(dst, t.data(), t.size(), dtype);
}

// bias + BatchNorm(inference) as one scale/shift per feature
void fuse_bn(const std::vector<float> &b1, const std::vector<float> &bn, int m, float eps, float *s, float *t) {
    for (int j = 0; j < m; ++j) {
        double gamma = bn[j], beta = bn[m + j], mean = bn[2 * m + j], var = bn[3 * m + j];
        double sc = gamma / std::sqrt(var + (double)eps);
        s[j] = (float)sc;
        t[j] = (float)(((double)b1[j] - mean) * sc + beta);
    }
}

bool check_seqs(kvcar_ctx *c, const int32_t *seqs, int n) {
    if (!seqs || n <= 0 || n > KVCAR_MAX_BATCH) return false;
    for (int i = 0; i < n; ++i) {
        if (seqs[i] < 0 || seqs[i] >= c->cfg.max_seqs || !c->open[seqs[i]]) return false;
    }
    return true;
}

kvcar_status reserve_pages(kvcar_ctx *c, const int32_t *seqs, int n, int n_tokens) {
    const int P = c->cfg.page_tokens;
    size_t need_total = 0;
    std::vector<int> need(n);
    for (int i = 0; i < n; ++i) {
        int s = seqs[i];
        int want = (c->len[s] + n_tokens + P - 1) / P;
        if (want > c->cfg.max_pages_per_seq) return fail(c, KVCAR_ERR_OOM_PAGES, "sequence exceeds max_pages_per_seq");
        need[i] = std::max(0, want - (int)c->table[s].size());
        need_total += need[i];
    }
    if (need_total > c->free_pages.size()) return fail(c, KVCAR_ERR_OOM_PAGES, "page pool exhausted");
    for (int i = 0; i < n; ++i) {
        int s = seqs[i];
        for (int k = 0; k < need[i]; ++k) {
            int page = c->free_pages.back();
            c->free_pages.pop_back();
            c->pending.push_back(make_int4(0, s, (int)c->table[s].size(), page));
            c->table[s].push_back(page);
        }
    }
    return KVCAR_OK;
}

// bring the device copies of the page table and sequence lengths up to date, in stream order
kvcar_status flush_tables(kvcar_ctx *c, cudaStream_t st) {
    if (c->pending.empty()) return KVCAR_OK;
    int32_t *bt = reinterpret_cast<int32_t *>(c->ws + c->bt_off);
    int32_t *ln = reinterpret_cast<int32_t *>(c->ws + c->len_off);
    if (c->pending.size() > 4 * 240) {
        // many changes: re-send both tables whole (pageable source: staged before the call returns)
        const int mp = c->cfg.max_pages_per_seq;
        std::vector<int32_t> full((size_t)c->cfg.max_seqs * mp, 0);
        for (int s = 0; s < c->cfg.max_seqs; ++s)
            for (size_t i = 0; i < c->table[s].size(); ++i) full[(size_t)s * mp + i] = c->table[s][i];
        // the host mirror of the lengths is what the device must see once every pending update is applied
        cudaError_t e = cudaMemcpyAsync(bt, full.data(), full.size() * 4, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(ln, c->len.data(), c->len.size() * 4, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) return cuda_fail(c, e, "upload tables");
        c->pending.clear();
        return KVCAR_OK;
    }
    size_t done = 0;
    while (done < c->pending.size()) {
        TableUpdates u;
        u.max_pages_per_seq = c->cfg.max_pages_per_seq;
        u.n = (int)std::min<size_t>(240, c->pending.size() - done);
        memcpy(u.e, c->pending.data() + done, (size_t)u.n * sizeof(int4));
        cudaError_t e = launch_table_updates(bt, ln, u, st);
        if (e != cudaSuccess) return cuda_fail(c, e, "table update launch");
        ++c->launches;
        done += u.n;
    }
    c->pending.clear();
    return KVCAR_OK;
}

// every K and V head of the layer reads raw rows, and the shape fits the streaming kernel
bool layer_is_raw(const kvcar_ctx *c, int layer) {
    if (c->cfg.head_dim != 64 || c->cfg.n_q_heads / c->cfg.n_kv_heads > 8) return false;
    const LayerPlan &lp = c->plans_host[layer];
    for (int w = 0; w < 2; ++w)
        for (int s = 0; s < lp.w[w].n_src; ++s)
            if (lp.w[w].src[s].compressed) return false;
    return true;
}

bool use_tensor_kernel(const kvcar_ctx *c) {
    if (c->kernel == KVCAR_KERNEL_GENERIC) return false;
    return c->tc.available;
}

// device address of the library's built-in scratch array on the current device (defined with the array, below)
cudaError_t static_scratch_for_current_device(float **out);

}  // namespace

// =============================================================================
extern "C" {

kvcar_status kvcar_create(const kvcar_config *cfg, kvcar_ctx **out_ctx) {
    if (!cfg || !out_ctx) return KVCAR_ERR_INVALID_ARG;
    const kvcar_config &g = *cfg;
    if (g.n_layers <= 0 || g.n_q_heads <= 0 || g.n_kv_heads <= 0 || g.head_dim <= 0 || g.page_tokens <= 0 ||
        g.max_seqs <= 0 || g.max_pages <= 0 || g.max_pages_per_seq <= 0)
        return KVCAR_ERR_INVALID_ARG;
    if (g.n_q_heads % g.n_kv_heads != 0 || g.n_kv_heads > KVCAR_MAX_KV_HEADS || g.n_q_heads > KVCAR_MAX_Q_HEADS ||
        g.head_dim > KVCAR_MAX_HEAD_DIM || g.head_dim % 4 != 0)
        return KVCAR_ERR_INVALID_ARG;
    if (g.storage != KVCAR_F32 && g.storage != KVCAR_BF16) return KVCAR_ERR_INVALID_ARG;
    kvcar_ctx *c = new (std::nothrow) kvcar_ctx();
    if (!c) return KVCAR_ERR_INVALID_ARG;
    c->cfg = g;
    c->elem = g.storage == KVCAR_F32 ? 4 : 2;
    for (int w = 0; w < 2; ++w) c->src[w].assign((size_t)g.n_layers * g.n_kv_heads, -1);
    c->ae.resize((size_t)g.n_layers * 2);
    c->free_pages.resize(g.max_pages);
    for (int i = 0; i < g.max_pages; ++i) c->free_pages[i] = g.max_pages - 1 - i;  // back() pops 0 first
    c->table.resize(g.max_seqs);
    c->len.assign(g.max_seqs, 0);
    c->open.assign(g.max_seqs, 0);
    *out_ctx = c;
    return KVCAR_OK;
}

kvcar_status kvcar_destroy(kvcar_ctx *ctx) {
    if (!ctx) return KVCAR_ERR_INVALID_ARG;
    tc_destroy(ctx->tc);
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    if (ctx->side) cudaStreamDestroy(ctx->side);
    for (cudaEvent_t e : ctx->ev_h)
        if (e) cudaEventDestroy(e);
    if (ctx->hstage) cudaFreeHost(ctx->hstage);
    delete ctx;
    return KVCAR_OK;
}

kvcar_status kvcar_set_reuse_map(kvcar_ctx *c, const int32_t *src_k, const int32_t *src_v) {
    if (!c || !src_k || !src_v) return fail(c, KVCAR_ERR_INVALID_ARG, "null argument");
    if (c->bound) return fail(c, KVCAR_ERR_STATE, "reuse map is frozen after kvcar_bind_memory");
    for (const AEHost &a : c->ae)
        if (a.set) return fail(c, KVCAR_ERR_STATE, "set the reuse map before the autoencoders");
    const int hkv = c->cfg.n_kv_heads, n = c->cfg.n_layers * hkv;
    const int32_t *in[2] = {src_k, src_v};
    for (int w = 0; w < 2; ++w)
        for (int i = 0; i < n; ++i) {
            int v = in[w][i];
            if (v < -1 || v >= hkv) return fail(c, KVCAR_ERR_INVALID_ARG, "reuse entry out of range");
            if (i < hkv && v != -1) return fail(c, KVCAR_ERR_INVALID_ARG, "layer 0 has no layer below it");
        }
    for (int w = 0; w < 2; ++w) c->src[w].assign(in[w], in[w] + n);
    return KVCAR_OK;
}

kvcar_status kvcar_set_autoencoder(kvcar_ctx *c, int32_t layer, int32_t which, const kvcar_ae *ae) {
    if (!c || !ae) return fail(c, KVCAR_ERR_INVALID_ARG, "null argument");
    if (c->bound) return fail(c, KVCAR_ERR_STATE, "autoencoders are frozen after kvcar_bind_memory");
    if (layer < 0 || layer >= c->cfg.n_layers || (which != 0 && which != 1))
        return fail(c, KVCAR_ERR_INVALID_ARG, "layer/which out of range");
    const int n_stored = (int)stored_heads(c, layer, which).size();
    if (ae->in_dim != n_stored * c->cfg.head_dim || ae->in_dim <= 0)
        return fail(c, KVCAR_ERR_INVALID_ARG, "in_dim must equal stored heads * head_dim");
    if (ae->hidden <= 0 || ae->latent <= 0) return fail(c, KVCAR_ERR_INVALID_ARG, "non-positive width");
    const float *ptrs[] = {ae->enc_w1, ae->enc_b1, ae->enc_bn, ae->enc_w2, ae->enc_b2,
                           ae->dec_w1, ae->dec_b1, ae->dec_bn, ae->dec_w2, ae->dec_b2};
    for (const float *p : ptrs)
        if (!p) return fail(c, KVCAR_ERR_INVALID_ARG, "null weight pointer");
    AEHost &a = c->ae[layer * 2 + which];
    a.set = true;
    a.in_dim = ae->in_dim;
    a.hidden = ae->hidden;
    a.latent = ae->latent;
    a.slope = ae->leaky_slope;
    a.eps = ae->bn_eps;
    const size_t I = a.in_dim, M = a.hidden, D = a.latent;
    a.enc_w1.assign(ae->enc_w1, ae->enc_w1 + M * I);
    a.enc_b1.assign(ae->enc_b1, ae->enc_b1 + M);
    a.enc_bn.assign(ae->enc_bn, ae->enc_bn + 4 * M);
    a.enc_w2.assign(ae->enc_w2, ae->enc_w2 + D * M);
    a.enc_b2.assign(ae->enc_b2, ae->enc_b2 + D);
    a.dec_w1.assign(ae->dec_w1, ae->dec_w1 + M * D);
    a.dec_b1.assign(ae->dec_b1, ae->dec_b1 + M);
    a.dec_bn.assign(ae->dec_bn, ae->dec_bn + 4 * M);
    a.dec_w2.assign(ae->dec_w2, ae->dec_w2 + I * M);
    a.dec_b2.assign(ae->dec_b2, ae->dec_b2 + I);
    return KVCAR_OK;
}

kvcar_status kvcar_required_bytes(kvcar_ctx *c, size_t *pool, size_t *weights, size_t *workspace) {
    if (!c || !pool || !weights || !workspace) return fail(c, KVCAR_ERR_INVALID_ARG, "null argument");
    if (!c->bound) compute_layout(c);
    *pool = c->pool_bytes;
    *weights = c->weights_bytes;
    *workspace = c->ws_bytes;
    return KVCAR_OK;
}

kvcar_status kvcar_bind_memory(kvcar_ctx *c, void *pool, size_t pool_bytes, void *weights, size_t weights_bytes,
                               void *workspace, size_t workspace_bytes, void *stream) {
    Range range_("kvcar_bind_memory");
    if (!c || !pool || !weights || !workspace) return fail(c, KVCAR_ERR_INVALID_ARG, "null argument");
    if (c->bound) return fail(c, KVCAR_ERR_STATE, "memory already bound");
    if (((uintptr_t)pool | (uintptr_t)weights | (uintptr_t)workspace) & 255)
        return fail(c, KVCAR_ERR_INVALID_ARG, "buffers must be 256-byte aligned");
    if (c->cfg.latent_quant) {
        if (c->cfg.storage != KVCAR_BF16) return fail(c, KVCAR_ERR_UNSUPPORTED, "int8 latent rows need bf16 storage");
        for (int i = 0; i < c->cfg.n_layers * 2; ++i) {
            const AEHost &a = c->ae[i];
            if (!a.set && !stored_heads(c, i / 2, i % 2).empty())
                return fail(c, KVCAR_ERR_UNSUPPORTED, "int8 latent rows need an autoencoder wherever heads are stored");
            if (a.set && (a.latent % 16 != 0 || a.latent > a.in_dim))
                return fail(c, KVCAR_ERR_UNSUPPORTED,
                            "int8 latent rows need latent widths that are multiples of 16 and no wider than the input");
        }
    }
    compute_layout(c);
    if (pool_bytes < c->pool_bytes || weights_bytes < c->weights_bytes || workspace_bytes < c->ws_bytes)
        return fail(c, KVCAR_ERR_WORKSPACE, "a bound buffer is smaller than kvcar_required_bytes reports");
    cudaStream_t st = (cudaStream_t)stream;
    const kvcar_config &g = c->cfg;
    const int nl = g.n_layers, hkv = g.n_kv_heads, hd = g.head_dim;
    c->pool = (char *)pool;
    c->weights = (char *)weights;
    c->ws = (char *)workspace;

    std::vector<char> img(c->weights_bytes, 0);
    struct Packed {
        size_t enc_w1t, enc_w2t, dec_w1t, dec_w2t, enc_s, enc_t, enc_b2, dec_s, dec_t, dec_b2, w1k, w2k, enc_w1r, enc_w2r;
    };
    std::vector<Packed> pk(nl * 2);
    size_t w = 0;
    for (int i = 0; i < nl * 2; ++i) {
        const AEHost &a = c->ae[i];
        if (!a.set) continue;
        const size_t I = a.in_dim, M = a.hidden, D = a.latent, E = c->elem;
        Packed &p = pk[i];
        p.enc_w1t = w;
        p.enc_w2t = p.enc_w1t + I * M * E;
        p.dec_w1t = p.enc_w2t + M * D * E;
        p.dec_w2t = p.dec_w1t + D * M * E;
        w = align_up(w + 2 * (I * M + M * D) * E, 256);
        p.enc_s = w;
        p.enc_t = p.enc_s + M * 4;
        p.dec_s = p.enc_t + M * 4;
        p.dec_t = p.dec_s + M * 4;
        p.enc_b2 = p.dec_t + M * 4;
        p.dec_b2 = p.enc_b2 + D * 4;
        w = align_up(w + (4 * M + D + I) * 4, 256);
        put_transposed(&img[p.enc_w1t], a.enc_w1.data(), (int)M, (int)I, g.storage);  // [M][I] -> [I][M]
        put_transposed(&img[p.enc_w2t], a.enc_w2.data(), (int)D, (int)M, g.storage);  // [D][M] -> [M][D]
        put_transposed(&img[p.dec_w1t], a.dec_w1.data(), (int)M, (int)D, g.storage);  // [M][D] -> [D][M]
        put_transposed(&img[p.dec_w2t], a.dec_w2.data(), (int)I, (int)M, g.storage);  // [I][M] -> [M][I]
        fuse_bn(a.enc_b1, a.enc_bn, (int)M, a.eps, (float *)&img[p.enc_s], (float *)&img[p.enc_t]);
        fuse_bn(a.dec_b1, a.dec_bn, (int)M, a.eps, (float *)&img[p.dec_s], (float *)&img[p.dec_t]);
        memcpy(&img[p.enc_b2], a.enc_b2.data(), D * 4);
        memcpy(&img[p.dec_b2], a.dec_b2.data(), I * 4);
        if (g.storage == KVCAR_BF16) {
            p.w1k = w;
            p.w2k = p.w1k + M * D * 2;
            w = align_up(w + (M * D + I * M) * 2, 256);
            put_elems(&img[p.w1k], a.dec_w1.data(), M * D, KVCAR_BF16);
            put_elems(&img[p.w2k], a.dec_w2.data(), I * M, KVCAR_BF16);
        }
        p.enc_w1r = w;
        p.enc_w2r = p.enc_w1r + M * I * E;
        w = align_up(w + (M * I + D * M) * E, 256);
        put_elems(&img[p.enc_w1r], a.enc_w1.data(), M * I, g.storage);
        put_elems(&img[p.enc_w2r], a.enc_w2.data(), D * M, g.storage);
    }

    // per-layer decode plans
    c->plans_host.assign(nl, LayerPlan{});
    LayerPlan *plans = c->plans_host.data();
    for (int l = 0; l < nl; ++l) {
        LayerPlan &lp = plans[l];
        memset(&lp, 0, sizeof(lp));
        for (int which = 0; which < 2; ++which) {
            WhichPlan &wp = lp.w[which];
            wp.n_src = 0;
            for (int h = 0; h < hkv; ++h) {
                Resolved r = resolve(c, l, h, which);
                lp.cur[which][h] = c->pool + c->cur_off[r.root_layer * 2 + which];
                lp.cur_head[which][h] = r.root_head;
                int s = 0;
                for (; s < wp.n_src; ++s)
                    if (wp.src[s].src_layer == r.root_layer) break;
                if (s == wp.n_src) {
                    SourcePlan &sp = wp.src[wp.n_src++];
                    const int idx = r.root_layer * 2 + which;
                    const AEHost &a = c->ae[idx];
                    sp.src_layer = r.root_layer;
                    sp.pool = c->pool + c->pool_off[idx];
                    sp.width = c->width[idx];
                    sp.compressed = a.set ? 1 : 0;
                    sp.qparam = c->quant[idx] ? (const float *)(c->pool + c->qparam_off[idx]) : nullptr;
                    sp.n_need = 0;
                    if (a.set) {
                        sp.d = a.latent;
                        sp.m = a.hidden;
                        sp.in_dim = a.in_dim;
                        sp.slope = a.slope;
                        sp.w1t = c->weights + pk[idx].dec_w1t;
                        sp.w2t = c->weights + pk[idx].dec_w2t;
                        sp.s1 = (const float *)(c->weights + pk[idx].dec_s);
                        sp.t1 = (const float *)(c->weights + pk[idx].dec_t);
                        sp.b2 = (const float *)(c->weights + pk[idx].dec_b2);
                        if (g.storage == KVCAR_BF16) {
                            sp.w1k = c->weights + pk[idx].w1k;
                            sp.w2k = c->weights + pk[idx].w2k;
                        }
                    } else {
                        sp.d = sp.in_dim = sp.width;
                        sp.m = 0;
                    }
                }
                SourcePlan &sp = wp.src[s];
                sp.kv_head[sp.n_need] = (int8_t)h;
                sp.slot[sp.n_need] = (int8_t)r.slot;
                ++sp.n_need;
            }
        }
    }
    // tensor maps and job tables of the tensor-core kernel (fills their regions of the image)
    tc_setup(c->tc, c->cfg, plans, nl, c->weights, c->tmap_off, c->tcpart_off, img.data(),
             (size_t)g.max_pages * g.page_tokens);
    {
        const size_t slot = c->tmap_off + (size_t)nl * 2 * 3 * 128;
        tc_setup_absorb(c->tc, c->cfg, c->max_k_sources, c->max_m, std::min(g.max_seqs, KVCAR_MAX_BATCH), c->max_chunks,
                        c->ws + c->abs_off, img.data() + slot, c->weights + slot);
    }
    // descriptors of the raw pools (their three slots are otherwise unused: a raw pool has no decoder)
    c->raw_maps = g.storage == KVCAR_BF16;
    for (int i = 0; i < nl * 2 && c->raw_maps; ++i) {
        if (c->ae[i].set || c->width[i] == 0) continue;
        c->raw_maps = raw_build_map(img.data() + c->tmap_off + (size_t)i * 3 * 128, c->pool + c->pool_off[i],
                                    (size_t)g.max_pages * g.page_tokens, (uint64_t)c->width[i]);
    }
    c->tc.pbuf = reinterpret_cast<float *>(c->ws + c->kvsplit_off);
    c->tc.pflags = reinterpret_cast<uint32_t *>(c->ws + c->kvsplit_off +
                                                (size_t)TC_SPLIT_TILES * g.n_q_heads * 132 * sizeof(float));
    memcpy(&img[c->plan_off], plans, (size_t)nl * sizeof(LayerPlan));

    std::vector<EncPlan> enc(nl * 2);
    for (int i = 0; i < nl * 2; ++i) {
        EncPlan &e = enc[i];
        memset(&e, 0, sizeof(e));
        const AEHost &a = c->ae[i];
        std::vector<int> heads = stored_heads(c, i / 2, i % 2);
        e.pool = c->pool + c->pool_off[i];
        e.cur = c->pool + c->cur_off[i];
        e.width = c->width[i];
        e.n_stored = (int)heads.size();
        for (size_t k = 0; k < heads.size(); ++k) e.heads[k] = (int8_t)heads[k];
        e.in_dim = e.n_stored * hd;
        e.compressed = a.set ? 1 : 0;
        e.qparam = c->quant[i] ? (float *)(c->pool + c->qparam_off[i]) : nullptr;
        if (a.set) {
            e.d = a.latent;
            e.m = a.hidden;
            e.slope = a.slope;
            e.w1t = c->weights + pk[i].enc_w1t;
            e.w2t = c->weights + pk[i].enc_w2t;
            e.w1r = c->weights + pk[i].enc_w1r;
            e.w2r = c->weights + pk[i].enc_w2r;
            e.s1 = (const float *)(c->weights + pk[i].enc_s);
            e.t1 = (const float *)(c->weights + pk[i].enc_t);
            e.b2 = (const float *)(c->weights + pk[i].enc_b2);
        } else {
            e.d = e.in_dim;
        }
    }
    memcpy(&img[c->enc_off], enc.data(), enc.size() * sizeof(EncPlan));
    c->enc_host = enc;

    cudaError_t e = cudaMemcpyAsync(c->weights, img.data(), img.size(), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->ws, 0, c->part_off, st);  // tables, lengths, status
    if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + c->kvsplit_off, 0, tc_split_bytes(g), st);  // hand-over flags
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(c, e, "upload of packed weights");
    if (!c->side) {  // for kvcar_step_layer; without them it runs its launches in order on the caller's stream
        if (cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            if (c->side) cudaStreamDestroy(c->side);
            c->side = nullptr;
        }
    }
    {   // kvcar_decode_attention_static: take the built-in scratch array's address now, at set-up time (the first
        // lookup on a device loads the array's module, which is when the driver sets its memory aside)
        float *p = nullptr;
        if (static_scratch_for_current_device(&p) != cudaSuccess) cudaGetLastError();
        c->static_scratch = p;
    }
    if (!c->hstage) {  // set-up time: the host-buffer entry point's staging slots (without them it copies k, v, q singly)
        const size_t nbatch = (size_t)std::min(g.max_seqs, KVCAR_MAX_BATCH);
        const size_t kvb = align_up(nbatch * hkv * hd * c->elem, 256), qb = align_up(nbatch * g.n_q_heads * hd * c->elem, 256);
        c->hslot_bytes = 2 * kvb + qb;
        bool ok = cudaHostAlloc((void **)&c->hstage, c->hslot_bytes * kvcar_ctx::H_SLOTS, cudaHostAllocDefault) == cudaSuccess;
        for (int i = 0; ok && i < kvcar_ctx::H_SLOTS; ++i)
            ok = cudaEventCreateWithFlags(&c->ev_h[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) {
            cudaGetLastError();
            if (c->hstage) cudaFreeHost(c->hstage);
            c->hstage = nullptr;
        }
    }
    for (size_t off : c->guard_off)
        if (cudaMemsetAsync(c->pool + off, GUARD_FILL, GUARD_BYTES, st) != cudaSuccess)
            return cuda_fail(c, cudaGetLastError(), "guard fill");
    c->bound = true;
    c->pending.clear();
    // re-queue what host bookkeeping already holds (sequences opened / pages reserved before binding)
    for (int s = 0; s < g.max_seqs; ++s) {
        for (size_t i = 0; i < c->table[s].size(); ++i) c->pending.push_back(make_int4(0, s, (int)i, c->table[s][i]));
        if (c->len[s]) c->pending.push_back(make_int4(1, s, 0, c->len[s]));
    }
    return KVCAR_OK;
}

kvcar_status kvcar_set_kernel(kvcar_ctx *c, int32_t kernel) {
    if (!c || kernel < 0 || kernel > 2) return fail(c, KVCAR_ERR_INVALID_ARG, "unknown kernel family");
    if (kernel == KVCAR_KERNEL_TENSOR && c->bound && !c->tc.available)
        return fail(c, KVCAR_ERR_UNSUPPORTED, std::string("tensor-core kernel unavailable: ") + c->tc.why);
    c->kernel = kernel;
    return KVCAR_OK;
}

kvcar_status kvcar_seq_open(kvcar_ctx *c, int32_t seq) {
    if (!c || seq < 0 || seq >= c->cfg.max_seqs) return fail(c, KVCAR_ERR_INVALID_ARG, "sequence id out of range");
    if (c->open[seq]) return fail(c, KVCAR_ERR_STATE, "sequence already open");
    c->open[seq] = 1;
    c->len[seq] = 0;
    c->pending.push_back(make_int4(1, seq, 0, 0));
    return KVCAR_OK;
}

kvcar_status kvcar_seq_close(kvcar_ctx *c, int32_t seq) {
    if (!c || seq < 0 || seq >= c->cfg.max_seqs) return fail(c, KVCAR_ERR_INVALID_ARG, "sequence id out of range");
    if (!c->open[seq]) return fail(c, KVCAR_ERR_STATE, "sequence not open");
    for (int32_t p : c->table[seq]) c->free_pages.push_back(p);
    c->table[seq].clear();
    c->open[seq] = 0;
    c->len[seq] = 0;
    c->pending.push_back(make_int4(1, seq, 0, 0));
    return KVCAR_OK;
}

kvcar_status kvcar_reserve(kvcar_ctx *c, const int32_t *seqs, int32_t n_seqs, int32_t n_tokens) {
    if (!c) return KVCAR_ERR_INVALID_ARG;
    if (!check_seqs(c, seqs, n_seqs) || n_tokens <= 0) return fail(c, KVCAR_ERR_INVALID_ARG, "bad sequence list");
    return reserve_pages(c, seqs, n_seqs, n_tokens);
}

static kvcar_status enqueue_encode(kvcar_ctx *c, int32_t layer, const int32_t *seqs, int32_t n_seqs, int32_t n_tokens,
                                   const void *k, const void *v, cudaStream_t st);

kvcar_status kvcar_encode_append(kvcar_ctx *c, int32_t layer, const int32_t *seqs, int32_t n_seqs, int32_t n_tokens,
                                 const void *k, const void *v, void *stream) {
    Range range_("kvcar_encode_append");
    if (!c) return KVCAR_ERR_INVALID_ARG;
    if (!c->bound) return fail(c, KVCAR_ERR_STATE, "bind memory first");
    if (layer < 0 || layer >= c->cfg.n_layers || !k || !v || n_tokens <= 0)
        return fail(c, KVCAR_ERR_INVALID_ARG, "bad layer, pointer or token count");
    if (!check_seqs(c, seqs, n_seqs)) return fail(c, KVCAR_ERR_INVALID_ARG, "bad sequence list");
    if (((uintptr_t)k | (uintptr_t)v) & 15) return fail(c, KVCAR_ERR_INVALID_ARG, "k/v must be 16-byte aligned");
    kvcar_status s = reserve_pages(c, seqs, n_seqs, n_tokens);
    if (s != KVCAR_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    s = flush_tables(c, st);
    if (s != KVCAR_OK) return s;
    return enqueue_encode(c, layer, seqs, n_seqs, n_tokens, k, v, st);
}

// the encoder launches of one layer (arguments checked, pages reserved and tables flushed by the caller)
static kvcar_status enqueue_encode(kvcar_ctx *c, int32_t layer, const int32_t *seqs, int32_t n_seqs, int32_t n_tokens,
                                   const void *k, const void *v, cudaStream_t st) {
    EncodeArgs a{};
    a.plan = reinterpret_cast<const EncPlan *>(c->weights + c->enc_off) + layer * 2;
    a.block_table = reinterpret_cast<const int32_t *>(c->ws + c->bt_off);
    a.seq_len = reinterpret_cast<const int32_t *>(c->ws + c->len_off);
    a.k = k;
    a.v = v;
    a.max_pages_per_seq = c->cfg.max_pages_per_seq;
    a.page_tokens = c->cfg.page_tokens;
    a.n_tokens = n_tokens;
    a.kv_width = c->cfg.n_kv_heads * c->cfg.head_dim;
    a.hd = c->cfg.head_dim;
    SeqList sl;
    sl.n = n_seqs;
    memcpy(sl.id, seqs, (size_t)n_seqs * 4);
    // one token per sequence: one launch per fully connected layer, features spread over all SMs
    // (needs 16-byte loadable weight rows and its row block in shared memory)
    const int vl = 16 / c->elem;
    bool split_ok = n_tokens == 1 && !c->cfg.latent_quant && c->cfg.head_dim % vl == 0 && encode_split_smem(c->max_in, c->max_m) <= 200 * 1024;
    for (int w = 0; w < 2 && split_ok; ++w) {
        const AEHost &ae = c->ae[layer * 2 + w];
        if (ae.set && (ae.in_dim % vl || ae.hidden % vl)) split_ok = false;
    }
    const int nb = std::min(c->cfg.max_seqs, KVCAR_MAX_BATCH);
    cudaError_t e = split_ok ? launch_encode_split(a, sl, c->cfg.storage, c->max_in, c->max_m, c->max_d,
                                                   reinterpret_cast<float *>(c->ws + c->enchid_off), nb, st)
                             : launch_encode_generic(a, sl, c->cfg.storage, c->max_in, c->max_m, st);
    if (e != cudaSuccess) return cuda_fail(c, e, "encode launch");
    c->launches += split_ok ? 2 : 1;
    return KVCAR_OK;
}

kvcar_status kvcar_encode_append_tensor(kvcar_ctx *c, int32_t layer, const int32_t *seqs, int32_t n_seqs,
                                        int32_t n_tokens, const void *k, const void *v, void *stream) {
    Range range_("kvcar_encode_append_tensor");
    if (!c) return KVCAR_ERR_INVALID_ARG;
    if (!c->bound) return fail(c, KVCAR_ERR_STATE, "bind memory first");
    if (layer < 0 || layer >= c->cfg.n_layers || !k || !v || n_tokens <= 0)
        return fail(c, KVCAR_ERR_INVALID_ARG, "bad layer, pointer or token count");
    if (!check_seqs(c, seqs, n_seqs)) return fail(c, KVCAR_ERR_INVALID_ARG, "bad sequence list");
    if (((uintptr_t)k | (uintptr_t)v) & 15) return fail(c, KVCAR_ERR_INVALID_ARG, "k/v must be 16-byte aligned");
    const kvcar_config &g = c->cfg;
    if (g.storage != KVCAR_BF16 || g.head_dim != 64 || g.latent_quant)
        return fail(c, KVCAR_ERR_UNSUPPORTED, "the tensor-core encoder takes bf16 storage, bf16 latent rows and 64-wide heads");
    for (int w = 0; w < 2; ++w) {
        const AEHost &ae = c->ae[layer * 2 + w];
        if (!ae.set || ae.hidden % 16 || ae.latent % 16 || ae.hidden > 1024 || ae.latent > 1024)
            return fail(c, KVCAR_ERR_UNSUPPORTED,
                        "the tensor-core encoder needs an autoencoder for K and for V with widths that are multiples of 16");
    }
    if ((int64_t)n_seqs * n_tokens > 0x7fffffff) return fail(c, KVCAR_ERR_INVALID_ARG, "too many rows");
    kvcar_status s = reserve_pages(c, seqs, n_seqs, n_tokens);
    if (s != KVCAR_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    s = flush_tables(c, st);
    if (s != KVCAR_OK) return s;
    PrefillTcArgs a{};
    a.plan_dev = reinterpret_cast<const EncPlan *>(c->weights + c->enc_off) + layer * 2;
    a.plan_host = c->enc_host.data() + layer * 2;
    a.block_table = reinterpret_cast<const int32_t *>(c->ws + c->bt_off);
    a.seq_len = reinterpret_cast<const int32_t *>(c->ws + c->len_off);
    a.status = reinterpret_cast<int32_t *>(c->ws + c->status_off);
    a.src[0] = k;
    a.src[1] = v;
    a.hid = c->ws + c->pfhid_off;
    a.max_m = c->max_m;
    a.max_pages_per_seq = g.max_pages_per_seq;
    a.page_tokens = g.page_tokens;
    a.n_tokens = n_tokens;
    a.kv_width = g.n_kv_heads * g.head_dim;
    SeqList sl;
    sl.n = n_seqs;
    memcpy(sl.id, seqs, (size_t)n_seqs * 4);
    cudaError_t e = launch_prefill_tc(a, sl, st);
    if (e != cudaSuccess) return cuda_fail(c, e, "tensor-core encoder launch");
    c->launches += 2 * (((int64_t)n_seqs * n_tokens + PREFILL_TC_ROWS - 1) / PREFILL_TC_ROWS);
    return KVCAR_OK;
}

kvcar_status kvcar_advance(kvcar_ctx *c, const int32_t *seqs, int32_t n_seqs, int32_t n_tokens, void *stream) {
    Range range_("kvcar_advance");
    if (!c) return KVCAR_ERR_INVALID_ARG;
    if (!check_seqs(c, seqs, n_seqs) || n_tokens <= 0) return fail(c, KVCAR_ERR_INVALID_ARG, "bad sequence list");
    const int P = c->cfg.page_tokens;
    for (int i = 0; i < n_seqs; ++i)
        if (c->len[seqs[i]] + n_tokens > (int)c->table[seqs[i]].size() * P)
            return fail(c, KVCAR_ERR_STATE, "advance beyond reserved pages");
    for (int i = 0; i < n_seqs; ++i) {
        c->len[seqs[i]] += n_tokens;
        c->pending.push_back(make_int4(1, seqs[i], 0, c->len[seqs[i]]));
    }
    if (c->bound) return flush_tables(c, (cudaStream_t)stream);
    return KVCAR_OK;
}

// launch arguments of one layer's decode; returns the number of tiles along the longest listed sequence
static int prepare_decode(kvcar_ctx *c, int32_t layer, const int32_t *seqs, int32_t n_seqs, const void *q, void *out,
                          uint32_t flags, DecodeArgs &a, SeqList &sl) {
    const kvcar_config &g = c->cfg;
    int max_len = 0;
    for (int i = 0; i < n_seqs; ++i) max_len = std::max(max_len, c->len[seqs[i]]);
    a = DecodeArgs{};
    a.plan = reinterpret_cast<const LayerPlan *>(c->weights + c->plan_off) + layer;
    a.block_table = reinterpret_cast<const int32_t *>(c->ws + c->bt_off);
    a.seq_len = reinterpret_cast<const int32_t *>(c->ws + c->len_off);
    a.q = q;
    a.out = out;
    a.partials = reinterpret_cast<float *>(c->ws + c->part_off);
    a.status = reinterpret_cast<int32_t *>(c->ws + c->status_off);
    a.max_pages_per_seq = g.max_pages_per_seq;
    a.page_tokens = g.page_tokens;
    a.hq = g.n_q_heads;
    a.hkv = g.n_kv_heads;
    a.hd = g.head_dim;
    a.chunk_tokens = c->chunk_tokens;
    a.max_chunks = c->max_chunks;
    a.flags = flags;
    a.scale = 1.0f / std::sqrt((float)g.head_dim);
    a.raw_tmaps = c->raw_maps ? c->weights + c->tmap_off : nullptr;
    sl.n = n_seqs;
    memcpy(sl.id, seqs, (size_t)n_seqs * 4);
    return (max_len + c->chunk_tokens - 1) / c->chunk_tokens;
}

// The kernel that works through the cached tokens tile by tile (tensor-core, raw or generic) and leaves one partial
// result per tile.  It reads the cache rows below the sequences' lengths, the tables and q - nothing that this
// step's encoder writes (the exact current token enters in the combine kernel).
static kvcar_status enqueue_decode_tiles(kvcar_ctx *c, int32_t layer, const DecodeArgs &a, const SeqList &sl,
                                         int n_chunks, cudaStream_t st) {
    c->tc.last_mode = 0;
    if (n_chunks <= 0) return KVCAR_OK;
    const kvcar_config &g = c->cfg;
    const bool want_tc = use_tensor_kernel(c) && tc_layer_supported(c->tc, layer);
    if (c->kernel == KVCAR_KERNEL_TENSOR && !want_tc)
        return fail(c, KVCAR_ERR_UNSUPPORTED, std::string("tensor-core kernel cannot run this layer: ") + c->tc.why);
    cudaError_t e;
    if (c->kernel != KVCAR_KERNEL_GENERIC && layer_is_raw(c, layer)) {
        e = launch_decode_raw(a, sl, g.storage, n_chunks, st);
    } else if (want_tc) {
        int32_t lens[KVCAR_MAX_BATCH];
        for (int i = 0; i < sl.n; ++i) lens[i] = c->len[sl.id[i]];
        int n_launches = 1;
        e = tc_launch_decode(c->tc, a, sl, lens, layer, st, &n_launches);
        if (e == cudaSuccess) c->launches += n_launches - 1;
    } else {
        if (decode_generic_smem(a.hq, a.hd, c->max_d, c->max_m) > 227 * 1024)
            return fail(c, KVCAR_ERR_UNSUPPORTED, "shape needs more shared memory than one SM has");
        e = launch_decode_generic(a, sl, g.storage, c->max_d, c->max_m, n_chunks, st);
    }
    if (e != cudaSuccess) return cuda_fail(c, e, "decode launch");
    ++c->launches;
    return KVCAR_OK;
}

static kvcar_status enqueue_combine(kvcar_ctx *c, const DecodeArgs &a, const SeqList &sl, int n_chunks, cudaStream_t st) {
    // a tile launch in the absorbed V form left U vectors, not weighted values: its own merge kernel reads them
    cudaError_t e = c->tc.last_mode == 2 ? tc_launch_combine_absorbed(c->tc, a, sl, st)
                                         : launch_combine(a, sl, c->cfg.storage, n_chunks, st);
    if (e != cudaSuccess) return cuda_fail(c, e, "combine launch");
    ++c->launches;
    return KVCAR_OK;
}

static kvcar_status check_decode_args(kvcar_ctx *c, int32_t layer, const int32_t *seqs, int32_t n_seqs, const void *q,
                                      const void *out, uint32_t flags) {
    if (!c->bound) return fail(c, KVCAR_ERR_STATE, "bind memory first");
    if (layer < 0 || layer >= c->cfg.n_layers || !q || !out)
        return fail(c, KVCAR_ERR_INVALID_ARG, "bad layer or pointer");
    if (!check_seqs(c, seqs, n_seqs)) return fail(c, KVCAR_ERR_INVALID_ARG, "bad sequence list");
    if (((uintptr_t)q | (uintptr_t)out) & 15) return fail(c, KVCAR_ERR_INVALID_ARG, "q/out must be 16-byte aligned");
    if (flags & ~(KVCAR_INCLUDE_CURRENT_EXACT | KVCAR_ABSORBED | KVCAR_ABSORBED_V)) return fail(c, KVCAR_ERR_INVALID_ARG, "unknown flag");
    return KVCAR_OK;
}

kvcar_status kvcar_decode_attention(kvcar_ctx *c, int32_t layer, const int32_t *seqs, int32_t n_seqs, const void *q,
                                    void *out, uint32_t flags, void *stream) {
    Range range_("kvcar_decode_attention");
    if (!c) return KVCAR_ERR_INVALID_ARG;
    kvcar_status s = check_decode_args(c, layer, seqs, n_seqs, q, out, flags);
    if (s != KVCAR_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    s = flush_tables(c, st);
    if (s != KVCAR_OK) return s;
    DecodeArgs a;
    SeqList sl;
    const int n_chunks = prepare_decode(c, layer, seqs, n_seqs, q, out, flags, a, sl);
    s = enqueue_decode_tiles(c, layer, a, sl, n_chunks, st);
    if (s != KVCAR_OK) return s;
    return enqueue_combine(c, a, sl, n_chunks, st);
}

kvcar_status kvcar_step_layer(kvcar_ctx *c, int32_t layer, const int32_t *seqs, int32_t n_seqs, const void *k,
                              const void *v, const void *q, void *out, uint32_t flags, void *stream) {
    Range range_("kvcar_step_layer");
    if (!c) return KVCAR_ERR_INVALID_ARG;
    kvcar_status s = check_decode_args(c, layer, seqs, n_seqs, q, out, flags);
    if (s != KVCAR_OK) return s;
    if (!k || !v) return fail(c, KVCAR_ERR_INVALID_ARG, "null k or v");
    if (((uintptr_t)k | (uintptr_t)v) & 15) return fail(c, KVCAR_ERR_INVALID_ARG, "k/v must be 16-byte aligned");
    s = reserve_pages(c, seqs, n_seqs, 1);
    if (s != KVCAR_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    s = flush_tables(c, st);
    if (s != KVCAR_OK) return s;
    DecodeArgs a;
    SeqList sl;
    const int n_chunks = prepare_decode(c, layer, seqs, n_seqs, q, out, flags, a, sl);
    // The tile kernel does not depend on this step's encoder, so it goes to a side stream that forks here and
    // joins before the combine kernel: the encoder's two short launches overlap it instead of running in front
    // of it.  (The other way round - encoder on the side stream behind the fork event - measured no gain: the
    // encoder then finds a small grid's few idle SMs only and outlasts the tile kernel.)
    const bool fork = c->side != nullptr && n_chunks > 0;
    if (fork) {
        cudaError_t e = cudaEventRecord(c->ev_fork, st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(c->side, c->ev_fork, 0);
        if (e != cudaSuccess) return cuda_fail(c, e, "stream fork");
        s = enqueue_decode_tiles(c, layer, a, sl, n_chunks, c->side);
        cudaError_t e2 = cudaEventRecord(c->ev_join, c->side);  // recorded even after a failed launch: the join below
        if (s != KVCAR_OK) {                                     // must not leave the side stream detached
            cudaStreamWaitEvent(st, c->ev_join, 0);
            return s;
        }
        if (e2 != cudaSuccess) return cuda_fail(c, e2, "stream join");
    }
    s = enqueue_encode(c, layer, seqs, n_seqs, 1, k, v, st);
    if (fork) {
        cudaError_t e = cudaStreamWaitEvent(st, c->ev_join, 0);
        if (e != cudaSuccess) return cuda_fail(c, e, "stream join");
    }
    if (s != KVCAR_OK) return s;
    if (!fork) {
        s = enqueue_decode_tiles(c, layer, a, sl, n_chunks, st);
        if (s != KVCAR_OK) return s;
    }
    return enqueue_combine(c, a, sl, n_chunks, st);
}

kvcar_status kvcar_step_layer_host(kvcar_ctx *c, int32_t layer, const int32_t *seqs, int32_t n_seqs,
                                   const void *k_host, const void *v_host, const void *q_host, void *out_host,
                                   uint32_t flags, void *stream) {
    Range range_("kvcar_step_layer_host");
    if (!c) return KVCAR_ERR_INVALID_ARG;
    if (!c->bound) return fail(c, KVCAR_ERR_STATE, "bind memory first");
    if (!k_host || !v_host || !q_host || !out_host) return fail(c, KVCAR_ERR_INVALID_ARG, "null host buffer");
    if (!check_seqs(c, seqs, n_seqs)) return fail(c, KVCAR_ERR_INVALID_ARG, "bad sequence list");
    const kvcar_config &g = c->cfg;
    const size_t kvb = align_up((size_t)n_seqs * g.n_kv_heads * g.head_dim * c->elem, 256);
    const size_t qb = align_up((size_t)n_seqs * g.n_q_heads * g.head_dim * c->elem, 256);
    char *dk = c->ws + c->stage_off, *dv = dk + kvb, *dq = dv + kvb, *dout = dq + qb;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t kv_bytes = (size_t)n_seqs * g.n_kv_heads * g.head_dim * c->elem;
    const size_t q_bytes = (size_t)n_seqs * g.n_q_heads * g.head_dim * c->elem;
    cudaError_t e;
    if (c->hstage && 2 * kvb + q_bytes <= c->hslot_bytes) {
        // one copy: k, v, q gathered in a pinned slot with the device staging area's layout
        const unsigned slot = c->hslot++ % kvcar_ctx::H_SLOTS;
        if (c->ev_h_used[slot]) {
            e = cudaEventSynchronize(c->ev_h[slot]);  // the copy that read this slot eight calls ago
            if (e != cudaSuccess) return cuda_fail(c, e, "staging slot");
        }
        char *h = c->hstage + (size_t)slot * c->hslot_bytes;
        memcpy(h, k_host, kv_bytes);
        memcpy(h + kvb, v_host, kv_bytes);
        memcpy(h + 2 * kvb, q_host, q_bytes);
        e = cudaMemcpyAsync(dk, h, 2 * kvb + q_bytes, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaEventRecord(c->ev_h[slot], st);
        c->ev_h_used[slot] = e == cudaSuccess;
    } else {
        e = cudaMemcpyAsync(dk, k_host, kv_bytes, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(dv, v_host, kv_bytes, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(dq, q_host, q_bytes, cudaMemcpyHostToDevice, st);
    }
    if (e != cudaSuccess) return cuda_fail(c, e, "host to device copy");
    kvcar_status s = kvcar_step_layer(c, layer, seqs, n_seqs, dk, dv, dq, dout, flags, stream);
    if (s != KVCAR_OK) return s;
    e = cudaMemcpyAsync(out_host, dout, (size_t)n_seqs * g.n_q_heads * g.head_dim * c->elem, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(c, e, "device to host copy");
    return KVCAR_OK;
}

kvcar_status kvcar_debug_resolve(kvcar_ctx *c, int32_t layer, int32_t kv_head, int32_t which, int32_t *root_layer,
                                 int32_t *root_head, int32_t *slot) {
    if (!c || !root_layer || !root_head || !slot) return fail(c, KVCAR_ERR_INVALID_ARG, "null argument");
    if (layer < 0 || layer >= c->cfg.n_layers || kv_head < 0 || kv_head >= c->cfg.n_kv_heads || (which & ~1))
        return fail(c, KVCAR_ERR_INVALID_ARG, "index out of range");
    Resolved r = resolve(c, layer, kv_head, which);
    *root_layer = r.root_layer;
    *root_head = r.root_head;
    *slot = r.slot;
    return KVCAR_OK;
}

kvcar_status kvcar_debug_locate(kvcar_ctx *c, int32_t seq, int32_t token, int32_t *page, int64_t *row) {
    if (!c || !page || !row) return fail(c, KVCAR_ERR_INVALID_ARG, "null argument");
    if (seq < 0 || seq >= c->cfg.max_seqs || !c->open[seq] || token < 0)
        return fail(c, KVCAR_ERR_INVALID_ARG, "sequence not open or token negative");
    const int P = c->cfg.page_tokens;
    if (token / P >= (int)c->table[seq].size()) return fail(c, KVCAR_ERR_INVALID_ARG, "token lies in no reserved page");
    *page = c->table[seq][token / P];
    *row = (int64_t)*page * P + token % P;
    return KVCAR_OK;
}

kvcar_status kvcar_seq_len(kvcar_ctx *c, int32_t seq, int32_t *len) {
    if (!c || !len || seq < 0 || seq >= c->cfg.max_seqs || !c->open[seq])
        return fail(c, KVCAR_ERR_INVALID_ARG, "sequence not open");
    *len = c->len[seq];
    return KVCAR_OK;
}

kvcar_status kvcar_pool_layout(kvcar_ctx *c, int32_t layer, int32_t which, size_t *offset, size_t *row_pitch,
                               int32_t *width) {
    if (!c || !offset || !row_pitch || !width) return fail(c, KVCAR_ERR_INVALID_ARG, "null argument");
    if (layer < 0 || layer >= c->cfg.n_layers || (which & ~1)) return fail(c, KVCAR_ERR_INVALID_ARG, "index out of range");
    if (!c->bound) compute_layout(c);
    const int i = layer * 2 + which;
    *offset = c->pool_off[i];
    *width = c->width[i];
    *row_pitch = (size_t)c->width[i] * (c->quant[i] ? 1 : c->elem);
    return KVCAR_OK;
}

kvcar_status kvcar_pool_quant_layout(kvcar_ctx *c, int32_t layer, int32_t which, size_t *param_offset) {
    if (!c || !param_offset) return fail(c, KVCAR_ERR_INVALID_ARG, "null argument");
    if (layer < 0 || layer >= c->cfg.n_layers || (which & ~1)) return fail(c, KVCAR_ERR_INVALID_ARG, "index out of range");
    if (!c->bound) compute_layout(c);
    if (!c->quant[layer * 2 + which]) return fail(c, KVCAR_ERR_STATE, "this (layer, K/V) holds no int8 rows");
    *param_offset = c->qparam_off[layer * 2 + which];
    return KVCAR_OK;
}

kvcar_status kvcar_cache_bytes_per_token(kvcar_ctx *c, double *compressed, double *uncompressed) {
    if (!c || !compressed || !uncompressed) return fail(c, KVCAR_ERR_INVALID_ARG, "null argument");
    double comp = 0;
    for (int i = 0; i < c->cfg.n_layers * 2; ++i) {
        const int w = stored_width(c, i / 2, i % 2);
        // int8 rows (Eq. 4): one byte per element plus the row's scale and zero-point, where anything is stored
        comp += (c->cfg.latent_quant && c->ae[i].set) ? (w ? w + 8.0 : 0.0) : (double)w * c->elem;
    }
    *compressed = comp;
    *uncompressed = 2.0 * c->cfg.n_layers * c->cfg.n_kv_heads * c->cfg.head_dim * c->elem;
    return KVCAR_OK;
}

kvcar_status kvcar_layer_work_per_token(kvcar_ctx *c, int32_t layer, double *bytes, double *flops) {
    if (!c || !bytes || !flops || layer < 0 || layer >= c->cfg.n_layers)
        return fail(c, KVCAR_ERR_INVALID_ARG, "bad argument");
    const int hkv = c->cfg.n_kv_heads, hd = c->cfg.head_dim;
    double b = 0, f = 0;
    for (int which = 0; which < 2; ++which) {
        std::vector<int> need(c->cfg.n_layers, 0);
        for (int h = 0; h < hkv; ++h) ++need[resolve(c, layer, h, which).root_layer];
        for (int s = 0; s < c->cfg.n_layers; ++s) {
            if (!need[s]) continue;
            const AEHost &a = c->ae[s * 2 + which];
            // a latent row mixes all heads of its layer and is read whole; of a raw row only the needed heads' slices
            if (a.set && c->cfg.latent_quant)
                b += stored_width(c, s, which) + 8.0;
            else
                b += a.set ? (double)stored_width(c, s, which) * c->elem : (double)need[s] * hd * c->elem;
            if (a.set) f += 2.0 * a.latent * a.hidden + 2.0 * a.hidden * hd * need[s];
        }
    }
    f += 4.0 * c->cfg.n_q_heads * hd;  // q.K and p.V
    *bytes = b;
    *flops = f;
    return KVCAR_OK;
}

kvcar_status kvcar_layer_work_absorbed(kvcar_ctx *c, int32_t layer, int32_t both_sides, double *flops) {
    if (!c || !flops || layer < 0 || layer >= c->cfg.n_layers) return fail(c, KVCAR_ERR_INVALID_ARG, "bad argument");
    const int hkv = c->cfg.n_kv_heads, hd = c->cfg.head_dim, group = c->cfg.n_q_heads / hkv;
    double f = 0;
    for (int which = 0; which < 2; ++which) {
        std::vector<int> need(c->cfg.n_layers, 0);
        for (int h = 0; h < hkv; ++h) ++need[resolve(c, layer, h, which).root_layer];
        for (int s = 0; s < c->cfg.n_layers; ++s) {
            if (!need[s]) continue;
            const AEHost &a = c->ae[s * 2 + which];
            if (!a.set) {
                f += 2.0 * need[s] * group * hd;  // raw rows: plain q.k / p.v
                continue;
            }
            f += 2.0 * a.latent * a.hidden;
            if (which == 0 || both_sides)
                f += 2.0 * a.hidden * need[s] * group;
            else
                f += 2.0 * a.hidden * hd * need[s] + 2.0 * need[s] * group * hd;  // second layer + p.v'
        }
    }
    *flops = f;
    return KVCAR_OK;
}

kvcar_status kvcar_launch_count(kvcar_ctx *c, int64_t *count) {
    if (!c || !count) return KVCAR_ERR_INVALID_ARG;
    *count = c->launches;
    return KVCAR_OK;
}

kvcar_status kvcar_layer_kernel(kvcar_ctx *c, int32_t layer, int32_t *kernel) {
    if (!c || !kernel || layer < 0 || layer >= c->cfg.n_layers) return fail(c, KVCAR_ERR_INVALID_ARG, "bad argument");
    if (!c->bound) return fail(c, KVCAR_ERR_STATE, "bind memory first");
    if (c->kernel != KVCAR_KERNEL_GENERIC && layer_is_raw(c, layer))
        *kernel = KVCAR_KERNEL_RAW;
    else
        *kernel = (use_tensor_kernel(c) && tc_layer_supported(c->tc, layer)) ? KVCAR_KERNEL_TENSOR : KVCAR_KERNEL_GENERIC;
    return KVCAR_OK;
}

kvcar_status kvcar_sync_status(kvcar_ctx *c, void *stream) {
    if (!c) return KVCAR_ERR_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "stream synchronize");
    if (c->bound) {
        int32_t status = 0;
        e = cudaMemcpy(&status, c->ws + c->status_off, 4, cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return cuda_fail(c, e, "status read");
        if (status != 0) {
            cudaMemset(c->ws + c->status_off, 0, 4);
            char buf[96];
            snprintf(buf, sizeof buf, "device-side bounded wait ran out (code 0x%x)", status);
            return fail(c, KVCAR_ERR_DEVICE_TIMEOUT, buf);
        }
    }
    return KVCAR_OK;
}

const char *kvcar_last_error(kvcar_ctx *c) { return c ? c->err.c_str() : "null context"; }

kvcar_status kvcar_debug_expire_wait(kvcar_ctx *c, uint64_t limit_ns, void *stream) {
    if (!c) return KVCAR_ERR_INVALID_ARG;
    if (!c->bound) return fail(c, KVCAR_ERR_STATE, "bind memory first");
    if (limit_ns == 0 || limit_ns > 1000000000ull) return fail(c, KVCAR_ERR_INVALID_ARG, "limit must be 1 ns .. 1 s");
    cudaError_t e = tc_launch_expire_wait(reinterpret_cast<int32_t *>(c->ws + c->status_off), limit_ns, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "launch");
    ++c->launches;
    return KVCAR_OK;
}

kvcar_status kvcar_debug_check(kvcar_ctx *c, void *stream, int32_t *what, int64_t *where) {
    if (!c || !what || !where) return fail(c, KVCAR_ERR_INVALID_ARG, "null argument");
    if (!c->bound) return fail(c, KVCAR_ERR_STATE, "bind memory first");
    *what = 0;
    *where = -1;
    cudaStream_t st = (cudaStream_t)stream;
    kvcar_status fs = flush_tables(c, st);
    if (fs != KVCAR_OK) return fs;
    const kvcar_config &g = c->cfg;
    const int mp = g.max_pages_per_seq;
    std::vector<unsigned char> guards(c->guard_off.size() * GUARD_BYTES);
    std::vector<int32_t> bt((size_t)g.max_seqs * mp), ln(g.max_seqs);
    cudaError_t e = cudaSuccess;
    for (size_t i = 0; i < c->guard_off.size() && e == cudaSuccess; ++i)
        e = cudaMemcpyAsync(&guards[i * GUARD_BYTES], c->pool + c->guard_off[i], GUARD_BYTES, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(bt.data(), c->ws + c->bt_off, bt.size() * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ln.data(), c->ws + c->len_off, ln.size() * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(c, e, "read-back for the check");
    for (size_t i = 0; i < guards.size(); ++i)
        if (guards[i] != GUARD_FILL) {
            *what = 1;
            *where = (int64_t)(c->guard_off[i / GUARD_BYTES] + i % GUARD_BYTES);
            return fail(c, KVCAR_ERR_GUARD, "a guard region of the pool buffer was written");
        }
    for (int s = 0; s < g.max_seqs; ++s) {
        if (!c->open[s]) continue;
        for (size_t i = 0; i < c->table[s].size(); ++i)
            if (bt[(size_t)s * mp + i] != c->table[s][i]) {
                *what = 2;
                *where = (int64_t)s * mp + (int64_t)i;
                return fail(c, KVCAR_ERR_GUARD, "the device page table differs from the allocator's");
            }
        if (ln[s] != c->len[s]) {
            *what = 3;
            *where = s;
            return fail(c, KVCAR_ERR_GUARD, "a device sequence length differs from the host's");
        }
    }
    return KVCAR_OK;
}

}  // extern "C"

// =============================================================================
// Allocation-free decode attention: split-KV partials in a fixed array that is
// part of the library image.  In host code `g_static_scratch` is only a handle
// for the runtime, never an address a kernel may use: the device address is
// looked up once per device with cudaGetSymbolAddress and that pointer is what
// the kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[KVCAR_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
float *g_static_scratch_ptr[kMaxDevices] = {};  // per device; filled by the first kvcar_bind_memory there

// Device address of the scratch array on the current device.
cudaError_t static_scratch_for_current_device(float **out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    float *p = __atomic_load_n(&g_static_scratch_ptr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        void *sym = nullptr;
        e = cudaGetSymbolAddress(&sym, g_static_scratch);
        if (e != cudaSuccess) return e;
        p = reinterpret_cast<float *>(sym);
        __atomic_store_n(&g_static_scratch_ptr[dev], p, __ATOMIC_RELEASE);  // same value from any thread
    }
    *out = p;
    return cudaSuccess;
}
}  // namespace

extern "C" kvcar_status kvcar_decode_attention_static(kvcar_ctx *c, int32_t layer, const int32_t *seqs,
                                                      int32_t n_seqs, const void *q, void *out, uint32_t flags,
                                                      void *stream) {
    Range range_("kvcar_decode_attention_static");
    if (!c) return KVCAR_ERR_INVALID_ARG;
    if (!c->bound) return fail(c, KVCAR_ERR_STATE, "bind memory first");
    if (layer < 0 || layer >= c->cfg.n_layers || !q || !out)
        return fail(c, KVCAR_ERR_INVALID_ARG, "bad layer or pointer");
    if (!check_seqs(c, seqs, n_seqs)) return fail(c, KVCAR_ERR_INVALID_ARG, "bad sequence list");
    if (((uintptr_t)q | (uintptr_t)out) & 15) return fail(c, KVCAR_ERR_INVALID_ARG, "q/out must be 16-byte aligned");
    if (flags & ~(KVCAR_INCLUDE_CURRENT_EXACT | KVCAR_ABSORBED | KVCAR_ABSORBED_V)) return fail(c, KVCAR_ERR_INVALID_ARG, "unknown flag");
    const kvcar_config &g = c->cfg;
    int max_len = 0;
    for (int i = 0; i < n_seqs; ++i) max_len = std::max(max_len, c->len[seqs[i]]);
    const int chunk_tokens = 128;
    const int n_chunks = (max_len + chunk_tokens - 1) / chunk_tokens;
    const size_t need = (size_t)n_seqs * std::max(n_chunks, 1) * g.n_q_heads * (g.head_dim + 2) * sizeof(float);
    if (need > (size_t)KVCAR_STATIC_SCRATCH_BYTES) {
        char buf[160];
        snprintf(buf, sizeof buf, "static scratch too small: this call needs %zu bytes of split-KV partials, the "
                 "built-in array holds %u", need, (unsigned)KVCAR_STATIC_SCRATCH_BYTES);
        return fail(c, KVCAR_ERR_WORKSPACE, buf);
    }
    if (decode_generic_smem(g.n_q_heads, g.head_dim, c->max_d, c->max_m) > 227 * 1024)
        return fail(c, KVCAR_ERR_UNSUPPORTED, "shape needs more shared memory than one SM has");
    float *scratch = c->static_scratch;
    if (!scratch) return fail(c, KVCAR_ERR_STATE, "the built-in scratch array could not be located when memory was bound");
    cudaError_t e;
    cudaStream_t st = (cudaStream_t)stream;
    kvcar_status s = flush_tables(c, st);
    if (s != KVCAR_OK) return s;
    DecodeArgs a{};
    a.plan = reinterpret_cast<const LayerPlan *>(c->weights + c->plan_off) + layer;
    a.block_table = reinterpret_cast<const int32_t *>(c->ws + c->bt_off);
    a.seq_len = reinterpret_cast<const int32_t *>(c->ws + c->len_off);
    a.q = q;
    a.out = out;
    a.partials = scratch;
    a.status = reinterpret_cast<int32_t *>(c->ws + c->status_off);
    a.max_pages_per_seq = g.max_pages_per_seq;
    a.page_tokens = g.page_tokens;
    a.hq = g.n_q_heads;
    a.hkv = g.n_kv_heads;
    a.hd = g.head_dim;
    a.chunk_tokens = chunk_tokens;
    a.max_chunks = std::max(n_chunks, 1);  // partials are packed for this call's longest sequence
    a.flags = flags;
    a.scale = 1.0f / std::sqrt((float)g.head_dim);
    SeqList sl;
    sl.n = n_seqs;
    memcpy(sl.id, seqs, (size_t)n_seqs * 4);
    if (n_chunks > 0) {
        e = launch_decode_generic(a, sl, g.storage, c->max_d, c->max_m, n_chunks, st);
        if (e != cudaSuccess) return cuda_fail(c, e, "decode launch");
        ++c->launches;
    }
    e = launch_combine(a, sl, g.storage, n_chunks, st);
    if (e != cudaSuccess) return cuda_fail(c, e, "combine launch");
    ++c->launches;
    return KVCAR_OK;
}
