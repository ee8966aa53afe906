// Host side of libh1b: the C ABI declared in include/h1b.h. Validation,
// workspace carving, the host mirror of the lengths, launches. All device
// arithmetic is in h1b_kernels.cu.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include <cuda_runtime.h>

#include "../../include/h1b.h"
#include "h1b_kernels.h"

using namespace h1b;

namespace {

constexpr long kTargetItems = 8192;   // decode work items aimed for (one warp each)
constexpr int kMinSplitTokens = 256;
constexpr int kMaxQueryTokens = H1B_MAX_QUERY_TOKENS;
constexpr int kMaxGroupHeads = 16;        // query heads per KV head: the attention kernel takes them four at a time
constexpr int kPromptMinTokens = 32;    // prompt attention: runs of at least this many query tokens take the tile kernel
constexpr int kPrefillMinTokens = 64;   // appends of at least this many tokens per sequence take the tensor-core path

struct Plan {
    size_t rt, rh, len, status, qwords, partial, stage_k, stage_v, stage_q, stage_out, dbg_q, dbg_row, dbg_s, cache, total;
    size_t partial_bytes, slab_bytes;
    size_t qwords_words, cache_bytes;       // words of the query-sketch scratch, bytes of the cache region
    size_t rope;                            // rotary table [cap_tokens][head_dim / 2][2] fp32 (H1B_FLAG_ROPE only)
    size_t table, seq_cap, layer_bytes;     // paged cache: block tables [max_batch][table_stride], capacities [max_batch]
    int table_stride, page_chunks;          // 0 when the cache is contiguous
    int cap_tokens, m_words, gq, groups;
};

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int check_config(const h1b_config *c) {
    if (!c) return H1B_ERR_NULL;
    if (c->n_layers < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->max_batch < 1 || c->max_seq < 1 ||
        c->head_dim < 1 || c->sketch_bits < 1 || c->group_size < 1 || c->device < 0 ||
        (c->flags & ~(H1B_FLAG_FP16_VALUES | H1B_FLAG_ROPE)) != 0)
        return H1B_ERR_INVALID_ARG;
    if (c->n_q_heads % c->n_kv_heads != 0 || c->head_dim % c->group_size != 0 || c->sketch_bits % 32 != 0)
        return H1B_ERR_INVALID_ARG;
    if (c->max_batch > 256) return H1B_ERR_INVALID_ARG;
    const int gq = c->n_q_heads / c->n_kv_heads;
    if (gq > kMaxGroupHeads) return H1B_ERR_UNSUPPORTED;
    if (c->sketch_bits != 64 && c->sketch_bits != 128 && c->sketch_bits != 256 && c->sketch_bits != 512)
        return H1B_ERR_UNSUPPORTED;
    if (c->head_dim == kHeadDim / 2) {
        // 64-wide heads travel in pairs through the 128-wide kernels: an even number of KV heads, groups of 32
        // channels (or fp16 values), and both sketches of a pair within 512 bits
        if ((c->n_kv_heads & 1) || c->group_size != kGroup || c->sketch_bits > 256) return H1B_ERR_UNSUPPORTED;
    } else if (c->head_dim != kHeadDim || (c->group_size != kGroup && c->group_size != kHeadDim)) {
        return H1B_ERR_UNSUPPORTED;
    }
    if ((long)c->n_layers * c->max_batch * c->n_kv_heads > (1L << 28)) return H1B_ERR_INVALID_ARG;
    if (c->page_tokens < 0 || c->n_pages < 0) return H1B_ERR_INVALID_ARG;
    if (c->page_tokens > 0) {
        if (c->page_tokens % kChunkTokens != 0 || c->n_pages < 1) return H1B_ERR_INVALID_ARG;
    } else if (c->n_pages != 0) {
        return H1B_ERR_INVALID_ARG;
    }
    return H1B_OK;
}

// The configuration the kernels see. Head dimension 128: the caller's. Head dimension 64: heads 2s and 2s+1 form
// slab s of 128 channels, so there are half as many slabs as heads (which the kernels call KV heads), the sketch
// words of both heads sit side by side (twice the bits), and the projection is the block-diagonal [[R, 0], [0, R]].
bool is_paired(const h1b_config *c) { return c->head_dim == kHeadDim / 2; }
h1b_config internal_config(const h1b_config *c) {
    h1b_config ic = *c;
    if (is_paired(c)) {
        ic.head_dim = kHeadDim;
        ic.n_kv_heads = c->n_kv_heads / 2;
        ic.sketch_bits = 2 * c->sketch_bits;
    }
    return ic;
}

// (query token, query head) pairs that share a KV head ("virtual heads": gq * Tq of them) go through the attention
// kernel `gqk` at a time, one work item per group of them: vgroups items per slab and split. 128-wide heads: one, two
// or four per item. Two 64-wide heads per slab: an item takes one or four virtual heads of EACH KV head of the pair
// (gq counts both KV heads' query heads there), so two or eight.
void heads_per_item(int gq, int Tq, bool paired, int *gqk, int *vgroups) {
    const int vheads = gq * Tq;
    *gqk = paired ? (vheads >= 4 ? 8 : 2) : (vheads >= 3 ? 4 : vheads);
    *vgroups = (vheads + *gqk - 1) / *gqk;
}

int make_plan(const h1b_config *user, Plan *p) {
    const int rc = check_config(user);
    if (rc != H1B_OK) return rc;
    const h1b_config ic = internal_config(user), *c = &ic;
    p->m_words = c->sketch_bits / 32;
    p->gq = c->n_q_heads / c->n_kv_heads;
    p->groups = (c->flags & H1B_FLAG_FP16_VALUES) ? 0 : c->head_dim / c->group_size;   // 0: values stay fp16
    const ChunkLayout cl = chunk_layout(p->m_words, p->groups);
    p->cap_tokens = (c->max_seq + kChunkTokens - 1) / kChunkTokens * kChunkTokens;
    p->slab_bytes = (size_t)(p->cap_tokens / kChunkTokens) * cl.bytes;
    p->page_chunks = c->page_tokens / kChunkTokens;
    p->table_stride = c->page_tokens > 0 ? (c->max_seq + c->page_tokens - 1) / c->page_tokens : 0;
    p->layer_bytes = (size_t)c->n_pages * c->n_kv_heads * p->page_chunks * cl.bytes;
    const size_t L = c->n_layers, B = c->max_batch, Hq = c->n_q_heads, Hkv = c->n_kv_heads, d = c->head_dim;
    const size_t slabs = L * B * Hkv;
    // split-K scratch, counted in head slots (one partial of kPartStride floats each; a work item takes the slots of
    // its heads). Room for the largest of: kTargetItems work items of four heads (the split count aimed for), one
    // item per slab of all layers (a decode call then never needs a second pass), and ONE layer of the largest
    // multi-query call the interface allows (H1B_MAX_QUERY_TOKENS query tokens on max_batch sequences), so that
    // no call the header allows runs out of scratch.
    {
        const bool paired = is_paired(user);
        int gqk1, vg1, gqkm, vgm;
        heads_per_item(p->gq, 1, paired, &gqk1, &vg1);
        heads_per_item(p->gq, kMaxQueryTokens, paired, &gqkm, &vgm);
        size_t slots = (size_t)kTargetItems * 4;
        slots = std::max(slots, slabs * (size_t)vg1 * gqk1);
        slots = std::max(slots, B * Hkv * (size_t)vgm * gqkm);
        p->partial_bytes = slots * kPartStride * sizeof(float);
    }
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    p->rt = take(L * d * c->sketch_bits * sizeof(float));
    p->rh = take(L * 2 * d * c->sketch_bits * sizeof(uint16_t));     // fp16 pieces of Rt for the tensor-core prefill
    p->len = take(L * B * sizeof(int32_t));
    p->status = take(64);
    p->qwords_words = L * B * Hq * kMaxQueryTokens * p->m_words;
    p->qwords = take(p->qwords_words * sizeof(uint32_t));
    p->partial = take(p->partial_bytes);
    p->stage_k = take(L * B * Hkv * d * 2);
    p->stage_v = take(L * B * Hkv * d * 2);
    p->stage_q = take(L * B * Hq * d * 2);
    p->stage_out = take(L * B * Hq * d * 4);
    p->dbg_q = take(p->m_words * sizeof(uint32_t));
    p->dbg_row = take(kHeadDim * 2);
    p->dbg_s = take((size_t)p->cap_tokens * sizeof(int32_t));
    p->table = take((size_t)c->max_batch * (p->table_stride ? p->table_stride : 1) * sizeof(int32_t));
    p->seq_cap = take((size_t)c->max_batch * sizeof(int32_t));
    p->rope = take((c->flags & H1B_FLAG_ROPE) ? (size_t)p->cap_tokens * (user->head_dim / 2) * 2 * sizeof(float) : 0);
    p->cache_bytes = c->page_tokens > 0 ? L * p->layer_bytes : slabs * p->slab_bytes;
    p->cache = take(p->cache_bytes);
    p->total = o;
    return H1B_OK;
}

thread_local std::string g_init_error;

// N(0,1) from a counter-based stream (splitmix64 + Box-Muller), host only.
uint64_t splitmix64(uint64_t x) {
    x += 0x9E3779B97F4A7C15ull;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}
void fill_gaussian(float *dst, size_t n, uint64_t seed) {
    for (size_t i = 0; i < n; i += 2) {
        const uint64_t a = splitmix64(seed * 0x100000001B3ull + i), b = splitmix64(a ^ 0xD1B54A32D192ED03ull);
        const double u1 = ((double)(a >> 11) + 1.0) / 9007199254740993.0;   // (0, 1)
        const double u2 = (double)(b >> 11) / 9007199254740992.0;           // [0, 1)
        const double r = std::sqrt(-2.0 * std::log(u1)), th = 6.283185307179586476925 * u2;
        dst[i] = (float)(r * std::cos(th));
        if (i + 1 < n) dst[i + 1] = (float)(r * std::sin(th));
    }
}

}  // namespace

struct h1b_ctx {
    h1b_config cfg;                    // what the kernels see (see internal_config)
    h1b_config ucfg;                   // what the caller asked for
    bool paired;                       // head dimension 64: two heads per slab
    Plan plan;
    ChunkLayout cl;
    unsigned char *ws;
    std::vector<int32_t> len_host;     // [L][max_batch], mirror of the device lengths
    std::vector<int32_t> table_host;   // paged cache: mirror of the block tables [max_batch][table_stride], -1 = none
    std::vector<int32_t> cap_host;     // tokens each sequence has room for (max_seq, or what its pages hold)
    int rope_positions;                // positions the rotary table holds (0: not set yet)
    int forced_splits;
    int64_t launches;
    bool profiling;
    std::vector<cudaEvent_t> events;   // pairs (before, after) around the split-K kernel
    size_t events_used;
    cudaStream_t side;                 // long appends: the value kernel runs here, beside the key kernel
    cudaEvent_t fork, join;            // ... forked from and joined back into the caller's stream
    bool no_prompt_tiles;              // test helper: prompt attention through the 16-token route whatever the run's length
    int32_t *dbg_scores;               // test helper: where the next prompt-attention call exports one head's scores
    uint64_t dbg_prompt_stall_ns;      // test helper: the next tile-route prompt-attention call runs with its issuing warp idle
    int dbg_layer, dbg_seq, dbg_head, dbg_T;
    DecodeParams last_decode;          // the most recent attention launch (test helper: h1b_debug_partials)
    bool have_last_decode;
    std::string err;
};

namespace {

int fail(h1b_ctx *ctx, int code, const char *fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    if (ctx) ctx->err = buf; else g_init_error = buf;
    return code;
}

#define H1B_CUDA(ctx, expr)                                                                   \
    do {                                                                                      \
        cudaError_t e_ = (expr);                                                              \
        if (e_ != cudaSuccess)                                                                \
            return fail(ctx, H1B_ERR_CUDA, "%s: %s (%s:%d)", #expr, cudaGetErrorString(e_),   \
                        __FILE__, __LINE__);                                                  \
    } while (0)

template <class T>
T *at(h1b_ctx *ctx, size_t off) { return reinterpret_cast<T *>(ctx->ws + off); }

CacheAddr cache_addr(h1b_ctx *ctx) {
    CacheAddr a;
    a.base = ctx->ws + ctx->plan.cache;
    a.table = ctx->plan.page_chunks ? at<int32_t>(ctx, ctx->plan.table) : nullptr;
    a.slab_bytes = ctx->plan.slab_bytes;
    a.layer_bytes = ctx->plan.layer_bytes;
    a.table_stride = ctx->plan.table_stride; a.page_chunks = ctx->plan.page_chunks;
    a.Hkv = ctx->cfg.n_kv_heads; a.max_batch = ctx->cfg.max_batch; a.chunk_bytes = ctx->cl.bytes;
    a.cache_bytes = ctx->plan.cache_bytes;
    return a;
}

// Chunks [c_lo, c_hi] of one slab, copied to the host (one copy when they are contiguous, one per chunk when paged).
int fetch_chunks(h1b_ctx *ctx, int layer, int seq, int slab, int c_lo, int c_hi, std::vector<unsigned char> *raw) {
    const CacheAddr a = cache_addr(ctx);
    const size_t cb = ctx->cl.bytes;
    raw->resize((size_t)(c_hi - c_lo + 1) * cb);
    H1B_CUDA(ctx, cudaDeviceSynchronize());
    if (!a.table) {
        H1B_CUDA(ctx, cudaMemcpy(raw->data(), a.base + chunk_offset(a, nullptr, layer, seq, slab, c_lo), raw->size(),
                                 cudaMemcpyDeviceToHost));
        return H1B_OK;
    }
    for (int c = c_lo; c <= c_hi; ++c)
        H1B_CUDA(ctx, cudaMemcpy(raw->data() + (size_t)(c - c_lo) * cb,
                                 a.base + chunk_offset(a, ctx->table_host.data(), layer, seq, slab, c), cb,
                                 cudaMemcpyDeviceToHost));
    return H1B_OK;
}

int check_layers(h1b_ctx *ctx, int layer_begin, int n_layers, int B) {
    if (!ctx) return H1B_ERR_NULL;
    if (layer_begin < 0 || n_layers < 1 || layer_begin + n_layers > ctx->cfg.n_layers)
        return fail(ctx, H1B_ERR_INVALID_ARG, "layers [%d, %d) outside [0, %d)", layer_begin,
                    layer_begin + n_layers, ctx->cfg.n_layers);
    if (B < 1 || B > ctx->cfg.max_batch)
        return fail(ctx, H1B_ERR_INVALID_ARG, "B = %d outside [1, %d]", B, ctx->cfg.max_batch);
    return H1B_OK;
}

}  // namespace

extern "C" {

static cudaError_t resolve_static_scratch(int dev);

size_t h1b_entry_bytes(const h1b_config *cfg) {
    if (check_config(cfg) != H1B_OK) return 0;
    if (cfg->flags & H1B_FLAG_FP16_VALUES) return (size_t)cfg->sketch_bits / 8 + (size_t)cfg->head_dim * 2;
    return (size_t)cfg->sketch_bits / 8 + (size_t)cfg->head_dim / 2 + (size_t)(cfg->head_dim / cfg->group_size) * 4;
}

size_t h1b_cache_bytes(const h1b_config *cfg) {
    Plan p;
    if (make_plan(cfg, &p) != H1B_OK) return 0;
    return p.total;
}

int h1b_init_projection(const h1b_config *cfg, uint64_t seed, const float *Rt_host, void *workspace,
                        size_t workspace_bytes, void *stream, h1b_ctx **out) {
    if (!cfg || !out) return fail(nullptr, H1B_ERR_NULL, "cfg or out is NULL");
    *out = nullptr;
    Plan plan;
    const int rc = make_plan(cfg, &plan);
    if (rc != H1B_OK) return fail(nullptr, rc, "invalid or unsupported configuration");
    if (!workspace) return fail(nullptr, H1B_ERR_NULL, "workspace is NULL");
    if (workspace_bytes < plan.total || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return fail(nullptr, H1B_ERR_WORKSPACE, "workspace needs %zu bytes, 256-byte aligned (got %zu at %p)",
                    plan.total, workspace_bytes, workspace);
    h1b_ctx *ctx = new (std::nothrow) h1b_ctx();
    if (!ctx) return fail(nullptr, H1B_ERR_INVALID_ARG, "out of host memory");
    ctx->ucfg = *cfg;
    ctx->cfg = internal_config(cfg);
    ctx->paired = is_paired(cfg);
    ctx->plan = plan;
    ctx->cl = chunk_layout(plan.m_words, plan.groups);
    ctx->ws = static_cast<unsigned char *>(workspace);
    ctx->len_host.assign((size_t)cfg->n_layers * cfg->max_batch, 0);
    ctx->table_host.assign((size_t)cfg->max_batch * (plan.table_stride ? plan.table_stride : 1), -1);
    ctx->cap_host.assign((size_t)cfg->max_batch, plan.page_chunks ? 0 : cfg->max_seq);
    ctx->forced_splits = 0;
    ctx->rope_positions = 0;
    ctx->launches = 0;
    ctx->profiling = false;
    ctx->events_used = 0;
    ctx->side = nullptr; ctx->fork = nullptr; ctx->join = nullptr;
    ctx->have_last_decode = false;
    ctx->dbg_scores = nullptr;
    ctx->dbg_prompt_stall_ns = 0;
    ctx->no_prompt_tiles = false;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto bail = [&](cudaError_t e, const char *what) {
        fail(nullptr, H1B_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
        delete ctx;
        return H1B_ERR_CUDA;
    };
    cudaError_t e = cudaSetDevice(cfg->device);
    if (e != cudaSuccess) return bail(e, "cudaSetDevice");
    // Every byte of the cache is a finite fp16 / small integer from here on, so
    // tokens past a sequence's end can be read and weighted by zero.
    e = cudaMemsetAsync(workspace, 0, plan.total, st);
    if (e != cudaSuccess) return bail(e, "cudaMemsetAsync");
    const size_t nR = (size_t)cfg->n_layers * cfg->head_dim * cfg->sketch_bits;
    std::vector<float> gen, wide;
    if (!Rt_host) {
        gen.resize(nR);
        fill_gaussian(gen.data(), nR, seed);
        Rt_host = gen.data();
    }
    size_t nR_dev = nR;
    if (ctx->paired) {                          // [[R, 0], [0, R]] per layer: [128][2m]
        const size_t d = cfg->head_dim, m = cfg->sketch_bits;
        nR_dev = (size_t)cfg->n_layers * 2 * d * 2 * m;
        wide.assign(nR_dev, 0.f);
        for (size_t l = 0; l < (size_t)cfg->n_layers; ++l)
            for (size_t i = 0; i < d; ++i)
                for (size_t j = 0; j < m; ++j) {
                    const float r = Rt_host[(l * d + i) * m + j];
                    wide[(l * 2 * d + i) * 2 * m + j] = r;
                    wide[(l * 2 * d + d + i) * 2 * m + m + j] = r;
                }
        Rt_host = wide.data();
    }
    e = cudaMemcpyAsync(ctx->ws + plan.rt, Rt_host, nR_dev * sizeof(float), cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return bail(e, "cudaMemcpyAsync(Rt)");
    e = cudaMemcpyAsync(ctx->ws + plan.table, ctx->table_host.data(), ctx->table_host.size() * sizeof(int32_t),
                        cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return bail(e, "cudaMemcpyAsync(block tables)");
    e = cudaMemcpyAsync(ctx->ws + plan.seq_cap, ctx->cap_host.data(), ctx->cap_host.size() * sizeof(int32_t),
                        cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return bail(e, "cudaMemcpyAsync(capacities)");
    e = launch_split_projection(at<float>(ctx, plan.rt), at<uint16_t>(ctx, plan.rh), cfg->n_layers, ctx->cfg.sketch_bits, st);
    if (e != cudaSuccess) return bail(e, "split_projection_kernel");
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return bail(e, "cudaStreamSynchronize");
    // Set-up that would otherwise fall to the first call of some kind: the launch attributes of every kernel this
    // cache can reach, and the device address of the built-in scratch array of h1b_decode_attention_static().
    // Done here, no later call has anything to prepare (none needs a warm-up before a stream capture, and the
    // array's module is loaded, its memory backed, before any region in which the caller may not allocate).
    e = warm_kernel_attributes(plan.m_words, plan.groups, ctx->paired, plan.page_chunks > 0, (cfg->flags & H1B_FLAG_ROPE) != 0);
    if (e != cudaSuccess) return bail(e, "kernel attributes");
    if (prompt_attention_supported(plan.m_words, plan.groups, ctx->paired)) {
        PromptParams pw = {};
        pw.m_words = plan.m_words; pw.groups = plan.groups;
        e = launch_prompt_attention(pw, nullptr, nullptr, true);
        if (e != cudaSuccess) return bail(e, "kernel attributes (prompt attention)");
    }
    e = resolve_static_scratch(cfg->device);
    if (e != cudaSuccess) return bail(e, "cudaGetSymbolAddress(built-in scratch array)");
    // without these three the two long-append kernels simply run one after the other
    if (cudaStreamCreateWithFlags(&ctx->side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->join, cudaEventDisableTiming) != cudaSuccess) {
        (void)cudaGetLastError();
        if (ctx->join) cudaEventDestroy(ctx->join);
        if (ctx->fork) cudaEventDestroy(ctx->fork);
        if (ctx->side) cudaStreamDestroy(ctx->side);
        ctx->side = nullptr; ctx->fork = nullptr; ctx->join = nullptr;
    }
    *out = ctx;
    return H1B_OK;
}

// ---------------------------------------------------------------------------
// Shared pieces of append, decode and step (static: not part of the ABI).
// ---------------------------------------------------------------------------
static int check_rope(h1b_ctx *ctx, int layer_begin, int n_layers, int B, const NewCounts *nn);
static int make_new_counts(h1b_ctx *ctx, int layer_begin, int n_layers, const int32_t *n_new_host, int B, int Tn,
                           NewCounts *nn) {
    std::memset(nn, 0, sizeof *nn);
    for (int b = 0; b < B; ++b) {
        const int n = n_new_host ? n_new_host[b] : Tn;
        if (n < 0 || n > Tn) return fail(ctx, H1B_ERR_INVALID_ARG, "n_new[%d] = %d outside [0, %d]", b, n, Tn);
        nn->v[b] = n;
    }
    for (int l = layer_begin; l < layer_begin + n_layers; ++l)
        for (int b = 0; b < B; ++b)
            if ((long)ctx->len_host[(size_t)l * ctx->cfg.max_batch + b] + nn->v[b] > ctx->cap_host[b])
                return fail(ctx, H1B_ERR_CAPACITY, "layer %d sequence %d: %d + %d tokens exceed its capacity of %d", l, b,
                            ctx->len_host[(size_t)l * ctx->cfg.max_batch + b], nn->v[b], ctx->cap_host[b]);
    return check_rope(ctx, layer_begin, n_layers, B, nn);
}

static bool uses_rope(const h1b_ctx *ctx) { return (ctx->ucfg.flags & H1B_FLAG_ROPE) != 0; }
static RopeRef rope_ref(h1b_ctx *ctx) {
    RopeRef r;
    r.table = uses_rope(ctx) ? at<float>(ctx, ctx->plan.rope) : nullptr;
    r.half = ctx->ucfg.head_dim / 2;
    r.n_pos = ctx->rope_positions;
    return r;
}
// With rotary embedding every position that a call touches must be in the table.
static int check_rope(h1b_ctx *ctx, int layer_begin, int n_layers, int B, const NewCounts *nn) {
    if (!uses_rope(ctx)) return H1B_OK;
    if (ctx->rope_positions < 1) return fail(ctx, H1B_ERR_INVALID_ARG, "H1B_FLAG_ROPE: h1b_set_rope_table has not been called");
    for (int l = layer_begin; l < layer_begin + n_layers; ++l)
        for (int b = 0; b < B; ++b) {
            const int end = ctx->len_host[(size_t)l * ctx->cfg.max_batch + b] + (nn ? nn->v[b] : 0);
            if (end > ctx->rope_positions)
                return fail(ctx, H1B_ERR_CAPACITY, "layer %d sequence %d reaches position %d, the rotary table holds %d",
                            l, b, end, ctx->rope_positions);
        }
    return H1B_OK;
}

static AppendParams append_params(h1b_ctx *ctx, int layer_begin, int n_layers, const void *k, const void *v, int B,
                                  int Tn) {
    AppendParams p;
    p.k = static_cast<const uint16_t *>(k);
    p.v = static_cast<const uint16_t *>(v);
    p.Rt = at<float>(ctx, ctx->plan.rt);
    p.ca = cache_addr(ctx);
    p.len = at<int32_t>(ctx, ctx->plan.len);
    p.done = at<int32_t>(ctx, ctx->plan.status) + 4;
    p.status = at<int32_t>(ctx, ctx->plan.status);
    p.seq_cap = at<int32_t>(ctx, ctx->plan.seq_cap);
    p.layer_begin = layer_begin; p.n_layers = n_layers; p.B = B; p.Tn = Tn;
    p.Hkv = ctx->cfg.n_kv_heads; p.max_batch = ctx->cfg.max_batch; p.m_words = ctx->plan.m_words;
    p.groups = ctx->plan.groups;
    p.rope = rope_ref(ctx);
    return p;
}

static SketchParams sketch_params(h1b_ctx *ctx, int layer_begin, int n_layers, const void *q, int B,
                                  uint32_t *qwords, size_t qwords_words = 0 /* 0: the workspace's sketch scratch */) {
    SketchParams sp;
    sp.qwords_words = qwords_words ? qwords_words : ctx->plan.qwords_words;
    sp.status = at<int32_t>(ctx, ctx->plan.status);
    sp.q = static_cast<const uint16_t *>(q);
    sp.Rt = at<float>(ctx, ctx->plan.rt);
    sp.qwords = qwords;
    // (paired heads: a row of the sketch is a pair of query heads, 128 channels, and yields both heads' words)
    sp.layer_begin = layer_begin; sp.n_layers = n_layers; sp.B = B;
    sp.Hq = ctx->paired ? ctx->cfg.n_q_heads / 2 : ctx->cfg.n_q_heads;
    sp.max_batch = ctx->cfg.max_batch; sp.m_words = ctx->plan.m_words;
    sp.rope = rope_ref(ctx);
    sp.len = at<int32_t>(ctx, ctx->plan.len);
    sp.Tq = 1;
    sp.q_seq_rows = sp.Hq;
    sp.q_tail = 0;
    sp.qw_row_words = 0;
    return sp;
}

static void commit_lengths(h1b_ctx *ctx, int layer_begin, int n_layers, int B, const NewCounts &nn) {
    for (int l = layer_begin; l < layer_begin + n_layers; ++l)
        for (int b = 0; b < B; ++b) ctx->len_host[(size_t)l * ctx->cfg.max_batch + b] += nn.v[b];
}

// How one attention call goes through the split-K scratch: decided on the host before anything is launched.
struct DecodePlan {
    int gqk, vgroups;       // heads per work item, items per (slab, split)
    int pass_layers;        // layers per pass through the scratch (all of them unless the scratch is small)
    int splits;             // work items per (slab, group of heads)
    size_t partial_bytes;   // what the scratch holds: partials, and words of query sketches
    size_t qwords_words;
};

// Every sequence is split so that there are about kTargetItems work items, capped by what the scratch holds. The
// host only chooses how many splits; which chunks a split takes is worked out on the device from the sequence's
// length at that moment, so the result does not depend on how well the host's view of the lengths matches the
// device's. `extra_tokens`: tokens the same call appends before it attends (the host's lengths do not have them yet).
// Fails (nothing launched, nothing changed) when one layer's units do not fit the scratch.
static int plan_decode(h1b_ctx *ctx, int layer_begin, int n_layers, int B, size_t partial_bytes, int Tq, int q_tail,
                       int extra_tokens, DecodePlan *dpl) {
    heads_per_item(ctx->plan.gq, Tq, ctx->paired, &dpl->gqk, &dpl->vgroups);
    dpl->partial_bytes = partial_bytes;
    dpl->qwords_words = ctx->plan.qwords_words;
    const size_t max_items = partial_bytes / ((size_t)dpl->gqk * kPartStride * sizeof(float));
    // slabs x groups of virtual heads: the units a split divides. When the scratch cannot hold one partial for
    // every unit of the call (many query tokens on a large batch), the layers go through it in several passes,
    // one behind the other on the stream.
    const long per_layer = (long)B * ctx->cfg.n_kv_heads * dpl->vgroups;
    if ((size_t)per_layer > max_items)
        return fail(ctx, H1B_ERR_CAPACITY, "%ld (sequence, KV head, head group) units of one layer exceed the split-K "
                    "scratch (%zu items of %d heads)", per_layer, max_items, dpl->gqk);
    dpl->pass_layers = (int)std::min<size_t>((size_t)n_layers, max_items / (size_t)per_layer);
    const long slabs = per_layer * dpl->pass_layers;
    int maxlen = 1;
    for (int l = layer_begin; l < layer_begin + n_layers; ++l)
        for (int b = 0; b < B; ++b)
            maxlen = std::max(maxlen, ctx->len_host[(size_t)l * ctx->cfg.max_batch + b] + extra_tokens - q_tail);
    long splits = ctx->forced_splits > 0 ? ctx->forced_splits : kTargetItems / slabs;
    const long max_splits = std::max(1, maxlen / kMinSplitTokens);
    if (ctx->forced_splits <= 0 && splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    if ((size_t)(slabs * splits) > max_items) {
        if (ctx->forced_splits > 0)
            return fail(ctx, H1B_ERR_CAPACITY, "%ld splits of %ld slabs exceed the split-K scratch (%zu items)",
                        splits, slabs, max_items);
        splits = (long)(max_items / (size_t)slabs);
    }
    dpl->splits = (int)splits;
    return H1B_OK;
}

// Enqueue the split-K attention kernel and the combine over scratch (qwords, partial) as planned.
static int enqueue_decode(h1b_ctx *ctx, const DecodePlan &dpl, int layer_begin, int n_layers, float inv_tau, void *out,
                          int B, cudaStream_t st, uint32_t *qwords, float *partial, bool may_profile, int *launches,
                          int Tq = 1, int q_tail = 0, int out_seq_tokens = 0) {
    DecodeParams dp;
    dp.ca = cache_addr(ctx);
    dp.len = at<int32_t>(ctx, ctx->plan.len);
    dp.qwords = qwords;
    dp.partial = partial;
    dp.partial_floats = dpl.partial_bytes / sizeof(float);
    dp.qwords_words = dpl.qwords_words;
    dp.status = at<int32_t>(ctx, ctx->plan.status);
    dp.B = B; dp.Hkv = ctx->cfg.n_kv_heads;
    dp.Hq = ctx->cfg.n_q_heads; dp.max_batch = ctx->cfg.max_batch; dp.m_words = ctx->plan.m_words;
    dp.groups = ctx->plan.groups;
    dp.splits = dpl.splits;
    dp.Tq = Tq; dp.gqk = dpl.gqk; dp.vgroups = dpl.vgroups;
    dp.q_tail = q_tail;
    dp.out_seq_rows = (out_seq_tokens > 0 ? out_seq_tokens : Tq) * ctx->cfg.n_q_heads;
    dp.paired = ctx->paired ? 1 : 0;
    dp.out_dim = ctx->ucfg.head_dim;
    dp.c2 = (float)(2.0 * (double)inv_tau * 1.4426950408889634 / (double)ctx->ucfg.sketch_bits);
    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
    if (may_profile && dpl.pass_layers == n_layers && ctx->profiling && ctx->events_used + 2 <= ctx->events.size()) {
        ev0 = ctx->events[ctx->events_used];
        ev1 = ctx->events[ctx->events_used + 1];
        ctx->events_used += 2;
    }
    const size_t layer_out = (size_t)B * dp.out_seq_rows * (size_t)ctx->ucfg.head_dim;           // floats of one layer
    for (int done = 0; done < n_layers; done += dpl.pass_layers) {
        dp.layer_begin = layer_begin + done;
        dp.n_layers = std::min(dpl.pass_layers, n_layers - done);
        dp.out = static_cast<float *>(out) + (size_t)done * layer_out;
        H1B_CUDA(ctx, launch_decode(dp, st, launches, ev0, ev1));
        ctx->last_decode = dp;
        ctx->have_last_decode = true;
    }
    return H1B_OK;
}

static int check_decode_args(h1b_ctx *ctx, int layer_begin, int n_layers, const void *q, float inv_tau,
                             const void *out, int B) {
    int rc = check_layers(ctx, layer_begin, n_layers, B);
    if (rc != H1B_OK) return rc;
    if (!q || !out) return fail(ctx, H1B_ERR_NULL, "q or out is NULL");
    // the kernels read rows with 16-byte loads: a misaligned tensor would fault on the device, so it stops here
    if ((reinterpret_cast<uintptr_t>(q) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u))
        return fail(ctx, H1B_ERR_INVALID_ARG, "q and out must be 16-byte aligned (got %p, %p)", q, out);
    if (!(inv_tau > 0.f) || !std::isfinite(inv_tau))
        return fail(ctx, H1B_ERR_INVALID_ARG, "inv_tau must be finite and > 0");
    return check_rope(ctx, layer_begin, n_layers, B, nullptr);
}

int h1b_append_kv(h1b_ctx *ctx, int layer_begin, int n_layers, const void *k, const void *v,
                  const int32_t *n_new_host, int B, int Tn, void *stream) {
    int rc = check_layers(ctx, layer_begin, n_layers, B);
    if (rc != H1B_OK) return rc;
    if (!k || !v) return fail(ctx, H1B_ERR_NULL, "k or v is NULL");
    if ((reinterpret_cast<uintptr_t>(k) & 15u) || (reinterpret_cast<uintptr_t>(v) & 15u))
        return fail(ctx, H1B_ERR_INVALID_ARG, "k and v must be 16-byte aligned (got %p, %p)", k, v);
    if (Tn < 1) return fail(ctx, H1B_ERR_INVALID_ARG, "Tn = %d < 1", Tn);
    NewCounts nn;
    rc = make_new_counts(ctx, layer_begin, n_layers, n_new_host, B, Tn, &nn);
    if (rc != H1B_OK) return rc;
    int launches = 0;
    if (Tn >= kPrefillMinTokens) {
        // long append: tensor-core projection over tiles of 128 cache positions
        PrefillParams pp;
        pp.k = static_cast<const uint16_t *>(k);
        pp.v = static_cast<const uint16_t *>(v);
        pp.Rh = at<uint16_t>(ctx, ctx->plan.rh);
        pp.ca = cache_addr(ctx);
        pp.seq_cap = at<int32_t>(ctx, ctx->plan.seq_cap);
        pp.rope = rope_ref(ctx);
        pp.len = at<int32_t>(ctx, ctx->plan.len);
        pp.status = at<int32_t>(ctx, ctx->plan.status);
        pp.layer_begin = layer_begin; pp.n_layers = n_layers; pp.B = B; pp.Tn = Tn;
        pp.Hkv = ctx->cfg.n_kv_heads; pp.max_batch = ctx->cfg.max_batch; pp.m_words = ctx->plan.m_words;
        pp.groups = ctx->plan.groups;
        int tiles = 1;
        for (int l = layer_begin; l < layer_begin + n_layers; ++l)
            for (int b = 0; b < B; ++b) {
                const int len0 = ctx->len_host[(size_t)l * ctx->cfg.max_batch + b];
                if (nn.v[b] > 0) tiles = std::max(tiles, (len0 + nn.v[b] + 127) / 128 - len0 / 128);
            }
        pp.tiles_per_seq = tiles;
        // one block streams consecutive tiles of a slab through a two-deep pipeline: long runs amortise its start-up,
        // as long as there are still several blocks for every SM
        const long slabs = (long)n_layers * B * ctx->cfg.n_kv_heads * ((ctx->cfg.sketch_bits + 127) / 128);
        int tpb = std::min(tiles, 32);
        while (tpb > 4 && slabs * ((tiles + tpb - 1) / tpb) < 148 * 4) tpb = (tpb + 1) / 2;
        pp.tiles_per_block = tpb;
        pp.heads_per_item = ctx->cfg.n_kv_heads;
        H1B_CUDA(ctx, launch_prefill(pp, nn, static_cast<cudaStream_t>(stream), ctx->side, ctx->fork, ctx->join, &launches));
    } else {
        const AppendParams ap = append_params(ctx, layer_begin, n_layers, k, v, B, Tn);
        H1B_CUDA(ctx, launch_prepare(&ap, nullptr, nn, static_cast<cudaStream_t>(stream), &launches));
    }
    ctx->launches += launches;
    commit_lengths(ctx, layer_begin, n_layers, B, nn);
    return H1B_OK;
}

int h1b_decode_attention(h1b_ctx *ctx, int layer_begin, int n_layers, const void *q, float inv_tau, void *out,
                         int B, void *stream) {
    int rc = check_decode_args(ctx, layer_begin, n_layers, q, inv_tau, out, B);
    if (rc != H1B_OK) return rc;
    DecodePlan dpl;
    rc = plan_decode(ctx, layer_begin, n_layers, B, ctx->plan.partial_bytes, 1, 0, 0, &dpl);
    if (rc != H1B_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int launches = 0;
    const SketchParams sp = sketch_params(ctx, layer_begin, n_layers, q, B, at<uint32_t>(ctx, ctx->plan.qwords));
    NewCounts none;
    std::memset(&none, 0, sizeof none);
    H1B_CUDA(ctx, launch_prepare(nullptr, &sp, none, st, &launches));
    rc = enqueue_decode(ctx, dpl, layer_begin, n_layers, inv_tau, out, B, st, sp.qwords, at<float>(ctx, ctx->plan.partial),
                        true, &launches);
    ctx->launches += launches;
    return rc;
}

int h1b_decode_attention_multi(h1b_ctx *ctx, int layer_begin, int n_layers, const void *q, int Tq, float inv_tau,
                               void *out, int B, void *stream) {
    int rc = check_decode_args(ctx, layer_begin, n_layers, q, inv_tau, out, B);
    if (rc != H1B_OK) return rc;
    if (Tq < 1 || Tq > kMaxQueryTokens)
        return fail(ctx, H1B_ERR_INVALID_ARG, "Tq = %d outside [1, %d]", Tq, kMaxQueryTokens);
    for (int l = layer_begin; l < layer_begin + n_layers; ++l)
        for (int b = 0; b < B; ++b)
            if (ctx->len_host[(size_t)l * ctx->cfg.max_batch + b] < Tq)
                return fail(ctx, H1B_ERR_INVALID_ARG, "layer %d sequence %d holds %d < Tq = %d tokens", l, b,
                            ctx->len_host[(size_t)l * ctx->cfg.max_batch + b], Tq);
    DecodePlan dpl;
    rc = plan_decode(ctx, layer_begin, n_layers, B, ctx->plan.partial_bytes, Tq, 0, 0, &dpl);
    if (rc != H1B_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int launches = 0;
    // rows of the sketch are (sequence, query token, query head): Tq * Hq "heads" per sequence
    SketchParams sp = sketch_params(ctx, layer_begin, n_layers, q, B, at<uint32_t>(ctx, ctx->plan.qwords));
    sp.Hq = Tq * sp.Hq;                                 // (n_q_heads, or with 64-wide heads the pairs of them)
    sp.Tq = Tq;
    sp.q_seq_rows = sp.Hq;
    NewCounts none;
    std::memset(&none, 0, sizeof none);
    H1B_CUDA(ctx, launch_prepare(nullptr, &sp, none, st, &launches));
    rc = enqueue_decode(ctx, dpl, layer_begin, n_layers, inv_tau, out, B, st, sp.qwords, at<float>(ctx, ctx->plan.partial),
                        true, &launches, Tq);
    ctx->launches += launches;
    return rc;
}

int h1b_prefill_attention(h1b_ctx *ctx, int layer_begin, int n_layers, const void *q, int Tn, float inv_tau, void *out,
                          int B, void *stream) {
    int rc = check_decode_args(ctx, layer_begin, n_layers, q, inv_tau, out, B);
    if (rc != H1B_OK) return rc;
    if (Tn < 1) return fail(ctx, H1B_ERR_INVALID_ARG, "Tn = %d < 1", Tn);
    for (int l = layer_begin; l < layer_begin + n_layers; ++l)
        for (int b = 0; b < B; ++b)
            if (ctx->len_host[(size_t)l * ctx->cfg.max_batch + b] < Tn)
                return fail(ctx, H1B_ERR_INVALID_ARG, "layer %d sequence %d holds %d < Tn = %d tokens", l, b,
                            ctx->len_host[(size_t)l * ctx->cfg.max_batch + b], Tn);
    // Runs of at least kPromptMinTokens query tokens on a cache format the tile kernel serves: scores and P.V as
    // dense contractions over blocks of 128 queries x 64 cached tokens. The sketches of all query tokens are kept in
    // the first words of the output rows they belong to (the kernel reads a row's words before it writes the row).
    if (Tn >= kPromptMinTokens && !ctx->no_prompt_tiles && prompt_attention_supported(ctx->plan.m_words, ctx->plan.groups, ctx->paired) &&
        (size_t)n_layers * B * Tn * ctx->cfg.n_q_heads < (size_t)0x7fffffff) {
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        int launches = 0;
        NewCounts none;
        std::memset(&none, 0, sizeof none);
        SketchParams sp = sketch_params(ctx, layer_begin, n_layers, q, B, static_cast<uint32_t *>(out),
                                        (size_t)n_layers * B * Tn * ctx->cfg.n_q_heads * kHeadDim);
        sp.Hq = Tn * sp.Hq;
        sp.Tq = Tn;
        sp.q_seq_rows = sp.Hq;
        sp.qw_row_words = kHeadDim;                     // one output row (128 floats) per (token, head)
        H1B_CUDA(ctx, launch_prepare(nullptr, &sp, none, st, &launches));
        PromptParams pp = {};
        pp.ca = cache_addr(ctx);
        pp.len = at<int32_t>(ctx, ctx->plan.len);
        pp.qstash = static_cast<const uint32_t *>(out);
        pp.qstash_row_words = kHeadDim;
        pp.out = static_cast<float *>(out);
        pp.status = at<int32_t>(ctx, ctx->plan.status);
        pp.layer_begin = layer_begin; pp.n_layers = n_layers; pp.B = B; pp.Hkv = ctx->cfg.n_kv_heads; pp.Hq = ctx->cfg.n_q_heads;
        pp.max_batch = ctx->cfg.max_batch; pp.m_words = ctx->plan.m_words; pp.groups = ctx->plan.groups; pp.Tn = Tn;
        pp.c = (float)(2.0 * (double)inv_tau * 1.4426950408889634 / (double)ctx->ucfg.sketch_bits);
        pp.dbg_scores = ctx->dbg_scores; pp.dbg_layer = ctx->dbg_layer; pp.dbg_b = ctx->dbg_seq; pp.dbg_h = ctx->dbg_head;
        pp.dbg_T = ctx->dbg_T;
        ctx->dbg_scores = nullptr;                      // one call only
        pp.dbg_no_issue = ctx->dbg_prompt_stall_ns ? 1 : 0;
        pp.wait_ns = ctx->dbg_prompt_stall_ns;
        ctx->dbg_prompt_stall_ns = 0;
        H1B_CUDA(ctx, launch_prompt_attention(pp, st, &launches));
        ctx->launches += launches;
        return H1B_OK;
    }
    // every block of the walk is planned before the first one is launched: a call that cannot run launches nothing
    std::vector<DecodePlan> plans;
    for (int t0 = 0; t0 < Tn; t0 += kMaxQueryTokens) {
        const int Tq = std::min(kMaxQueryTokens, Tn - t0), q_tail = Tn - t0 - Tq;
        DecodePlan dpl;
        rc = plan_decode(ctx, layer_begin, n_layers, B, ctx->plan.partial_bytes, Tq, q_tail, 0, &dpl);
        if (rc != H1B_OK) return rc;
        plans.push_back(dpl);
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int launches = 0;
    NewCounts none;
    std::memset(&none, 0, sizeof none);
    const size_t d = ctx->ucfg.head_dim, Hq = ctx->ucfg.n_q_heads;
    // blocks of up to kMaxQueryTokens query tokens, first to last; block j ends q_tail tokens before the sequences' ends
    for (int t0 = 0; t0 < Tn && rc == H1B_OK; t0 += kMaxQueryTokens) {
        const int Tq = std::min(kMaxQueryTokens, Tn - t0), q_tail = Tn - t0 - Tq;
        const DecodePlan &dpl = plans[(size_t)(t0 / kMaxQueryTokens)];
        SketchParams sp = sketch_params(ctx, layer_begin, n_layers,
                                        static_cast<const uint16_t *>(q) + (size_t)t0 * Hq * d, B,
                                        at<uint32_t>(ctx, ctx->plan.qwords));
        const int rows_per_token = sp.Hq;               // query heads, or with 64-wide heads pairs of them
        sp.Hq = Tq * rows_per_token;
        sp.Tq = Tq;
        sp.q_seq_rows = Tn * rows_per_token;
        sp.q_tail = q_tail;
        H1B_CUDA(ctx, launch_prepare(nullptr, &sp, none, st, &launches));
        rc = enqueue_decode(ctx, dpl, layer_begin, n_layers, inv_tau, static_cast<float *>(out) + (size_t)t0 * Hq * d, B, st,
                            sp.qwords, at<float>(ctx, ctx->plan.partial), false, &launches, Tq, q_tail, Tn);
    }
    ctx->launches += launches;
    return rc;
}

int h1b_decode_step_layers(h1b_ctx *ctx, int layer_begin, int n_layers, const void *k, const void *v, const void *q,
                           float inv_tau, void *out, int B, void *stream) {
    int rc = check_decode_args(ctx, layer_begin, n_layers, q, inv_tau, out, B);
    if (rc != H1B_OK) return rc;
    if (!k || !v) return fail(ctx, H1B_ERR_NULL, "k or v is NULL");
    if ((reinterpret_cast<uintptr_t>(k) & 15u) || (reinterpret_cast<uintptr_t>(v) & 15u))
        return fail(ctx, H1B_ERR_INVALID_ARG, "k and v must be 16-byte aligned (got %p, %p)", k, v);
    NewCounts nn;
    rc = make_new_counts(ctx, layer_begin, n_layers, nullptr, B, 1, &nn);
    if (rc != H1B_OK) return rc;
    DecodePlan dpl;                                     // before anything is launched or the lengths move
    rc = plan_decode(ctx, layer_begin, n_layers, B, ctx->plan.partial_bytes, 1, 0, 1, &dpl);
    if (rc != H1B_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int launches = 0;
    const AppendParams ap = append_params(ctx, layer_begin, n_layers, k, v, B, 1);
    const SketchParams sp = sketch_params(ctx, layer_begin, n_layers, q, B, at<uint32_t>(ctx, ctx->plan.qwords));
    H1B_CUDA(ctx, launch_prepare(&ap, &sp, nn, st, &launches));
    commit_lengths(ctx, layer_begin, n_layers, B, nn);
    rc = enqueue_decode(ctx, dpl, layer_begin, n_layers, inv_tau, out, B, st, sp.qwords, at<float>(ctx, ctx->plan.partial),
                        true, &launches);
    ctx->launches += launches;
    return rc;
}

int h1b_decode_step(h1b_ctx *ctx, const void *k, const void *v, const void *q, float inv_tau, void *out, int B,
                    void *stream) {
    if (!ctx) return H1B_ERR_NULL;
    return h1b_decode_step_layers(ctx, 0, ctx->cfg.n_layers, k, v, q, inv_tau, out, B, stream);
}

int h1b_sync_lengths(h1b_ctx *ctx, void *stream) {
    if (!ctx) return H1B_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    H1B_CUDA(ctx, cudaMemcpyAsync(ctx->len_host.data(), at<int32_t>(ctx, ctx->plan.len),
                                  ctx->len_host.size() * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    H1B_CUDA(ctx, cudaStreamSynchronize(st));
    return H1B_OK;
}

// ---------------------------------------------------------------------------
// Decode attention without touching the workspace's scratch region and without
// allocating anything: the query sketches and the split-K partials live in a
// fixed array that is part of the library image. Every device that loads the
// library carries these bytes until the process exits.
// ---------------------------------------------------------------------------
#define H1B_STATIC_SCRATCH_BYTES (8u << 20)
static __device__ __align__(256) unsigned char h1b_static_scratch[H1B_STATIC_SCRATCH_BYTES];

// In host code the name above is only a stand-in for the symbol, not a device
// address; the address each device gave the array is looked up once per device,
// when the first context on that device is created (h1b_init_projection, a
// synchronous set-up call made with that device current), and kept here.
static void *g_static_scratch_addr[64] = {};
static std::mutex g_static_scratch_mutex;

// Never launched: a device-side reference, so that the array is certain to be kept in the image.
__global__ void h1b_static_scratch_anchor(unsigned char *dst) {
    if (dst) *dst = h1b_static_scratch[0];
}

static cudaError_t resolve_static_scratch(int dev) {
    if (dev < 0 || dev >= 64) return cudaSuccess;       // such a device simply has no static entry point (refused there)
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (g_static_scratch_addr[dev]) return cudaSuccess;
    void *p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, h1b_static_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    g_static_scratch_addr[dev] = p;
    return cudaSuccess;
}

int h1b_decode_attention_static(h1b_ctx *ctx, int layer_begin, int n_layers, const void *q, float inv_tau,
                                void *out, int B, void *stream) {
    int rc = check_decode_args(ctx, layer_begin, n_layers, q, inv_tau, out, B);
    if (rc != H1B_OK) return rc;
    const int dev = ctx->cfg.device;
    if (dev < 0 || dev >= 64) return fail(ctx, H1B_ERR_UNSUPPORTED, "device ordinal %d outside [0, 64)", dev);
    int cur = -1;
    H1B_CUDA(ctx, cudaGetDevice(&cur));
    if (cur != dev)
        return fail(ctx, H1B_ERR_INVALID_ARG, "device %d must be current (current is %d)", dev, cur);
    unsigned char *scratch;
    {
        std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
        scratch = static_cast<unsigned char *>(g_static_scratch_addr[dev]);     // resolved when the context was made
    }
    if (!scratch) return fail(ctx, H1B_ERR_CUDA, "the built-in scratch array has no address on device %d", dev);

    // carve: query sketches for every (layer, sequence, head) slot the kernels index, then the partials. What must
    // fit is ONE layer of the call (more layers than fit go through the array in passes, fewer splits are used
    // when the automatic choice would not fit): the same planning as the ordinary entry point, over this array.
    const size_t qw_bytes = align_up((size_t)ctx->cfg.n_layers * ctx->cfg.max_batch * ctx->cfg.n_q_heads *
                                         ctx->plan.m_words * sizeof(uint32_t), 256);
    int gqk, vgroups;
    heads_per_item(ctx->plan.gq, 1, ctx->paired, &gqk, &vgroups);
    const size_t need = qw_bytes + (size_t)B * ctx->cfg.n_kv_heads * vgroups * gqk * kPartStride * sizeof(float);
    if (need > H1B_STATIC_SCRATCH_BYTES)
        return fail(ctx, H1B_ERR_CAPACITY,
                    "static scratch too small: this call needs at least %zu bytes, the built-in array holds %u",
                    need, (unsigned)H1B_STATIC_SCRATCH_BYTES);
    DecodePlan dpl;
    rc = plan_decode(ctx, layer_begin, n_layers, B, H1B_STATIC_SCRATCH_BYTES - qw_bytes, 1, 0, 0, &dpl);
    if (rc != H1B_OK) return rc;
    dpl.qwords_words = qw_bytes / sizeof(uint32_t);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int launches = 0;
    const SketchParams sp = sketch_params(ctx, layer_begin, n_layers, q, B, reinterpret_cast<uint32_t *>(scratch),
                                          qw_bytes / sizeof(uint32_t));
    NewCounts none;
    std::memset(&none, 0, sizeof none);
    H1B_CUDA(ctx, launch_prepare(nullptr, &sp, none, st, &launches));
    rc = enqueue_decode(ctx, dpl, layer_begin, n_layers, inv_tau, out, B, st, sp.qwords,
                        reinterpret_cast<float *>(scratch + qw_bytes), false, &launches);
    ctx->launches += launches;
    return rc;
}

int h1b_decode_step_host(h1b_ctx *ctx, const void *k_host, const void *v_host, const void *q_host, float inv_tau,
                         void *out_host, int B, void *stream) {
    if (!ctx) return H1B_ERR_NULL;
    if (!k_host || !v_host || !q_host || !out_host) return fail(ctx, H1B_ERR_NULL, "a host buffer is NULL");
    int rc = check_layers(ctx, 0, ctx->cfg.n_layers, B);
    if (rc != H1B_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t L = ctx->ucfg.n_layers, d = ctx->ucfg.head_dim;
    const size_t kv_bytes = L * B * ctx->ucfg.n_kv_heads * d * 2, q_bytes = L * B * ctx->ucfg.n_q_heads * d * 2;
    const unsigned char *kh = static_cast<const unsigned char *>(k_host);
    bool one_copy = false;
    if (static_cast<const unsigned char *>(v_host) == kh + kv_bytes &&
        static_cast<const unsigned char *>(q_host) == kh + 2 * kv_bytes &&
        ctx->plan.stage_v == ctx->plan.stage_k + kv_bytes && ctx->plan.stage_q == ctx->plan.stage_v + kv_bytes) {
        // the three inputs lie back to back in host memory (and so does the staging): one copy instead of three.
        // Neighbours that belong to different page-locked allocations are refused by the runtime before anything
        // is enqueued: then the three copies below do the job.
        one_copy = cudaMemcpyAsync(ctx->ws + ctx->plan.stage_k, k_host, 2 * kv_bytes + q_bytes, cudaMemcpyHostToDevice, st) ==
                   cudaSuccess;
        if (!one_copy) (void)cudaGetLastError();
    }
    if (!one_copy) {
        H1B_CUDA(ctx, cudaMemcpyAsync(ctx->ws + ctx->plan.stage_k, k_host, kv_bytes, cudaMemcpyHostToDevice, st));
        H1B_CUDA(ctx, cudaMemcpyAsync(ctx->ws + ctx->plan.stage_v, v_host, kv_bytes, cudaMemcpyHostToDevice, st));
        H1B_CUDA(ctx, cudaMemcpyAsync(ctx->ws + ctx->plan.stage_q, q_host, q_bytes, cudaMemcpyHostToDevice, st));
    }
    rc = h1b_decode_step(ctx, ctx->ws + ctx->plan.stage_k, ctx->ws + ctx->plan.stage_v, ctx->ws + ctx->plan.stage_q,
                         inv_tau, ctx->ws + ctx->plan.stage_out, B, stream);
    if (rc != H1B_OK) return rc;
    H1B_CUDA(ctx, cudaMemcpyAsync(out_host, ctx->ws + ctx->plan.stage_out, q_bytes * 2, cudaMemcpyDeviceToHost, st));
    H1B_CUDA(ctx, cudaStreamSynchronize(st));
    return H1B_OK;
}

int h1b_free(h1b_ctx *ctx) {
    if (!ctx) return H1B_ERR_NULL;
    int rc = H1B_OK;
    if (cudaSetDevice(ctx->cfg.device) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) rc = H1B_ERR_CUDA;
    for (cudaEvent_t e : ctx->events) cudaEventDestroy(e);
    if (ctx->join) cudaEventDestroy(ctx->join);
    if (ctx->fork) cudaEventDestroy(ctx->fork);
    if (ctx->side) cudaStreamDestroy(ctx->side);
    delete ctx;
    return rc;
}

int h1b_get_projection(h1b_ctx *ctx, int layer, float *Rt_host) {
    if (!ctx) return H1B_ERR_NULL;
    if (!Rt_host) return fail(ctx, H1B_ERR_NULL, "Rt_host is NULL");
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, H1B_ERR_INVALID_ARG, "layer %d out of range", layer);
    const size_t n = (size_t)ctx->cfg.head_dim * ctx->cfg.sketch_bits;
    H1B_CUDA(ctx, cudaDeviceSynchronize());
    if (!ctx->paired) {
        H1B_CUDA(ctx, cudaMemcpy(Rt_host, at<float>(ctx, ctx->plan.rt) + (size_t)layer * n, n * sizeof(float),
                                 cudaMemcpyDeviceToHost));
        return H1B_OK;
    }
    // the caller's [64][m] is the upper left block of the block-diagonal [128][2m] the device holds
    std::vector<float> wide(n);
    H1B_CUDA(ctx, cudaMemcpy(wide.data(), at<float>(ctx, ctx->plan.rt) + (size_t)layer * n, n * sizeof(float),
                             cudaMemcpyDeviceToHost));
    const size_t d = ctx->ucfg.head_dim, m = ctx->ucfg.sketch_bits;
    for (size_t i = 0; i < d; ++i) std::memcpy(Rt_host + i * m, wide.data() + i * 2 * m, m * sizeof(float));
    return H1B_OK;
}

int h1b_get_lengths(h1b_ctx *ctx, int layer, int32_t *len_host) {
    if (!ctx) return H1B_ERR_NULL;
    if (!len_host) return fail(ctx, H1B_ERR_NULL, "len_host is NULL");
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, H1B_ERR_INVALID_ARG, "layer %d out of range", layer);
    const int mb = ctx->cfg.max_batch;
    H1B_CUDA(ctx, cudaDeviceSynchronize());
    H1B_CUDA(ctx, cudaMemcpy(len_host, at<int32_t>(ctx, ctx->plan.len) + (size_t)layer * mb, mb * sizeof(int32_t),
                             cudaMemcpyDeviceToHost));
    for (int b = 0; b < mb; ++b)
        if (len_host[b] != ctx->len_host[(size_t)layer * mb + b])
            return fail(ctx, H1B_ERR_INVALID_ARG, "layer %d sequence %d: device length %d, host mirror %d", layer, b,
                        len_host[b], ctx->len_host[(size_t)layer * mb + b]);
    return H1B_OK;
}

static int truncate_impl(h1b_ctx *ctx, int seq, int new_len, bool whole_device, cudaStream_t st) {
    if (!ctx) return H1B_ERR_NULL;
    const int mb = ctx->cfg.max_batch;
    if (seq < -1 || seq >= mb) return fail(ctx, H1B_ERR_INVALID_ARG, "sequence %d out of range", seq);
    if (new_len < 0) return fail(ctx, H1B_ERR_INVALID_ARG, "new_len %d < 0", new_len);
    for (int l = 0; l < ctx->cfg.n_layers; ++l)
        for (int b = 0; b < mb; ++b)
            if ((seq < 0 || b == seq) && new_len > 0 && ctx->len_host[(size_t)l * mb + b] < new_len)
                return fail(ctx, H1B_ERR_INVALID_ARG, "layer %d sequence %d holds %d < %d tokens", l, b,
                            ctx->len_host[(size_t)l * mb + b], new_len);
    if (whole_device) H1B_CUDA(ctx, cudaDeviceSynchronize());
    H1B_CUDA(ctx, launch_set_len(at<int32_t>(ctx, ctx->plan.len), ctx->cfg.n_layers, mb, seq, new_len, st));
    if (whole_device) H1B_CUDA(ctx, cudaDeviceSynchronize());
    for (int l = 0; l < ctx->cfg.n_layers; ++l)
        for (int b = 0; b < mb; ++b)
            if (seq < 0 || b == seq) ctx->len_host[(size_t)l * mb + b] = new_len;
    return H1B_OK;
}

int h1b_truncate(h1b_ctx *ctx, int seq, int new_len) { return truncate_impl(ctx, seq, new_len, true, nullptr); }

int h1b_truncate_async(h1b_ctx *ctx, int seq, int new_len, void *stream) {
    return truncate_impl(ctx, seq, new_len, false, static_cast<cudaStream_t>(stream));
}

int h1b_reset(h1b_ctx *ctx, int seq) { return h1b_truncate(ctx, seq, 0); }

int h1b_export_cache(h1b_ctx *ctx, int layer, int seq, int kv_head, int t0, int n, uint32_t *words, uint8_t *codes,
                     uint16_t *scale, uint16_t *zero) {
    if (!ctx) return H1B_ERR_NULL;
    if (layer < 0 || layer >= ctx->cfg.n_layers || seq < 0 || seq >= ctx->cfg.max_batch || kv_head < 0 ||
        kv_head >= ctx->ucfg.n_kv_heads)
        return fail(ctx, H1B_ERR_INVALID_ARG, "(layer %d, seq %d, kv_head %d) out of range", layer, seq, kv_head);
    const int len = ctx->len_host[(size_t)layer * ctx->cfg.max_batch + seq];
    if (t0 < 0 || n < 0 || t0 + n > len)
        return fail(ctx, H1B_ERR_INVALID_ARG, "tokens [%d, %d) outside the cached [0, %d)", t0, t0 + n, len);
    if (ctx->plan.groups == 0 && (codes || scale || zero))
        return fail(ctx, H1B_ERR_INVALID_ARG, "this cache keeps fp16 values: it has no codes, scales or zero-points");
    if (n == 0) return H1B_OK;
    const ChunkLayout &cl = ctx->cl;
    const int c_lo = t0 / kChunkTokens, c_hi = (t0 + n - 1) / kChunkTokens;
    std::vector<unsigned char> raw;
    // with paired heads, head kv_head is half `half` of slab kv_head / 2: its share of the words, channel blocks and groups
    const int slab = ctx->paired ? kv_head / 2 : kv_head, half = ctx->paired ? (kv_head & 1) : 0;
    { const int rcf = fetch_chunks(ctx, layer, seq, slab, c_lo, c_hi, &raw); if (rcf != H1B_OK) return rcf; }
    const int d = ctx->ucfg.head_dim, mw = ctx->ucfg.sketch_bits / 32;
    const int ng = ctx->paired ? cl.groups / 2 : cl.groups;
    const int w0 = half * mw, cb0 = half * (d / 16), g0 = half * ng;
    for (int i = 0; i < n; ++i) {
        const int t = t0 + i, tt = t % kChunkTokens;
        const unsigned char *ch = raw.data() + (size_t)(t / kChunkTokens - c_lo) * cl.bytes;
        if (words)
            for (int w = 0; w < mw; ++w) std::memcpy(&words[(size_t)i * mw + w], ch + key_word_off(w0 + w, tt), 4);
        if (codes)
            for (int cb = 0; cb < d / 16; ++cb)
                for (int r = 0; r < 8; ++r) {
                    const unsigned char byte = ch[code_byte_off(cl, tt, cb0 + cb, r)];
                    codes[(size_t)i * d + cb * 16 + r] = byte & 15;
                    codes[(size_t)i * d + cb * 16 + r + 8] = byte >> 4;
                }
        for (int g = 0; g < ng; ++g) {
            if (scale) std::memcpy(&scale[(size_t)i * ng + g], ch + scale_off(cl, tt, g0 + g), 2);
            if (zero) std::memcpy(&zero[(size_t)i * ng + g], ch + zero_off(cl, tt, g0 + g), 2);
        }
    }
    return H1B_OK;
}

int h1b_export_values(h1b_ctx *ctx, int layer, int seq, int kv_head, int t0, int n, uint16_t *values) {
    if (!ctx) return H1B_ERR_NULL;
    if (ctx->plan.groups != 0) return fail(ctx, H1B_ERR_INVALID_ARG, "this cache keeps 4-bit codes, not fp16 values");
    if (!values) return fail(ctx, H1B_ERR_NULL, "values is NULL");
    if (layer < 0 || layer >= ctx->cfg.n_layers || seq < 0 || seq >= ctx->cfg.max_batch || kv_head < 0 ||
        kv_head >= ctx->ucfg.n_kv_heads)
        return fail(ctx, H1B_ERR_INVALID_ARG, "(layer %d, seq %d, kv_head %d) out of range", layer, seq, kv_head);
    const int len = ctx->len_host[(size_t)layer * ctx->cfg.max_batch + seq];
    if (t0 < 0 || n < 0 || t0 + n > len)
        return fail(ctx, H1B_ERR_INVALID_ARG, "tokens [%d, %d) outside the cached [0, %d)", t0, t0 + n, len);
    if (n == 0) return H1B_OK;
    const ChunkLayout &cl = ctx->cl;
    const int c_lo = t0 / kChunkTokens, c_hi = (t0 + n - 1) / kChunkTokens;
    std::vector<unsigned char> raw;
    const int slab = ctx->paired ? kv_head / 2 : kv_head, half = ctx->paired ? (kv_head & 1) : 0;
    { const int rcf = fetch_chunks(ctx, layer, seq, slab, c_lo, c_hi, &raw); if (rcf != H1B_OK) return rcf; }
    const int d = ctx->ucfg.head_dim;
    for (int i = 0; i < n; ++i) {
        const int t = t0 + i, tt = t % kChunkTokens;
        const unsigned char *ch = raw.data() + (size_t)(t / kChunkTokens - c_lo) * cl.bytes;
        for (int c = 0; c < d; ++c) std::memcpy(&values[(size_t)i * d + c], ch + value_half_off(cl, tt, half * d + c), 2);
    }
    return H1B_OK;
}

int h1b_debug_scores(h1b_ctx *ctx, int layer, int seq, int kv_head, const void *q, uint32_t *qwords_host,
                     int32_t *score_host) {
    if (!ctx) return H1B_ERR_NULL;
    if (!q) return fail(ctx, H1B_ERR_NULL, "q is NULL");
    if (layer < 0 || layer >= ctx->cfg.n_layers || seq < 0 || seq >= ctx->cfg.max_batch || kv_head < 0 ||
        kv_head >= ctx->ucfg.n_kv_heads)
        return fail(ctx, H1B_ERR_INVALID_ARG, "(layer %d, seq %d, kv_head %d) out of range", layer, seq, kv_head);
    const int len = ctx->len_host[(size_t)layer * ctx->cfg.max_batch + seq];
    const int mw = ctx->plan.m_words, mwh = ctx->ucfg.sketch_bits / 32;
    const int slab = ctx->paired ? kv_head / 2 : kv_head, half = ctx->paired ? (kv_head & 1) : 0;
    H1B_CUDA(ctx, cudaDeviceSynchronize());
    if (ctx->paired) {
        // a 128-channel row with the 64-channel query in front and zeros behind: the upper left block of the
        // block-diagonal projection then gives the query's sketch in the first m/32 words
        H1B_CUDA(ctx, cudaMemset(ctx->ws + ctx->plan.dbg_row, 0, kHeadDim * 2));
        H1B_CUDA(ctx, cudaMemcpy(ctx->ws + ctx->plan.dbg_row, q, (size_t)ctx->ucfg.head_dim * 2, cudaMemcpyDeviceToDevice));
        q = ctx->ws + ctx->plan.dbg_row;
    }
    // sketch the single query row with the layer's projection into the debug slot
    SketchParams sp;
    sp.q = static_cast<const uint16_t *>(q);
    sp.Rt = at<float>(ctx, ctx->plan.rt) + (size_t)layer * ctx->cfg.head_dim * ctx->cfg.sketch_bits;
    sp.qwords = at<uint32_t>(ctx, ctx->plan.dbg_q);
    sp.qwords_words = (size_t)mw;
    sp.status = at<int32_t>(ctx, ctx->plan.status);
    sp.layer_begin = 0; sp.n_layers = 1; sp.B = 1; sp.Hq = 1; sp.max_batch = 1; sp.m_words = mw;
    // with rotary embedding the row is turned like the query of a decode call: at the sequence's last position
    sp.rope = rope_ref(ctx);
    sp.len = at<int32_t>(ctx, ctx->plan.len) + (size_t)layer * ctx->cfg.max_batch + seq;
    sp.Tq = 1;
    sp.q_seq_rows = 1;
    sp.q_tail = 0;
    sp.qw_row_words = 0;
    if (uses_rope(ctx) && ctx->rope_positions < 1)
        return fail(ctx, H1B_ERR_INVALID_ARG, "H1B_FLAG_ROPE: h1b_set_rope_table has not been called");
    int launches = 0;
    NewCounts none;
    std::memset(&none, 0, sizeof none);
    H1B_CUDA(ctx, launch_prepare(nullptr, &sp, none, nullptr, &launches));
    H1B_CUDA(ctx, launch_debug_scores(cache_addr(ctx), layer, seq, slab, sp.qwords, len, half * mwh, mwh,
                                      at<int32_t>(ctx, ctx->plan.dbg_s), nullptr));
    H1B_CUDA(ctx, cudaDeviceSynchronize());
    if (qwords_host)
        H1B_CUDA(ctx, cudaMemcpy(qwords_host, sp.qwords, mwh * sizeof(uint32_t), cudaMemcpyDeviceToHost));
    if (score_host && len > 0)
        H1B_CUDA(ctx, cudaMemcpy(score_host, at<int32_t>(ctx, ctx->plan.dbg_s), (size_t)len * sizeof(int32_t),
                                 cudaMemcpyDeviceToHost));
    return H1B_OK;
}

int h1b_set_rope_table(h1b_ctx *ctx, const float *cos_sin_host, int n_positions, void *stream) {
    if (!ctx) return H1B_ERR_NULL;
    if (!cos_sin_host) return fail(ctx, H1B_ERR_NULL, "cos_sin_host is NULL");
    if (!uses_rope(ctx)) return fail(ctx, H1B_ERR_INVALID_ARG, "the cache was not made with H1B_FLAG_ROPE");
    if (n_positions < 1) return fail(ctx, H1B_ERR_INVALID_ARG, "n_positions = %d < 1", n_positions);
    n_positions = std::min(n_positions, ctx->plan.cap_tokens);      // positions the cache can never reach are not kept
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t bytes = (size_t)n_positions * (ctx->ucfg.head_dim / 2) * 2 * sizeof(float);
    H1B_CUDA(ctx, cudaMemcpyAsync(ctx->ws + ctx->plan.rope, cos_sin_host, bytes, cudaMemcpyHostToDevice, st));
    H1B_CUDA(ctx, cudaStreamSynchronize(st));
    ctx->rope_positions = n_positions;
    return H1B_OK;
}

int h1b_set_block_table(h1b_ctx *ctx, int seq, const int32_t *pages_host, int n, void *stream) {
    if (!ctx) return H1B_ERR_NULL;
    if (!ctx->plan.page_chunks) return fail(ctx, H1B_ERR_INVALID_ARG, "this cache is not paged");
    if (seq < 0 || seq >= ctx->cfg.max_batch) return fail(ctx, H1B_ERR_INVALID_ARG, "sequence %d out of range", seq);
    if (n < 0 || n > ctx->plan.table_stride)
        return fail(ctx, H1B_ERR_INVALID_ARG, "%d pages outside [0, %d]", n, ctx->plan.table_stride);
    if (n > 0 && !pages_host) return fail(ctx, H1B_ERR_NULL, "pages_host is NULL");
    for (int i = 0; i < n; ++i)
        if (pages_host[i] < 0 || pages_host[i] >= ctx->cfg.n_pages)
            return fail(ctx, H1B_ERR_INVALID_ARG, "page %d (entry %d) outside the pool of %d", pages_host[i], i, ctx->cfg.n_pages);
    // no page may belong to two sequences (or twice to one): their appends would overwrite each other
    for (int i = 0; i < n; ++i) {
        for (int j = 0; j < i; ++j)
            if (pages_host[j] == pages_host[i])
                return fail(ctx, H1B_ERR_INVALID_ARG, "page %d appears twice (entries %d and %d)", pages_host[i], j, i);
        for (int b = 0; b < ctx->cfg.max_batch; ++b) {
            if (b == seq) continue;
            const int32_t *other = ctx->table_host.data() + (size_t)b * ctx->plan.table_stride;
            for (int j = 0; j < ctx->plan.table_stride; ++j)
                if (other[j] == pages_host[i])
                    return fail(ctx, H1B_ERR_INVALID_ARG, "page %d (entry %d) already belongs to sequence %d", pages_host[i], i, b);
        }
    }
    const int page_tokens = ctx->cfg.page_tokens;
    int held = 0;
    for (int l = 0; l < ctx->cfg.n_layers; ++l) held = std::max(held, ctx->len_host[(size_t)l * ctx->cfg.max_batch + seq]);
    if ((long)n * page_tokens < held)
        return fail(ctx, H1B_ERR_INVALID_ARG, "sequence %d holds %d tokens: %d pages of %d are too few", seq, held, n, page_tokens);
    int32_t *row = ctx->table_host.data() + (size_t)seq * ctx->plan.table_stride;
    for (int i = 0; i < ctx->plan.table_stride; ++i) row[i] = i < n ? pages_host[i] : -1;
    ctx->cap_host[seq] = (int)std::min<long>((long)n * page_tokens, ctx->cfg.max_seq);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // (the host copies are the source, and they may change before the copies run: synchronise)
    H1B_CUDA(ctx, cudaMemcpyAsync(at<int32_t>(ctx, ctx->plan.table) + (size_t)seq * ctx->plan.table_stride, row,
                                  (size_t)ctx->plan.table_stride * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    H1B_CUDA(ctx, cudaMemcpyAsync(at<int32_t>(ctx, ctx->plan.seq_cap) + seq, &ctx->cap_host[seq], sizeof(int32_t),
                                  cudaMemcpyHostToDevice, st));
    H1B_CUDA(ctx, cudaStreamSynchronize(st));
    return H1B_OK;
}

int h1b_set_splits(h1b_ctx *ctx, int splits) {
    if (!ctx) return H1B_ERR_NULL;
    int gqk, vgroups;
    heads_per_item(ctx->plan.gq, 1, ctx->paired, &gqk, &vgroups);
    const size_t most = ctx->plan.partial_bytes / ((size_t)gqk * kPartStride * sizeof(float));
    if (splits < 0 || (size_t)splits > most)
        return fail(ctx, H1B_ERR_INVALID_ARG, "splits %d outside [0, %zu]", splits, most);
    ctx->forced_splits = splits;
    return H1B_OK;
}

int h1b_poll_status(h1b_ctx *ctx) {
    if (!ctx) return H1B_ERR_NULL;
    int32_t s = 0;
    H1B_CUDA(ctx, cudaMemcpy(&s, at<int32_t>(ctx, ctx->plan.status), sizeof s, cudaMemcpyDeviceToHost));
    if (s == kStatusOk) return H1B_OK;
    H1B_CUDA(ctx, cudaMemset(at<int32_t>(ctx, ctx->plan.status), 0, sizeof s));
    if (s == kStatusCapacity)
        return fail(ctx, H1B_ERR_CAPACITY, "a replayed append found a sequence full: its rows were dropped");
    if (s >= kStatusBounds)
        return fail(ctx, H1B_ERR_BOUNDS, "bounds-checked build: index check %d of a kernel failed; the access was skipped",
                    s - kStatusBounds);
    return fail(ctx, H1B_ERR_TIMEOUT, "a kernel gave up a bounded wait (status %d)", s);
}

int h1b_debug_prompt_scores(h1b_ctx *ctx, int layer, int seq, int q_head, int32_t *score_dev, int n_tokens) {
    if (!ctx) return H1B_ERR_NULL;
    if (score_dev && (layer < 0 || layer >= ctx->cfg.n_layers || seq < 0 || seq >= ctx->cfg.max_batch || q_head < 0 ||
                      q_head >= ctx->cfg.n_q_heads || n_tokens < 1))
        return fail(ctx, H1B_ERR_INVALID_ARG, "(layer %d, seq %d, head %d, %d tokens) out of range", layer, seq, q_head, n_tokens);
    ctx->dbg_scores = score_dev;
    ctx->dbg_layer = layer; ctx->dbg_seq = seq; ctx->dbg_head = q_head; ctx->dbg_T = n_tokens;
    return H1B_OK;
}

int h1b_debug_prompt_stall(h1b_ctx *ctx, uint64_t limit_ns) {
    if (!ctx) return H1B_ERR_NULL;
    if (limit_ns < 1 || limit_ns > 1000000000ull)
        return fail(ctx, H1B_ERR_INVALID_ARG, "limit_ns = %llu outside [1, 1e9]", (unsigned long long)limit_ns);
    ctx->dbg_prompt_stall_ns = limit_ns;
    return H1B_OK;
}

int h1b_debug_prompt_route(h1b_ctx *ctx, int tiles) {
    if (!ctx) return H1B_ERR_NULL;
    ctx->no_prompt_tiles = tiles == 0;
    return H1B_OK;
}

int h1b_bounds_checked(void) { return bounds_checked_build() ? 1 : 0; }

int h1b_debug_bounds_probe(h1b_ctx *ctx, void *stream) {
    if (!ctx) return H1B_ERR_NULL;
    if (!bounds_checked_build())
        return fail(ctx, H1B_ERR_UNSUPPORTED, "this library was built without the kernels' index checks (H1B_DEBUG_BOUNDS)");
    // the word the probe would write if its check did not stop it: the debug query slot, cleared first
    int32_t *target = at<int32_t>(ctx, ctx->plan.dbg_q);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    H1B_CUDA(ctx, cudaMemsetAsync(target, 0, sizeof(int32_t), st));
    H1B_CUDA(ctx, launch_debug_bounds_probe(at<int32_t>(ctx, ctx->plan.status), target, st));
    ++ctx->launches;
    int32_t wrote = 0;
    H1B_CUDA(ctx, cudaMemcpyAsync(&wrote, target, sizeof wrote, cudaMemcpyDeviceToHost, st));
    H1B_CUDA(ctx, cudaStreamSynchronize(st));
    if (wrote != 0) return fail(ctx, H1B_ERR_INVALID_ARG, "the guarded store of the probe was made: the checks are not in effect");
    return H1B_OK;
}

int h1b_debug_wait_timeout(h1b_ctx *ctx, uint64_t limit_ns, void *stream) {
    if (!ctx) return H1B_ERR_NULL;
    if (limit_ns < 1 || limit_ns > 1000000000ull)
        return fail(ctx, H1B_ERR_INVALID_ARG, "limit_ns = %llu outside [1, 1e9]", (unsigned long long)limit_ns);
    H1B_CUDA(ctx, launch_debug_wait_timeout(at<int32_t>(ctx, ctx->plan.status), limit_ns, static_cast<cudaStream_t>(stream)));
    ++ctx->launches;
    return H1B_OK;
}

int h1b_debug_partials(h1b_ctx *ctx, int layer, int seq, int q_token, int q_head, int32_t *n_splits_host,
                       float *hmin_host, float *wsum_host, int max_splits) {
    if (!ctx) return H1B_ERR_NULL;
    if (!n_splits_host || !hmin_host || !wsum_host) return fail(ctx, H1B_ERR_NULL, "an output pointer is NULL");
    if (!ctx->have_last_decode) return fail(ctx, H1B_ERR_INVALID_ARG, "no attention call has been made on this context");
    const DecodeParams &p = ctx->last_decode;
    if (layer < p.layer_begin || layer >= p.layer_begin + p.n_layers || seq < 0 || seq >= p.B || q_token < 0 ||
        q_token >= p.Tq || q_head < 0 || q_head >= p.Hq)
        return fail(ctx, H1B_ERR_INVALID_ARG, "(layer %d, seq %d, query token %d, head %d) is not part of the last attention launch",
                    layer, seq, q_token, q_head);
    if (max_splits < p.splits) return fail(ctx, H1B_ERR_INVALID_ARG, "%d splits, room for %d", p.splits, max_splits);
    // where the combine kernel finds this head's partials (the same arithmetic)
    const int gq = p.Hq / p.Hkv, kvh = q_head / gq, jj = q_head % gq, gqu = gq >> 1, gqh = p.gqk >> 1;
    const int v = q_token * gq + jj;
    const int vp = p.paired ? q_token * gqu + jj % gqu : 0;
    const int vg = p.paired ? vp / gqh : v / p.gqk, hh = p.paired ? (jj / gqu) * gqh + vp % gqh : v % p.gqk;
    const long slab_local = ((long)(layer - p.layer_begin) * p.B + seq) * p.Hkv + kvh;
    const float *base = p.partial + (((size_t)slab_local * p.vgroups + vg) * p.splits * p.gqk + hh) * kPartStride;
    const size_t stride = (size_t)p.gqk * kPartStride;
    H1B_CUDA(ctx, cudaDeviceSynchronize());
    for (int s = 0; s < p.splits; ++s) {
        float pair[2];
        H1B_CUDA(ctx, cudaMemcpy(pair, base + (size_t)s * stride + 128, sizeof pair, cudaMemcpyDeviceToHost));
        hmin_host[s] = pair[0];
        wsum_host[s] = 0.5f * pair[1];                  // the kernel's weights carry a factor 2 (it cancels in the division)
    }
    *n_splits_host = p.splits;
    return H1B_OK;
}

int h1b_set_profiling(h1b_ctx *ctx, int enable) {
    if (!ctx) return H1B_ERR_NULL;
    if (enable && ctx->events.empty()) {
        ctx->events.reserve(8192);
        for (int i = 0; i < 8192; ++i) {
            cudaEvent_t e;
            H1B_CUDA(ctx, cudaEventCreate(&e));
            ctx->events.push_back(e);
        }
    }
    ctx->profiling = enable != 0;
    return H1B_OK;
}

int h1b_read_profile(h1b_ctx *ctx, double *decode_ms, int64_t *decode_launches) {
    if (!ctx) return H1B_ERR_NULL;
    if (!decode_ms || !decode_launches) return fail(ctx, H1B_ERR_NULL, "an output pointer is NULL");
    H1B_CUDA(ctx, cudaDeviceSynchronize());
    double sum = 0.0;
    for (size_t i = 0; i + 1 < ctx->events_used; i += 2) {
        float ms = 0.f;
        H1B_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->events[i], ctx->events[i + 1]));
        sum += ms;
    }
    *decode_ms = sum;
    *decode_launches = (int64_t)(ctx->events_used / 2);
    ctx->events_used = 0;
    return H1B_OK;
}

int64_t h1b_launch_count(const h1b_ctx *ctx) { return ctx ? ctx->launches : 0; }

const char *h1b_last_error(const h1b_ctx *ctx) { return ctx ? ctx->err.c_str() : g_init_error.c_str(); }

}  // extern "C"
