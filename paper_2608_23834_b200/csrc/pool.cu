// Host side of libmkv: pool bookkeeping, per-format free lists, sequence rows (Algorithm 1),
// argument validation and the C ABI entry points.  No arithmetic of the method lives here.
#include <cstdio>
#include <algorithm>
#include <cstring>
#include <new>
#include <string>

#include "mkv_internal.cuh"

namespace mkv {

static thread_local std::string g_last_error;

int32_t cuda_fail(cudaError_t e, const char* what)
{
    g_last_error = std::string(what) + ": " + cudaGetErrorString(e);
    return MKV_E_CUDA;
}

void set_last_error(const char* msg) { g_last_error = msg; }

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

static int32_t check_cfg(const mkv_pool_config* c)
{
    if (!c) return MKV_E_INVALID;
    if (c->page_size < kPage || c->page_size % kPage || c->page_size > kPage * kMaxTiles) return MKV_E_INVALID;
    if (c->head_dim != 128 && c->head_dim != 256) return MKV_E_INVALID;
    if (c->n_kv_heads < 1 || c->n_q_heads < c->n_kv_heads) return MKV_E_INVALID;
    if (c->n_q_heads % c->n_kv_heads) return MKV_E_INVALID;
    if (c->n_q_heads / c->n_kv_heads > kMaxGroup) return MKV_E_INVALID;
    if (c->fp8_pages < 0 || c->tq3_pages < 0) return MKV_E_INVALID;
    if (!(c->k_scale > 0.f) || !(c->v_scale > 0.f)) return MKV_E_INVALID;
    if (c->tq3_format < 0 || c->tq3_format > 2) return MKV_E_INVALID;
    return MKV_OK;
}

size_t decode_ws_header_bytes(int B, int hkv)
{
    // 256 reserved bytes, then the row tickets of the tensor-core scan (one word per possible block)
    (void)B; (void)hkv;
    size_t b = 256 + sizeof(uint32_t) * (size_t)kMaxCtas;
    return (b + 255) / 256 * 256;
}

}  // namespace mkv

using namespace mkv;

extern "C" {

const char* mkv_last_cuda_error(void) { return g_last_error.c_str(); }

int32_t mkv_pool_query(const mkv_pool_config* cfg, size_t* fp8_bytes, size_t* tq3_bytes)
{
    int32_t rc = check_cfg(cfg);
    if (rc) return rc;
    if (!fp8_bytes || !tq3_bytes) return MKV_E_INVALID;
    const int tiles = cfg->page_size / kPage;
    *fp8_bytes = (size_t)cfg->fp8_pages * cfg->n_kv_heads * fp8_page_bytes(cfg->head_dim, tiles) + kStatusTail;
    *tq3_bytes = (size_t)cfg->tq3_pages * cfg->n_kv_heads * tq3_page_bytes(cfg->head_dim, tiles);
    if (*tq3_bytes == 0) *tq3_bytes = 256;
    return MKV_OK;
}

int32_t mkv_decode_workspace_bytes(const mkv_pool_config* cfg, int32_t max_batch, size_t* bytes)
{
    int32_t rc = check_cfg(cfg);
    if (rc) return rc;
    if (!bytes || max_batch < 1) return MKV_E_INVALID;
    int group = cfg->n_q_heads / cfg->n_kv_heads;
    size_t a = decode_ws_scalar_bytes(max_batch, cfg->n_kv_heads, group, cfg->head_dim);
    size_t b = decode_ws_tensor_bytes(max_batch, cfg->n_kv_heads, group, cfg->head_dim);
    *bytes = decode_ws_header_bytes(max_batch, cfg->n_kv_heads) + (a > b ? a : b);
    return MKV_OK;
}

int32_t mkv_workspace_init(void* ws, size_t bytes, void* stream)
{
    if (!ws || bytes < 256 || !aligned(ws, 256)) return MKV_E_INVALID;
    // the ticket words in the header must start at zero; partial slots need no initialisation
    MKV_CUDA(cudaMemsetAsync(ws, 0, bytes, (cudaStream_t)stream));
    return MKV_OK;
}

static mkv_pool* new_pool(const mkv_pool_config* cfg, void* fp8_arena, void* tq3_arena);

int32_t mkv_pool_create_host_only(const mkv_pool_config* cfg, mkv_pool** out)
{
    int32_t rc = check_cfg(cfg);
    if (rc) return rc;
    if (!out) return MKV_E_INVALID;
    mkv_pool* p = new_pool(cfg, nullptr, nullptr);
    if (!p) return MKV_E_INVALID;
    *out = p;
    return MKV_OK;
}

static mkv_pool* new_pool(const mkv_pool_config* cfg, void* fp8_arena, void* tq3_arena)
{
    mkv_pool* p = new (std::nothrow) mkv_pool();
    if (!p) return nullptr;
    p->cfg = *cfg;
    p->cfg.k_rot_signs = nullptr;
    p->d = cfg->head_dim;
    p->hkv = cfg->n_kv_heads;
    p->hq = cfg->n_q_heads;
    p->group = cfg->n_q_heads / cfg->n_kv_heads;
    p->tiles = cfg->page_size / kPage;
    p->fmt = cfg->tq3_format == 2 ? 2 : 1;
    p->fp8 = static_cast<uint8_t*>(fp8_arena);
    p->tq3 = static_cast<uint8_t*>(tq3_arena);
    p->variant = MKV_DECODE_TENSOR;
    p->wait_ns = 20000000ull;
    std::memset(&p->sigma, 0, sizeof p->sigma);
    for (int i = 0; cfg->k_rot_signs && i < cfg->head_dim; ++i)
        if (cfg->k_rot_signs[i] < 0) p->sigma.w[i >> 5] |= 1u << (i & 31);
    for (int f = 0; f < 2; ++f) {
        int n = f == MKV_FMT_FP8 ? cfg->fp8_pages : cfg->tq3_pages;
        p->free_list[f].reserve(n);
        for (int i = n - 1; i >= 0; --i) p->free_list[f].push_back(i);   // pops 0, 1, 2, ...
        p->allocated[f].assign(n, 0);
    }
    p->status_dev = nullptr;
    p->device = -1;
    return p;
}

int32_t mkv_pool_create(const mkv_pool_config* cfg, void* fp8_arena, void* tq3_arena, void* stream,
                        mkv_pool** out)
{
    int32_t rc = check_cfg(cfg);
    if (rc) return rc;
    if (!out || !fp8_arena || !tq3_arena || !cfg->k_rot_signs) return MKV_E_INVALID;
    if (!aligned(fp8_arena, 256) || !aligned(tq3_arena, 256)) return MKV_E_INVALID;
    for (int i = 0; i < cfg->head_dim; ++i)
        if (cfg->k_rot_signs[i] != 1 && cfg->k_rot_signs[i] != -1) return MKV_E_INVALID;
    mkv_pool* p = new_pool(cfg, fp8_arena, tq3_arena);
    if (!p) return MKV_E_INVALID;
    size_t fp8_bytes, tq3_bytes;
    mkv_pool_query(cfg, &fp8_bytes, &tq3_bytes);
    p->status_dev = reinterpret_cast<uint32_t*>(p->fp8 + fp8_bytes - kStatusTail);

    cudaError_t e = cudaGetDevice(&p->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&p->dev.sm_count, cudaDevAttrMultiProcessorCount, p->device);
    if (e == cudaSuccess)
        e = cudaDeviceGetAttribute(&p->dev.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, p->device);
    cudaStream_t s = (cudaStream_t)stream;
    if (e == cudaSuccess) e = cudaMemsetAsync(p->fp8, 0, fp8_bytes, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(p->tq3, 0, tq3_bytes, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) {
        delete p;
        return cuda_fail(e, "mkv_pool_create");
    }
    *out = p;
    return MKV_OK;
}

int32_t mkv_pool_destroy(mkv_pool* pool)
{
    if (!pool) return MKV_E_INVALID;
    delete pool;
    return MKV_OK;
}

int32_t mkv_page_alloc(mkv_pool* pool, int32_t fmt, int32_t* ids, int32_t n)
{
    if (!pool || (fmt != MKV_FMT_FP8 && fmt != MKV_FMT_TQ3) || n < 0 || (n > 0 && !ids)) return MKV_E_INVALID;
    std::lock_guard<std::mutex> lk(pool->mu);
    auto& fl = pool->free_list[fmt];
    if ((size_t)n > fl.size()) return fmt == MKV_FMT_FP8 ? MKV_E_OOM_FP8 : MKV_E_OOM_TQ3;
    for (int i = 0; i < n; ++i) {
        ids[i] = fl.back();
        fl.pop_back();
        pool->allocated[fmt][ids[i]] = 1;
    }
    return MKV_OK;
}

int32_t mkv_page_free(mkv_pool* pool, int32_t fmt, const int32_t* ids, int32_t n)
{
    if (!pool || (fmt != MKV_FMT_FP8 && fmt != MKV_FMT_TQ3) || n < 0 || (n > 0 && !ids)) return MKV_E_INVALID;
    std::lock_guard<std::mutex> lk(pool->mu);
    auto& al = pool->allocated[fmt];
    for (int i = 0; i < n; ++i) {
        if (ids[i] < 0 || (size_t)ids[i] >= al.size()) return MKV_E_BOUNDS;
        if (al[ids[i]] != 1) return MKV_E_STATE;          // free already, or retiring (mkv_seq_release frees those)
        for (int j = 0; j < i; ++j)
            if (ids[j] == ids[i]) return MKV_E_STATE;
    }
    for (int i = 0; i < n; ++i) {
        al[ids[i]] = 0;
        pool->free_list[fmt].push_back(ids[i]);
    }
    return MKV_OK;
}

int32_t mkv_pool_stats(const mkv_pool* pool, mkv_stats* out)
{
    if (!pool || !out) return MKV_E_INVALID;
    mkv_pool* p = const_cast<mkv_pool*>(pool);
    std::lock_guard<std::mutex> lk(p->mu);
    out->fp8_pages_total = p->cfg.fp8_pages;
    out->tq3_pages_total = p->cfg.tq3_pages;
    out->fp8_pages_used = p->cfg.fp8_pages - (int64_t)p->free_list[0].size();
    out->tq3_pages_used = p->cfg.tq3_pages - (int64_t)p->free_list[1].size();
    out->fp8_bytes_used = out->fp8_pages_used * p->hkv * (int64_t)fp8_page_bytes(p->d, p->tiles);
    out->tq3_bytes_used = out->tq3_pages_used * p->hkv * (int64_t)tq3_page_bytes(p->d, p->tiles);
    out->bf16_bytes_equivalent = (out->fp8_pages_used + out->tq3_pages_used) * p->hkv * (int64_t)p->cfg.page_size * p->d * 4;
    return MKV_OK;
}

int32_t mkv_pool_status(mkv_pool* pool, void* stream)
{
    if (!pool || !pool->fp8) return MKV_E_INVALID;
    uint32_t st = 0;
    cudaStream_t s = (cudaStream_t)stream;
    MKV_CUDA(cudaMemcpyAsync(&st, pool->status_dev, sizeof st, cudaMemcpyDeviceToHost, s));
    MKV_CUDA(cudaStreamSynchronize(s));
    if (st) {
        MKV_CUDA(cudaMemsetAsync(pool->status_dev, 0, sizeof st, s));
        MKV_CUDA(cudaStreamSynchronize(s));
    }
    if (st & kStTimeout) return MKV_E_TIMEOUT;
    if (st & kStBounds) return MKV_E_BOUNDS;
    if (st & kStState) return MKV_E_STATE;
    return MKV_OK;
}

int32_t mkv_pool_set_decode_variant(mkv_pool* pool, int32_t variant)
{
    if (!pool || (variant != MKV_DECODE_TENSOR && variant != MKV_DECODE_SCALAR && variant != MKV_DECODE_TMEM)) return MKV_E_INVALID;
    pool->variant = variant;
    return MKV_OK;
}

int32_t mkv_pool_set_wait_limit_ns(mkv_pool* pool, uint64_t ns)
{
    if (!pool) return MKV_E_INVALID;
    pool->wait_ns = ns;
    return MKV_OK;
}

static int32_t raw_span(mkv_pool* pool, int32_t fmt, int32_t id, uint8_t** ptr, size_t* bytes)
{
    if (!pool || !pool->fp8 || (fmt != MKV_FMT_FP8 && fmt != MKV_FMT_TQ3)) return MKV_E_INVALID;
    int cap = fmt == MKV_FMT_FP8 ? pool->cfg.fp8_pages : pool->cfg.tq3_pages;
    if (id < 0 || id >= cap) return MKV_E_BOUNDS;
    size_t rec = fmt == MKV_FMT_FP8 ? fp8_page_bytes(pool->d, pool->tiles) : tq3_page_bytes(pool->d, pool->tiles);
    *bytes = rec * pool->hkv;
    *ptr = (fmt == MKV_FMT_FP8 ? pool->fp8 : pool->tq3) + (size_t)id * *bytes;
    return MKV_OK;
}

int32_t mkv_page_read_raw(mkv_pool* pool, int32_t fmt, int32_t id, void* host_buf, void* stream)
{
    uint8_t* ptr;
    size_t bytes;
    int32_t rc = raw_span(pool, fmt, id, &ptr, &bytes);
    if (rc) return rc;
    if (!host_buf) return MKV_E_INVALID;
    MKV_CUDA(cudaMemcpyAsync(host_buf, ptr, bytes, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    MKV_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    return MKV_OK;
}

int32_t mkv_page_write_raw(mkv_pool* pool, int32_t fmt, int32_t id, const void* host_buf, void* stream)
{
    uint8_t* ptr;
    size_t bytes;
    int32_t rc = raw_span(pool, fmt, id, &ptr, &bytes);
    if (rc) return rc;
    if (!host_buf) return MKV_E_INVALID;
    MKV_CUDA(cudaMemcpyAsync(ptr, host_buf, bytes, cudaMemcpyHostToDevice, (cudaStream_t)stream));
    MKV_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    return MKV_OK;
}

// ---- hot-path entry points: validate on the host, then enqueue ---------------------------------

int32_t mkv_append(mkv_pool* pool, const void* k, const void* v, const int32_t* slots, int32_t n, void* stream)
{
    if (!pool || !pool->fp8 || n < 0) return MKV_E_INVALID;
    if (n == 0) return MKV_OK;
    if (!k || !v || !slots || !aligned(k, 16) || !aligned(v, 16) || !aligned(slots, 4)) return MKV_E_INVALID;
    return launch_append(pool, k, v, slots, n, (cudaStream_t)stream);
}

int32_t mkv_demote(mkv_pool* pool, const int32_t* src, const int32_t* dst, int32_t n, int32_t* bt,
                   uint8_t* tags, const int64_t* entry, int64_t table_entries, void* stream)
{
    if (!pool || !pool->fp8 || n < 0) return MKV_E_INVALID;
    if (n == 0) return MKV_OK;
    if (!src || !dst) return MKV_E_INVALID;
    if (entry && (!bt || !tags || table_entries < 1)) return MKV_E_INVALID;
    return launch_demote(pool, src, dst, n, bt, tags, entry, table_entries, (cudaStream_t)stream);
}

int32_t mkv_promote(mkv_pool* pool, const int32_t* src, const int32_t* dst, int32_t n, int32_t* bt, uint8_t* tags,
                    const int64_t* entry, int64_t table_entries, void* stream)
{
    if (!pool || !pool->fp8 || n < 0) return MKV_E_INVALID;
    if (n == 0) return MKV_OK;
    if (!src || !dst) return MKV_E_INVALID;
    if (entry && (!bt || !tags || table_entries < 1)) return MKV_E_INVALID;
    return launch_promote(pool, src, dst, n, bt, tags, entry, table_entries, (cudaStream_t)stream);
}

int32_t mkv_set_anchor(mkv_pool* pool, uint8_t* tags, int64_t table_entries, int64_t entry, int32_t flag, void* stream)
{
    if (!pool || !pool->fp8 || !tags || entry < 0 || table_entries < 1) return MKV_E_INVALID;
    if (entry >= table_entries) return MKV_E_BOUNDS;
    return launch_set_anchor(pool, tags, entry, flag, (cudaStream_t)stream);
}

int32_t mkv_decode_attention(mkv_pool* pool, const void* q, const int32_t* bt, const uint8_t* tags,
                             const int32_t* lens, int32_t B, int32_t max_pages, float scale, float* out,
                             float* lse, void* ws, size_t ws_bytes, void* stream)
{
    if (!pool || !pool->fp8 || B < 0 || max_pages < 0) return MKV_E_INVALID;
    if (B == 0) return MKV_OK;
    if (!q || !bt || !tags || !lens || !out || !ws) return MKV_E_INVALID;
    if (!aligned(q, 16) || !aligned(out, 16) || !aligned(ws, 256) || !aligned(bt, 4) || !aligned(lens, 4))
        return MKV_E_INVALID;
    size_t need;
    if (mkv_decode_workspace_bytes(&pool->cfg, B, &need) != MKV_OK || ws_bytes < need) return MKV_E_INVALID;
    if (!(scale == scale)) return MKV_E_INVALID;
    if (pool->variant == MKV_DECODE_SCALAR)
        return launch_decode_scalar(pool, q, bt, tags, lens, B, max_pages, scale, out, lse, ws, ws_bytes,
                                    (cudaStream_t)stream);
    return launch_decode_tensor(pool, q, bt, tags, lens, B, max_pages, scale, out, lse, ws, ws_bytes,
                                (cudaStream_t)stream);
}

int32_t mkv_decode_attention_layers(const mkv_layer_call* L, int32_t n_layers, const int32_t* lens, int32_t B,
                                    int32_t max_pages, float scale, size_t ws_bytes, void* stream)
{
    if (!L || n_layers < 1 || n_layers > MKV_MAX_LAYERS_PER_CALL || B < 0 || max_pages < 0) return MKV_E_INVALID;
    if (B == 0) return MKV_OK;
    if (!lens || !aligned(lens, 4) || !(scale == scale)) return MKV_E_INVALID;
    mkv_pool* pools[MKV_MAX_LAYERS_PER_CALL];
    const void* q[MKV_MAX_LAYERS_PER_CALL];
    const int32_t* bt[MKV_MAX_LAYERS_PER_CALL];
    const uint8_t* tags[MKV_MAX_LAYERS_PER_CALL];
    float* out[MKV_MAX_LAYERS_PER_CALL];
    float* lse[MKV_MAX_LAYERS_PER_CALL];
    void* ws[MKV_MAX_LAYERS_PER_CALL];
    for (int i = 0; i < n_layers; ++i) {
        const mkv_layer_call& c = L[i];
        if (!c.pool || !c.pool->fp8 || !c.q_dev || !c.block_table_dev || !c.tier_tag_dev || !c.out_dev || !c.workspace_dev)
            return MKV_E_INVALID;
        if (!aligned(c.q_dev, 16) || !aligned(c.out_dev, 16) || !aligned(c.workspace_dev, 256) || !aligned(c.block_table_dev, 4))
            return MKV_E_INVALID;
        const mkv_pool* p0 = L[0].pool;
        if (c.pool->d != p0->d || c.pool->hkv != p0->hkv || c.pool->hq != p0->hq || c.pool->tiles != p0->tiles ||
            c.pool->device != p0->device || c.pool->variant != MKV_DECODE_TENSOR || c.pool->fmt != p0->fmt) {
            set_last_error("mkv_decode_attention_layers: pools of one geometry, page size, record format, one device and the tensor-core variant");
            return MKV_E_INVALID;
        }
        for (int j = 0; j < i; ++j)
            if (L[j].workspace_dev == c.workspace_dev) {
                set_last_error("mkv_decode_attention_layers: every layer needs its own workspace");
                return MKV_E_INVALID;
            }
        pools[i] = c.pool; q[i] = c.q_dev; bt[i] = c.block_table_dev; tags[i] = c.tier_tag_dev;
        out[i] = c.out_dev; lse[i] = c.lse_dev; ws[i] = c.workspace_dev;
    }
    size_t need;
    if (mkv_decode_workspace_bytes(&L[0].pool->cfg, B, &need) != MKV_OK || ws_bytes < need) return MKV_E_INVALID;
    return launch_decode_tensor_layers(pools, q, bt, tags, lens, B, max_pages, scale, out, lse, ws, n_layers,
                                       (cudaStream_t)stream);
}

int32_t mkv_append_layers(const mkv_layer_append* L, int32_t n_layers, const int32_t* slots, int32_t n, void* stream)
{
    if (!L || n_layers < 1 || n_layers > MKV_MAX_LAYERS_PER_CALL || n < 0 || n > 64) return MKV_E_INVALID;
    if (n == 0) return MKV_OK;
    if (!slots || !aligned(slots, 4)) return MKV_E_INVALID;
    mkv_pool* pools[MKV_MAX_LAYERS_PER_CALL];
    const void* k[MKV_MAX_LAYERS_PER_CALL];
    const void* v[MKV_MAX_LAYERS_PER_CALL];
    for (int i = 0; i < n_layers; ++i) {
        const mkv_layer_append& c = L[i];
        if (!c.pool || !c.pool->fp8 || !c.k_dev || !c.v_dev || !aligned(c.k_dev, 16) || !aligned(c.v_dev, 16)) return MKV_E_INVALID;
        const mkv_pool* p0 = L[0].pool;
        if (c.pool->d != p0->d || c.pool->hkv != p0->hkv || c.pool->tiles != p0->tiles || c.pool->device != p0->device) {
            set_last_error("mkv_append_layers: pools of one geometry on one device");
            return MKV_E_INVALID;
        }
        pools[i] = c.pool; k[i] = c.k_dev; v[i] = c.v_dev;
    }
    return launch_append_layers(pools, k, v, slots, n, n_layers, (cudaStream_t)stream);
}

int32_t mkv_decode_attention_scored(mkv_pool* pool, const void* q, const int32_t* bt, const uint8_t* tags,
                                    const int32_t* lens, int32_t B, int32_t max_pages, float scale, float* out,
                                    float* lse, float* page_mass, void* ws, size_t ws_bytes, void* stream)
{
    if (!pool || !pool->fp8 || B < 0 || max_pages < 0) return MKV_E_INVALID;
    if (B == 0) return MKV_OK;
    if (!q || !bt || !tags || !lens || !out || !ws || !lse || !page_mass) return MKV_E_INVALID;
    if (!aligned(q, 16) || !aligned(out, 16) || !aligned(ws, 256) || !aligned(bt, 4) || !aligned(lens, 4) ||
        !aligned(page_mass, 4) || !aligned(lse, 4))
        return MKV_E_INVALID;
    size_t need;
    if (mkv_decode_workspace_bytes(&pool->cfg, B, &need) != MKV_OK || ws_bytes < need) return MKV_E_INVALID;
    if (!(scale == scale)) return MKV_E_INVALID;
    uint32_t* tickets = reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(ws) + 256);
    float* partials = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + decode_ws_header_bytes(B, pool->hkv));
    return launch_decode_tensor_at(pool, q, bt, tags, lens, B, max_pages, scale, out, lse, partials, tickets, kMaxCtas,
                                   page_mass, (cudaStream_t)stream);
}

int32_t mkv_page_score_update_paged(const float* page_mass, const int32_t* lens, int32_t B, int32_t n_q_heads,
                                    int32_t max_pages, int32_t page_size, uint64_t head_mask, float beta, float* score,
                                    void* stream)
{
    if (B < 0 || max_pages < 0 || n_q_heads < 1 || n_q_heads > 64) return MKV_E_INVALID;
    if (page_size < kPage || page_size % kPage || page_size > kPage * kMaxTiles) return MKV_E_INVALID;
    if (B == 0 || max_pages == 0) return MKV_OK;
    if (!page_mass || !lens || !score || !(beta >= 0.f && beta <= 1.f)) return MKV_E_INVALID;
    if (n_q_heads < 64) head_mask &= (1ull << n_q_heads) - 1ull;
    return launch_page_score(page_mass, lens, B, n_q_heads, max_pages, head_mask, beta, score, page_size,
                             (cudaStream_t)stream);
}

int32_t mkv_page_score_update(const float* page_mass, const int32_t* lens, int32_t B, int32_t n_q_heads,
                              int32_t max_pages, uint64_t head_mask, float beta, float* score, void* stream)
{
    return mkv_page_score_update_paged(page_mass, lens, B, n_q_heads, max_pages, kPage, head_mask, beta, score, stream);
}

// ---- sequence rows (Algorithm 1, host bookkeeping only) ----------------------------------------

int32_t mkv_seq_create(mkv_pool* pool, mkv_seq** out)
{
    if (!pool || !out) return MKV_E_INVALID;
    mkv_seq* s = new (std::nothrow) mkv_seq();
    if (!s) return MKV_E_INVALID;
    s->pool = pool;
    s->len = 0;
    *out = s;
    return MKV_OK;
}

int32_t mkv_seq_finish(mkv_seq* seq)
{
    if (!seq) return MKV_E_INVALID;
    int32_t rc = MKV_OK;
    for (size_t i = 0; i < seq->ids.size(); ++i) {
        int fmt = seq->tags[i] == MKV_TAG_STALE ? MKV_FMT_TQ3 : MKV_FMT_FP8;
        int32_t r = mkv_page_free(seq->pool, fmt, &seq->ids[i], 1);
        if (r != MKV_OK) rc = r;
    }
    // sources still retiring go back too, in (format, id) order
    std::sort(seq->retiring.begin(), seq->retiring.end());
    while (!seq->retiring.empty()) {
        const std::pair<int32_t, int32_t> e = seq->retiring.front();
        int32_t r = mkv_seq_release(seq, e.first, e.second);
        if (r != MKV_OK) { rc = r; break; }
    }
    delete seq;
    return rc;
}

int32_t mkv_seq_append(mkv_seq* seq, int32_t* page_id, int32_t* slot, int32_t* opened)
{
    if (!seq || !page_id || !slot) return MKV_E_INVALID;
    const int T = seq->pool->cfg.page_size;
    bool open = seq->len % T == 0;
    if (open) {
        int32_t id;
        int32_t rc = mkv_page_alloc(seq->pool, MKV_FMT_FP8, &id, 1);
        if (rc) return rc;
        seq->ids.push_back(id);
        seq->tags.push_back(MKV_TAG_RECENT);
    }
    *page_id = seq->ids.back();
    *slot = seq->len % T;
    if (opened) *opened = open ? 1 : 0;
    seq->len += 1;
    return MKV_OK;
}

int32_t mkv_seq_protect(mkv_seq* seq, int32_t lp, int32_t flag)
{
    if (!seq) return MKV_E_INVALID;
    if (lp < 0 || (size_t)lp >= seq->ids.size()) return MKV_E_BOUNDS;
    if (seq->tags[lp] == MKV_TAG_STALE) return MKV_E_STATE;
    if (!flag && seq->tags[lp] != MKV_TAG_ANCHOR) return MKV_E_STATE;
    seq->tags[lp] = flag ? MKV_TAG_ANCHOR : MKV_TAG_RECENT;
    return MKV_OK;
}

// The source of a planned conversion: it leaves the row but stays out of the free list (state 2) until the
// caller reports, with mkv_seq_release, that earlier readers and the conversion are ordered before any later writer.
static int32_t retire_source(mkv_seq* seq, int32_t fmt, int32_t id)
{
    std::lock_guard<std::mutex> lk(seq->pool->mu);
    seq->pool->allocated[fmt][id] = 2;
    seq->retiring.emplace_back(fmt, id);
    return MKV_OK;
}

int32_t mkv_seq_demote(mkv_seq* seq, int32_t lp, int32_t* src, int32_t* dst)
{
    if (!seq || !src || !dst) return MKV_E_INVALID;
    if (lp < 0 || (size_t)lp >= seq->ids.size()) return MKV_E_BOUNDS;
    if (seq->tags[lp] == MKV_TAG_STALE) return MKV_E_STATE;
    if ((int64_t)(lp + 1) * seq->pool->cfg.page_size > seq->len) return MKV_E_STATE;   // only full pages may become TQ3
    int32_t id;
    int32_t rc = mkv_page_alloc(seq->pool, MKV_FMT_TQ3, &id, 1);
    if (rc) return rc;
    *src = seq->ids[lp];
    *dst = id;
    seq->ids[lp] = id;
    seq->tags[lp] = MKV_TAG_STALE;
    return retire_source(seq, MKV_FMT_FP8, *src);
}

int32_t mkv_seq_promote(mkv_seq* seq, int32_t lp, int32_t* src, int32_t* dst)
{
    if (!seq || !src || !dst) return MKV_E_INVALID;
    if (lp < 0 || (size_t)lp >= seq->ids.size()) return MKV_E_BOUNDS;
    if (seq->tags[lp] != MKV_TAG_STALE) return MKV_E_STATE;
    int32_t id;
    int32_t rc = mkv_page_alloc(seq->pool, MKV_FMT_FP8, &id, 1);
    if (rc) return rc;
    *src = seq->ids[lp];
    *dst = id;
    seq->ids[lp] = id;
    seq->tags[lp] = MKV_TAG_ANCHOR;
    return retire_source(seq, MKV_FMT_TQ3, *src);
}

int32_t mkv_seq_release(mkv_seq* seq, int32_t fmt, int32_t id)
{
    if (!seq || (fmt != MKV_FMT_FP8 && fmt != MKV_FMT_TQ3)) return MKV_E_INVALID;
    mkv_pool* pool = seq->pool;
    std::lock_guard<std::mutex> lk(pool->mu);
    if (id < 0 || (size_t)id >= pool->allocated[fmt].size()) return MKV_E_BOUNDS;
    for (size_t i = 0; i < seq->retiring.size(); ++i)
        if (seq->retiring[i].first == fmt && seq->retiring[i].second == id) {
            seq->retiring.erase(seq->retiring.begin() + (long)i);
            pool->allocated[fmt][id] = 0;
            pool->free_list[fmt].push_back(id);
            return MKV_OK;
        }
    return MKV_E_STATE;                                    // not a retiring source of this sequence
}

int32_t mkv_seq_age(mkv_seq* seq, int32_t recent_tokens, int32_t* lps, int32_t* srcs, int32_t* dsts,
                    int32_t cap, int32_t* n)
{
    if (!seq || !n || recent_tokens < 0 || cap < 0) return MKV_E_INVALID;
    const int T = seq->pool->cfg.page_size;
    int first_recent = (seq->len - recent_tokens > 0 ? seq->len - recent_tokens : 0) / T;
    if ((size_t)first_recent > seq->ids.size()) first_recent = (int)seq->ids.size();
    int need = 0;
    for (int lp = 0; lp < first_recent; ++lp)
        if (seq->tags[lp] == MKV_TAG_RECENT && (int64_t)(lp + 1) * T <= seq->len) ++need;
    if (need > cap || (need > 0 && (!lps || !srcs || !dsts))) return MKV_E_INVALID;
    {
        std::lock_guard<std::mutex> lk(seq->pool->mu);
        if ((size_t)need > seq->pool->free_list[MKV_FMT_TQ3].size()) return MKV_E_OOM_TQ3;
    }
    int k = 0;
    for (int lp = 0; lp < first_recent; ++lp)
        if (seq->tags[lp] == MKV_TAG_RECENT && (int64_t)(lp + 1) * T <= seq->len) {
            int32_t rc = mkv_seq_demote(seq, lp, &srcs[k], &dsts[k]);
            if (rc) return rc;
            lps[k++] = lp;
        }
    *n = k;
    return MKV_OK;
}

int32_t mkv_seq_len(const mkv_seq* seq, int32_t* len, int32_t* n_pages)
{
    if (!seq) return MKV_E_INVALID;
    if (len) *len = seq->len;
    if (n_pages) *n_pages = (int32_t)seq->ids.size();
    return MKV_OK;
}

int32_t mkv_seq_row(const mkv_seq* seq, int32_t* ids, uint8_t* tags, int32_t cap)
{
    if (!seq || cap < (int32_t)seq->ids.size()) return MKV_E_INVALID;
    for (size_t i = 0; i < seq->ids.size(); ++i) {
        if (ids) ids[i] = seq->ids[i];
        if (tags) tags[i] = seq->tags[i];
    }
    return MKV_OK;
}

}  // extern "C"
