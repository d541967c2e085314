// C-ABI layer: argument validation, layer offsets, dispatch to the kernels.
// Nothing here touches device memory on the host side or allocates any.
#include <math.h>

#include "../../include/bt.h"
#include "bt_kernels.h"

namespace {

constexpr float kLog2e = 1.4426950408889634f;

bool config_ok(const bt_config* c)
{
    return c && c->batch > 0 && c->heads > 0 && c->head_dim > 0 && c->block_len > 0 && c->prefix_len > 0 &&
           c->max_blocks > 0 && c->n_layers > 0 && c->decode_splits >= 0 && c->softmax_scale >= 0.f &&
           isfinite(c->softmax_scale);
}

bt_status check_config(const bt_config* c, int layer)
{
    if (!c) return BT_ERR_NULL;
    if (!config_ok(c)) return BT_ERR_SHAPE;
    if (layer < 0 || layer >= c->n_layers) return BT_ERR_SHAPE;
    if (c->head_dim != 64 && c->head_dim != 128) return BT_ERR_UNSUPPORTED;
    if (c->heads * (c->head_dim / 8) > 256) return BT_ERR_UNSUPPORTED;  // one CTA must cover a sequence
    if (c->decode_splits > 64) return BT_ERR_UNSUPPORTED;
    return BT_OK;
}

float scale_log2(const bt_config* c)
{
    const float s = c->softmax_scale > 0.f ? c->softmax_scale : 1.0f / sqrtf((float)c->head_dim);
    return s * kLog2e;
}

int choose_splits(const bt_config* c)
{
    if (c->decode_splits > 0) return c->decode_splits;
    // enough work items to reach every SM several times over, each of at least 128 rows (four chunks of the
    // streaming kernel; below that the per-item costs show) - short caches may still be cut into up to 4
    // parts of at least 16 rows
    const long long bh = (long long)c->batch * c->heads;
    const long long target = 512;
    long long s = (target + bh - 1) / bh;
    long long by_rows = c->max_blocks / 128;
    const long long small = c->max_blocks / 16 < 4 ? c->max_blocks / 16 : 4;
    if (by_rows < small) by_rows = small;
    if (by_rows < 1) by_rows = 1;
    if (s > by_rows) s = by_rows;
    if (s > 32) s = 32;
    if (s < 1) s = 1;
    return (int)s;
}

inline size_t block_layer_elems(const bt_config* c) { return (size_t)c->batch * c->heads * c->max_blocks * c->head_dim; }
inline int local_cap(const bt_config* c) { return c->prefix_len + c->block_len; }
inline size_t local_layer_elems(const bt_config* c) { return (size_t)c->batch * c->heads * local_cap(c) * 2 * c->head_dim; }

bt::CacheView block_view(const bt_config* c, const bt_block_cache* cache, int layer)
{
    bt::CacheView v;
    v.k = (char*)cache->k + block_layer_elems(c) * layer * 2;
    v.v = (char*)cache->v + block_layer_elems(c) * layer * 2;
    v.len = cache->len + (size_t)layer * c->batch;
    v.slab_stride = (int64_t)c->max_blocks * c->head_dim;
    v.row_stride = c->head_dim;
    v.cap = c->max_blocks;
    return v;
}

bt::CacheView local_view(const bt_config* c, const bt_local_cache* cache, int layer)
{
    bt::CacheView v;
    char* base = (char*)cache->kv + local_layer_elems(c) * layer * 2;
    v.k = base;
    v.v = base + (size_t)c->head_dim * 2;
    v.len = cache->len + (size_t)layer * c->batch;
    v.slab_stride = (int64_t)local_cap(c) * 2 * c->head_dim;
    v.row_stride = 2 * c->head_dim;
    v.cap = local_cap(c);
    return v;
}

inline bt_status cuda_status(cudaError_t e) { return e == cudaSuccess ? BT_OK : BT_ERR_CUDA; }

// The kernels move data in 16-byte pieces (128-bit loads and stores, cp.async, bulk and tensor copies):
// every tensor base must sit on a 16-byte boundary, length arrays on a 4-byte one.  NULL passes (it
// is either optional or refused as BT_ERR_NULL elsewhere).
inline bool al16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool al4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }
inline bool block_cache_aligned(const bt_block_cache* c) { return al16(c->k) && al16(c->v) && al4(c->len); }
inline bool local_cache_aligned(const bt_local_cache* c) { return al16(c->kv) && al4(c->len); }

// what bt_block_decode_attn (k_new == NULL) and bt_block_decode_step check before anything is enqueued
bt_status decode_validate(const bt_config* cfg, const bt_block_cache* cache, int layer, const void* q, const void* k_new,
                                 const void* v_new, bool step, const void* out, const void* workspace, size_t workspace_bytes,
                                 const uint32_t* dev_status)
{
    bt_status st = check_config(cfg, layer);
    if (st != BT_OK) return st;
    if (!cache || !cache->k || !cache->v || !cache->len || !q || !out) return BT_ERR_NULL;
    if (step && (!k_new || !v_new)) return BT_ERR_NULL;
    const bool need_ws = choose_splits(cfg) > 1 || step;
    if (need_ws && (!workspace || workspace_bytes < bt_workspace_bytes(cfg))) return BT_ERR_WORKSPACE;
    if (!block_cache_aligned(cache) || !al16(q) || !al16(out) || !al16(k_new) || !al16(v_new) || !al4(dev_status) ||
        (need_ws && !al16(workspace)))
        return BT_ERR_UNSUPPORTED;
    return BT_OK;
}

}  // namespace

namespace bt {
bt_status validate_decode_attn_args(const bt_config* cfg, const bt_block_cache* cache, int layer, const void* q, const void* out,
                                    const uint32_t* dev_status)
{
    // a workspace that cannot be refused: only the other arguments are judged
    return decode_validate(cfg, cache, layer, q, nullptr, nullptr, false, out, reinterpret_cast<const void*>(uintptr_t(16)),
                           ~size_t(0), dev_status);
}
}  // namespace bt

extern "C" {

int bt_version(void) { return 200; }

const char* bt_status_string(bt_status s)
{
    switch (s) {
        case BT_OK: return "BT_OK";
        case BT_ERR_NULL: return "BT_ERR_NULL";
        case BT_ERR_SHAPE: return "BT_ERR_SHAPE";
        case BT_ERR_UNSUPPORTED: return "BT_ERR_UNSUPPORTED";
        case BT_ERR_CAPACITY: return "BT_ERR_CAPACITY";
        case BT_ERR_WORKSPACE: return "BT_ERR_WORKSPACE";
        case BT_ERR_CUDA: return "BT_ERR_CUDA";
    }
    return "BT_ERR_?";
}

int bt_decode_splits(const bt_config* cfg)
{
    if (check_config(cfg, 0) != BT_OK) return 0;
    return choose_splits(cfg);
}

// Workspace layout: the split partials ([B*H][splits][hd+4] floats, absent when the row range is not
// split), then the arrival counters ([B*H] + [B] int32).
static size_t partial_bytes(const bt_config* cfg)
{
    const int s = choose_splits(cfg);
    return s <= 1 ? 0 : (size_t)s * cfg->batch * cfg->heads * (cfg->head_dim + 4) * sizeof(float);
}
static size_t counter_bytes(const bt_config* cfg) { return ((size_t)cfg->batch * cfg->heads + cfg->batch) * sizeof(int32_t); }

size_t bt_workspace_bytes(const bt_config* cfg)
{
    if (check_config(cfg, 0) != BT_OK) return 0;
    return partial_bytes(cfg) + counter_bytes(cfg);
}

bt_status bt_workspace_init(const bt_config* cfg, void* workspace, size_t workspace_bytes, void* stream)
{
    bt_status st = check_config(cfg, 0);
    if (st != BT_OK) return st;
    if (!workspace) return BT_ERR_NULL;
    if (workspace_bytes < bt_workspace_bytes(cfg)) return BT_ERR_WORKSPACE;
    if (!al16(workspace)) return BT_ERR_UNSUPPORTED;
    return cuda_status(cudaMemsetAsync((char*)workspace + partial_bytes(cfg), 0, counter_bytes(cfg), (cudaStream_t)stream));
}

bt_status bt_block_kv_append(const bt_config* cfg, bt_block_cache* cache, int layer, const void* k_new,
                             const void* v_new, int n_new, uint32_t* dev_status, void* stream)
{
    bt_status st = check_config(cfg, layer);
    if (st != BT_OK) return st;
    if (!cache || !cache->k || !cache->v || !cache->len || !k_new || !v_new) return BT_ERR_NULL;
    if (n_new <= 0) return BT_ERR_SHAPE;
    if (n_new > cfg->max_blocks) return BT_ERR_CAPACITY;
    if (!block_cache_aligned(cache) || !al16(k_new) || !al16(v_new) || !al4(dev_status)) return BT_ERR_UNSUPPORTED;
    return cuda_status(bt::launch_kv_append(block_view(cfg, cache, layer), cfg->batch, cfg->heads, cfg->head_dim,
                                            k_new, v_new, n_new, dev_status, (cudaStream_t)stream));
}

// append (optional) + attention in one launch; the arguments have passed decode_validate
static bt_status decode_launch(const bt_config* cfg, bt_block_cache* cache, int layer, const void* q, const void* k_new,
                               const void* v_new, void* out, void* workspace, size_t workspace_bytes,
                               uint32_t* dev_status, void* stream)
{
    const int splits = choose_splits(cfg);
    const bool need_ws = splits > 1 || k_new != nullptr;
    (void)workspace_bytes;
    bt::CacheView v = block_view(cfg, cache, layer);
    bt::DecodeArgs a;
    a.q = q;
    a.k = v.k;
    a.v = v.v;
    a.len = v.len;
    a.out = out;
    a.ws = (float*)workspace;
    a.counters = need_ws ? (int32_t*)((char*)workspace + partial_bytes(cfg)) : nullptr;
    a.k_new = k_new;
    a.v_new = v_new;
    a.dev_status = dev_status;
    a.B = cfg->batch;
    a.H = cfg->heads;
    a.hd = cfg->head_dim;
    a.n_max = cfg->max_blocks;
    a.splits = splits;
    a.scale_log2 = scale_log2(cfg);
    return cuda_status(bt::launch_block_decode(a, (cudaStream_t)stream));
}

bt_status bt_block_decode_attn(const bt_config* cfg, const bt_block_cache* cache, int layer, const void* q,
                               void* out, void* workspace, size_t workspace_bytes, uint32_t* dev_status,
                               void* stream)
{
    bt_status st = decode_validate(cfg, cache, layer, q, nullptr, nullptr, false, out, workspace, workspace_bytes, dev_status);
    if (st != BT_OK) return st;
    // without a row to append the kernel only reads the cache
    return decode_launch(cfg, const_cast<bt_block_cache*>(cache), layer, q, nullptr, nullptr, out, workspace,
                         workspace_bytes, dev_status, stream);
}

bt_status bt_block_decode_step(const bt_config* cfg, bt_block_cache* cache, int layer, const void* q,
                               const void* k_new, const void* v_new, void* out, void* workspace,
                               size_t workspace_bytes, uint32_t* dev_status, void* stream)
{
    bt_status st = decode_validate(cfg, cache, layer, q, k_new, v_new, true, out, workspace, workspace_bytes, dev_status);
    if (st != BT_OK) return st;
    return decode_launch(cfg, cache, layer, q, k_new, v_new, out, workspace, workspace_bytes, dev_status, stream);
}

bt_status bt_block_decode_step_multi(const bt_config* cfg, bt_block_cache* cache, int layer, const void* q,
                                     const void* k_new, const void* v_new, int n_q, void* out, void* workspace,
                                     size_t workspace_bytes, uint32_t* dev_status, void* stream)
{
    bt_status st = check_config(cfg, layer);
    if (st != BT_OK) return st;
    if (!cache || !cache->k || !cache->v || !cache->len || !q || !k_new || !v_new || !out) return BT_ERR_NULL;
    if (n_q <= 0) return BT_ERR_SHAPE;
    if (n_q > cfg->max_blocks) return BT_ERR_CAPACITY;
    if (!workspace || workspace_bytes < bt_workspace_bytes(cfg)) return BT_ERR_WORKSPACE;
    if (!block_cache_aligned(cache) || !al16(workspace) || !al4(dev_status)) return BT_ERR_UNSUPPORTED;
    bt::CacheView v = block_view(cfg, cache, layer);
    bt::MultiDecodeArgs a;
    a.q = q;
    a.k_new = k_new;
    a.v_new = v_new;
    a.k = v.k;
    a.v = v.v;
    a.len = v.len;
    a.out = out;
    a.counters = (int32_t*)((char*)workspace + partial_bytes(cfg));
    a.dev_status = dev_status;
    a.B = cfg->batch;
    a.H = cfg->heads;
    a.hd = cfg->head_dim;
    a.n_max = cfg->max_blocks;
    a.m = n_q;
    a.scale_log2 = scale_log2(cfg);
    if (!bt::multi_decode_supported(a)) return BT_ERR_UNSUPPORTED;
    return cuda_status(bt::launch_block_decode_multi(a, (cudaStream_t)stream));
}

bt_status bt_local_kv_reset(const bt_config* cfg, bt_local_cache* cache, int layer, const uint8_t* seq_mask,
                            void* stream)
{
    bt_status st = check_config(cfg, layer);
    if (st != BT_OK) return st;
    if (!cache || !cache->len) return BT_ERR_NULL;
    if (!al4(cache->len)) return BT_ERR_UNSUPPORTED;
    return cuda_status(bt::launch_len_reset(cache->len + (size_t)layer * cfg->batch, cfg->batch, seq_mask,
                                            (cudaStream_t)stream));
}

bt_status bt_local_kv_append(const bt_config* cfg, bt_local_cache* cache, int layer, const void* k_new,
                             const void* v_new, int n_new, uint32_t* dev_status, void* stream)
{
    bt_status st = check_config(cfg, layer);
    if (st != BT_OK) return st;
    if (!cache || !cache->kv || !cache->len || !k_new || !v_new) return BT_ERR_NULL;
    if (n_new <= 0) return BT_ERR_SHAPE;
    if (n_new > local_cap(cfg)) return BT_ERR_CAPACITY;
    if (!local_cache_aligned(cache) || !al16(k_new) || !al16(v_new) || !al4(dev_status)) return BT_ERR_UNSUPPORTED;
    return cuda_status(bt::launch_kv_append(local_view(cfg, cache, layer), cfg->batch, cfg->heads, cfg->head_dim,
                                            k_new, v_new, n_new, dev_status, (cudaStream_t)stream));
}

bt_status bt_token_decode_attn(const bt_config* cfg, bt_local_cache* cache, int layer, const void* q,
                               const void* k_new, const void* v_new, int n_q, int reset_first,
                               const uint8_t* reset_mask, void* out, uint32_t* dev_status, void* stream)
{
    bt_status st = check_config(cfg, layer);
    if (st != BT_OK) return st;
    if (!cache || !cache->kv || !cache->len || !q || !out) return BT_ERR_NULL;
    if ((k_new == nullptr) != (v_new == nullptr)) return BT_ERR_NULL;
    if (n_q <= 0) return BT_ERR_SHAPE;
    if (n_q > local_cap(cfg)) return BT_ERR_CAPACITY;
    if (!local_cache_aligned(cache) || !al16(q) || !al16(k_new) || !al16(v_new) || !al16(out) || !al4(dev_status))
        return BT_ERR_UNSUPPORTED;
    bt::TokenArgs a;
    a.kv = (char*)cache->kv + local_layer_elems(cfg) * layer * 2;
    a.len = cache->len + (size_t)layer * cfg->batch;
    a.q = q;
    a.k_new = k_new;
    a.v_new = v_new;
    a.out = out;
    a.reset_mask = reset_mask;
    a.dev_status = dev_status;
    a.B = cfg->batch;
    a.H = cfg->heads;
    a.hd = cfg->head_dim;
    a.cap = local_cap(cfg);
    a.n_q = n_q;
    a.reset_first = reset_first ? 1 : 0;
    a.scale_log2 = scale_log2(cfg);
    return cuda_status(bt::launch_token_decode(a, (cudaStream_t)stream));
}

bt_status bt_block_prefill_attn(const bt_config* cfg, const void* q, const void* k, const void* v, int n_blocks,
                                int64_t kv_seq_stride, void* out, uint32_t* dev_status, void* stream)
{
    bt_status st = check_config(cfg, 0);
    if (st != BT_OK) return st;
    if (!q || !k || !v || !out) return BT_ERR_NULL;
    if (n_blocks <= 0 || kv_seq_stride < n_blocks) return BT_ERR_SHAPE;
    if (!al16(q) || !al16(k) || !al16(v) || !al16(out) || !al4(dev_status)) return BT_ERR_UNSUPPORTED;
    bt::PrefillArgs a;
    a.q = q;
    a.k = k;
    a.v = v;
    a.out = out;
    a.B = cfg->batch;
    a.H = cfg->heads;
    a.hd = cfg->head_dim;
    a.T = n_blocks;
    a.kv_seq_stride = kv_seq_stride;
    a.scale_log2 = scale_log2(cfg);
    // the kernel is the caller's choice, never a silent switch: the tensor-core one unless the config asks
    // for the CUDA-core one
    if (cfg->prefill_plain) return cuda_status(bt::launch_block_prefill_simple(a, (cudaStream_t)stream));
    if (!bt::prefill_tc_supported(a)) return BT_ERR_UNSUPPORTED;  // no driver entry point for tensor maps
    return cuda_status(bt::launch_block_prefill_tc(a, dev_status, (cudaStream_t)stream));
}

bt_status bt_block_decode_step_host(const bt_config* cfg, bt_block_cache* cache, int layer, const void* q_host,
                                    const void* k_new_host, const void* v_new_host, void* out_host, void* q_dev,
                                    void* k_dev, void* v_dev, void* out_dev, void* workspace,
                                    size_t workspace_bytes, uint32_t* dev_status, void* stream)
{
    // everything bt_block_decode_step would refuse is refused here, before the first copy is enqueued
    bt_status st = check_config(cfg, layer);
    if (st != BT_OK) return st;
    if (!q_host || !k_new_host || !v_new_host || !out_host || !q_dev || !k_dev || !v_dev || !out_dev) return BT_ERR_NULL;
    st = decode_validate(cfg, cache, layer, q_dev, k_dev, v_dev, true, out_dev, workspace, workspace_bytes, dev_status);
    if (st != BT_OK) return st;
    const size_t bytes = (size_t)cfg->batch * cfg->heads * cfg->head_dim * 2;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemcpyAsync(k_dev, k_new_host, bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return BT_ERR_CUDA;
    if (cudaMemcpyAsync(v_dev, v_new_host, bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return BT_ERR_CUDA;
    if (cudaMemcpyAsync(q_dev, q_host, bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return BT_ERR_CUDA;
    st = decode_launch(cfg, cache, layer, q_dev, k_dev, v_dev, out_dev, workspace, workspace_bytes, dev_status, stream);
    if (st != BT_OK) return st;
    if (cudaMemcpyAsync(out_host, out_dev, bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return BT_ERR_CUDA;
    return BT_OK;
}

// ---- the linear maps either side of the attention path

static bt_status project_common(const bt_config* cfg, const void* x, const void* w, const void* bias, const void* out,
                                const uint32_t* dev_status)
{
    if (!x || !w || !out) return BT_ERR_NULL;
    if (!al16(x) || !al16(w) || !al16(bias) || !al16(out) || !al4(dev_status)) return BT_ERR_UNSUPPORTED;
    if ((long long)cfg->heads * cfg->head_dim > (1 << 20)) return BT_ERR_UNSUPPORTED;
    return BT_OK;
}

bt_status bt_prefix_project(const bt_config* cfg, const void* ctx, const void* w_prefix, const void* bias, void* prefix_out,
                            uint32_t* dev_status, void* stream)
{
    bt_status st = check_config(cfg, 0);
    if (st != BT_OK) return st;
    st = project_common(cfg, ctx, w_prefix, bias, prefix_out, dev_status);
    if (st != BT_OK) return st;
    const long long D = (long long)cfg->heads * cfg->head_dim;
    if (D * cfg->prefix_len > 0x7fffffffLL) return BT_ERR_UNSUPPORTED;
    bt::ProjectArgs a = {};
    a.x = ctx;
    a.w = w_prefix;
    a.bias = bias;
    a.out = prefix_out;
    a.M = cfg->batch;
    a.K = (int)D;
    a.N = (int)(D * cfg->prefix_len);
    a.mode = bt::kProjectPlain;
    a.dev_status = dev_status;
    if (!bt::project_supported(a)) return BT_ERR_UNSUPPORTED;
    return cuda_status(bt::launch_project(a, (cudaStream_t)stream));
}

static bt_status qkv_project(const bt_config* cfg, const bt::CacheView& view, const void* x, int n_rows, const void* w_qkv,
                             const void* bias, int reset_first, const uint8_t* reset_mask, void* q_out, uint32_t* dev_status,
                             void* stream)
{
    const long long D = (long long)cfg->heads * cfg->head_dim;
    if ((long long)cfg->batch * n_rows > 0x7fffffffLL / 2 || 3 * D > 0x7fffffffLL) return BT_ERR_UNSUPPORTED;
    bt::ProjectArgs a = {};
    a.x = x;
    a.w = w_qkv;
    a.bias = bias;
    a.out = q_out;
    a.M = cfg->batch * n_rows;
    a.K = (int)D;
    a.N = (int)(3 * D);
    a.mode = bt::kProjectQkv;
    a.cache = view;
    a.n_rows = n_rows;
    a.H = cfg->heads;
    a.hd = cfg->head_dim;
    a.reset_first = reset_first ? 1 : 0;
    a.reset_mask = reset_mask;
    a.dev_status = dev_status;
    if (!bt::project_supported(a)) return BT_ERR_UNSUPPORTED;
    return cuda_status(bt::launch_project(a, (cudaStream_t)stream));
}

bt_status bt_block_qkv_project_append(const bt_config* cfg, bt_block_cache* cache, int layer, const void* x, int n_rows,
                                      const void* w_qkv, const void* bias, void* q_out, uint32_t* dev_status, void* stream)
{
    bt_status st = check_config(cfg, layer);
    if (st != BT_OK) return st;
    if (!cache || !cache->k || !cache->v || !cache->len) return BT_ERR_NULL;
    st = project_common(cfg, x, w_qkv, bias, q_out, dev_status);
    if (st != BT_OK) return st;
    if (n_rows <= 0) return BT_ERR_SHAPE;
    if (n_rows > cfg->max_blocks) return BT_ERR_CAPACITY;
    if (!block_cache_aligned(cache)) return BT_ERR_UNSUPPORTED;
    return qkv_project(cfg, block_view(cfg, cache, layer), x, n_rows, w_qkv, bias, 0, nullptr, q_out, dev_status, stream);
}

bt_status bt_local_qkv_project_append(const bt_config* cfg, bt_local_cache* cache, int layer, const void* x, int n_rows,
                                      const void* w_qkv, const void* bias, int reset_first, const uint8_t* reset_mask,
                                      void* q_out, uint32_t* dev_status, void* stream)
{
    bt_status st = check_config(cfg, layer);
    if (st != BT_OK) return st;
    if (!cache || !cache->kv || !cache->len) return BT_ERR_NULL;
    st = project_common(cfg, x, w_qkv, bias, q_out, dev_status);
    if (st != BT_OK) return st;
    if (n_rows <= 0) return BT_ERR_SHAPE;
    if (n_rows > local_cap(cfg)) return BT_ERR_CAPACITY;
    if (!local_cache_aligned(cache)) return BT_ERR_UNSUPPORTED;
    return qkv_project(cfg, local_view(cfg, cache, layer), x, n_rows, w_qkv, bias, reset_first, reset_mask, q_out, dev_status, stream);
}

bt_status bt_selftest_bounded_wait(uint32_t* report, uint32_t* dev_status, void* stream)
{
    if (!dev_status) return BT_ERR_NULL;
    if (!al4(report) || !al4(dev_status)) return BT_ERR_UNSUPPORTED;
    return cuda_status(bt::launch_selftest_bounded_wait(report, dev_status, (cudaStream_t)stream));
}

}  // extern "C"
