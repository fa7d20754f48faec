// C ABI of the skv library (see include/skv.h): argument checking, the routed
// owner-only page allocator's bookkeeping, and kernel launches.  Host code only.
#include "../../include/skv.h"
#include "skv_common.cuh"

#include <math.h>
#include <new>
#include <stdlib.h>
#include <string.h>
#include <vector>

using namespace skv;

struct skv_cache {
    int n_layers = 0, kv_heads = 0, head_dim = 0, page_size = 0, n_owners = 0;
    int64_t max_pages = 0;
    std::vector<int32_t> r;          // routing map
    std::vector<int32_t> slot;       // layer -> rank among owners, or -1
    std::vector<int32_t> owners;     // owner layers in increasing order
    uint8_t *pool = nullptr;         // caller's device memory (header + pages), or null
    size_t pool_bytes = 0;
    size_t page_bytes = 0;           // one page of one owner layer
    int sm_count = 0;
    int max_smem_optin = 0;
    DecodeTuning tune{0, 8, 2, 1, 1, Balance{0, 2, 0}};
    int chunks_per_worker = 8;       // pool chunk slots per worker (sizes the workspace)
    // the decode workspace whose control words are known to be zero (see prepare_workspace)
    const void *ws_ready = nullptr;
    int ws_batch = 0, ws_q_heads = 0, ws_workers = 0, ws_chunks = 0;
    int64_t launches = 0;
    unsigned long long *trace = nullptr;   // optional per-worker timestamps (device)
    size_t trace_bytes = 0;

    int *status_word() const { return reinterpret_cast<int *>(pool); }
    uint8_t *layer_base(int owner_slot) const
    {
        return pool + HEADER_BYTES + (size_t)owner_slot * (size_t)max_pages * page_bytes;
    }
};

namespace {

int check_routing(int n_layers, const int32_t *r)
{
    if (n_layers <= 0 || !r) return SKV_ERR_ARG;
    if (r[0] != 0) return SKV_ERR_ROUTING;
    for (int l = 0; l < n_layers; ++l) {
        if (r[l] < 0 || r[l] > l) return SKV_ERR_ROUTING;
        if (r[r[l]] != r[l]) return SKV_ERR_ROUTING;
    }
    return SKV_OK;
}

int check_shape(int kv_heads, int head_dim, int page_size, int64_t max_pages)
{
    if (kv_heads <= 0 || head_dim <= 0 || page_size <= 0 || max_pages <= 0) return SKV_ERR_ARG;
    if (head_dim != 64 && head_dim != 128) return SKV_ERR_UNSUPPORTED;
    if (page_size != PAGE) return SKV_ERR_UNSUPPORTED;
    if (max_pages > 0x7FFFFFFFll) return SKV_ERR_UNSUPPORTED;   // page ids are int32
    return SKV_OK;
}

size_t page_bytes_of(int kv_heads, int head_dim) { return (size_t)kv_heads * block_bytes(head_dim); }

bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct WorkspaceLayout {
    size_t ctrl_off, seg_off, prefix_off, ml_off, o_off, total, zero_bytes;
    int64_t n_slots;
};

// control words | per-segment block counters | page-count prefix | partial (max,sum) | partial outputs
WorkspaceLayout workspace_layout(const skv_cache *c, int batch, int q_heads, int n_workers, int max_chunks)
{
    WorkspaceLayout w;
    const int G = q_heads / c->kv_heads;
    const int64_t n_seg = (int64_t)batch * c->kv_heads;
    w.n_slots = (int64_t)n_workers + n_seg + (int64_t)max_chunks + n_seg;
    w.ctrl_off = 0;
    w.seg_off = 256;
    w.prefix_off = w.seg_off + round_up((size_t)n_seg * sizeof(int32_t), 256);
    w.zero_bytes = w.prefix_off;
    w.ml_off = w.prefix_off + round_up((size_t)(batch + 1) * sizeof(int32_t), 256);
    w.o_off = w.ml_off + round_up((size_t)w.n_slots * G * 2 * sizeof(float), 256);
    w.total = w.o_off + round_up((size_t)w.n_slots * G * c->head_dim * sizeof(float), 256);
    return w;
}

int n_workers_of(const skv_cache *c) { return c->sm_count * c->tune.ctas_per_sm * c->tune.warps; }

int max_chunks_of(const skv_cache *c) { return c->tune.bal.pool_pct > 0 ? c->chunks_per_worker * n_workers_of(c) : 0; }

Balance balance_of(const skv_cache *c)
{
    Balance b = c->tune.bal;
    b.max_chunks = max_chunks_of(c);
    return b;
}

// The split-K kernel expects its control words and per-segment counters to be zero on entry and leaves
// them zero on exit, so they are cleared only when the workspace (or the layout in it) changes.
int prepare_workspace(skv_cache *c, void *workspace, const WorkspaceLayout &wl, int batch, int q_heads, cudaStream_t st)
{
    const int W = n_workers_of(c), ch = max_chunks_of(c);
    if (c->ws_ready == workspace && c->ws_batch == batch && c->ws_q_heads == q_heads && c->ws_workers == W &&
        c->ws_chunks == ch)
        return SKV_OK;
    if (cudaMemsetAsync(workspace, 0, wl.zero_bytes, st) != cudaSuccess) {
        (void)cudaGetLastError();
        return SKV_ERR_CUDA;
    }
    c->ws_ready = workspace;
    c->ws_batch = batch;
    c->ws_q_heads = q_heads;
    c->ws_workers = W;
    c->ws_chunks = ch;
    return SKV_OK;
}

int check_decode_args(const skv_cache *c, int layer, int batch, int q_heads)
{
    if (!c) return SKV_ERR_ARG;
    if (!c->pool) return SKV_ERR_ARG;
    if (layer < 0 || layer >= c->n_layers) return SKV_ERR_LAYER;
    if (batch <= 0 || q_heads <= 0) return SKV_ERR_ARG;
    if (q_heads % c->kv_heads != 0) return SKV_ERR_UNSUPPORTED;
    const int G = q_heads / c->kv_heads;
    if (G > 8) return SKV_ERR_UNSUPPORTED;
    if (c->tune.variant == 1 && G != 1) return SKV_ERR_UNSUPPORTED;
    if (batch > 16384) return SKV_ERR_UNSUPPORTED;
    return SKV_OK;
}

}  // namespace

extern "C" {

const char *skv_strerror(int status)
{
    switch (status) {
    case SKV_OK: return "ok";
    case SKV_ERR_ARG: return "invalid argument";
    case SKV_ERR_ROUTING: return "invalid routing map (need r[0]=0, 0<=r[l]<=l, r[r[l]]=r[l])";
    case SKV_ERR_UNSUPPORTED: return "unsupported shape";
    case SKV_ERR_NOMEM: return "caller-provided buffer too small";
    case SKV_ERR_LAYER: return "layer out of range or not an owner";
    case SKV_ERR_CUDA: return "CUDA runtime error";
    case SKV_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case SKV_ERR_BOUNDS: return "page or slot id out of range";
    case SKV_ERR_TOO_LARGE: return "batch x heads needs more scratch than the library's built-in scratch area holds";
    default: return "unknown status";
    }
}

int skv_routing_from_owners(int n_layers, const int32_t *owners, int n_owners, int32_t *r_out)
{
    if (n_layers <= 0 || !owners || n_owners <= 0 || !r_out) return SKV_ERR_ARG;
    std::vector<char> is_owner((size_t)n_layers, 0);
    for (int i = 0; i < n_owners; ++i) {
        if (owners[i] < 0 || owners[i] >= n_layers) return SKV_ERR_ARG;
        is_owner[(size_t)owners[i]] = 1;
    }
    if (!is_owner[0]) return SKV_ERR_ROUTING;
    int last = 0;
    for (int l = 0; l < n_layers; ++l) {
        if (is_owner[(size_t)l]) last = l;
        r_out[l] = last;
    }
    return SKV_OK;
}

int skv_routing_groups(int n_layers, int g, int32_t *r_out)
{
    if (n_layers <= 0 || g <= 0 || !r_out) return SKV_ERR_ARG;
    for (int l = 0; l < n_layers; ++l) r_out[l] = l - l % g;
    return SKV_OK;
}

int skv_cache_pool_bytes(int n_layers, const int32_t *r, int kv_heads, int head_dim, int page_size,
                         int64_t max_pages, size_t *out_bytes)
{
    if (!out_bytes) return SKV_ERR_ARG;
    int rc = check_routing(n_layers, r);
    if (rc) return rc;
    rc = check_shape(kv_heads, head_dim, page_size, max_pages);
    if (rc) return rc;
    size_t owners = 0;
    for (int l = 0; l < n_layers; ++l) owners += (r[l] == l);
    *out_bytes = HEADER_BYTES + owners * (size_t)max_pages * page_bytes_of(kv_heads, head_dim);
    return SKV_OK;
}

int skv_cache_create(skv_cache **out, int n_layers, const int32_t *r, int kv_heads, int head_dim,
                     int page_size, int64_t max_pages, void *device_pool, size_t pool_bytes, void *stream)
{
    if (!out) return SKV_ERR_ARG;
    *out = nullptr;
    size_t need = 0;
    int rc = skv_cache_pool_bytes(n_layers, r, kv_heads, head_dim, page_size, max_pages, &need);
    if (rc) return rc;
    if (device_pool) {
        if (!aligned(device_pool, 256)) return SKV_ERR_ARG;
        if (pool_bytes < need) return SKV_ERR_NOMEM;
    } else if (pool_bytes != 0) {
        return SKV_ERR_ARG;
    }
    skv_cache *c = new (std::nothrow) skv_cache;
    if (!c) return SKV_ERR_ARG;
    c->n_layers = n_layers;
    c->kv_heads = kv_heads;
    c->head_dim = head_dim;
    c->page_size = page_size;
    c->max_pages = max_pages;
    c->r.assign(r, r + n_layers);
    c->slot.assign((size_t)n_layers, -1);
    for (int l = 0; l < n_layers; ++l)
        if (r[l] == l) {
            c->slot[(size_t)l] = (int32_t)c->owners.size();
            c->owners.push_back(l);
        }
    c->n_owners = (int)c->owners.size();
    c->page_bytes = page_bytes_of(kv_heads, head_dim);
    c->pool = static_cast<uint8_t *>(device_pool);
    c->pool_bytes = device_pool ? need : 0;
    if (device_pool) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&c->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess ||
            cudaMemsetAsync(device_pool, 0, need, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
            (void)cudaGetLastError();
            delete c;
            return SKV_ERR_CUDA;
        }
    }
    *out = c;
    return SKV_OK;
}

void skv_cache_destroy(skv_cache *cache) { delete cache; }

int skv_layer_owner(const skv_cache *c, int layer)
{
    if (!c || layer < 0 || layer >= c->n_layers) return SKV_ERR_LAYER;
    return c->r[(size_t)layer];
}

int skv_is_owner(const skv_cache *c, int layer)
{
    if (!c || layer < 0 || layer >= c->n_layers) return SKV_ERR_LAYER;
    return c->r[(size_t)layer] == layer ? 1 : 0;
}

int skv_cache_stats(const skv_cache *c, int *n_owners, size_t *page_bytes, size_t *kv_bytes, size_t *bytes_per_token)
{
    if (!c) return SKV_ERR_ARG;
    if (n_owners) *n_owners = c->n_owners;
    if (page_bytes) *page_bytes = c->page_bytes;
    if (kv_bytes) *kv_bytes = (size_t)c->n_owners * (size_t)c->max_pages * c->page_bytes;
    if (bytes_per_token) *bytes_per_token = (size_t)2 * c->n_owners * c->kv_heads * c->head_dim * 2;
    return SKV_OK;
}

int skv_append(skv_cache *c, int layer, const void *K, const void *V, const int64_t *slot_map,
               int64_t n_tokens, void *stream)
{
    if (!c) return SKV_ERR_ARG;
    if (layer < 0 || layer >= c->n_layers) return SKV_ERR_LAYER;
    if (n_tokens < 0) return SKV_ERR_ARG;
    const int s = c->slot[(size_t)layer];
    if (s < 0) return SKV_OK;                    // not in S: Algorithm 2 skips the update
    if (!c->pool) return SKV_ERR_ARG;
    if (n_tokens == 0) return SKV_OK;
    if (!K || !V || !slot_map || !aligned(K, 16) || !aligned(V, 16)) return SKV_ERR_ARG;
    AppendParams p;
    p.layer_base = c->layer_base(s);
    p.K = static_cast<const uint4 *>(K);
    p.V = static_cast<const uint4 *>(V);
    p.slot_map = slot_map;
    p.n_tokens = n_tokens;
    p.n_slots = c->max_pages * PAGE;
    p.page_stride = (int64_t)c->page_bytes;
    p.Hkv = c->kv_heads;
    p.D = c->head_dim;
    p.status = c->status_word();
    if (launch_append(p, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SKV_ERR_CUDA;
    c->launches += 1;
    return SKV_OK;
}

int skv_gather(skv_cache *c, int layer, const int64_t *slot_ids, int64_t n, void *K_out, void *V_out, void *stream)
{
    if (!c || !c->pool) return SKV_ERR_ARG;
    if (layer < 0 || layer >= c->n_layers || c->slot[(size_t)layer] < 0) return SKV_ERR_LAYER;
    if (n < 0) return SKV_ERR_ARG;
    if (n == 0) return SKV_OK;
    if (!slot_ids || !K_out || !V_out || !aligned(K_out, 16) || !aligned(V_out, 16)) return SKV_ERR_ARG;
    GatherParams p;
    p.layer_base = c->layer_base(c->slot[(size_t)layer]);
    p.K_out = static_cast<uint4 *>(K_out);
    p.V_out = static_cast<uint4 *>(V_out);
    p.slot_ids = slot_ids;
    p.n = n;
    p.n_slots = c->max_pages * PAGE;
    p.page_stride = (int64_t)c->page_bytes;
    p.Hkv = c->kv_heads;
    p.D = c->head_dim;
    p.status = c->status_word();
    if (launch_gather(p, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SKV_ERR_CUDA;
    c->launches += 1;
    return SKV_OK;
}

int skv_decode_workspace_bytes(const skv_cache *c, int batch, int q_heads, size_t *out_bytes)
{
    if (!c || !out_bytes || batch <= 0 || q_heads <= 0) return SKV_ERR_ARG;
    if (q_heads % c->kv_heads != 0 || q_heads / c->kv_heads > 8) return SKV_ERR_UNSUPPORTED;
    const int sm = c->sm_count > 0 ? c->sm_count : 148;
    const int W = sm * c->tune.ctas_per_sm * c->tune.warps;
    const int ch = c->tune.bal.pool_pct > 0 ? c->chunks_per_worker * W : 0;
    *out_bytes = workspace_layout(c, batch, q_heads, W, ch).total;
    return SKV_OK;
}

namespace {
// launches the split-K kernel; `out` non-null selects the fused (in-kernel) merge
int launch_splitk(skv_cache *c, int layer, const void *Q, const int32_t *page_table, const int32_t *seq_lens,
                  void *out, int batch, int q_heads, int pt_stride, float scale, void *workspace,
                  size_t workspace_bytes, void *stream)
{
    int rc = check_decode_args(c, layer, batch, q_heads);
    if (rc) return rc;
    if (!Q || !page_table || !seq_lens || !workspace || pt_stride <= 0) return SKV_ERR_ARG;
    if (!aligned(Q, 16) || !aligned(workspace, 256) || (out && !aligned(out, 8))) return SKV_ERR_ARG;
    const int G = q_heads / c->kv_heads;
    const int W = n_workers_of(c);
    const WorkspaceLayout wl = workspace_layout(c, batch, q_heads, W, max_chunks_of(c));
    if (workspace_bytes < wl.total) return SKV_ERR_NOMEM;
    const size_t smem = decode_smem_bytes(c->head_dim, batch, c->tune.warps, c->tune.stages);
    if (smem == 0 || smem > (size_t)c->max_smem_optin) return SKV_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = prepare_workspace(c, workspace, wl, batch, q_heads, st);
    if (rc) return rc;
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    DecodeParams p;
    p.layer_base = c->layer_base(c->slot[(size_t)c->r[(size_t)layer]]);
    p.page_stride = (int64_t)c->page_bytes;
    p.max_pages = c->max_pages;
    p.Q = static_cast<const uint16_t *>(Q);
    p.page_table = page_table;
    p.seq_lens = seq_lens;
    p.part_o = reinterpret_cast<float *>(ws + wl.o_off);
    p.part_ml = reinterpret_cast<float *>(ws + wl.ml_off);
    p.prefix = reinterpret_cast<int32_t *>(ws + wl.prefix_off);
    p.ctrl = reinterpret_cast<int32_t *>(ws + wl.ctrl_off);
    p.seg_count = reinterpret_cast<int32_t *>(ws + wl.seg_off);
    p.out = static_cast<uint16_t *>(out);
    p.B = batch;
    p.Hq = q_heads;
    p.Hkv = c->kv_heads;
    p.pt_stride = pt_stride;
    const float sc = scale > 0.f ? scale : 1.0f / sqrtf((float)c->head_dim);
    p.scale_log2 = sc * 1.4426950408889634f;
    p.bal = balance_of(c);
    p.status = c->status_word();
    p.trace = (c->trace && c->trace_bytes >= (size_t)W * 32) ? c->trace : nullptr;
    const bool tensor_core = c->tune.variant == 2 || (c->tune.variant == 0 && G > 1);
    const int grid = c->sm_count * c->tune.ctas_per_sm;
    if (launch_decode_splitk(p, c->head_dim, G, tensor_core, grid, c->tune.warps, c->tune.stages, st) != cudaSuccess)
        return SKV_ERR_CUDA;
    c->launches += 1;
    return SKV_OK;
}
}  // namespace

int skv_decode_splitk(skv_cache *c, int layer, const void *Q, const int32_t *page_table, const int32_t *seq_lens,
                      int batch, int q_heads, int pt_stride, float scale, void *workspace,
                      size_t workspace_bytes, void *stream)
{
    return launch_splitk(c, layer, Q, page_table, seq_lens, nullptr, batch, q_heads, pt_stride, scale, workspace,
                         workspace_bytes, stream);
}

int skv_decode_merge(skv_cache *c, void *out, int batch, int q_heads, void *workspace, size_t workspace_bytes,
                     void *stream)
{
    int rc = check_decode_args(c, 0, batch, q_heads);
    if (rc) return rc;
    if (!out || !workspace || !aligned(out, 8) || !aligned(workspace, 256)) return SKV_ERR_ARG;
    const int W = n_workers_of(c);
    const WorkspaceLayout wl = workspace_layout(c, batch, q_heads, W, max_chunks_of(c));
    if (workspace_bytes < wl.total) return SKV_ERR_NOMEM;
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    MergeParams m;
    m.part_o = reinterpret_cast<const float *>(ws + wl.o_off);
    m.part_ml = reinterpret_cast<const float *>(ws + wl.ml_off);
    m.prefix = reinterpret_cast<const int32_t *>(ws + wl.prefix_off);
    m.out = static_cast<uint16_t *>(out);
    m.B = batch;
    m.Hq = q_heads;
    m.Hkv = c->kv_heads;
    m.D = c->head_dim;
    m.n_workers = W;
    m.bal = balance_of(c);
    if (launch_merge(m, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SKV_ERR_CUDA;
    c->launches += 1;
    return SKV_OK;
}

int skv_decode_attn(skv_cache *c, int layer, const void *Q, const int32_t *page_table, const int32_t *seq_lens,
                    void *out, int batch, int q_heads, int pt_stride, float scale, void *workspace,
                    size_t workspace_bytes, void *stream)
{
    if (!out) return SKV_ERR_ARG;
    if (c && c->tune.fused_merge)
        return launch_splitk(c, layer, Q, page_table, seq_lens, out, batch, q_heads, pt_stride, scale, workspace,
                             workspace_bytes, stream);
    int rc = skv_decode_splitk(c, layer, Q, page_table, seq_lens, batch, q_heads, pt_stride, scale, workspace,
                               workspace_bytes, stream);
    if (rc) return rc;
    return skv_decode_merge(c, out, batch, q_heads, workspace, workspace_bytes, stream);
}

}  // extern "C"

// Used by skv_decode_attn_static (skv_static.cu): the same launch as skv_decode_attn on a scratch area the
// library owns.  The area is shared by every handle and keeps whatever the last call left in it, so its
// control words are cleared on every call instead of being trusted.
namespace skv {
int decode_attn_on_scratch(skv_cache *c, int layer, const void *Q, const int32_t *page_table, const int32_t *seq_lens,
                           void *out, int batch, int q_heads, int pt_stride, float scale, void *scratch,
                           size_t scratch_bytes, void *stream)
{
    if (!out) return SKV_ERR_ARG;
    if (c) c->ws_ready = nullptr;
    if (c && c->tune.fused_merge)
        return launch_splitk(c, layer, Q, page_table, seq_lens, out, batch, q_heads, pt_stride, scale, scratch,
                             scratch_bytes, stream);
    int rc = launch_splitk(c, layer, Q, page_table, seq_lens, nullptr, batch, q_heads, pt_stride, scale, scratch,
                           scratch_bytes, stream);
    if (rc) return rc;
    return skv_decode_merge(c, out, batch, q_heads, scratch, scratch_bytes, stream);
}
}  // namespace skv

extern "C" {

int skv_decode_step(skv_cache *c, const void *Q, const void *K, const void *V, const int64_t *slot_map,
                    const int32_t *page_table, const int32_t *seq_lens, void *out, int batch, int q_heads,
                    int pt_stride, float scale, void *workspace, size_t workspace_bytes, void *stream)
{
    int rc = check_decode_args(c, 0, batch, q_heads);
    if (rc) return rc;
    if (!Q || !K || !V || !slot_map || !out) return SKV_ERR_ARG;
    const size_t q_layer = (size_t)batch * q_heads * c->head_dim * 2;
    const size_t kv_layer = (size_t)batch * c->kv_heads * c->head_dim * 2;
    const uint8_t *q = static_cast<const uint8_t *>(Q), *k = static_cast<const uint8_t *>(K),
                  *v = static_cast<const uint8_t *>(V);
    uint8_t *o = static_cast<uint8_t *>(out);
    for (int l = 0; l < c->n_layers; ++l) {
        const int os = c->slot[(size_t)l];
        if (os >= 0) {
            rc = skv_append(c, l, k + (size_t)os * kv_layer, v + (size_t)os * kv_layer, slot_map, batch, stream);
            if (rc) return rc;
        }
        rc = skv_decode_attn(c, l, q + (size_t)l * q_layer, page_table, seq_lens, o + (size_t)l * q_layer, batch,
                             q_heads, pt_stride, scale, workspace, workspace_bytes, stream);
        if (rc) return rc;
    }
    return SKV_OK;
}

// ---- whole decode step from host buffers -------------------------------------
namespace {
struct StagingLayout {
    size_t q, k, v, slot_map, page_table, seq_lens, out, ws, total, ws_bytes;
};
int staging_layout(const skv_cache *c, int batch, int q_heads, int pt_stride, StagingLayout *s)
{
    size_t ws_bytes = 0;
    int rc = skv_decode_workspace_bytes(c, batch, q_heads, &ws_bytes);
    if (rc) return rc;
    if (pt_stride <= 0) return SKV_ERR_ARG;
    const size_t q_bytes = (size_t)c->n_layers * batch * q_heads * c->head_dim * 2;
    const size_t kv_bytes = (size_t)c->n_owners * batch * c->kv_heads * c->head_dim * 2;
    size_t at = 0;
    s->q = at;          at += round_up(q_bytes, 256);
    s->k = at;          at += round_up(kv_bytes, 256);
    s->v = at;          at += round_up(kv_bytes, 256);
    s->slot_map = at;   at += round_up((size_t)batch * 8, 256);
    s->page_table = at; at += round_up((size_t)batch * pt_stride * 4, 256);
    s->seq_lens = at;   at += round_up((size_t)batch * 4, 256);
    s->out = at;        at += round_up(q_bytes, 256);
    s->ws = at;         at += round_up(ws_bytes, 256);
    s->ws_bytes = ws_bytes;
    s->total = at;
    return SKV_OK;
}
}  // namespace

int skv_decode_step_staging_bytes(const skv_cache *c, int batch, int q_heads, int pt_stride, size_t *out_bytes)
{
    if (!c || !out_bytes || batch <= 0 || q_heads <= 0) return SKV_ERR_ARG;
    StagingLayout s;
    int rc = staging_layout(c, batch, q_heads, pt_stride, &s);
    if (rc) return rc;
    *out_bytes = s.total;
    return SKV_OK;
}

int skv_decode_step_host(skv_cache *c, const void *hQ, const void *hK, const void *hV, const int64_t *h_slot_map,
                         const int32_t *h_page_table, const int32_t *h_seq_lens, void *h_out, int batch,
                         int q_heads, int pt_stride, float scale, void *staging, size_t staging_bytes, void *stream)
{
    int rc = check_decode_args(c, 0, batch, q_heads);
    if (rc) return rc;
    if (!hQ || !hK || !hV || !h_slot_map || !h_page_table || !h_seq_lens || !h_out || !staging) return SKV_ERR_ARG;
    if (!aligned(staging, 256)) return SKV_ERR_ARG;
    StagingLayout s;
    rc = staging_layout(c, batch, q_heads, pt_stride, &s);
    if (rc) return rc;
    if (staging_bytes < s.total) return SKV_ERR_NOMEM;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t *d = static_cast<uint8_t *>(staging);
    const size_t q_layer = (size_t)batch * q_heads * c->head_dim * 2;
    const size_t kv_layer = (size_t)batch * c->kv_heads * c->head_dim * 2;
    bool ok = true;
    ok &= cudaMemcpyAsync(d + s.q, hQ, q_layer * c->n_layers, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(d + s.k, hK, kv_layer * c->n_owners, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(d + s.v, hV, kv_layer * c->n_owners, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(d + s.slot_map, h_slot_map, (size_t)batch * 8, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(d + s.page_table, h_page_table, (size_t)batch * pt_stride * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(d + s.seq_lens, h_seq_lens, (size_t)batch * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (!ok) { (void)cudaGetLastError(); return SKV_ERR_CUDA; }
    rc = skv_decode_step(c, d + s.q, d + s.k, d + s.v, reinterpret_cast<const int64_t *>(d + s.slot_map),
                         reinterpret_cast<const int32_t *>(d + s.page_table),
                         reinterpret_cast<const int32_t *>(d + s.seq_lens), d + s.out, batch, q_heads, pt_stride,
                         scale, d + s.ws, s.ws_bytes, stream);
    if (rc) return rc;
    if (cudaMemcpyAsync(h_out, d + s.out, q_layer * c->n_layers, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
        (void)cudaGetLastError();
        return SKV_ERR_CUDA;
    }
    return SKV_OK;
}

// ---- status, tuning, counters --------------------------------------------------
int skv_get_status(skv_cache *c, void *stream, int *device_status)
{
    if (!c || !c->pool || !device_status) return SKV_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int word = 0;
    if (cudaMemcpyAsync(&word, c->status_word(), sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemsetAsync(c->status_word(), 0, sizeof(int), st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        (void)cudaGetLastError();
        return SKV_ERR_CUDA;
    }
    *device_status = (word & STATUS_TIMEOUT) ? SKV_ERR_TIMEOUT : (word & STATUS_BOUNDS) ? SKV_ERR_BOUNDS : SKV_OK;
    if (word & STATUS_TIMEOUT) c->ws_ready = nullptr;     // a worker gave up: counters may be left non-zero
    return SKV_OK;
}

int skv_set_decode_variant(skv_cache *c, int variant)
{
    if (!c || variant < 0 || variant > 2) return SKV_ERR_ARG;
    c->tune.variant = variant;
    return SKV_OK;
}

int skv_set_decode_tuning(skv_cache *c, int warps_per_cta, int stages, int ctas_per_sm)
{
    if (!c) return SKV_ERR_ARG;
    DecodeTuning t = c->tune;
    if (warps_per_cta) t.warps = warps_per_cta;
    if (stages) t.stages = stages;
    if (ctas_per_sm) t.ctas_per_sm = ctas_per_sm;
    if (t.warps < 1 || t.warps > 16 || t.stages < 2 || t.stages > 8 || t.ctas_per_sm < 1 || t.ctas_per_sm > 8)
        return SKV_ERR_ARG;
    if (c->pool) {
        const size_t smem = decode_smem_bytes(c->head_dim, 1, t.warps, t.stages);
        if (smem == 0 || smem > (size_t)c->max_smem_optin) return SKV_ERR_UNSUPPORTED;
    }
    c->tune = t;
    return SKV_OK;
}

int skv_set_decode_merge_mode(skv_cache *c, int fused)
{
    if (!c || fused < 0 || fused > 1) return SKV_ERR_ARG;
    c->tune.fused_merge = fused;
    return SKV_OK;
}

int skv_set_decode_balance(skv_cache *c, int pool_percent, int min_chunk_blocks, int chunks_per_worker)
{
    if (!c || pool_percent < 0 || pool_percent > 100 || min_chunk_blocks < 1 || chunks_per_worker < 1 ||
        chunks_per_worker > 64)
        return SKV_ERR_ARG;
    c->tune.bal.pool_pct = pool_percent;
    c->tune.bal.min_chunk = min_chunk_blocks;
    c->chunks_per_worker = chunks_per_worker;
    return SKV_OK;
}

int skv_set_trace_buffer(skv_cache *c, void *device_buffer, size_t bytes)
{
    if (!c || (device_buffer && !aligned(device_buffer, 8))) return SKV_ERR_ARG;
    c->trace = static_cast<unsigned long long *>(device_buffer);
    c->trace_bytes = device_buffer ? bytes : 0;
    return SKV_OK;
}

int skv_decode_worker_count(const skv_cache *c)
{
    if (!c || !c->pool) return SKV_ERR_ARG;
    return n_workers_of(c);
}

int skv_launch_count(const skv_cache *c, int64_t *out_count)
{
    if (!c || !out_count) return SKV_ERR_ARG;
    *out_count = c->launches;
    return SKV_OK;
}

int skv_plan_worker_range(int64_t n_blocks, int n_workers, int w, int64_t *begin, int64_t *end)
{
    if (n_blocks < 0 || n_workers <= 0 || w < 0 || w >= n_workers || !begin || !end) return SKV_ERR_ARG;
    *begin = worker_begin(w, n_blocks, n_workers);
    *end = worker_begin((int64_t)w + 1, n_blocks, n_workers);
    return SKV_OK;
}

int skv_plan_worker_of(int64_t n_blocks, int n_workers, int64_t x)
{
    if (n_blocks <= 0 || n_workers <= 0 || x < 0 || x >= n_blocks) return SKV_ERR_ARG;
    return worker_of(x, n_blocks, n_workers);
}

}  // extern "C"
