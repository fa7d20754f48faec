// C ABI of the skv library (see include/skv.h): argument checking, the routed
// owner-only page allocator's bookkeeping, and kernel launches.  Host code only.
#include "../../include/skv.h"
#include "skv_common.cuh"

#include <math.h>
#include <new>
#include <stdlib.h>
#include <string.h>
#include <vector>

#include <atomic>
#include <chrono>
#include <mutex>

using namespace skv;

namespace skv {
cudaError_t ensure_dynamic_smem_fn(const void *kernel, size_t smem)
{
    struct Granted { const void *kernel; int dev; int smem; };
    static Granted table[128];
    static int used = 0;
    static std::mutex lock;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> hold(lock);
    Granted *g = nullptr;
    for (int i = 0; i < used && !g; ++i)
        if (table[i].kernel == kernel && table[i].dev == dev) g = &table[i];
    if (g && (int)smem <= g->smem) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (!g && used < 128) {
        g = &table[used++];
        g->kernel = kernel;
        g->dev = dev;
        g->smem = 0;
    }
    if (g) g->smem = (int)smem;
    return cudaSuccess;
}
}  // namespace skv

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
    int l2_bytes = 0;
    DecodeTuning tune{0, 2, 2, 4, 1};
    bool fp8 = false;                // pages hold E4M3 codes + per-row scales instead of bf16
    int prefill_variant = 0;         // 0 auto (tcgen05 where supported), 1 mma.sync kernel, 2 tcgen05 kernel
    uint8_t *prefill_scratch = nullptr;   // FP8 cache: room for one owner layer's pages as bf16 (caller's device memory)
    size_t prefill_scratch_bytes = 0;
    bool shape_is_default = true;    // until skv_set_decode_tuning is called: the CUDA-core kernel runs as 1 x 2 x 8
    int l2_keep_pct = 35;            // > 0: consecutive layers that read one owner walk it in opposite directions
    bool early_fetch = false;        // stand-alone attention calls fill their rings before waiting for the kernel before them
    int worker_mode = 0;             // 0 auto (CTA per range for stand-alone calls, warp per range inside chains),
                                     // 1 warp per range always, 2 CTA per range wherever it applies
    int cta_consumers = 8;           // consumer warps per CTA of the CTA-per-range kernel
    int cta_stages = 0;              // its ring depth; 0 = as deep as shared memory allows, up to 20 per SM
    int cta_per_sm = 1;              // its CTAs resident per SM
    bool cta_in_turn = true;         // its consumers take the blocks in turn (reproducible) instead of first come first served
    int merge_mode = 0;              // 0 auto, 1 a merge launch after every split-K launch, 2 merged by the CTA-per-range
                                     // kernel itself wherever that kernel can
    unsigned long long epoch_nonce = 0, epoch_count = 0;   // tags of in-kernel merging: never the same value twice
    std::vector<uint8_t> walk_reverse;   // per layer, for l2_keep_pct > 0: walk the block ranges backwards
    std::vector<uint8_t> walk_keep;      // per layer: the next layer reads the same owner
    int64_t launches = 0;
    unsigned long long *trace = nullptr;   // optional per-worker timestamps (device)
    size_t trace_bytes = 0;
    // skv_decode_step_host: a copy stream and events that let host<->device copies of one part of the
    // step run beside the kernels of another (created on first use, destroyed with the handle)
    static constexpr int HOST_GROUPS = 8;
    int host_groups = 4;            // layer groups of skv_decode_step_host
    int host_ramp = 1;              // 1: small first and last groups (smoothstep cut), 0: equal groups
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_entry = nullptr, ev_exit = nullptr, ev_in[HOST_GROUPS] = {}, ev_done[HOST_GROUPS] = {};

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

size_t page_bytes_of(int kv_heads, int head_dim, bool fp8)
{
    return (size_t)kv_heads * (fp8 ? fp8_block_bytes(head_dim) : block_bytes(head_dim));
}

bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// The workspace holds two identical buffers so that two consecutive calls of a chain may overlap on the
// GPU; each buffer is  page-count prefix | partial (max,sum) | partial outputs.  Nothing in it has to be
// initialised: every slot the merge kernel reads was written by the split-K launch before it.
struct WorkspaceLayout {
    size_t prefix_off, ml_off, o_off, tag_off, buf_bytes, total;
    int64_t n_slots;
};

WorkspaceLayout workspace_layout(const skv_cache *c, int batch, int q_heads, int n_workers)
{
    WorkspaceLayout w;
    const int G = q_heads / c->kv_heads;
    const int64_t n_seg = (int64_t)batch * c->kv_heads;
    w.n_slots = (int64_t)n_workers + n_seg;          // a run of worker w in segment s writes slot w + s
    w.prefix_off = 0;
    w.ml_off = w.prefix_off + round_up((size_t)(batch + 1) * sizeof(int32_t), 256);
    w.o_off = w.ml_off + round_up((size_t)w.n_slots * G * 2 * sizeof(float), 256);
    w.tag_off = w.o_off + round_up((size_t)w.n_slots * G * c->head_dim * sizeof(float), 256);
    w.buf_bytes = w.tag_off + round_up((size_t)w.n_slots * sizeof(unsigned long long), 256);    // one tag per slot
    w.total = 2 * w.buf_bytes;
    return w;
}

// FP8 pages go to the tcgen05 kernel (a worker is a CTA there) unless the mma.sync variant is asked for
bool fp8_on_umma(const skv_cache *c) { return c->fp8 && c->tune.variant != 2 && decode_fp8_umma_supported(c->head_dim, 1); }

// Workers of a warp-per-range (or tcgen05) split-K launch under the current variant and launch shape.  A
// handle without device memory (accounting only) has no device to ask and counts a B200's 148 SMs.
int n_workers_of(const skv_cache *c)
{
    const int sm = c->sm_count > 0 ? c->sm_count : 148;
    if (fp8_on_umma(c)) return sm * decode_fp8_umma_ctas_per_sm();
    return sm * c->tune.ctas_per_sm * c->tune.warps;
}

// Workers of a CTA-per-range launch: the CTAs that are resident at once.
int n_cta_workers_of(const skv_cache *c) { return (c->sm_count > 0 ? c->sm_count : 148) * c->cta_per_sm; }

// The workspace is sized for whichever kernel leaves more partials (a call may run either).
int n_workers_max(const skv_cache *c)
{
    const int a = n_workers_of(c), b = n_cta_workers_of(c);
    return a > b ? a : b;
}

// Ring depth of the CTA-per-range kernel for this shape: the handle's setting, else as many stages as fit
// (at most 20); 0 if not even two fit.
int cta_stages_for(const skv_cache *c, int batch, int G)
{
    int S = c->cta_stages > 0 ? c->cta_stages : 20 / c->cta_per_sm;
    // (what one CTA may take when cta_per_sm of them share an SM: the SM's shared memory less 1 KB per CTA the system keeps)
    const size_t room = ((size_t)c->max_smem_optin + 1024) / c->cta_per_sm - 1024;
    while (S >= 2 && decode_cta_smem_bytes(c->head_dim, batch, G, c->cta_consumers, S, c->fp8) > room) --S;
    // by default a whole number of rounds of the consumers (a stage then always serves the same consumer)
    if (c->cta_stages == 0 && S >= 2 * c->cta_consumers) S -= S % c->cta_consumers;
    return S >= 2 ? S : 0;
}

// Walk directions for L2 reuse: a layer that reads the same owner as the layer before it walks every
// block range in the opposite direction, so that it starts on the blocks its predecessor read last.
void plan_walks(skv_cache *c)
{
    const size_t L = (size_t)c->n_layers;
    c->walk_reverse.assign(L, 0);
    c->walk_keep.assign(L, 0);
    for (size_t l = 0; l < L; ++l) {
        if (l > 0 && c->r[l] == c->r[l - 1]) c->walk_reverse[l] = !c->walk_reverse[l - 1];
        if (l + 1 < L && c->r[l + 1] == c->r[l]) c->walk_keep[l] = 1;
    }
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

int skv_routing_rcla(int n_layers, double p_self, const double *u, const double *v, int32_t *map_out)
{
    if (n_layers <= 0 || !u || !v || !map_out || !(p_self >= 0.0 && p_self <= 1.0)) return SKV_ERR_ARG;
    for (int l = 0; l < n_layers; ++l)
        if (!(u[l] >= 0.0 && u[l] < 1.0) || !(v[l] >= 0.0 && v[l] < 1.0)) return SKV_ERR_ARG;
    map_out[0] = 0;                                       // nothing precedes the first layer
    for (int l = 1; l < n_layers; ++l) {
        if (u[l] < p_self) {
            map_out[l] = l;                               // d = 1: the layer's own K,V
        } else {
            const int pick = (int)(v[l] * l);             // d = 0: uniform over the l layers before it
            map_out[l] = pick < l ? pick : l - 1;
        }
    }
    return SKV_OK;
}

int skv_routing_rdcla(int n_layers, int k, double p_self, const double *u, int32_t *map_out)
{
    if (n_layers <= 0 || k <= 0 || !u || !map_out || !(p_self >= 0.0 && p_self <= 1.0)) return SKV_ERR_ARG;
    for (int l = 0; l < n_layers; ++l) {
        if (!(u[l] >= 0.0 && u[l] < 1.0)) return SKV_ERR_ARG;
        map_out[l] = u[l] < p_self ? l : l - l % k;
    }
    return SKV_OK;
}

}  // extern "C"

namespace {
int pool_bytes_impl(int n_layers, const int32_t *r, int kv_heads, int head_dim, int page_size, int64_t max_pages,
                    bool fp8, size_t *out_bytes)
{
    if (!out_bytes) return SKV_ERR_ARG;
    int rc = check_routing(n_layers, r);
    if (rc) return rc;
    rc = check_shape(kv_heads, head_dim, page_size, max_pages);
    if (rc) return rc;
    size_t owners = 0;
    for (int l = 0; l < n_layers; ++l) owners += (r[l] == l);
    *out_bytes = HEADER_BYTES + owners * (size_t)max_pages * page_bytes_of(kv_heads, head_dim, fp8);
    return SKV_OK;
}

int create_impl(skv_cache **out, int n_layers, const int32_t *r, int kv_heads, int head_dim, int page_size,
                int64_t max_pages, void *device_pool, size_t pool_bytes, void *stream, bool fp8)
{
    if (!out) return SKV_ERR_ARG;
    *out = nullptr;
    size_t need = 0;
    int rc = pool_bytes_impl(n_layers, r, kv_heads, head_dim, page_size, max_pages, fp8, &need);
    if (rc) return rc;
    if (device_pool) {
        if (!aligned(device_pool, 256)) return SKV_ERR_ARG;
        if (pool_bytes < need) return SKV_ERR_NOMEM;
    } else if (pool_bytes != 0) {
        return SKV_ERR_ARG;
    }
    skv_cache *c = new (std::nothrow) skv_cache;
    if (!c) return SKV_ERR_ARG;
    {   // a number of the handle's own for the tags of in-kernel merging: two handles may take turns on one workspace
        static std::atomic<unsigned long long> handles{0};
        const unsigned long long t = (unsigned long long)std::chrono::steady_clock::now().time_since_epoch().count();
        c->epoch_nonce = ((t * 0x9E3779B97F4A7C15ull) >> 32) ^ (++handles * 0x85EBCA6Bull) ^ (unsigned long long)(uintptr_t)c;
        c->epoch_nonce &= 0xFFFFFFFFull;
    }
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
    c->fp8 = fp8;
    if (fp8) c->tune.ctas_per_sm = 6;          // the FP8 kernel is bound by instruction latency: 12 warps per SM
    c->page_bytes = page_bytes_of(kv_heads, head_dim, fp8);
    plan_walks(c);
    c->pool = static_cast<uint8_t *>(device_pool);
    c->pool_bytes = device_pool ? need : 0;
    if (device_pool) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&c->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&c->l2_bytes, cudaDevAttrL2CacheSize, dev) != cudaSuccess ||
            cudaMemsetAsync(device_pool, 0, need, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
            (void)cudaGetLastError();
            delete c;
            return SKV_ERR_CUDA;
        }
    }
    *out = c;
    return SKV_OK;
}

}  // namespace

extern "C" {

int skv_cache_pool_bytes(int n_layers, const int32_t *r, int kv_heads, int head_dim, int page_size,
                         int64_t max_pages, size_t *out_bytes)
{
    return pool_bytes_impl(n_layers, r, kv_heads, head_dim, page_size, max_pages, false, out_bytes);
}

int skv_cache_pool_bytes_fp8(int n_layers, const int32_t *r, int kv_heads, int head_dim, int page_size,
                             int64_t max_pages, size_t *out_bytes)
{
    return pool_bytes_impl(n_layers, r, kv_heads, head_dim, page_size, max_pages, true, out_bytes);
}

int skv_cache_create(skv_cache **out, int n_layers, const int32_t *r, int kv_heads, int head_dim,
                     int page_size, int64_t max_pages, void *device_pool, size_t pool_bytes, void *stream)
{
    return create_impl(out, n_layers, r, kv_heads, head_dim, page_size, max_pages, device_pool, pool_bytes, stream, false);
}

int skv_cache_create_fp8(skv_cache **out, int n_layers, const int32_t *r, int kv_heads, int head_dim,
                         int page_size, int64_t max_pages, void *device_pool, size_t pool_bytes, void *stream)
{
    return create_impl(out, n_layers, r, kv_heads, head_dim, page_size, max_pages, device_pool, pool_bytes, stream, true);
}

void skv_cache_destroy(skv_cache *cache)
{
    if (!cache) return;
    if (cache->copy_stream) {
        (void)cudaStreamSynchronize(cache->copy_stream);
        (void)cudaStreamDestroy(cache->copy_stream);
        (void)cudaEventDestroy(cache->ev_entry);
        (void)cudaEventDestroy(cache->ev_exit);
        for (int g = 0; g < skv_cache::HOST_GROUPS; ++g) {
            (void)cudaEventDestroy(cache->ev_in[g]);
            (void)cudaEventDestroy(cache->ev_done[g]);
        }
        (void)cudaGetLastError();
    }
    delete cache;
}

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
    if (bytes_per_token)      // bf16: 2 bytes per value; fp8: 1 byte per value + one fp32 scale per row
        *bytes_per_token = c->fp8 ? (size_t)2 * c->n_owners * c->kv_heads * (c->head_dim + 4)
                                  : (size_t)2 * c->n_owners * c->kv_heads * c->head_dim * 2;
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
    if (c->fp8) {
        AppendFp8Params q;
        q.layer_base = c->layer_base(s);
        q.K = static_cast<const uint16_t *>(K);
        q.V = static_cast<const uint16_t *>(V);
        q.slot_map = slot_map;
        q.n_tokens = n_tokens;
        q.n_slots = c->max_pages * PAGE;
        q.page_stride = (int64_t)c->page_bytes;
        q.layer_stride = 0;
        q.Hkv = c->kv_heads;
        q.D = c->head_dim;
        q.status = c->status_word();
        if (launch_append_fp8(q, 1, c->tune.pdl != 0, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SKV_ERR_CUDA;
        c->launches += 1;
        return SKV_OK;
    }
    AppendParams p;
    p.layer_base = c->layer_base(s);
    p.K = static_cast<const uint4 *>(K);
    p.V = static_cast<const uint4 *>(V);
    p.slot_map = slot_map;
    p.n_tokens = n_tokens;
    p.n_slots = c->max_pages * PAGE;
    p.page_stride = (int64_t)c->page_bytes;
    p.layer_stride = 0;
    p.Hkv = c->kv_heads;
    p.D = c->head_dim;
    p.status = c->status_word();
    if (launch_append(p, 1, c->tune.pdl != 0, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SKV_ERR_CUDA;
    c->launches += 1;
    return SKV_OK;
}

int skv_gather(skv_cache *c, int layer, const int64_t *slot_ids, int64_t n, void *K_out, void *V_out, void *stream)
{
    if (!c || !c->pool) return SKV_ERR_ARG;
    if (layer < 0 || layer >= c->n_layers || c->slot[(size_t)layer] < 0) return SKV_ERR_LAYER;
    if (c->fp8) return SKV_ERR_UNSUPPORTED;            // an FP8 cache is read back with skv_gather_fp8
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

int skv_gather_fp8(skv_cache *c, int layer, const int64_t *slot_ids, int64_t n, void *K_codes, void *V_codes,
                   float *K_scales, float *V_scales, void *stream)
{
    if (!c || !c->pool) return SKV_ERR_ARG;
    if (layer < 0 || layer >= c->n_layers || c->slot[(size_t)layer] < 0) return SKV_ERR_LAYER;
    if (!c->fp8) return SKV_ERR_UNSUPPORTED;
    if (n < 0) return SKV_ERR_ARG;
    if (n == 0) return SKV_OK;
    if (!slot_ids || !K_codes || !V_codes || !K_scales || !V_scales) return SKV_ERR_ARG;
    GatherFp8Params p;
    p.layer_base = c->layer_base(c->slot[(size_t)layer]);
    p.K_codes = static_cast<uint8_t *>(K_codes);
    p.V_codes = static_cast<uint8_t *>(V_codes);
    p.K_scales = K_scales;
    p.V_scales = V_scales;
    p.slot_ids = slot_ids;
    p.n = n;
    p.n_slots = c->max_pages * PAGE;
    p.page_stride = (int64_t)c->page_bytes;
    p.Hkv = c->kv_heads;
    p.D = c->head_dim;
    p.status = c->status_word();
    if (launch_gather_fp8(p, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SKV_ERR_CUDA;
    c->launches += 1;
    return SKV_OK;
}

int skv_decode_workspace_bytes(const skv_cache *c, int batch, int q_heads, size_t *out_bytes)
{
    if (!c || !out_bytes || batch <= 0 || q_heads <= 0) return SKV_ERR_ARG;
    if (q_heads % c->kv_heads != 0 || q_heads / c->kv_heads > 8) return SKV_ERR_UNSUPPORTED;
    *out_bytes = workspace_layout(c, batch, q_heads, n_workers_max(c)).total;
    return SKV_OK;
}

namespace {
// What a split-K launch tells the merge launch that follows it.
struct SplitkPlan {
    int n_workers = 0;       // ranges the block list was cut into
    int unit_tokens = PAGE;  // tokens per unit of the list
    int finished_single = 0; // segments inside one range were finished by the split-K launch itself
    int merged = 0;          // ... and so were all others: no merge launch is needed
};

// Launches the split-K kernel on buffer `buf` (0 or 1) of the workspace.  `chained` = the call follows
// another attention call of the same step whose inputs were all ready before that call was launched, so
// it need not wait for it before reading.  `out` (may be null) = where the call's result rows go: given
// it, the CTA-per-range kernel may run, which finishes the segments that lie inside one range.
int launch_splitk(skv_cache *c, int layer, const void *Q, const int32_t *page_table, const int32_t *seq_lens,
                  int batch, int q_heads, int pt_stride, float scale, void *workspace, size_t workspace_bytes,
                  void *stream, SplitkPlan *plan, void *out = nullptr, int buf = 0, bool chained = false)
{
    int rc = check_decode_args(c, layer, batch, q_heads);
    if (rc) return rc;
    if (!Q || !page_table || !seq_lens || !workspace || pt_stride <= 0) return SKV_ERR_ARG;
    if (!aligned(Q, 16) || !aligned(workspace, 256)) return SKV_ERR_ARG;
    if (out && !aligned(out, 8)) return SKV_ERR_ARG;
    const int G = q_heads / c->kv_heads;
    const WorkspaceLayout wl = workspace_layout(c, batch, q_heads, n_workers_max(c));
    if (workspace_bytes < wl.total) return SKV_ERR_NOMEM;
    const bool tensor_core = c->fp8 || c->tune.variant == 2 || (c->tune.variant == 0 && G > 1);
    const bool umma = fp8_on_umma(c) && decode_fp8_umma_supported(c->head_dim, G);
    // CTA per range: stand-alone calls whose result buffer is known (not the links of a chain, which overlap
    // by having many small CTAs; not the tcgen05 FP8 kernel, which has its own CTA-wide design)
    const int cta_S = cta_stages_for(c, batch, G);
    const bool cta = !umma && !chained && out && c->worker_mode != 1 && cta_S > 0;
    // Default launch shapes of the warp-per-range kernel (8 warps per SM, two 8 KB stages each, many small
    // CTAs so that the CTAs of the next launch can move in one by one): 2 warps x 4 CTAs per SM for the
    // tensor-core kernel, 1 warp x 8 CTAs per SM for the CUDA-core kernel (measured best for each on B200).
    int warps = c->tune.warps, ctas = c->tune.ctas_per_sm;
    if (c->shape_is_default && !tensor_core) {
        warps = 1;
        ctas = 8;
    }
    const int W = cta ? n_cta_workers_of(c) : n_workers_of(c);
    const size_t smem = umma  ? decode_fp8_umma_smem_bytes(c->head_dim, batch)
                        : cta ? decode_cta_smem_bytes(c->head_dim, batch, G, c->cta_consumers, cta_S, c->fp8)
                              : decode_smem_bytes(c->head_dim, batch, warps, c->tune.stages, c->fp8);
    if (smem == 0 || smem > (size_t)c->max_smem_optin) return SKV_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t *ws = static_cast<uint8_t *>(workspace) + (size_t)buf * wl.buf_bytes;
    DecodeParams p;
    p.layer_base = c->layer_base(c->slot[(size_t)c->r[(size_t)layer]]);
    p.page_stride = (int64_t)c->page_bytes;
    p.max_pages = c->max_pages;
    p.Q = static_cast<const uint16_t *>(Q);
    p.page_table = page_table;
    p.seq_lens = seq_lens;
    p.out = static_cast<uint16_t *>(out);
    p.part_o = reinterpret_cast<float *>(ws + wl.o_off);
    p.part_ml = reinterpret_cast<float *>(ws + wl.ml_off);
    p.prefix = reinterpret_cast<int32_t *>(ws + wl.prefix_off);
    p.B = batch;
    p.Hq = q_heads;
    p.Hkv = c->kv_heads;
    p.pt_stride = pt_stride;
    const float sc = scale > 0.f ? scale : 1.0f / sqrtf((float)c->head_dim);
    p.scale_log2 = sc * 1.4426950408889634f;
    p.flags = chained ? DECODE_LATE_WAIT : (c->early_fetch && c->tune.pdl) ? DECODE_EARLY_FETCH : 0;
    if (cta && c->cta_in_turn) p.flags |= DECODE_CLAIM_IN_TURN;
    // Merging inside the kernel hands partials from CTA to CTA along the block list, which is only quick when
    // few segments are cut more than once (a hand-over costs about 3 us, a merge launch 3 to 8): by default
    // where there are at least two thirds as many segments as ranges (measured break-even: half as many).
    // Every CTA must be resident at once (one per SM), because a CTA waits for its neighbour's partial.
    const int kernel = c->fp8 ? 2 : tensor_core ? 1 : 0;
    const bool in_kernel_merge = cta && decode_cta_can_merge(c->head_dim, kernel) && c->cta_per_sm == 1 && c->merge_mode != 1 &&
                                 (c->merge_mode == 2 || 3 * (int64_t)batch * c->kv_heads >= 2 * (int64_t)W);
    if (in_kernel_merge) p.flags |= DECODE_MERGE_IN_KERNEL;
    p.tags = reinterpret_cast<unsigned long long *>(ws + wl.tag_off);
    p.epoch = (c->epoch_nonce << 32) | (++c->epoch_count & 0xFFFFFFFFull);
    p.keep_pct = 0;
    // what one call streams fits in L2 beside everything else when it is under about a third of it
    p.l2_fit_blocks = (int64_t)(c->l2_bytes / 3) / (int64_t)(c->fp8 ? fp8_block_bytes(c->head_dim) : block_bytes(c->head_dim));
    if (c->l2_keep_pct > 0) {
        if (c->walk_reverse[(size_t)layer]) p.flags |= DECODE_REVERSE;
        if (c->walk_keep[(size_t)layer]) p.keep_pct = c->l2_keep_pct;
    }
    p.status = c->status_word();
    const size_t trace_need = (size_t)W * (cta ? c->cta_consumers : 1) * 32;
    p.trace = (c->trace && c->trace_bytes >= trace_need) ? c->trace : nullptr;
    const cudaError_t le =
        umma  ? launch_decode_fp8_umma(p, c->head_dim, G, W, c->tune.pdl != 0, st)
        : cta ? launch_decode_cta(p, c->head_dim, G, kernel, W, c->cta_consumers, cta_S, c->tune.pdl != 0, st)
              : launch_decode_splitk(p, c->head_dim, G, kernel, c->sm_count * ctas, warps, c->tune.stages,
                                     c->tune.pdl != 0, st);
    if (le != cudaSuccess) {
        (void)cudaGetLastError();
        // a launch shape with more warps per CTA than the register file holds for this kernel variant
        return le == cudaErrorLaunchOutOfResources ? SKV_ERR_UNSUPPORTED : SKV_ERR_CUDA;
    }
    c->launches += 1;
    if (plan) {
        plan->n_workers = W;
        plan->unit_tokens = umma ? decode_fp8_umma_tile_tokens() : PAGE;
        plan->finished_single = cta ? 1 : 0;
        plan->merged = in_kernel_merge ? 1 : 0;
    }
    return SKV_OK;
}
}  // namespace

int skv_decode_splitk(skv_cache *c, int layer, const void *Q, const int32_t *page_table, const int32_t *seq_lens,
                      int batch, int q_heads, int pt_stride, float scale, void *workspace,
                      size_t workspace_bytes, void *stream)
{
    return launch_splitk(c, layer, Q, page_table, seq_lens, batch, q_heads, pt_stride, scale, workspace,
                         workspace_bytes, stream, nullptr);
}

namespace {
// The merge kernel on buffer `buf` of the workspace.  `plan` = what the split-K launch before it did (null:
// a warp-per-range or tcgen05 launch under the handle's current settings); seq_lens / pt_stride (may be null
// / 0) let the kernel count the pages itself instead of reading the counts that launch left in the workspace.
int launch_merge_on(skv_cache *c, void *out, int batch, int q_heads, void *workspace, size_t workspace_bytes,
                    void *stream, int buf, const SplitkPlan *plan = nullptr, const int32_t *seq_lens = nullptr,
                    int pt_stride = 0)
{
    int rc = check_decode_args(c, 0, batch, q_heads);
    if (rc) return rc;
    if (!out || !workspace || !aligned(out, 8) || !aligned(workspace, 256)) return SKV_ERR_ARG;
    const WorkspaceLayout wl = workspace_layout(c, batch, q_heads, n_workers_max(c));
    if (workspace_bytes < wl.total) return SKV_ERR_NOMEM;
    uint8_t *ws = static_cast<uint8_t *>(workspace) + (size_t)buf * wl.buf_bytes;
    MergeParams m;
    m.part_o = reinterpret_cast<const float *>(ws + wl.o_off);
    m.part_ml = reinterpret_cast<const float *>(ws + wl.ml_off);
    m.prefix = reinterpret_cast<const int32_t *>(ws + wl.prefix_off);
    m.seq_lens = (seq_lens && pt_stride > 0 && batch <= 4096) ? seq_lens : nullptr;     // the counts go to shared memory
    m.unit_tokens = plan ? plan->unit_tokens : fp8_on_umma(c) ? decode_fp8_umma_tile_tokens() : PAGE;
    m.max_tokens = (int64_t)pt_stride * PAGE;
    m.out = static_cast<uint16_t *>(out);
    m.B = batch;
    m.Hq = q_heads;
    m.Hkv = c->kv_heads;
    m.D = c->head_dim;
    m.n_workers = plan ? plan->n_workers : n_workers_of(c);
    m.skip_single = plan ? plan->finished_single : 0;
    // with overlappable launches the merge grid must be resident in one wave (see merge_kernel)
    m.max_ctas = c->tune.pdl ? (c->sm_count > 0 ? c->sm_count : 1) : 0x7FFFFFFF;
    if (launch_merge(m, c->tune.pdl != 0, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return SKV_ERR_CUDA;
    }
    c->launches += 1;
    return SKV_OK;
}
}  // namespace

int skv_decode_merge(skv_cache *c, void *out, int batch, int q_heads, void *workspace, size_t workspace_bytes,
                     void *stream)
{
    return launch_merge_on(c, out, batch, q_heads, workspace, workspace_bytes, stream, 0);
}

int skv_decode_attn(skv_cache *c, int layer, const void *Q, const int32_t *page_table, const int32_t *seq_lens,
                    void *out, int batch, int q_heads, int pt_stride, float scale, void *workspace,
                    size_t workspace_bytes, void *stream)
{
    if (!out) return SKV_ERR_ARG;
    SplitkPlan plan;
    int rc = launch_splitk(c, layer, Q, page_table, seq_lens, batch, q_heads, pt_stride, scale, workspace,
                           workspace_bytes, stream, &plan, out);
    if (rc) return rc;
    if (plan.merged) return SKV_OK;
    return launch_merge_on(c, out, batch, q_heads, workspace, workspace_bytes, stream, 0, &plan, seq_lens, pt_stride);
}

}  // extern "C"

namespace {
// The updates of every owner layer of one step in one launch.  K, V: [n_owners][batch][kv_heads][head_dim].
int step_updates(skv_cache *c, const void *K, const void *V, const int64_t *slot_map, int batch, void *stream,
                 int first_owner = 0, int n_upd = -1)
{
    if (!aligned(K, 16) || !aligned(V, 16)) return SKV_ERR_ARG;
    if (n_upd < 0) n_upd = c->n_owners - first_owner;
    if (n_upd == 0) return SKV_OK;
    const size_t kv_off = (size_t)first_owner * batch * c->kv_heads * c->head_dim * 2;
    K = static_cast<const uint8_t *>(K) + kv_off;
    V = static_cast<const uint8_t *>(V) + kv_off;
    if (c->fp8) {
        AppendFp8Params q;
        q.layer_base = c->layer_base(first_owner);
        q.K = static_cast<const uint16_t *>(K);
        q.V = static_cast<const uint16_t *>(V);
        q.slot_map = slot_map;
        q.n_tokens = batch;
        q.n_slots = c->max_pages * PAGE;
        q.page_stride = (int64_t)c->page_bytes;
        q.layer_stride = (int64_t)c->max_pages * (int64_t)c->page_bytes;
        q.Hkv = c->kv_heads;
        q.D = c->head_dim;
        q.status = c->status_word();
        if (launch_append_fp8(q, n_upd, c->tune.pdl != 0, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
            (void)cudaGetLastError();
            return SKV_ERR_CUDA;
        }
        c->launches += 1;
        return SKV_OK;
    }
    AppendParams ap;
    ap.layer_base = c->layer_base(first_owner);
    ap.K = static_cast<const uint4 *>(K);
    ap.V = static_cast<const uint4 *>(V);
    ap.slot_map = slot_map;
    ap.n_tokens = batch;
    ap.n_slots = c->max_pages * PAGE;
    ap.page_stride = (int64_t)c->page_bytes;
    ap.layer_stride = (int64_t)c->max_pages * (int64_t)c->page_bytes;
    ap.Hkv = c->kv_heads;
    ap.D = c->head_dim;
    ap.status = c->status_word();
    if (launch_append(ap, n_upd, c->tune.pdl != 0, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return SKV_ERR_CUDA;
    }
    c->launches += 1;
    return SKV_OK;
}

// Attention of layers [l0, l1) of one step.  With overlappable launches: a chain in which the split-K launch
// of layer l+1 may start while that of layer l is finishing and its merge is running (they work on alternate
// workspace buffers; a split-K launch waits for everything before it half-way through its own work, which
// also keeps the launch of layer l+2 from starting before layer l has been merged); the first launch of
// the chain waits before it reads anything.  `updates_done` = the owners' updates of the step have been
// issued already (else each owner layer is updated just before its attention).
int step_layers(skv_cache *c, int l0, int l1, const uint8_t *q, const uint8_t *k, const uint8_t *v,
                const int64_t *slot_map, const int32_t *page_table, const int32_t *seq_lens, uint8_t *o, int batch,
                int q_heads, int pt_stride, float scale, void *workspace, size_t workspace_bytes, void *stream,
                bool updates_done)
{
    const size_t q_layer = (size_t)batch * q_heads * c->head_dim * 2;
    const size_t kv_layer = (size_t)batch * c->kv_heads * c->head_dim * 2;
    for (int l = l0; l < l1; ++l) {
        const int os = c->slot[(size_t)l];
        int rc;
        if (os >= 0 && !updates_done) {
            rc = skv_append(c, l, k + (size_t)os * kv_layer, v + (size_t)os * kv_layer, slot_map, batch, stream);
            if (rc) return rc;
        }
        const bool chained = c->tune.pdl && updates_done && l > l0;
        SplitkPlan plan;
        rc = launch_splitk(c, l, q + (size_t)l * q_layer, page_table, seq_lens, batch, q_heads, pt_stride, scale,
                           workspace, workspace_bytes, stream, &plan, updates_done && c->tune.pdl ? nullptr : o + (size_t)l * q_layer,
                           l & 1, chained);
        if (rc) return rc;
        // the merge kernel waits for that launch and lets the next split-K launch be scheduled at once
        rc = launch_merge_on(c, o + (size_t)l * q_layer, batch, q_heads, workspace, workspace_bytes, stream, l & 1, &plan,
                             seq_lens, pt_stride);
        if (rc) return rc;
    }
    return SKV_OK;
}
}  // namespace

extern "C" {

int skv_decode_step(skv_cache *c, const void *Q, const void *K, const void *V, const int64_t *slot_map,
                    const int32_t *page_table, const int32_t *seq_lens, void *out, int batch, int q_heads,
                    int pt_stride, float scale, void *workspace, size_t workspace_bytes, void *stream)
{
    int rc = check_decode_args(c, 0, batch, q_heads);
    if (rc) return rc;
    if (!Q || !K || !V || !slot_map || !out) return SKV_ERR_ARG;
    // All inputs of the step exist before it starts, and the update of layer l touches only layer l's
    // pages, which no layer before l reads: so (with overlappable launches) every owner's update goes
    // first, in one launch, and the attention calls form one chain.  Without them: layer by layer,
    // exactly as a caller of the per-layer entry points would.
    const bool batched = c->tune.pdl != 0;
    if (batched) {
        rc = step_updates(c, K, V, slot_map, batch, stream);
        if (rc) return rc;
    }
    return step_layers(c, 0, c->n_layers, static_cast<const uint8_t *>(Q), static_cast<const uint8_t *>(K),
                       static_cast<const uint8_t *>(V), slot_map, page_table, seq_lens, static_cast<uint8_t *>(out),
                       batch, q_heads, pt_stride, scale, workspace, workspace_bytes, stream, batched);
}

// ---- pre-fill attention -------------------------------------------------------
}  // extern "C"

namespace {
// pre-fill attention over the pages of owner layer `src` (already resolved and checked)
int prefill_over(skv_cache *c, int src, const void *Q, const int32_t *cu_q_lens, const int32_t *page_table,
                 const int32_t *seq_lens, void *out, int batch, int max_q_len, int q_heads, int pt_stride,
                 float scale, void *stream);
}  // namespace

extern "C" {

int skv_prefill_attn(skv_cache *c, int layer, const void *Q, const int32_t *cu_q_lens, const int32_t *page_table,
                     const int32_t *seq_lens, void *out, int batch, int max_q_len, int q_heads, int pt_stride,
                     float scale, void *stream)
{
    const int rc = check_decode_args(c, layer, batch, q_heads);
    if (rc) return rc;
    return prefill_over(c, c->r[(size_t)layer], Q, cu_q_lens, page_table, seq_lens, out, batch, max_q_len, q_heads,
                        pt_stride, scale, stream);
}

int skv_prefill_attn_src(skv_cache *c, int src_layer, const void *Q, const int32_t *cu_q_lens,
                         const int32_t *page_table, const int32_t *seq_lens, void *out, int batch, int max_q_len,
                         int q_heads, int pt_stride, float scale, void *stream)
{
    const int rc = check_decode_args(c, src_layer, batch, q_heads);
    if (rc) return rc;
    if (c->slot[(size_t)src_layer] < 0) return SKV_ERR_LAYER;        // only layers that keep their K,V can be read
    return prefill_over(c, src_layer, Q, cu_q_lens, page_table, seq_lens, out, batch, max_q_len, q_heads, pt_stride,
                        scale, stream);
}

}  // extern "C"

namespace {
int prefill_over(skv_cache *c, int src, const void *Q, const int32_t *cu_q_lens, const int32_t *page_table,
                 const int32_t *seq_lens, void *out, int batch, int max_q_len, int q_heads, int pt_stride,
                 float scale, void *stream)
{
    if (!Q || !cu_q_lens || !page_table || !seq_lens || !out || pt_stride <= 0 || max_q_len <= 0) return SKV_ERR_ARG;
    if (!aligned(Q, 4) || !aligned(out, 4)) return SKV_ERR_ARG;
    if (batch > 65535 || c->kv_heads > 65535) return SKV_ERR_UNSUPPORTED;      // grid.y / grid.z limits
    const int G = q_heads / c->kv_heads;
    // FP8 pages: with a scratch area for one layer's pages as bf16, the pages the call reaches are converted
    // there first and the tcgen05 kernel runs on the scratch; without one, the mma.sync kernel that converts
    // the codes on the way in
    const size_t bf16_page = page_bytes_of(c->kv_heads, c->head_dim, false);
    const bool via_scratch = c->fp8 && c->prefill_scratch && c->prefill_scratch_bytes >= (size_t)c->max_pages * bf16_page;
    const bool can_umma = (!c->fp8 || via_scratch) && prefill_umma_supported(c->head_dim, G) && aligned(Q, 16) && aligned(out, 16) &&
                          prefill_umma_smem_bytes(c->head_dim) <= (size_t)c->max_smem_optin;
    if (c->prefill_variant == 2 && !can_umma) return SKV_ERR_UNSUPPORTED;
    const bool umma = c->prefill_variant == 2 || (c->prefill_variant == 0 && can_umma);
    if (!umma && (c->fp8 ? prefill_fp8_smem_bytes(c->head_dim) : prefill_smem_bytes(c->head_dim)) > (size_t)c->max_smem_optin)
        return SKV_ERR_UNSUPPORTED;
    if (c->fp8 && !aligned(Q, 8)) return SKV_ERR_ARG;
    PrefillParams p;
    p.layer_base = c->layer_base(c->slot[(size_t)src]);
    p.page_stride = (int64_t)c->page_bytes;
    p.max_pages = c->max_pages;
    p.Q = static_cast<const uint16_t *>(Q);
    p.out = static_cast<uint16_t *>(out);
    p.cu_q = cu_q_lens;
    p.page_table = page_table;
    p.seq_lens = seq_lens;
    p.B = batch;
    p.Hq = q_heads;
    p.Hkv = c->kv_heads;
    p.pt_stride = pt_stride;
    const float sc = scale > 0.f ? scale : 1.0f / sqrtf((float)c->head_dim);
    p.scale_log2 = sc * 1.4426950408889634f;
    p.status = c->status_word();
    const int tq = umma ? prefill_umma_tile_tokens(G) : prefill_tile_tokens(G);
    const int q_tiles = (max_q_len + tq - 1) / tq;
    const cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (umma && c->fp8) {
        DequantParams dq;
        dq.fp8_base = p.layer_base;
        dq.bf16_base = c->prefill_scratch;
        dq.fp8_page_stride = (int64_t)c->page_bytes;
        dq.bf16_page_stride = (int64_t)bf16_page;
        dq.max_pages = c->max_pages;
        dq.page_table = page_table;
        dq.seq_lens = seq_lens;
        dq.B = batch;
        dq.Hkv = c->kv_heads;
        dq.pt_stride = pt_stride;
        if (launch_dequant_pages(dq, c->head_dim, pt_stride, st) != cudaSuccess) {
            (void)cudaGetLastError();
            return SKV_ERR_CUDA;
        }
        c->launches += 1;
        p.layer_base = c->prefill_scratch;
        p.page_stride = (int64_t)bf16_page;
    }
    const cudaError_t le = umma     ? launch_prefill_umma(p, c->head_dim, G, q_tiles, c->tune.pdl != 0, st)
                           : c->fp8 ? launch_prefill_fp8(p, c->head_dim, G, q_tiles, c->tune.pdl != 0, st)
                                    : launch_prefill(p, c->head_dim, G, q_tiles, c->tune.pdl != 0, st);
    if (le != cudaSuccess) {
        (void)cudaGetLastError();
        return SKV_ERR_CUDA;
    }
    c->launches += 1;
    return SKV_OK;
}
}  // namespace

extern "C" {

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

namespace {
bool host_step_resources(skv_cache *c)
{
    if (c->copy_stream) return true;
    bool ok = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_entry, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_exit, cudaEventDisableTiming) == cudaSuccess;
    for (int g = 0; ok && g < skv_cache::HOST_GROUPS; ++g) {
        ok = ok && cudaEventCreateWithFlags(&c->ev_in[g], cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&c->ev_done[g], cudaEventDisableTiming) == cudaSuccess;
    }
    if (!ok) (void)cudaGetLastError();
    return ok;
}
}  // namespace

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
    if (!host_step_resources(c)) return SKV_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream), cs = c->copy_stream;
    uint8_t *d = static_cast<uint8_t *>(staging);
    const uint8_t *hq = static_cast<const uint8_t *>(hQ);
    uint8_t *ho = static_cast<uint8_t *>(h_out);
    const size_t q_layer = (size_t)batch * q_heads * c->head_dim * 2;
    const size_t kv_layer = (size_t)batch * c->kv_heads * c->head_dim * 2;
    const int L = c->n_layers;
    // The layers are cut into NG groups.  Copy stream: the small inputs, then group by group the new K,V
    // rows of the group's owners and its queries; caller's stream: a group's kernels as soon as its inputs
    // have arrived; copy stream again: a group's result rows as soon as its kernels are done.  So only the
    // first group's inputs and the last group's results are not hidden behind kernels, and those two groups
    // are the small ones (cut points on a smoothstep curve).
    const int NG = L < c->host_groups ? L : c->host_groups;
    int bound[skv_cache::HOST_GROUPS + 1];
    bound[0] = 0;
    for (int g = 1; g <= NG; ++g) {
        const double x = (double)g / NG;
        int64_t b = c->host_ramp ? (int64_t)(L * x * x * (3.0 - 2.0 * x) + 0.5) : ((int64_t)g * L) / NG;
        if (b < bound[g - 1] + 1) b = bound[g - 1] + 1;
        if (b > L - (NG - g)) b = L - (NG - g);
        bound[g] = (int)b;
    }
    bound[NG] = L;
    auto owners_before = [&](int l) { int n = 0; for (int i = 0; i < l; ++i) n += c->slot[(size_t)i] >= 0; return n; };
    const bool batched = c->tune.pdl != 0;
    bool ok = cudaEventRecord(c->ev_entry, st) == cudaSuccess;             // staging may still be in use by
    ok = ok && cudaStreamWaitEvent(cs, c->ev_entry, 0) == cudaSuccess;     // earlier work on the caller's stream
    ok = ok && cudaMemcpyAsync(d + s.slot_map, h_slot_map, (size_t)batch * 8, cudaMemcpyHostToDevice, cs) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(d + s.page_table, h_page_table, (size_t)batch * pt_stride * 4, cudaMemcpyHostToDevice, cs) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(d + s.seq_lens, h_seq_lens, (size_t)batch * 4, cudaMemcpyHostToDevice, cs) == cudaSuccess;
    // K,V rows: those of the first group's owners with the first group, all the others with the second, so
    // that the updates are two launches at most and the attention launches of a group stay one chain.
    const int own0 = owners_before(bound[1]);
    for (int g = 0; ok && g < NG; ++g) {
        const int l0 = bound[g], l1 = bound[g + 1];
        const int o0 = g == 0 ? 0 : own0, o1 = g == 0 ? own0 : c->n_owners;
        if (g < 2 && o1 > o0) {
            ok = ok && cudaMemcpyAsync(d + s.k + o0 * kv_layer, static_cast<const uint8_t *>(hK) + o0 * kv_layer,
                                       (size_t)(o1 - o0) * kv_layer, cudaMemcpyHostToDevice, cs) == cudaSuccess;
            ok = ok && cudaMemcpyAsync(d + s.v + o0 * kv_layer, static_cast<const uint8_t *>(hV) + o0 * kv_layer,
                                       (size_t)(o1 - o0) * kv_layer, cudaMemcpyHostToDevice, cs) == cudaSuccess;
        }
        ok = ok && cudaMemcpyAsync(d + s.q + l0 * q_layer, hq + l0 * q_layer, (size_t)(l1 - l0) * q_layer,
                                   cudaMemcpyHostToDevice, cs) == cudaSuccess;
        ok = ok && cudaEventRecord(c->ev_in[g], cs) == cudaSuccess;
    }
    if (!ok) { (void)cudaGetLastError(); return SKV_ERR_CUDA; }
    const int64_t *slot_map = reinterpret_cast<const int64_t *>(d + s.slot_map);
    const int32_t *page_table = reinterpret_cast<const int32_t *>(d + s.page_table);
    const int32_t *seq_lens = reinterpret_cast<const int32_t *>(d + s.seq_lens);
    for (int g = 0; g < NG; ++g) {
        const int l0 = bound[g], l1 = bound[g + 1];
        if (cudaStreamWaitEvent(st, c->ev_in[g], 0) != cudaSuccess) { (void)cudaGetLastError(); return SKV_ERR_CUDA; }
        if (g < 2 && batched) {
            rc = g == 0 ? step_updates(c, d + s.k, d + s.v, slot_map, batch, stream, 0, own0)
                        : step_updates(c, d + s.k, d + s.v, slot_map, batch, stream, own0, c->n_owners - own0);
            if (rc) return rc;
        }
        rc = step_layers(c, l0, l1, d + s.q, d + s.k, d + s.v, slot_map, page_table, seq_lens, d + s.out, batch,
                         q_heads, pt_stride, scale, d + s.ws, s.ws_bytes, stream, batched);
        if (rc) return rc;
        ok = cudaEventRecord(c->ev_done[g], st) == cudaSuccess;
        ok = ok && cudaStreamWaitEvent(cs, c->ev_done[g], 0) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(ho + l0 * q_layer, d + s.out + l0 * q_layer, (size_t)(l1 - l0) * q_layer,
                                   cudaMemcpyDeviceToHost, cs) == cudaSuccess;
        if (!ok) { (void)cudaGetLastError(); return SKV_ERR_CUDA; }
    }
    // the caller's stream is complete only when the last rows are on the host
    ok = cudaEventRecord(c->ev_exit, cs) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(st, c->ev_exit, 0) == cudaSuccess;
    if (!ok) { (void)cudaGetLastError(); return SKV_ERR_CUDA; }
    return SKV_OK;
}

int skv_set_host_step(skv_cache *c, int groups, int ramp)
{
    if (!c || groups < 1 || groups > skv_cache::HOST_GROUPS || ramp < 0 || ramp > 1) return SKV_ERR_ARG;
    c->host_groups = groups;
    c->host_ramp = ramp;
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
    if (t.warps < 1 || t.warps > 16 || t.stages < 1 || t.stages > 8 || t.ctas_per_sm < 1 || t.ctas_per_sm > 8)
        return SKV_ERR_ARG;
    if (c->pool) {
        const size_t smem = decode_smem_bytes(c->head_dim, 1, t.warps, t.stages, c->fp8);
        if (smem == 0 || smem > (size_t)c->max_smem_optin) return SKV_ERR_UNSUPPORTED;
    }
    c->tune = t;
    c->shape_is_default = false;
    return SKV_OK;
}

int skv_prefill_scratch_bytes(const skv_cache *c, size_t *out_bytes)
{
    if (!c || !out_bytes) return SKV_ERR_ARG;
    *out_bytes = c->fp8 ? (size_t)c->max_pages * page_bytes_of(c->kv_heads, c->head_dim, false) : 0;
    return SKV_OK;
}

int skv_set_prefill_scratch(skv_cache *c, void *device_scratch, size_t bytes)
{
    if (!c || (device_scratch && !aligned(device_scratch, 256))) return SKV_ERR_ARG;
    c->prefill_scratch = static_cast<uint8_t *>(device_scratch);
    c->prefill_scratch_bytes = device_scratch ? bytes : 0;
    return SKV_OK;
}

int skv_set_prefill_variant(skv_cache *c, int variant)
{
    if (!c || variant < 0 || variant > 2) return SKV_ERR_ARG;
    c->prefill_variant = variant;
    return SKV_OK;
}

int skv_set_decode_overlap(skv_cache *c, int enabled)
{
    if (!c || enabled < 0 || enabled > 1) return SKV_ERR_ARG;
    c->tune.pdl = enabled;
    return SKV_OK;
}

int skv_set_decode_early_fetch(skv_cache *c, int enabled)
{
    if (!c || enabled < 0 || enabled > 1) return SKV_ERR_ARG;
    c->early_fetch = enabled != 0;
    return SKV_OK;
}

int skv_set_decode_worker(skv_cache *c, int mode, int consumers, int stages, int ctas_per_sm)
{
    if (!c || mode < 0 || mode > 3 || consumers < 0 || consumers > 8 || stages < 0 || stages == 1 || stages > 26 ||
        ctas_per_sm < 0 || ctas_per_sm > 4)
        return SKV_ERR_ARG;
    c->cta_in_turn = mode != 3;
    c->worker_mode = mode == 3 ? 2 : mode;
    if (consumers) c->cta_consumers = consumers;
    c->cta_stages = stages;
    if (ctas_per_sm) c->cta_per_sm = ctas_per_sm;
    return SKV_OK;
}

int skv_set_decode_merge(skv_cache *c, int mode)
{
    if (!c || mode < 0 || mode > 2) return SKV_ERR_ARG;
    c->merge_mode = mode;
    return SKV_OK;
}

int skv_set_decode_l2_reuse(skv_cache *c, int keep_percent)
{
    if (!c || keep_percent < 0 || keep_percent > 100) return SKV_ERR_ARG;
    c->l2_keep_pct = keep_percent;
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
    const int warp_ranges = n_workers_of(c), cta_warps = n_cta_workers_of(c) * c->cta_consumers;
    return warp_ranges > cta_warps ? warp_ranges : cta_warps;
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
