/*
 * skv.h -- C ABI of the routed (depth-wise shared) paged KV cache and its
 * decode-time attention step for NVIDIA B200 (sm_100a).
 *
 * What the library computes, in the paper's terms ("Stochastic KV Routing:
 * Enabling Adaptive Depth-Wise Cache Sharing", Section 3.1):
 *
 *   - A transformer decoder has L layers.  A cache sharing strategy S names
 *     the layers that keep a KV cache; every layer l reads the cache of its
 *     source layer mu(l) <= l (Eq. (3.2)).  This library takes the map itself,
 *     r[l] (0-based), and accepts any r with r[0] = 0, r[l] <= l and
 *     r[r[l]] = r[l]; layers with r[l] = l are the OWNERS.
 *   - Algorithm 2, one decode step, per layer:  "Update" (append the new
 *     token's K,V) happens only for owners; "Load" + "Attn" reads the owner's
 *     cache:  Output_l = Attn(Q_l, K_r[l], V_r[l])   (Eq. (3.1)).
 *     Attn is scaled dot-product softmax attention with grouped queries:
 *     query head h reads KV head floor(h / (q_heads / kv_heads)).
 *   - Cache memory is allocated for owners only, so its size is
 *     2 x |owners| x kv_heads x head_dim x 2 bytes per token (Section 1
 *     footnote with #layers -> |S|; Section 4.3: with groups of g layers the
 *     cache shrinks by the factor g).
 *
 * Conventions
 *   - Every function returns an int status: SKV_OK (0) or a negative
 *     skv_status.  Nothing throws or aborts.  Argument errors are found on the
 *     host before anything is launched.
 *   - "device" pointers are CUDA device memory of the current device, owned by
 *     the caller for the whole life of the handle; the library never allocates
 *     or frees device memory (except where a function says otherwise).
 *     "host" pointers are ordinary host memory.
 *   - All device work is enqueued on the caller's stream (a cudaStream_t passed
 *     as void*; NULL = the default stream) and the call returns without
 *     waiting, except skv_get_status which synchronises that stream.
 *   - bf16 tensors are dense, row-major, last index fastest.
 *   - Layers are 0-based (the paper counts from 1).
 *   - There is no CPU implementation behind these calls: without a usable
 *     CUDA device every call that needs one returns SKV_ERR_CUDA.
 *
 * Supported shapes: head_dim 64 or 128; page_size 16; q_heads a multiple of
 * kv_heads with q_heads / kv_heads <= 8.
 */
#ifndef SKV_H
#define SKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct skv_cache skv_cache; /* opaque host-side handle */

typedef enum skv_status {
    SKV_OK = 0,
    SKV_ERR_ARG = -1,         /* null pointer, non-positive size, misaligned buffer */
    SKV_ERR_ROUTING = -2,     /* r[0] != 0, r[l] > l, r[l] < 0 or r[r[l]] != r[l] */
    SKV_ERR_UNSUPPORTED = -3, /* shape outside the supported set */
    SKV_ERR_NOMEM = -4,       /* caller's pool or workspace is too small */
    SKV_ERR_LAYER = -5,       /* layer index out of range, or an owner is required */
    SKV_ERR_CUDA = -6,        /* a CUDA runtime call failed (no device, bad stream, ...) */
    SKV_ERR_TIMEOUT = -7,     /* device status: a bounded wait inside a kernel ran out */
    SKV_ERR_BOUNDS = -8,      /* device status: a page id or slot id was out of range */
    SKV_ERR_TOO_LARGE = -9    /* skv_decode_attn_static: the call needs more than SKV_STATIC_SCRATCH_BYTES */
} skv_status;

const char *skv_strerror(int status);

/* ---- routing maps (pure host) ------------------------------------------ */

/* Eq. (3.2): r_out[l] = l if l is in owners[], else the largest owner below l.
 * owners: host, n_owners distinct layer indices in [0, n_layers), any order;
 * layer 0 must be among them (otherwise mu is undefined for the layers below
 * the first owner -> SKV_ERR_ROUTING).  r_out: host, n_layers entries. */
int skv_routing_from_owners(int n_layers, const int32_t *owners, int n_owners, int32_t *r_out);

/* Section 4.3 "leaders": every g consecutive layers read the first one of
 * their group, r_out[l] = l - (l mod g); the last group may be short. */
int skv_routing_groups(int n_layers, int g, int32_t *r_out);

/* Section 3.2, training time: the cache source of every layer for ONE forward
 * pass of R-CLA.  For each layer l a decision d ~ Bernoulli(p_self) is drawn as
 * (u[l] < p_self): d = 1 keeps the layer's own K,V (map_out[l] = l), d = 0 takes
 * layer floor(v[l] * l), i.e. uniform over the l layers before it.  Layer 0 has
 * nothing before it and always reads itself.  The random numbers are the
 * caller's: u, v host arrays of n_layers doubles in [0, 1) (SKV_ERR_ARG else).
 * The map need not be a valid skv_cache_create map (a layer may read a layer
 * that itself reads elsewhere): at training time every layer's K,V exists, see
 * skv_prefill_attn_src. */
int skv_routing_rcla(int n_layers, double p_self, const double *u, const double *v, int32_t *map_out);

/* Section 4.2 ablation "RD-CLA@k": the fixed groups of skv_routing_groups(k),
 * applied stochastically: u[l] < p_self keeps the layer's own K,V, otherwise the
 * layer reads the first layer of its group. */
int skv_routing_rdcla(int n_layers, int k, double p_self, const double *u, int32_t *map_out);

/* ---- cache -------------------------------------------------------------- */

/* Bytes of device memory the caller must provide for the page pool:
 * a 256-byte header + |owners| * max_pages * page_bytes, where
 * page_bytes = 2 (K,V) * page_size * kv_heads * head_dim * 2.
 * max_pages is per owner layer; page ids are shared by all owner layers. */
int skv_cache_pool_bytes(int n_layers, const int32_t *r, int kv_heads, int head_dim,
                         int page_size, int64_t max_pages, size_t *out_bytes);

/* Create a handle (Algorithm 2's cache state for a strategy S).
 *   r           host, n_layers entries, copied.
 *   device_pool device, >= pool_bytes, 256-byte aligned; zero-filled on `stream`
 *               by this call; must outlive the handle.  If device_pool is NULL
 *               (and pool_bytes 0) the handle does accounting only: routing and
 *               byte queries work, every call that would launch returns
 *               SKV_ERR_ARG.  No CUDA call is made in that case.
 * Errors: SKV_ERR_ROUTING, SKV_ERR_UNSUPPORTED, SKV_ERR_NOMEM (pool_bytes too
 * small), SKV_ERR_ARG, SKV_ERR_CUDA. */
int skv_cache_create(skv_cache **out, int n_layers, const int32_t *r, int kv_heads, int head_dim,
                     int page_size, int64_t max_pages, void *device_pool, size_t pool_bytes,
                     void *stream);

/* The same cache with FP8 pages (the paper names KV quantisation as composable
 * with depth-wise sharing, Sections 2 and 5, and fixes no scheme; this is the
 * library's): OCP E4M3 codes and one fp32 scale per (token, kv head) row, for K
 * and for V separately.  skv_append quantises on the way in:
 *   amax = max |x| over the row's head_dim values,  scale = amax / 448,
 *   code = E4M3(x * (448 / amax)), round to nearest even, saturating at +-448
 * (a row of zeros: scale 0, codes 0; each step is one fp32 operation), and the
 * attention sees  code value x scale.  Cache bytes per token become
 * 2 x |owners| x kv_heads x (head_dim + 4).  skv_decode_attn, skv_decode_step and
 * skv_decode_step_host work on such a cache as on a bf16 one (any q_heads /
 * kv_heads <= 8; the scales are applied outside the contractions).  At
 * head_dim 128 both contractions run as FP8 tensor-core instructions (tcgen05,
 * kind f8f6f4) on the stored codes, with the queries and the probabilities each
 * split into two E4M3 terms; at head_dim 64, or with skv_set_decode_variant(2),
 * the codes are converted to f16 on the way into mma.sync.  The pre-fill calls
 * run an mma.sync kernel that converts the codes the same way, or, given a
 * scratch area (skv_set_prefill_scratch), the tcgen05 kernel on a bf16 copy of
 * the pages they reach (prefill variant 2 without one: SKV_ERR_UNSUPPORTED); skv_gather
 * returns SKV_ERR_UNSUPPORTED (use skv_gather_fp8).  Same arguments and errors
 * as skv_cache_pool_bytes / skv_cache_create. */
int skv_cache_pool_bytes_fp8(int n_layers, const int32_t *r, int kv_heads, int head_dim,
                             int page_size, int64_t max_pages, size_t *out_bytes);
int skv_cache_create_fp8(skv_cache **out, int n_layers, const int32_t *r, int kv_heads, int head_dim,
                         int page_size, int64_t max_pages, void *device_pool, size_t pool_bytes,
                         void *stream);

/* Frees host state (and the handle's copy stream and events, if
 * skv_decode_step_host created them); never touches device_pool. */
void skv_cache_destroy(skv_cache *cache);

/* r[layer] (>= 0) or SKV_ERR_LAYER. */
int skv_layer_owner(const skv_cache *cache, int layer);
/* 1 if r[layer] == layer, 0 if not, SKV_ERR_LAYER if out of range. */
int skv_is_owner(const skv_cache *cache, int layer);

/* Byte accounting; any out pointer may be NULL.
 *   page_bytes      bytes of one page of one owner layer
 *   kv_bytes        |owners| * max_pages * page_bytes (the KV storage proper)
 *   bytes_per_token 2 * |owners| * kv_heads * head_dim * 2
 *                   (FP8 cache: 2 * |owners| * kv_heads * (head_dim + 4)) */
int skv_cache_stats(const skv_cache *cache, int *n_owners, size_t *page_bytes, size_t *kv_bytes,
                    size_t *bytes_per_token);

/* ---- Algorithm 2 "Update": append ---------------------------------------- */

/* Store the K,V rows of n_tokens new tokens in `layer`'s cache.  If `layer`
 * is not an owner this is a no-op that launches nothing (its K,V are never
 * read: Algorithm 2 updates only layers in S) and K, V may be NULL.
 *   K, V      device bf16 [n_tokens][kv_heads][head_dim], 16-byte aligned
 *   slot_map  device int64 [n_tokens]; slot = page * page_size + offset;
 *             a negative slot skips the token; slots >= max_pages * page_size
 *             are skipped and raise SKV_ERR_BOUNDS in the device status.
 *             Duplicate slots in one call: unspecified which row is kept.
 * The copy is bit-exact. */
int skv_append(skv_cache *cache, int layer, const void *K, const void *V, const int64_t *slot_map,
               int64_t n_tokens, void *stream);

/* Inverse of skv_append for tests and snapshots: read rows back.
 *   layer     must be an owner (SKV_ERR_LAYER otherwise)
 *   slot_ids  device int64 [n]; negative -> the output row is left untouched
 *   K_out, V_out device bf16 [n][kv_heads][head_dim] */
int skv_gather(skv_cache *cache, int layer, const int64_t *slot_ids, int64_t n, void *K_out,
               void *V_out, void *stream);

/* Read-back of an FP8 cache (skv_cache_create_fp8): the stored codes and scales.
 *   K_codes, V_codes  device uint8 [n][kv_heads][head_dim]
 *   K_scales, V_scales device fp32 [n][kv_heads]
 * SKV_ERR_UNSUPPORTED on a bf16 cache. */
int skv_gather_fp8(skv_cache *cache, int layer, const int64_t *slot_ids, int64_t n, void *K_codes,
                   void *V_codes, float *K_scales, float *V_scales, void *stream);

/* ---- Algorithm 2 "Load + Attn": decode attention -------------------------- */

/* Bytes of device workspace skv_decode_attn needs for this batch / head count
 * under the CURRENT launch shape (ask again after skv_set_decode_tuning or
 * skv_set_decode_variant).
 * Independent of sequence lengths.  It holds, twice (two calls of a chain may
 * overlap), the split partials, one 8-byte tag per partial and a page-count
 * prefix. */
int skv_decode_workspace_bytes(const skv_cache *cache, int batch, int q_heads, size_t *out_bytes);

/* Eq. (3.1) for one layer and one new token per sequence:
 *   out[b,h,:] = sum_{t < seq_lens[b]} softmax_t(scale * <Q[b,h,:], K[b,t,kv(h),:]>) * V[b,t,kv(h),:]
 * with K,V the cache of layer r[layer] and token t of sequence b stored at
 * slot page_table[b][t / page_size] * page_size + t % page_size.
 *   Q           device bf16 [batch][q_heads][head_dim], 16-byte aligned
 *   page_table  device int32 [batch][pt_stride]; entries past a sequence's
 *               last page are never read
 *   seq_lens    device int32 [batch]; tokens to attend, including the one just
 *               appended; 0 gives an all-zero output row.  A length that needs
 *               more than pt_stride pages is cut to pt_stride * page_size tokens
 *               on the device and raises SKV_ERR_BOUNDS in the device status
 *               (no page id is read past the end of a page_table row)
 *   out         device bf16 [batch][q_heads][head_dim]
 *   scale       <= 0 selects 1/sqrt(head_dim)
 *   workspace   device, 256-byte aligned, >= skv_decode_workspace_bytes; needs
 *               no initialisation and may be shared by calls on one stream.
 * One or two launches.  Split-K (flash-decoding): the (sequence, kv head, page) blocks
 * of the call form one list that is cut into equal contiguous ranges, one per
 * worker, whatever the mix of lengths; a worker streams its range through
 * shared memory and leaves, for each (sequence, kv head) its range touches, an
 * fp32 partial (max, sum, output).  Merge: one warp per (sequence, kv head)
 * combines its partials by log-sum-exp and writes the bf16 rows.  The worker is
 * a CTA per SM whose warps share one ring of stages and combine their states in
 * shared memory -- it then finishes every (sequence, kv head) that lies inside
 * its range itself and the merge launch has only the others left, or, where
 * skv_set_decode_merge lets it, finishes those too and no merge launch follows
 * -- or a single warp (skv_set_decode_worker).  Slots past seq_lens[b] in the last page contribute nothing
 * whatever they contain.  No host synchronisation; sequence lengths are read
 * on the device.  The split-K launch waits for the work before it in the
 * stream before it reads anything; with skv_set_decode_overlap on, the merge
 * kernel is already resident when the split-K launch ends and the kernel after
 * the call may be scheduled while the call is still running.
 * Errors: SKV_ERR_ARG, SKV_ERR_LAYER, SKV_ERR_UNSUPPORTED (head ratio),
 * SKV_ERR_NOMEM (workspace), SKV_ERR_CUDA.  Device-side problems (page id out
 * of range, a bounded wait that ran out) are reported by skv_get_status; after
 * SKV_ERR_TIMEOUT the outputs of that call are undefined. */
int skv_decode_attn(skv_cache *cache, int layer, const void *Q, const int32_t *page_table,
                    const int32_t *seq_lens, void *out, int batch, int q_heads, int pt_stride,
                    float scale, void *workspace, size_t workspace_bytes, void *stream);

/* (No counterpart in the paper; an integration convenience.)
 * skv_decode_attn for callers that cannot hand the library a workspace because
 * they cannot allocate device memory at the point of the call: code running
 * inside a serving engine after it has frozen its memory pool (the engine
 * pre-allocates every byte it will ever use and treats a later cudaMalloc as a
 * bug, or has none left to give), plugins loaded into a host process that
 * forbids allocation on its hot path, and callers without an allocator of
 * their own (a plain C program handed only the input and output buffers).
 * Same arguments, result and errors as skv_decode_attn minus the workspace:
 * the split-K partials and control words live in a fixed area of
 * SKV_STATIC_SCRATCH_BYTES that is part of the library image, so every GPU
 * that loads the library gives up that much memory until the process exits.
 *   - Neither this call nor anything it uses allocates or frees device memory.
 *   - A call whose skv_decode_workspace_bytes(cache, batch, q_heads) exceeds
 *     SKV_STATIC_SCRATCH_BYTES is refused with SKV_ERR_TOO_LARGE before
 *     anything is launched (under the default launch shape the need is about
 *     2 * (SMs * 8 + batch * kv_heads) * (q_heads / kv_heads) * (head_dim + 2) * 4
 *     bytes: 6.0 MB for batch 32 of the Llama-3-8B head shape).
 *   - The first call on each device looks up the area's device address (with
 *     that device current); make that first call outside any stream capture.
 *   - All calls on a device, from every handle and every stream, share the one
 *     area, and it keeps the previous call's contents.  Nothing in it has to
 *     start at zero (the merge only reads what the split-K launch of the same
 *     call wrote), so nothing is cleared; but two calls that overlap on the GPU
 *     (different streams without an ordering between them) race on it and give
 *     undefined results.  Calls on one stream are safe. */
#define SKV_STATIC_SCRATCH_BYTES ((size_t)8 << 20)
int skv_decode_attn_static(skv_cache *cache, int layer, const void *Q, const int32_t *page_table,
                           const int32_t *seq_lens, void *out, int batch, int q_heads, int pt_stride,
                           float scale, void *stream);

/* The two launches of skv_decode_attn separately (profiling, sequence-sharded
 * use): the split-K pass fills `workspace` with partials; the merge kernel
 * turns the partials in `workspace` into `out`.  Same arguments and errors. */
int skv_decode_splitk(skv_cache *cache, int layer, const void *Q, const int32_t *page_table,
                      const int32_t *seq_lens, int batch, int q_heads, int pt_stride, float scale,
                      void *workspace, size_t workspace_bytes, void *stream);
int skv_decode_merge(skv_cache *cache, void *out, int batch, int q_heads, void *workspace,
                     size_t workspace_bytes, void *stream);

/* ---- pre-fill attention (Section 3.1.1 "Pre-fill") ------------------------ */

/* Eq. (3.1) for the tokens of a prompt (or of a chunk of it) processed in
 * parallel: query row i of sequence b is the token at position
 *   pos = seq_lens[b] - q_len_b + i,   q_len_b = cu_q_lens[b+1] - cu_q_lens[b],
 * i.e. the rows of a sequence are its LAST q_len_b cached tokens, and it attends
 * the tokens 0..pos of the cache of layer r[layer] (a decoder is causal):
 *   out[row,h,:] = sum_{t <= pos} softmax_t(scale * <Q[row,h,:], K[b,t,kv(h),:]>) * V[b,t,kv(h),:]
 * The rows' own K,V must have been appended before (skv_append takes any number
 * of tokens), so q_len_b <= seq_lens[b].  One row per sequence gives the decode
 * step of skv_decode_attn.
 *   Q          device bf16 [n_q][q_heads][head_dim], sequences concatenated,
 *              n_q = cu_q_lens[batch]; 4-byte aligned
 *   cu_q_lens  device int32 [batch+1], non-decreasing, cu_q_lens[0] = first row
 *   page_table, seq_lens   as in skv_decode_attn
 *   out        device bf16 [n_q][q_heads][head_dim]
 *   max_q_len  host bound on q_len_b (sizes the grid; no host synchronisation)
 * One launch, no workspace: a CTA owns 64 or 128 query rows (that many /
 * (q_heads/kv_heads) tokens x the query heads of one kv head) and streams the
 * pages they see (skv_set_prefill_variant).
 * Errors as skv_decode_attn; a sequence with q_len_b > seq_lens[b],
 * q_len_b > max_q_len or seq_lens[b] > pt_stride * page_size raises
 * SKV_ERR_BOUNDS in the device status and its rows are left untouched. */
int skv_prefill_attn(skv_cache *cache, int layer, const void *Q, const int32_t *cu_q_lens,
                     const int32_t *page_table, const int32_t *seq_lens, void *out, int batch,
                     int max_q_len, int q_heads, int pt_stride, float scale, void *stream);

/* skv_prefill_attn with the source named by the caller instead of the routing
 * map: the rows attend the pages of `src_layer`, which must be an owner
 * (SKV_ERR_LAYER otherwise).  This is the routed attention of a training-time
 * forward pass (Section 3.2): with a cache in which every layer owns its pages
 * (identity map), layer l of a pass calls it with src_layer = map[l] from
 * skv_routing_rcla / skv_routing_rdcla.  Forward only. */
int skv_prefill_attn_src(skv_cache *cache, int src_layer, const void *Q, const int32_t *cu_q_lens,
                         const int32_t *page_table, const int32_t *seq_lens, void *out, int batch,
                         int max_q_len, int q_heads, int pt_stride, float scale, void *stream);

/* Pre-fill on an FP8 cache through the bf16 tensor-core kernel.  Given a scratch
 * area of skv_prefill_scratch_bytes (room for the pages of ONE owner layer as
 * bf16: max_pages * 2 * page_size * kv_heads * head_dim * 2 bytes; device,
 * 256-byte aligned, the caller's, kept until it is taken back with NULL),
 * skv_prefill_attn / skv_prefill_attn_src on an FP8 cache first turn the pages
 * that the call's sequences reach back into bf16 (code value x the row's scale,
 * rounded to nearest even) in that area -- one more launch, a pass over the
 * pages that costs a few per cent of a prompt's attention -- and then run the
 * tcgen05 kernel on it.  Without a scratch area (the default), or where that
 * kernel does not apply, they run the mma.sync kernel that converts the codes on
 * the way in.  Calls that use the area must not overlap on the GPU.
 * skv_prefill_scratch_bytes gives 0 for a bf16 cache. */
int skv_prefill_scratch_bytes(const skv_cache *cache, size_t *out_bytes);
int skv_set_prefill_scratch(skv_cache *cache, void *device_scratch, size_t bytes);

/* One whole decode step of Algorithm 2 with inputs already on the device:
 * for l = 0..L-1: append (owners only) then decode attention, on `stream`.
 * Because every input of the step exists when it starts, and the update of
 * layer l writes only layer l's pages (which no earlier layer reads), the
 * library issues all owners' updates first, in one launch, and then the L
 * attention calls as a chain in which the split-K launch of layer l+1 may begin
 * while layer l is finishing (skv_set_decode_overlap; results are the same as
 * layer by layer).
 *   Q        device bf16 [n_layers][batch][q_heads][head_dim]
 *   K, V     device bf16 [n_owners][batch][kv_heads][head_dim], owner layers in
 *            increasing layer order
 *   slot_map device int64 [batch]: slot of each sequence's new token
 *   out      device bf16 [n_layers][batch][q_heads][head_dim]
 * Other arguments as in skv_decode_attn. */
int skv_decode_step(skv_cache *cache, const void *Q, const void *K, const void *V,
                    const int64_t *slot_map, const int32_t *page_table, const int32_t *seq_lens,
                    void *out, int batch, int q_heads, int pt_stride, float scale, void *workspace,
                    size_t workspace_bytes, void *stream);

/* One whole decode step of Algorithm 2 from HOST buffers: copies the step's
 * inputs to the device, runs append + decode attention for layers 0..L-1 in
 * order, and copies the outputs back.  Everything is ordered after the work
 * already on `stream`, and `stream` is complete only when the outputs are in
 * h_out (the caller synchronises `stream`); inside, the layers are cut into
 * groups and a copy stream owned by the handle (created on the first call,
 * destroyed by skv_cache_destroy) moves the next group's inputs in while a
 * group's kernels run and takes each group's results back while the next group
 * runs.  Host buffers should be pinned for the copies to be asynchronous.
 *   hQ          host bf16 [n_layers][batch][q_heads][head_dim]
 *   hK, hV      host bf16 [n_owners][batch][kv_heads][head_dim], owner layers
 *               in increasing layer order
 *   h_slot_map  host int64 [batch]  (slot of each sequence's new token)
 *   h_page_table host int32 [batch][pt_stride];  h_seq_lens host int32 [batch]
 *   h_out       host bf16 [n_layers][batch][q_heads][head_dim]
 *   staging     device, 256-byte aligned, >= skv_decode_step_staging_bytes;
 *               holds the device copies of all of the above plus the decode
 *               workspace */
int skv_decode_step_staging_bytes(const skv_cache *cache, int batch, int q_heads, int pt_stride,
                                  size_t *out_bytes);
int skv_decode_step_host(skv_cache *cache, const void *hQ, const void *hK, const void *hV,
                         const int64_t *h_slot_map, const int32_t *h_page_table,
                         const int32_t *h_seq_lens, void *h_out, int batch, int q_heads,
                         int pt_stride, float scale, void *staging, size_t staging_bytes,
                         void *stream);

/* ---- status, tuning, counters ------------------------------------------- */

/* Synchronises `stream`, reads and clears the device status word.
 * *device_status receives SKV_OK, SKV_ERR_TIMEOUT or SKV_ERR_BOUNDS. */
int skv_get_status(skv_cache *cache, void *stream, int *device_status);

/* Split-K kernel variant: 0 = automatic (CUDA-core kernel when
 * q_heads == kv_heads, tensor-core (mma) kernel otherwise), 1 = CUDA-core
 * kernel (only q_heads == kv_heads), 2 = tensor-core kernel.  On an FP8 cache:
 * 0 or 1 = the tcgen05 kernel where it applies (head_dim 128; its worker count
 * and launch shape are fixed, skv_set_decode_tuning does not apply to it),
 * 2 = the mma.sync kernel. */
int skv_set_decode_variant(skv_cache *cache, int variant);

/* Launch shape of the split-K kernel (default: 8 warps per SM with two 8 KB
 * stages each, as 2 warps x 4 CTAs per SM for the tensor-core kernel and
 * 1 warp x 8 CTAs per SM for the CUDA-core kernel): warps per CTA (1..16), pipeline stages
 * per warp (1..8) and CTAs per SM (1..8); 0 keeps the current value (other values: SKV_ERR_ARG).
 * SKV_ERR_UNSUPPORTED if the combination does not fit in shared memory. */
int skv_set_decode_tuning(skv_cache *cache, int warps_per_cta, int stages, int ctas_per_sm);

/* Pre-fill kernel variant: 0 = automatic (the tcgen05 kernel when head_dim is
 * 128, q_heads / kv_heads divides 128 and Q, out are 16-byte aligned; else the
 * mma.sync kernel), 1 = mma.sync kernel (64 query rows per CTA), 2 = tcgen05
 * kernel (128 query rows per CTA, accumulators in tensor memory;
 * SKV_ERR_UNSUPPORTED from skv_prefill_attn where it does not apply). */
int skv_set_prefill_variant(skv_cache *cache, int variant);

/* 1 (default): split-K and merge launches carry the programmatic-dependent-
 * launch attribute, so the GPU may schedule a launch while the one before it
 * in the stream is still running (each still waits for the work it depends on
 * before reading it), and skv_decode_step chains its attention calls; 0: plain
 * launches, and skv_decode_step goes layer by layer through skv_append /
 * skv_decode_attn. */
int skv_set_decode_overlap(skv_cache *cache, int enabled);

/* Which worker the split-K pass of a stand-alone attention call uses
 * (skv_decode_attn, skv_decode_attn_static; the two-call form skv_decode_splitk +
 * skv_decode_merge and the chained launches of skv_decode_step always use warps).
 *   mode 0 (default) or 2: CTAs that own a range each -- `consumers` warps
 *        (1..8; 0 keeps the current value) share one ring of `stages` stages of
 *        one (page, kv head) block (2..26; 0, the default: as many as fit, at
 *        most 20 per SM) filled by a producer warp, take its blocks in turn and
 *        combine their running states in shared memory at the end of every
 *        (sequence, kv head).  The grid is `ctas_per_sm` (1..4; 0 keeps the current
 *        value, default 1) CTAs per SM, all resident at once;
 *   mode 3: as 2, but a consumer takes the ring's next block whenever it is free
 *        instead of every consumers-th one (results then vary in their last bits
 *        from run to run);
 *   mode 1: a warp per range, launch shape from skv_set_decode_tuning.
 * FP8 pages at head_dim 128 keep their tcgen05 kernel either way.  Results of
 * the modes agree to rounding (the order of the sums differs). */
int skv_set_decode_worker(skv_cache *cache, int mode, int consumers, int stages, int ctas_per_sm);

/* Early fetch for stand-alone attention calls (skv_decode_attn, skv_decode_attn_static,
 * skv_decode_splitk; needs skv_set_decode_overlap on).  0 (default): a split-K
 * launch waits for the kernel before it in the stream before it reads anything.
 * 1: it reads seq_lens and page_table, and starts copying pages, while that
 * kernel is still running, and waits for it only before it reads Q and before it
 * copies the LAST page of any sequence.  In a decoder this is what the data flow
 * allows (Algorithm 2: Q of layer l is computed from the output of layer l-1, and
 * the Update of layer l adds one token, which lands in the sequence's last page;
 * everything else the call reads is older), and it takes the launch, the length
 * scan and the first page copies off the critical path: skv_append lets the
 * launch after it start at once, so on an owner layer they run beside the update.
 * The caller's promise when switching it on: the kernel directly before each such
 * call in its stream writes neither seq_lens nor page_table nor any cached token
 * other than tokens in the last page of a sequence (skv_append of the step's new
 * token is such a kernel; so is any kernel that only produces Q).  If that kernel
 * was itself launched with the programmatic stream-serialisation attribute and
 * releases its dependents before it has waited for the kernel before it (as
 * skv_append's decode-step kernel does), the promise covers that earlier kernel
 * too, and so on up the chain: with a decoder whose own kernels between two
 * attention calls behave like that, the next layer's attention kernel moves into
 * the SMs that this layer's leaves and fills its ring while the rest still work.
 * Results are identical. */
int skv_set_decode_early_fetch(skv_cache *cache, int enabled);

/* Who combines the partials of a stand-alone attention call (skv_decode_attn,
 * skv_decode_attn_static).  mode 1: the merge kernel, launched after every split-K
 * launch.  mode 2: the CTA-per-range kernel itself, wherever it runs and its variant
 * has the warp for it (not: one query head per kv head at head_dim 128; not with
 * more than one CTA per SM; not the tcgen05 FP8 kernel): a segment cut by range
 * ends is finished by handing its partial from range to range through the
 * workspace, each hand-over marked by a tag the next CTA waits for (bounded;
 * SKV_ERR_TIMEOUT in the status word when it runs out) and clears, and no merge
 * launch follows.  That is quick when few segments are cut more than once and slow when a
 * segment spans many ranges.  mode 0 (default): mode 2 when the call has at least
 * two thirds as many (sequence, kv head) segments as CTAs, else mode 1.  Results agree within
 * the rounding of a different summation order.  SKV_ERR_ARG for other modes. */
int skv_set_decode_merge(skv_cache *cache, int mode);

/* L2 reuse between consecutive layers that read the same owner (the paper's
 * depth-wise sharing makes them stream identical pages): with keep_percent > 0
 * such layers walk every worker's block range in alternating directions, and a
 * layer whose successor reads the same owner loads the last keep_percent % of
 * each range with normal L2 priority (everything else is loaded evict-first),
 * so the successor starts on blocks that are still in L2.  Default 35;
 * 0 = every layer walks forward, everything evict-first.  Results do not depend
 * on it beyond floating-point summation order. */
int skv_set_decode_l2_reuse(skv_cache *cache, int keep_percent);

/* How skv_decode_step_host cuts the step: `groups` layer groups (1..8, default
 * 4), of equal size (ramp 0) or with small first and last groups, whose copies
 * nothing hides (ramp 1, default).  Results do not depend on either. */
int skv_set_host_step(skv_cache *cache, int groups, int ramp);

/* Tracing: while a device buffer of at least 32 * skv_decode_worker_count bytes
 * is set, every split-K launch records four uint64 per worker (warp): SM id,
 * kernel-entry time, time its first page arrived, exit time (global timer, ns).
 * NULL switches tracing off.  skv_decode_worker_count = the larger of SMs *
 * CTAs per SM * warps per CTA under the current tuning and SMs * consumer warps
 * of the CTA-per-SM kernel (which records one entry per consumer warp). */
int skv_set_trace_buffer(skv_cache *cache, void *device_buffer, size_t bytes);
int skv_decode_worker_count(const skv_cache *cache);

/* Number of kernels this handle has launched so far. */
int skv_launch_count(const skv_cache *cache, int64_t *out_count);

/* The split-K work partition (pure host arithmetic, same code the kernels use):
 * the n_blocks (sequence, kv head, page) blocks of a call are cut into
 * n_workers contiguous ranges of equal size +-1.  skv_plan_worker_range gives
 * worker w's [begin, end); skv_plan_worker_of gives the worker whose range
 * holds block x, or SKV_ERR_ARG. */
int skv_plan_worker_range(int64_t n_blocks, int n_workers, int w, int64_t *begin, int64_t *end);
int skv_plan_worker_of(int64_t n_blocks, int n_workers, int64_t x);

#ifdef __cplusplus
}
#endif
#endif /* SKV_H */
