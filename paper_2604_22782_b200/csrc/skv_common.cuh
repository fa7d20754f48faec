// Shared declarations of the skv CUDA library (sm_100a): page geometry, kernel
// parameter blocks, PTX helpers and the host-side launcher prototypes.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace skv {

// ---- page geometry ---------------------------------------------------------
// One page holds PAGE tokens of every kv head of one owner layer.  Within the
// page, each (kv head) owns one contiguous block [K half | V half]; a half is
// stored "chunk-major": [D/8 chunks][PAGE tokens][8 bf16], i.e. element
// (token t, dim d) of a half sits at byte ((d/8)*PAGE + t)*16 + (d%8)*2.
// A 128-byte run is thus 8 tokens x 8 dims: exactly one 8x8 tensor-core
// operand matrix, so ldmatrix reads it without bank conflicts and the whole
// block is moved by a single linear bulk copy.
constexpr int PAGE = 16;
constexpr int CHUNK_ELEMS = 8;                   // bf16 per 16-byte chunk
constexpr int HEADER_BYTES = 256;                // pool header (device status word)

__host__ __device__ constexpr int half_bytes(int D) { return PAGE * D * 2; }
__host__ __device__ constexpr int block_bytes(int D) { return 2 * half_bytes(D); }

// FP8 pages (E4M3 codes, one fp32 scale per (token, kv head) row for K and for V).  The block of
// one (page, kv head):  K codes | V codes | K scales [PAGE] fp32 | V scales [PAGE] fp32.
//   K codes: [2 groups of 8 tokens][D/16 chunks of 16 dims][8 tokens][16 B]
//   V codes: [D dims][PAGE tokens]  =  [D/8 groups of 8 dims][8 dims][16 B]
// Both are the tensor cores' K-major core-matrix layout (8 rows x 16 bytes, contiguous) for the
// operand they are used as: K with the tokens as rows and the dims contracted, V^T with the dims as
// rows and the tokens contracted (see skv_decode_fp8_umma.cu); the mma.sync kernel reads the same
// layout with plain shared-memory loads (Fp8State in skv_decode.cu).
__host__ __device__ constexpr int fp8_k_pos(int D, int t, int d) { return (t >> 3) * 8 * D + (d >> 4) * 128 + (t & 7) * 16 + (d & 15); }
__host__ __device__ constexpr int fp8_v_off(int D) { return PAGE * D; }
__host__ __device__ constexpr int fp8_ks_off(int D) { return 2 * PAGE * D; }
__host__ __device__ constexpr int fp8_vs_off(int D) { return 2 * PAGE * D + PAGE * 4; }
__host__ __device__ constexpr int fp8_block_bytes(int D) { return 2 * PAGE * D + 2 * PAGE * 4; }

// device status bits
constexpr int STATUS_TIMEOUT = 1;
constexpr int STATUS_BOUNDS = 2;

struct AppendParams {
    uint8_t *layer_base;        // first page of the (first) owner layer written
    const uint4 *K;             // [n_layers_here][n_tokens][Hkv][D] bf16 viewed as 16-byte chunks
    const uint4 *V;
    const int64_t *slot_map;    // [n_tokens], shared by all layers of the launch
    int64_t n_tokens;
    int64_t n_slots;            // max_pages * PAGE
    int64_t page_stride;        // bytes between pages of one layer
    int64_t layer_stride;       // bytes between consecutive owner layers in the pool (grid.z walks them)
    int Hkv, D;
    int *status;
};

struct AppendFp8Params {
    uint8_t *layer_base;
    const uint16_t *K;          // [n_layers_here][n_tokens][Hkv][D] bf16 bits
    const uint16_t *V;
    const int64_t *slot_map;
    int64_t n_tokens;
    int64_t n_slots;
    int64_t page_stride;
    int64_t layer_stride;
    int Hkv, D;
    int *status;
};

struct GatherFp8Params {
    const uint8_t *layer_base;
    uint8_t *K_codes;           // [n][Hkv][D]
    uint8_t *V_codes;           // [n][Hkv][D]
    float *K_scales;            // [n][Hkv]
    float *V_scales;
    const int64_t *slot_ids;
    int64_t n;
    int64_t n_slots;
    int64_t page_stride;
    int Hkv, D;
    int *status;
};

struct GatherParams {
    const uint8_t *layer_base;
    uint4 *K_out;
    uint4 *V_out;
    const int64_t *slot_ids;
    int64_t n;
    int64_t n_slots;
    int64_t page_stride;
    int Hkv, D;
    int *status;
};

// DecodeParams::flags
constexpr int DECODE_REVERSE = 1;     // every worker walks its block range from the last block to the first
constexpr int DECODE_LATE_WAIT = 2;   // inputs are known to be ready: the wait on the previous kernel in the
                                      // stream is taken half-way through the range instead of before the first read

constexpr int DECODE_EARLY_FETCH = 4;  // the lengths, the page table and all cached tokens except each sequence's
                                      // newest one were complete before the kernel before this one started: the
                                      // ring is filled before the wait on that kernel, the queries are read after it

constexpr int DECODE_CLAIM_IN_TURN = 8; // CTA-per-range kernel: block j of a range goes to consumer j mod C instead
                                      // of to whichever consumer is free first

constexpr int DECODE_MERGE_IN_KERNEL = 16; // CTA-per-range kernel: segments cut by range ends are finished by the CTAs
                                          // themselves, handing partials from range to range (no merge launch follows)

struct DecodeParams {
    const uint8_t *layer_base;  // first page of the owner layer that is read
    int64_t page_stride;
    int64_t max_pages;
    const uint16_t *Q;          // [B][Hq][D] bf16 bits
    const int32_t *page_table;  // [B][pt_stride]
    const int32_t *seq_lens;    // [B]
    uint16_t *out;              // [B][Hq][D] bf16 bits (CTA-per-range kernel only: segments inside one range are finished there)
    float *part_o;              // [n_slots][G][D]
    float *part_ml;             // [n_slots][G][2]  (running max in log2 units, sum)
    int32_t *prefix;            // [B+1] cumulative page counts (written by CTA 0 for the merge kernel)
    int B, Hq, Hkv, pt_stride;
    float scale_log2;           // scale * log2(e)
    int flags;
    int keep_pct;               // share of each worker's range, at the END of its walk, that is loaded with
                                // normal L2 priority; the rest is loaded evict-first
    int64_t l2_fit_blocks;      // a call with at most this many blocks in all is small enough to stay in L2 for
                                // the next layer that reads the same owner: all of it is loaded with normal priority
    int *status;
    unsigned long long *trace;  // optional [n_workers][4]: sm id, entry ns, first-page ns, exit ns
    unsigned long long *tags;   // [n_slots]: `epoch` once the partial at that slot is complete (DECODE_MERGE_IN_KERNEL)
    unsigned long long epoch;   // a value no earlier call on this workspace has used
};

struct MergeParams {
    const float *part_o;
    const float *part_ml;
    const int32_t *prefix;      // [B+1] page (or tile) counts as the split-K launch left them
    const int32_t *seq_lens;    // [B], or null.  Not null: the kernel counts the pages itself, before it waits
                                // for the split-K launch (the lengths are an input of the call, older than that launch)
    int unit_tokens;            // tokens per unit of the flattened list (a page, or a tile of several pages)
    int64_t max_tokens;         // pt_stride * PAGE: longer sequences were cut to this by the split-K launch
    uint16_t *out;              // [B][Hq][D] bf16 bits
    int B, Hq, Hkv, D;
    int n_workers;
    int max_ctas;               // grid limit (one CTA per SM)
    int skip_single;            // 1: segments with a single partial were finished by the split-K launch itself
};

struct PrefillParams {
    const uint8_t *layer_base;  // first page of the owner layer that is read
    int64_t page_stride;
    int64_t max_pages;
    const uint16_t *Q;          // [n_q][Hq][D] bf16 bits, sequences concatenated
    uint16_t *out;              // [n_q][Hq][D] bf16 bits
    const int32_t *cu_q;        // [B+1] first query row of every sequence
    const int32_t *page_table;  // [B][pt_stride]
    const int32_t *seq_lens;    // [B] cached tokens including the new ones
    int B, Hq, Hkv, pt_stride;
    float scale_log2;
    int *status;
};

struct DequantParams {
    const uint8_t *fp8_base;    // first page of the FP8 owner layer
    uint8_t *bf16_base;         // scratch: the same pages in the bf16 layout
    int64_t fp8_page_stride, bf16_page_stride;
    int64_t max_pages;
    const int32_t *page_table;  // [B][pt_stride]
    const int32_t *seq_lens;    // [B]
    int B, Hkv, pt_stride;
};

struct DecodeTuning {
    int variant;                // 0 auto, 1 CUDA-core (G=1), 2 tensor-core
    int warps;                  // per CTA
    int stages;                 // per warp
    int ctas_per_sm;
    int pdl;                    // 1: launches carry the programmatic-dependent-launch attribute
};

// host launchers (each returns a cudaError_t from the launch)
cudaError_t launch_append(const AppendParams &p, int n_layers, bool pdl, cudaStream_t s);
cudaError_t launch_gather(const GatherParams &p, cudaStream_t s);
// decode attention over FP8 pages on tcgen05 (skv_decode_fp8_umma.cu): a worker is a CTA, grid = worker count
bool decode_fp8_umma_supported(int D, int G);
int decode_fp8_umma_ctas_per_sm();
int decode_fp8_umma_tile_tokens();           // tokens per unit of its flattened list
size_t decode_fp8_umma_smem_bytes(int D, int B);
cudaError_t launch_decode_fp8_umma(const DecodeParams &p, int D, int G, int grid, bool pdl, cudaStream_t s);
cudaError_t launch_append_fp8(const AppendFp8Params &p, int n_layers, bool pdl, cudaStream_t s);
cudaError_t launch_gather_fp8(const GatherFp8Params &p, cudaStream_t s);
// smem bytes the split-K kernel needs for this shape, or 0 if unsupported
size_t decode_smem_bytes(int D, int B, int warps, int stages, bool fp8);
// kernel variant: 0 = CUDA-core (G = 1), 1 = tensor-core (bf16 pages), 2 = FP8 pages (tensor-core, any G)
cudaError_t launch_decode_splitk(const DecodeParams &p, int D, int G, int kernel, int grid,
                                 int warps, int stages, bool pdl, cudaStream_t s);
cudaError_t launch_merge(const MergeParams &p, bool pdl, cudaStream_t s);
// the CTA-per-range split-K kernel (skv_decode_cta.cu): grid = worker count, consumers + 1 warps per CTA
size_t decode_cta_smem_bytes(int D, int B, int G, int consumers, int stages, bool fp8);
bool decode_cta_can_merge(int D, int kernel);   // the variant (kernel: 0 CUDA cores, 1 tensor cores, 2 FP8 pages) can finish cut segments itself
cudaError_t launch_decode_cta(const DecodeParams &p, int D, int G, int kernel, int grid, int consumers, int stages,
                              bool pdl, cudaStream_t s);
// FP8 pages of the sequences' pages -> bf16 pages in a scratch area (skv_dequant.cu); grid covers max_pages_per_seq
cudaError_t launch_dequant_pages(const DequantParams &p, int D, int max_pages_per_seq, cudaStream_t s);
size_t prefill_smem_bytes(int D);
size_t prefill_fp8_smem_bytes(int D);
cudaError_t launch_prefill_fp8(const PrefillParams &p, int D, int G, int q_tiles, bool pdl, cudaStream_t s);
int prefill_tile_tokens(int G);                 // query tokens per CTA tile
cudaError_t launch_prefill(const PrefillParams &p, int D, int G, int q_tiles, bool pdl, cudaStream_t s);
// the tcgen05 (UMMA / tensor-memory) variant
size_t prefill_umma_smem_bytes(int D);
bool prefill_umma_supported(int D, int G);
int prefill_umma_tile_tokens(int G);
cudaError_t launch_prefill_umma(const PrefillParams &p, int D, int G, int q_tiles, bool pdl, cudaStream_t s);

// Raise a kernel's dynamic shared-memory limit to `smem` bytes (skv_api.cu).  The limit only ever has to
// grow, and asking the runtime on every launch costs more than the launch itself, so what has been granted
// is remembered per kernel and device.
cudaError_t ensure_dynamic_smem_fn(const void *kernel, size_t smem);
template <class Kernel>
inline cudaError_t ensure_dynamic_smem(Kernel kern, size_t smem)
{
    return ensure_dynamic_smem_fn(reinterpret_cast<const void *>(kern), smem);
}

// ---- worker <-> work-range arithmetic (shared by split-K and merge) --------
// The flattened work space orders (sequence b, kv head h, page pg) b-major:
// position x = prefix[b]*Hkv + h*pages_b + pg,  total T = prefix[B]*Hkv.
// Worker w of W owns [w*T/W, (w+1)*T/W).
__host__ __device__ inline int64_t worker_begin(int64_t w, int64_t T, int64_t W) { return (w * T) / W; }

// first worker whose range contains position x (0 <= x < T)
__host__ __device__ inline int worker_of(int64_t x, int64_t T, int64_t W)
{
    int64_t w = (x * W) / T;
    if (w >= W) w = W - 1;
    while (w > 0 && worker_begin(w, T, W) > x) --w;
    while (w + 1 < W && worker_begin(w + 1, T, W) <= x) ++w;
    return (int)w;
}

// ---- PTX helpers -------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait: gives up after limit_ns nanoseconds and returns false.
__device__ __forceinline__ bool mbar_wait_limited(uint32_t bar, uint32_t parity, uint64_t limit_ns)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > limit_ns) return false;
    }
}

// The kernels' limit: about two seconds.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity)
{
    return mbar_wait_limited(bar, parity, 2000000000ull);
}

// linear bulk copy global -> this CTA's shared memory, completion on an mbarrier
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}

// same, with an L2 eviction-priority policy (from make_policy_*)
__device__ __forceinline__ void bulk_copy_g2s_hint(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar,
                                                   uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}

__device__ __forceinline__ uint64_t make_policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ uint64_t make_policy_evict_normal()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

// Programmatic dependent launch: wait for the kernel before this one in the stream (a no-op when the
// launch carried no such attribute); let the kernel after this one start being scheduled.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}

// D(16x8,f32) += A(16x16,bf16,row) * B(16x8,bf16,col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1)
{
    asm(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// D(16x8,f32) += A(16x16,f16,row) * B(16x8,f16,col)  (a function of its register operands only: not
// volatile, so that the compiler may move it among the shared-memory loads)
__device__ __forceinline__ void mma_f16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1)
{
    asm(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// four E4M3 codes (one 32-bit word) -> two f16x2 registers: lo = codes 0,1; hi = codes 2,3 (exact)
__device__ __forceinline__ void e4m3x4_to_f16x2(uint32_t w, uint32_t &lo, uint32_t &hi)
{
    asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\t"
        "cvt.rn.f16x2.e4m3x2 %0, a;\n\tcvt.rn.f16x2.e4m3x2 %1, b;\n\t}"
        : "=r"(lo), "=r"(hi)
        : "r"(w));
}

// two fp32 -> packed f16x2 (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// two fp32 -> two E4M3 codes in the low 16 bits (lo in bits 0-7), round to nearest even, saturating at +-448
__device__ __forceinline__ uint32_t pack_e4m3x2(float lo, float hi)
{
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return (uint32_t)r;
}

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// two fp32 -> packed bf16x2 (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

}  // namespace skv
