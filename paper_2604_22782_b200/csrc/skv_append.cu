// "Update" of Algorithm 2: scatter the new tokens' K,V rows into the pages of an
// owner layer, and the inverse read-back.  Pure 16-byte copies, bit-exact.
#include "skv_common.cuh"

namespace skv {

namespace {

constexpr int COPY_THREADS = 256;

// One thread moves one 16-byte chunk (8 bf16 of one head of one token); grid.y picks K or V,
// grid.z the owner layer when one launch serves several.  A warp takes 16 tokens x 2 adjacent
// chunks of one head: lane = token (low 4 bits) + 16 * chunk parity, so that the reads of a token's
// two chunks fill one 32-byte sector and, when the 16 tokens sit in consecutive slots of a page
// (pre-fill), each half-warp writes one contiguous 256-byte run of the chunk-major page layout.
struct CopyCoord {
    int64_t tok;
    int h, c;
    bool in_range;
};

__device__ __forceinline__ CopyCoord coord_of(int64_t n_tok, int Hkv, int CH)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * COPY_THREADS + threadIdx.x) >> 5;
    const int pairs = CH / 2;                             // head_dim is 64 or 128: CH is even
    const int64_t per_group = (int64_t)Hkv * pairs;       // warps per group of 16 tokens
    const int64_t g16 = warp / per_group;
    const int rem = (int)(warp - g16 * per_group);
    CopyCoord k;
    k.h = rem / pairs;
    k.c = 2 * (rem - k.h * pairs) + (lane >> 4);
    k.tok = g16 * 16 + (lane & 15);
    k.in_range = k.tok < n_tok;
    return k;
}

__global__ void __launch_bounds__(COPY_THREADS) append_kernel(AppendParams p)
{
    pdl_trigger();      // an attention launch right after this one may set itself up while the rows are copied
    pdl_wait();         // (launched ahead of the end of the kernel before it: the rows and the slot map may be that
                        // kernel's, and whoever waits for this kernel's end must be able to take the other's for granted)
    const int CH = p.D / CHUNK_ELEMS;
    const CopyCoord k = coord_of(p.n_tokens, p.Hkv, CH);
    if (!k.in_range) return;
    const int which = blockIdx.y;                       // 0 = K, 1 = V
    const int64_t layer = blockIdx.z;                   // owner layers of one launch, consecutive in the pool
    const int64_t row_chunks = (int64_t)p.Hkv * CH;
    const uint4 *src = (which ? p.V : p.K) + (layer * p.n_tokens + k.tok) * row_chunks + (int64_t)k.h * CH + k.c;
    // the row's piece and the token's slot are asked for together (neither address depends on the other: one
    // trip to memory instead of two, in a kernel that is nothing but that trip)
    const uint4 piece = __ldg(src);
    const int64_t slot = p.slot_map[k.tok];
    if (slot < 0) return;
    if (slot >= p.n_slots) {
        if (k.h == 0 && k.c == 0) atomicOr(p.status, STATUS_BOUNDS);
        return;
    }
    const int64_t page = slot / PAGE;
    const int off = (int)(slot - page * PAGE);
    uint8_t *dst = p.layer_base + layer * p.layer_stride + page * p.page_stride + (int64_t)k.h * block_bytes(p.D) +
                   (int64_t)which * half_bytes(p.D) + ((int64_t)k.c * PAGE + off) * 16;
    *reinterpret_cast<uint4 *>(dst) = piece;
}

// Large calls (a prompt): one warp per (group of 16 consecutive tokens of the call, kv head), grid.y = K or V,
// grid.z = owner layer.  The warp reads the group's 16 rows of that head as whole rows (two 256-byte rows per
// load instruction at head_dim 128: full lines, where the kernel above reads 32 bytes per token and
// instruction).  If the 16 tokens are the 16 slots of one page, in order -- what a prompt's tokens are -- the
// rows are turned into the page's chunk-major half through shared memory and written as one contiguous run
// (4 KB at head_dim 128); the shared-memory positions are XOR-swizzled so that neither the row-major writes
// nor the chunk-major reads conflict.  Any other slot pattern (loose tokens, holes, reversed pages, the
// ragged end of the call) takes the rows the same way and scatters their 16-byte chunks one by one, as the
// kernel above does: the same cache for every slot map.
constexpr int PAGE_WARPS = 8;

__global__ void __launch_bounds__(PAGE_WARPS * 32, 4) append_pages_kernel(AppendParams p)
{
    pdl_trigger();
    __shared__ __align__(16) uint4 stage[PAGE_WARPS][PAGE * 16];
    constexpr unsigned ALL = 0xFFFFFFFFu;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int CH = p.D / CHUNK_ELEMS;                     // 16-byte chunks per row of one head: 16 or 8
    const int rows_per_load = 32 / CH, loads = PAGE / rows_per_load;
    const int c = lane % CH, t_in_load = lane / CH;
    const int64_t n_groups = (p.n_tokens + PAGE - 1) / PAGE, n_items = n_groups * p.Hkv;
    const int which = blockIdx.y;
    const int64_t layer = blockIdx.z;
    const uint4 *rows = (which ? p.V : p.K) + layer * p.n_tokens * p.Hkv * CH;
    uint8_t *half = p.layer_base + layer * p.layer_stride + (int64_t)which * half_bytes(p.D);
    for (int64_t item = (int64_t)blockIdx.x * PAGE_WARPS + warp; item < n_items; item += (int64_t)gridDim.x * PAGE_WARPS) {
        const int64_t g = item / p.Hkv;
        const int h = (int)(item - g * p.Hkv);
        const int64_t i0 = g * PAGE;
        // the rows first (their addresses do not depend on the slots), so that both trips to memory overlap
        uint4 v[PAGE / 2];                                // at most 8 loads (head_dim 128)
#pragma unroll
        for (int i = 0; i < PAGE / 2; ++i) {
            const int64_t tok = i0 + i * rows_per_load + t_in_load;
            v[i] = (i < loads && tok < p.n_tokens) ? __ldg(rows + (tok * p.Hkv + h) * CH + c) : make_uint4(0u, 0u, 0u, 0u);
        }
        const int64_t mine = (lane < PAGE && i0 + lane < p.n_tokens) ? p.slot_map[i0 + lane] : -1;
        const int64_t first = __shfl_sync(ALL, mine, 0);
        const bool whole = __all_sync(ALL, lane >= PAGE || (first >= 0 && first % PAGE == 0 && first + PAGE <= p.n_slots &&
                                                             mine == first + lane));
        if (whole) {
#pragma unroll
            for (int i = 0; i < PAGE / 2; ++i)
                if (i < loads) {
                    const int t = i * rows_per_load + t_in_load;
                    stage[warp][c * PAGE + (t ^ (c & (PAGE - 1)))] = v[i];
                }
            __syncwarp();
            uint4 *dst = reinterpret_cast<uint4 *>(half + (first / PAGE) * p.page_stride + (int64_t)h * block_bytes(p.D));
            for (int u = lane; u < CH * PAGE; u += 32) {
                const int c2 = u / PAGE, t2 = u % PAGE;
                dst[u] = stage[warp][c2 * PAGE + (t2 ^ (c2 & (PAGE - 1)))];
            }
            __syncwarp();
        } else {
#pragma unroll
            for (int i = 0; i < PAGE / 2; ++i) {
                const int t = i * rows_per_load + t_in_load;             // (< PAGE also for i >= loads: a lane that exists)
                const int64_t slot = __shfl_sync(ALL, mine, t & (PAGE - 1));
                if (i >= loads || i0 + t >= p.n_tokens || slot < 0) continue;
                if (slot >= p.n_slots) {
                    if (h == 0 && c == 0 && which == 0) atomicOr(p.status, STATUS_BOUNDS);
                    continue;
                }
                const int64_t page = slot / PAGE;
                const int off = (int)(slot - page * PAGE);
                *reinterpret_cast<uint4 *>(half + page * p.page_stride + (int64_t)h * block_bytes(p.D) + ((int64_t)c * PAGE + off) * 16) = v[i];
            }
        }
    }
}

__global__ void __launch_bounds__(COPY_THREADS) gather_kernel(GatherParams p)
{
    const int CH = p.D / CHUNK_ELEMS;
    const CopyCoord k = coord_of(p.n, p.Hkv, CH);
    if (!k.in_range) return;
    const int64_t slot = p.slot_ids[k.tok];
    if (slot < 0) return;
    if (slot >= p.n_slots) {
        if (k.h == 0 && k.c == 0) atomicOr(p.status, STATUS_BOUNDS);
        return;
    }
    const int64_t page = slot / PAGE;
    const int off = (int)(slot - page * PAGE);
    const int which = blockIdx.y;
    const uint8_t *src = p.layer_base + page * p.page_stride + (int64_t)k.h * block_bytes(p.D) +
                         (int64_t)which * half_bytes(p.D) + ((int64_t)k.c * PAGE + off) * 16;
    uint4 *dst = (which ? p.V_out : p.K_out) + (k.tok * p.Hkv + k.h) * CH + k.c;
    *dst = *reinterpret_cast<const uint4 *>(src);
}

// ---- FP8 pages -----------------------------------------------------------------------------
// One row (token, kv head) by one warp: the D values are spread over the lanes (PER = D/32 each,
// dims lane*PER ..); amax by shuffles; scale = amax / 448, codes = E4M3(x * (448 / amax))
// round-to-nearest-even, saturating; every step a single fp32 operation.  Returns the lane's codes
// (c01: dims 0,1 of the lane, c23: dims 2,3) and the row's amax.
__device__ __forceinline__ void quantize_row(const uint16_t *row, int PER, int lane, uint32_t &c01, uint32_t &c23, float &amax)
{
    float x[4] = {0.f, 0.f, 0.f, 0.f};
    if (PER == 4) {
        const uint2 w = __ldg(reinterpret_cast<const uint2 *>(row + lane * 4));
        x[0] = bf16_lo(w.x); x[1] = bf16_hi(w.x); x[2] = bf16_lo(w.y); x[3] = bf16_hi(w.y);
    } else {
        const uint32_t w = __ldg(reinterpret_cast<const uint32_t *>(row + lane * 2));
        x[0] = bf16_lo(w); x[1] = bf16_hi(w);
    }
    amax = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
    const float inv = amax > 0.f ? __fdiv_rn(448.f, amax) : 0.f;
    c01 = pack_e4m3x2(__fmul_rn(x[0], inv), __fmul_rn(x[1], inv));
    c23 = pack_e4m3x2(__fmul_rn(x[2], inv), __fmul_rn(x[3], inv));
}

// The 16 rows of a whole page (tokens t0 .. t0+15 of the call, in slot order) by one warp, 16 bytes per store.
__device__ __forceinline__ void append_fp8_page(const AppendFp8Params &p, int64_t t0, int64_t page, int h, int which,
                                                int64_t layer, int lane)
{
    const int D = p.D, PER = D / 32;
    const uint16_t *rows = (which ? p.V : p.K) + (layer * p.n_tokens * p.Hkv + h) * D;      // row of token t: + t * Hkv * D
    uint8_t *blk = p.layer_base + layer * p.layer_stride + page * p.page_stride + (int64_t)h * fp8_block_bytes(D);
    if (which == 0) {
        // K: lane = (token q of this round, 16-dim chunk c); a chunk of a token is one 16-byte piece of the page
        const int CH = D / 16, TPI = 32 / CH;          // 8 chunks x 4 tokens per round at D = 128
        const int c = lane % CH, q = lane / CH;
        for (int t = q; t < PAGE; t += TPI) {
            const uint4 *src = reinterpret_cast<const uint4 *>(rows + (t0 + t) * p.Hkv * D + 16 * c);
            const uint4 a = __ldg(src), b = __ldg(src + 1);
            const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
            float x[16];
            float amax = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                x[2 * i] = bf16_lo(w[i]);
                x[2 * i + 1] = bf16_hi(w[i]);
                amax = fmaxf(amax, fmaxf(fabsf(x[2 * i]), fabsf(x[2 * i + 1])));
            }
            for (int d = 1; d < CH; d <<= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
            const float inv = amax > 0.f ? __fdiv_rn(448.f, amax) : 0.f;
            uint32_t o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                o[i] = pack_e4m3x2(__fmul_rn(x[4 * i], inv), __fmul_rn(x[4 * i + 1], inv)) |
                       (pack_e4m3x2(__fmul_rn(x[4 * i + 2], inv), __fmul_rn(x[4 * i + 3], inv)) << 16);
            *reinterpret_cast<uint4 *>(blk + fp8_k_pos(D, t, 16 * c)) = make_uint4(o[0], o[1], o[2], o[3]);
            if (c == 0) *reinterpret_cast<float *>(blk + fp8_ks_off(D) + 4 * t) = __fdiv_rn(amax, 448.f);
        }
        return;
    }
    uint32_t v[4][4] = {};                 // [dim of the lane][4 tokens per word]
    float my_scale = 0.f;
#pragma unroll
    for (int t = 0; t < PAGE; ++t) {
        uint32_t c01, c23;
        float amax;
        quantize_row(rows + (t0 + t) * p.Hkv * D, PER, lane, c01, c23, amax);
        const int sh = 8 * (t & 3);
        v[0][t >> 2] |= (c01 & 0xFFu) << sh;
        v[1][t >> 2] |= (c01 >> 8) << sh;
        v[2][t >> 2] |= (c23 & 0xFFu) << sh;
        v[3][t >> 2] |= (c23 >> 8) << sh;
        if (lane == t) my_scale = __fdiv_rn(amax, 448.f);
    }
    uint4 *dst = reinterpret_cast<uint4 *>(blk + fp8_v_off(D) + (lane * PER) * PAGE);
#pragma unroll
    for (int d = 0; d < 4; ++d)
        if (d < PER) dst[d] = make_uint4(v[d][0], v[d][1], v[d][2], v[d][3]);
    if (lane < PAGE) *reinterpret_cast<float *>(blk + fp8_vs_off(D) + 4 * lane) = my_scale;
}

// The same page, all 16 rows at once (the large-call kernel).  The rows come in as whole rows (coalesced)
// through shared memory; then lane (token t = lane % 16, half hf = lane / 16) owns half a row: its maximum
// needs ONE shuffle with the other half's (instead of five per row, row after row), and it quantises D/2
// values.  K codes leave as the 16-byte pieces of the page layout; V codes are turned dim-major through shared
// memory (a piece = one dim x 16 tokens).  in_rows: PAGE x (2 D + 16) bytes, codes: PAGE x (D + 4) bytes of
// shared memory of this warp (the paddings keep the column accesses off one bank).
__device__ __forceinline__ void append_fp8_page_wide(const AppendFp8Params &p, int64_t t0, int64_t page, int h, int which,
                                                     int64_t layer, int lane, uint8_t *in_rows, uint8_t *codes)
{
    const int D = p.D, row_bytes = 2 * D, in_stride = row_bytes + 16, code_stride = D + 4;
    const uint16_t *rows = (which ? p.V : p.K) + (layer * p.n_tokens * p.Hkv + h) * D;      // row of token t: + t * Hkv * D
    uint8_t *blk = p.layer_base + layer * p.layer_stride + page * p.page_stride + (int64_t)h * fp8_block_bytes(D);
    // ---- rows -> shared memory: 32 lanes x 16 bytes per load, PAGE * row_bytes / 512 loads (8 at head_dim 128)
    const int units = row_bytes / 16, n_loads = PAGE * units / 32;
    uint4 v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
        if (i < n_loads) {
            const int u = i * 32 + lane, r = u / units, cu = u - r * units;
            v[i] = __ldg(reinterpret_cast<const uint4 *>(rows + (t0 + r) * p.Hkv * D) + cu);
        }
#pragma unroll
    for (int i = 0; i < 8; ++i)
        if (i < n_loads) {
            const int u = i * 32 + lane, r = u / units, cu = u - r * units;
            *reinterpret_cast<uint4 *>(in_rows + r * in_stride + cu * 16) = v[i];
        }
    __syncwarp();
    // ---- half a row per lane: maximum and scale (a first pass over the lane's values in shared memory) ...
    const int t = lane & 15, hf = lane >> 4, half_vals = D / 2;                    // 64 or 32 values
    const uint8_t *mine = in_rows + t * in_stride + hf * D;                        // (D bytes = D/2 bf16)
    float amax = 0.f;
    for (int i = 0; i < half_vals / 8; ++i) {
        const uint4 q = *reinterpret_cast<const uint4 *>(mine + 16 * i);
        amax = fmaxf(amax, fmaxf(fmaxf(fabsf(bf16_lo(q.x)), fabsf(bf16_hi(q.x))), fmaxf(fabsf(bf16_lo(q.y)), fabsf(bf16_hi(q.y)))));
        amax = fmaxf(amax, fmaxf(fmaxf(fabsf(bf16_lo(q.z)), fabsf(bf16_hi(q.z))), fmaxf(fabsf(bf16_lo(q.w)), fabsf(bf16_hi(q.w)))));
    }
    amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 16));
    const float inv = amax > 0.f ? __fdiv_rn(448.f, amax) : 0.f;
    if (hf == 0) *reinterpret_cast<float *>(blk + (which ? fp8_vs_off(D) : fp8_ks_off(D)) + 4 * t) = __fdiv_rn(amax, 448.f);
    // ... and the codes (a second pass), 16 values = one 16-byte piece of codes at a time
    auto piece = [&](int j) -> uint4 {                                             // values 16j .. 16j+15 of the lane's half
        const uint4 a = *reinterpret_cast<const uint4 *>(mine + 32 * j), b2 = *reinterpret_cast<const uint4 *>(mine + 32 * j + 16);
        const uint32_t wv[8] = {a.x, a.y, a.z, a.w, b2.x, b2.y, b2.z, b2.w};
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            o[i] = pack_e4m3x2(__fmul_rn(bf16_lo(wv[2 * i]), inv), __fmul_rn(bf16_hi(wv[2 * i]), inv)) |
                   (pack_e4m3x2(__fmul_rn(bf16_lo(wv[2 * i + 1]), inv), __fmul_rn(bf16_hi(wv[2 * i + 1]), inv)) << 16);
        return make_uint4(o[0], o[1], o[2], o[3]);
    };
    if (which == 0) {
        // K: 16 dims of a token are one 16-byte piece of the page; the lane has half_vals / 16 of them
        for (int j = 0; j < half_vals / 16; ++j)
            *reinterpret_cast<uint4 *>(blk + fp8_k_pos(D, t, hf * half_vals + 16 * j)) = piece(j);
        __syncwarp();                                                              // (in_rows is free again)
        return;
    }
    // V: token-major codes into shared memory, dim-major pieces out
    for (int j = 0; j < half_vals / 16; ++j) {
        const uint4 o = piece(j);
        uint32_t *dstw = reinterpret_cast<uint32_t *>(codes + t * code_stride + hf * half_vals + 16 * j);   // (4-byte aligned rows)
        dstw[0] = o.x; dstw[1] = o.y; dstw[2] = o.z; dstw[3] = o.w;
    }
    __syncwarp();
    for (int d = lane; d < D; d += 32) {
        uint32_t o[4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
            o[q] = (uint32_t)codes[(4 * q) * code_stride + d] | ((uint32_t)codes[(4 * q + 1) * code_stride + d] << 8) |
                   ((uint32_t)codes[(4 * q + 2) * code_stride + d] << 16) | ((uint32_t)codes[(4 * q + 3) * code_stride + d] << 24);
        *reinterpret_cast<uint4 *>(blk + fp8_v_off(D) + d * PAGE) = make_uint4(o[0], o[1], o[2], o[3]);
    }
    __syncwarp();
}

// 4 x 4 bytes transposed: word i of the input holds bytes [i][0..3], word j of the output bytes [0..3][j]
__device__ __forceinline__ void transpose_4x4_bytes(uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                    uint32_t &o0, uint32_t &o1, uint32_t &o2, uint32_t &o3)
{
    const uint32_t t0 = __byte_perm(a0, a1, 0x5140), t1 = __byte_perm(a0, a1, 0x7362);
    const uint32_t t2 = __byte_perm(a2, a3, 0x5140), t3 = __byte_perm(a2, a3, 0x7362);
    o0 = __byte_perm(t0, t2, 0x5410);
    o1 = __byte_perm(t0, t2, 0x7632);
    o2 = __byte_perm(t1, t3, 0x5410);
    o3 = __byte_perm(t1, t3, 0x7632);
}

// A whole page at head_dim 128 in registers only.  Lane = (token r of a round of four, 16-dim chunk c):
// in round k the lane holds dims 16c .. 16c+15 of token 4k + r, read as 32 contiguous bytes (a warp-wide load
// covers four whole rows).  A row's maximum is three shuffles among the eight lanes of the row.  K: the lane's
// 16 codes ARE one 16-byte piece of the page.  V (dim-major pages): the four lanes that share a chunk swap
// words so that lane r ends up with dims 16c+4r .. 16c+4r+3 of all 16 tokens (two exchange steps of a
// four-way transpose per round, then byte transposes in registers), 64 contiguous bytes of the page.
__device__ __forceinline__ void append_fp8_page_regs128(const AppendFp8Params &p, int64_t t0, int64_t page, int h, int which,
                                                        int64_t layer, int lane)
{
    constexpr int D = 128;
    constexpr unsigned ALL = 0xFFFFFFFFu;
    const uint16_t *rows = (which ? p.V : p.K) + (layer * p.n_tokens * p.Hkv + h) * D;      // row of token t: + t * Hkv * D
    uint8_t *blk = p.layer_base + layer * p.layer_stride + page * p.page_stride + (int64_t)h * fp8_block_bytes(D);
    const int c = lane & 7, r = lane >> 3;
    uint4 in[4][2];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint4 *src = reinterpret_cast<const uint4 *>(rows + (t0 + 4 * k + r) * p.Hkv * D + 16 * c);
        in[k][0] = __ldg(src);
        in[k][1] = __ldg(src + 1);
    }
    uint32_t code[4][4];                   // [round][dim quad of the chunk]: four codes per word
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t w[8] = {in[k][0].x, in[k][0].y, in[k][0].z, in[k][0].w, in[k][1].x, in[k][1].y, in[k][1].z, in[k][1].w};
        float amax = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fmaxf(fabsf(bf16_lo(w[i])), fabsf(bf16_hi(w[i]))));
        amax = fmaxf(amax, __shfl_xor_sync(ALL, amax, 1));
        amax = fmaxf(amax, __shfl_xor_sync(ALL, amax, 2));
        amax = fmaxf(amax, __shfl_xor_sync(ALL, amax, 4));
        const float inv = amax > 0.f ? __fdiv_rn(448.f, amax) : 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            code[k][j] = pack_e4m3x2(__fmul_rn(bf16_lo(w[2 * j]), inv), __fmul_rn(bf16_hi(w[2 * j]), inv)) |
                         (pack_e4m3x2(__fmul_rn(bf16_lo(w[2 * j + 1]), inv), __fmul_rn(bf16_hi(w[2 * j + 1]), inv)) << 16);
        if (c == 0)
            *reinterpret_cast<float *>(blk + (which ? fp8_vs_off(D) : fp8_ks_off(D)) + 4 * (4 * k + r)) = __fdiv_rn(amax, 448.f);
    }
    if (which == 0) {
#pragma unroll
        for (int k = 0; k < 4; ++k)
            *reinterpret_cast<uint4 *>(blk + fp8_k_pos(D, 4 * k + r, 16 * c)) = make_uint4(code[k][0], code[k][1], code[k][2], code[k][3]);
        return;
    }
    // four-way transpose of the dim quads across the lanes r = 0..3 of a chunk: afterwards code[k][q] of lane r is
    // what lane q held as code[k][r] (token 4k + q, dims 16c + 4r ..)
#pragma unroll
    for (int bit = 0; bit < 2; ++bit) {
        const bool up = (r >> bit) & 1;
#pragma unroll
        for (int k = 0; k < 4; ++k)
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (!((j >> bit) & 1)) {
                    const int jl = j, jh = j | (1 << bit);
                    const uint32_t give = up ? code[k][jl] : code[k][jh];
                    const uint32_t got = __shfl_xor_sync(ALL, give, 8 << bit);
                    if (up) code[k][jl] = got;
                    else code[k][jh] = got;
                }
    }
    // bytes: round k's four words (tokens 4k .. 4k+3) -> word k of each of the lane's four dims
    uint32_t piece[4][4];                  // [dim of the lane][tokens 4k .. 4k+3]
#pragma unroll
    for (int k = 0; k < 4; ++k)
        transpose_4x4_bytes(code[k][0], code[k][1], code[k][2], code[k][3], piece[0][k], piece[1][k], piece[2][k], piece[3][k]);
    uint4 *dst = reinterpret_cast<uint4 *>(blk + fp8_v_off(D) + (16 * c + 4 * r) * PAGE);
#pragma unroll
    for (int b = 0; b < 4; ++b) dst[b] = make_uint4(piece[b][0], piece[b][1], piece[b][2], piece[b][3]);
}

// One row (token tok at offset off of its page) by one warp: scattered small stores (V is dim-major: one byte
// in each of D rows; K: 4 bytes per lane).
__device__ __forceinline__ void append_fp8_token(const AppendFp8Params &p, int64_t tok, int64_t page, int off, int h,
                                                 int which, int64_t layer, int lane)
{
    const int D = p.D, PER = D / 32;                  // 4 values per lane at D = 128, 2 at D = 64
    const uint16_t *rows = (which ? p.V : p.K) + (layer * p.n_tokens * p.Hkv + h) * D;
    uint8_t *blk = p.layer_base + layer * p.layer_stride + page * p.page_stride + (int64_t)h * fp8_block_bytes(D);
    uint32_t c01, c23;
    float amax;
    quantize_row(rows + tok * p.Hkv * D, PER, lane, c01, c23, amax);
    if (which == 0) {                                  // K: a lane's dims are neighbours inside one 16-byte piece
        uint8_t *dst = blk + fp8_k_pos(D, off, lane * PER);
        if (PER == 4) *reinterpret_cast<uint32_t *>(dst) = c01 | (c23 << 16);
        else *reinterpret_cast<uint16_t *>(dst) = (uint16_t)c01;
    } else {                                           // V: dim-major, this token's column
        uint8_t *dst = blk + fp8_v_off(D) + (lane * PER) * PAGE + off;
        dst[0] = (uint8_t)(c01 & 0xFF);
        dst[PAGE] = (uint8_t)(c01 >> 8);
        if (PER == 4) {
            dst[2 * PAGE] = (uint8_t)(c23 & 0xFF);
            dst[3 * PAGE] = (uint8_t)(c23 >> 8);
        }
    }
    if (lane == 0)
        *reinterpret_cast<float *>(blk + (which ? fp8_vs_off(D) : fp8_ks_off(D)) + 4 * off) = __fdiv_rn(amax, 448.f);
}

// Small calls (a decode step: one token per sequence): one warp per (token, kv head) row, the warps of a
// bounded grid looping over the rows; grid.y picks K or V, grid.z the owner layer.  When the 16 tokens of a
// whole page do arrive together and in order, the warp of the page's first row does the page and the other
// 15 rows have nothing to do.
__global__ void __launch_bounds__(COPY_THREADS) append_fp8_kernel(AppendFp8Params p)
{
    pdl_trigger();
    pdl_wait();         // (as in append_kernel)
    const int lane = threadIdx.x & 31;
    // (rows counted head-major and an odd number of warps in the grid: a warp then meets every position inside
    // a page in turn, instead of always the pages' first rows or never one)
    const int64_t n_rows = p.n_tokens * p.Hkv, stride = (int64_t)gridDim.x * (blockDim.x >> 5);
    for (int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); warp < n_rows; warp += stride) {
        const int h = (int)(warp / p.n_tokens);
        const int64_t tok = warp - (int64_t)h * p.n_tokens;
        const int64_t slot = p.slot_map[tok];
        if (slot < 0) continue;
        if (slot >= p.n_slots) {
            if (h == 0 && lane == 0) atomicOr(p.status, STATUS_BOUNDS);
            continue;
        }
        const int64_t page = slot / PAGE;
        const int off = (int)(slot - page * PAGE);
        // do tokens tok-off .. tok-off+15 of this call carry the page's 16 slots in order?
        const int64_t t0 = tok - off;
        bool whole_page = t0 >= 0 && t0 + PAGE <= p.n_tokens;
        if (whole_page) {
            const int64_t s_l = lane < PAGE ? p.slot_map[t0 + lane] : 0;
            whole_page = __all_sync(0xFFFFFFFFu, lane >= PAGE || s_l == page * PAGE + lane);
        }
        if (!whole_page) append_fp8_token(p, tok, page, off, h, (int)blockIdx.y, blockIdx.z, lane);
        else if (off == 0) append_fp8_page(p, t0, page, h, (int)blockIdx.y, blockIdx.z, lane);
    }
}

// Large calls (a prompt): one warp per (group of 16 consecutive tokens of the call, kv head).  The warp looks at
// the slots of its tokens and of the 15 tokens on either side, finds the whole page that starts inside its group
// (at most one: its 16 tokens arrive together and in slot order), does that page 16 bytes per store, and does
// its tokens that belong to no whole page one row at a time.  Same result as the kernel above for any slot map.
constexpr int FP8_GROUP_WARPS = 7;
constexpr int FP8_IN_BYTES = PAGE * (2 * 128 + 16), FP8_CODE_BYTES = PAGE * (128 + 4);     // per warp, head_dim <= 128

// REGS128: head_dim 128, whole pages in registers (no shared memory, more warps per SM); otherwise through shared memory.
template <bool REGS128>
__global__ void __launch_bounds__(FP8_GROUP_WARPS * 32, REGS128 ? 4 : 3) append_fp8_groups_kernel(AppendFp8Params p)
{
    pdl_trigger();
    __shared__ __align__(16) uint8_t wide_in[REGS128 ? 1 : FP8_GROUP_WARPS][REGS128 ? 16 : FP8_IN_BYTES];
    __shared__ __align__(16) uint8_t wide_codes[REGS128 ? 1 : FP8_GROUP_WARPS][REGS128 ? 16 : FP8_CODE_BYTES];
    constexpr unsigned ALL = 0xFFFFFFFFu;
    const int lane = threadIdx.x & 31;
    const int64_t n_groups = (p.n_tokens + PAGE - 1) / PAGE, n_items = n_groups * p.Hkv;
    const int64_t stride = (int64_t)gridDim.x * (blockDim.x >> 5);
    for (int64_t item = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); item < n_items; item += stride) {
        const int h = (int)(item / n_groups);
        const int64_t i0 = (item - (int64_t)h * n_groups) * PAGE;
        if (REGS128 && i0 + PAGE <= p.n_tokens) {
            // the usual case first: the group's 16 tokens are one page, in order, from its first slot on
            const long long s_l = (long long)p.slot_map[i0 + (lane & 15)];
            const long long s_0 = __shfl_sync(ALL, s_l, 0);
            if (s_0 >= 0 && (s_0 & (PAGE - 1)) == 0 && s_0 + PAGE <= p.n_slots && __all_sync(ALL, s_l == s_0 + (lane & 15))) {
                append_fp8_page_regs128(p, i0, s_0 / PAGE, h, (int)blockIdx.y, blockIdx.z, lane);
                continue;
            }
        }
        // slots of tokens i0-15 .. i0+30: window index x = -15 .. 16 in w0 (lane x+15), 17 .. 30 in w1 (lane x-17)
        auto slot_of = [&](int64_t i) -> long long { return (i >= 0 && i < p.n_tokens) ? (long long)p.slot_map[i] : -1ll; };
        const long long w0 = slot_of(i0 - 15 + lane), w1 = lane < 14 ? slot_of(i0 + 17 + lane) : -1ll;
        auto at = [&](int x) -> long long {               // every lane calls it (with its own x)
            const long long a = __shfl_sync(ALL, w0, (x + 15) & 31), b = __shfl_sync(ALL, w1, (x - 17) & 31);
            return x <= 16 ? a : b;
        };
        const int l = lane & 15;                          // lanes 16..31 repeat lanes 0..15
        const long long mine = at(l);
        const bool valid = i0 + l < p.n_tokens && mine >= 0 && mine < p.n_slots;
        if (lane < PAGE && i0 + l < p.n_tokens && mine >= p.n_slots && h == 0 && blockIdx.y == 0) atomicOr(p.status, STATUS_BOUNDS);
        const int off = (int)(mine & (PAGE - 1));
        const int c = l - off;                            // where the token's page would start in the window (>= -15)
        bool covered = valid;
#pragma unroll
        for (int k = 0; k < PAGE; ++k) covered = (at(c + k) == mine - off + k) && covered;
        const unsigned starts = __ballot_sync(ALL, lane < PAGE && covered && off == 0);
        const unsigned loose = __ballot_sync(ALL, lane < PAGE && valid && !covered);
        if (starts) {
            const int ls = __ffs(starts) - 1;
            const long long s0 = __shfl_sync(ALL, mine, ls);
            if (REGS128) append_fp8_page_regs128(p, i0 + ls, s0 / PAGE, h, (int)blockIdx.y, blockIdx.z, lane);
            else append_fp8_page_wide(p, i0 + ls, s0 / PAGE, h, (int)blockIdx.y, blockIdx.z, lane, wide_in[threadIdx.x >> 5],
                                      wide_codes[threadIdx.x >> 5]);
        }
        for (unsigned m = loose; m; m &= m - 1) {
            const int lt = __ffs(m) - 1;
            const long long st = __shfl_sync(ALL, mine, lt);
            append_fp8_token(p, i0 + lt, st / PAGE, (int)(st & (PAGE - 1)), h, (int)blockIdx.y, blockIdx.z, lane);
        }
    }
}

// read-back: codes as [n][Hkv][D] for both K and V, scales as [n][Hkv]
__global__ void __launch_bounds__(COPY_THREADS) gather_fp8_kernel(GatherFp8Params p)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * COPY_THREADS + threadIdx.x) >> 5;
    if (warp >= p.n * p.Hkv) return;
    const int64_t tok = warp / p.Hkv;
    const int h = (int)(warp - tok * p.Hkv);
    const int64_t slot = p.slot_ids[tok];
    if (slot < 0) return;
    if (slot >= p.n_slots) {
        if (h == 0 && lane == 0) atomicOr(p.status, STATUS_BOUNDS);
        return;
    }
    const int64_t page = slot / PAGE;
    const int off = (int)(slot - page * PAGE);
    const int which = blockIdx.y;
    const int D = p.D;
    const uint8_t *blk = p.layer_base + page * p.page_stride + (int64_t)h * fp8_block_bytes(D);
    uint8_t *out = (which ? p.V_codes : p.K_codes) + (tok * p.Hkv + h) * D;
    for (int d = lane; d < D; d += 32)
        out[d] = which ? blk[fp8_v_off(D) + d * PAGE + off] : blk[fp8_k_pos(D, off, d)];
    if (lane == 0)
        (which ? p.V_scales : p.K_scales)[tok * p.Hkv + h] =
            *reinterpret_cast<const float *>(blk + (which ? fp8_vs_off(D) : fp8_ks_off(D)) + 4 * off);
}

// blocks needed for n tokens: one warp per (16 tokens, head, chunk pair)
int64_t copy_blocks(int64_t n, int Hkv, int D)
{
    const int64_t warps = ((n + 15) / 16) * Hkv * (D / CHUNK_ELEMS / 2);
    return (warps * 32 + COPY_THREADS - 1) / COPY_THREADS;
}

}  // namespace

// n_layers consecutive owner layers (grid.z) take rows from K/V [n_layers][n_tokens][Hkv][D] with one slot map
cudaError_t launch_append(const AppendParams &p, int n_layers, bool pdl, cudaStream_t s)
{
    const int64_t blocks = copy_blocks(p.n_tokens, p.Hkv, p.D);
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    if (n_layers < 1 || n_layers > 65535) return cudaErrorInvalidConfiguration;
    if (p.n_tokens >= 256) {                              // a prompt: rows read whole, pages written whole
        const int64_t items = ((p.n_tokens + PAGE - 1) / PAGE) * p.Hkv;
        int64_t ctas = (items + PAGE_WARPS - 1) / PAGE_WARPS;
        if (ctas > 65535 * 4) ctas = 65535 * 4;           // (the warps loop over their items)
        append_pages_kernel<<<dim3((unsigned)ctas, 2, (unsigned)n_layers), PAGE_WARPS * 32, 0, s>>>(p);
        return cudaGetLastError();
    }
    // A decode step's rows: with the attribute the launch may be brought forward to where the kernel before it
    // releases its dependents (the kernel waits for that kernel's end itself before it touches anything).
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks, 2, (unsigned)n_layers);
    cfg.blockDim = dim3(COPY_THREADS);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, append_kernel, p);
}

cudaError_t launch_gather(const GatherParams &p, cudaStream_t s)
{
    const int64_t blocks = copy_blocks(p.n, p.Hkv, p.D);
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    gather_kernel<<<dim3((unsigned)blocks, 2), COPY_THREADS, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace skv

namespace skv {

cudaError_t launch_append_fp8(const AppendFp8Params &p, int n_layers, bool pdl, cudaStream_t s)
{
    if (p.n_tokens == 0) return cudaSuccess;
    if (n_layers < 1 || n_layers > 65535) return cudaErrorInvalidConfiguration;
    // 7 warps per CTA and at most 4095 CTAs: the kernels' warps loop over their items, and 7 x 4095 is odd
    const bool groups = p.n_tokens >= 512;
    const int64_t items = groups ? ((p.n_tokens + PAGE - 1) / PAGE) * p.Hkv : p.n_tokens * p.Hkv;
    int64_t blocks = (items + 6) / 7;
    if (blocks > 4095) blocks = 4095;
    const dim3 grid((unsigned)blocks, 2, (unsigned)n_layers);
    if (groups && p.D == 128) append_fp8_groups_kernel<true><<<grid, 224, 0, s>>>(p);
    else if (groups) append_fp8_groups_kernel<false><<<grid, 224, 0, s>>>(p);
    else {                                                // a decode step's rows (launched as append_kernel is)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = grid;
        cfg.blockDim = dim3(224);
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = pdl ? 1 : 0;
        return cudaLaunchKernelEx(&cfg, append_fp8_kernel, p);
    }
    return cudaGetLastError();
}

cudaError_t launch_gather_fp8(const GatherFp8Params &p, cudaStream_t s)
{
    const int64_t warps = p.n * p.Hkv;
    const int64_t blocks = (warps * 32 + 255) / 256;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    gather_fp8_kernel<<<dim3((unsigned)blocks, 2), 256, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace skv
