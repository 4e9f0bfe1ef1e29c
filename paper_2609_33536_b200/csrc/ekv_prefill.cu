// Chunked-prefill attention over a mixed-fidelity paged prefix (dense QK^T / PV tiles).
//
// CTA = (request, kv head, tile of 64 query rows); a row is (query token, query head of the
// group), so the G heads that share a kv head are packed into the M dimension and every K/V
// tile fetched from HBM serves all of them. 4 warps x 16 rows. The KV axis is walked in tiles
// of 64 tokens (4 pages), double-buffered in shared memory with cp.async:
//   TARGET page : 16-byte chunks copied straight into the bf16 tile (XOR-swizzled rows);
//   BASE page   : the packed bytes are copied into a raw staging area and expanded
//                 (byte << 8, Sec. 3.2 / App. B.3 load rule) into the same bf16 tile, so the MMA
//                 loop is identical for both modes.
// S = QK^T and O += PV run on tensor cores (mma.sync m16n8k16, bf16 in, fp32 accumulate) with
// ldmatrix-fed operands, online softmax in registers, causal mask only on tiles that reach the
// diagonal. Rows past the end of the sequence are zero-filled in the tile.
#include "ekv_common.cuh"
#include <math.h>

namespace ekv {

constexpr int kPfThreads = 128;
constexpr int kPfRows = 64;        // query rows per CTA
constexpr int kPfKv = 64;          // KV tokens per tile
constexpr int kPfMaxPages = 8192;  // block-table entries kept in shared memory (131072 tokens)

struct PrefillParams {
    const uint8_t *k_layer, *v_layer;
    const uint8_t *tags;
    const int32_t *block_table, *seq_lens, *q_start;
    const __nv_bfloat16 *q;
    __nv_bfloat16 *out;
    int64_t block_bytes;
    int batch, num_q_heads, num_kv_heads, group, max_blocks;
    int group_rows;                    // rows a token takes in a tile: the group size rounded up to a power of two
    int q_tiles;                       // tiles per request: ceil(max_q_len / (64 / group_rows))
    float scale_log2;
    int out_f32;                       // debug: `out` is float and receives the unrounded result
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}

template <int D>
struct PfSmem {
    static constexpr int kRowB = D * 2;                 // bytes per token row of a bf16 tile
    static constexpr int kTile = kPfKv * kRowB;         // one K or V tile
    static constexpr int kRaw = kPfKv * D;              // packed bytes of one K or V tile
    static constexpr int kStage = 2 * kTile + 2 * kRaw; // K, V, raw K, raw V
    static constexpr int kTotal = 2 * kStage;
};

template <int D, bool HAS_BASE, bool F16>
__global__ void __launch_bounds__(kPfThreads, 2) prefill_chunk_kernel(PrefillParams p)
{
    using SM = PfSmem<D>;
    constexpr int CPR = D / 8;          // 16-byte chunks per bf16 row
    constexpr int KS = D / 16;          // k-steps of QK^T
    constexpr int NT = D / 8;           // n-tiles of the output
    extern __shared__ __align__(128) uint8_t smem[];
    int32_t *pages = (int32_t *)(smem + SM::kTotal);      // (phys << 1 | tag) per logical block

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int c = lane >> 2, j = lane & 3;
    // A token's query heads of this kv head take group_rows consecutive rows (the group size rounded up
    // to a power of two); rows past the real group are dead: zero queries, fully masked, no store.
    const int G = p.group, Gp = p.group_rows;
    const int tok_m = kPfRows / Gp;                       // query tokens per tile

    int idx = blockIdx.x;
    const int qt = p.q_tiles - 1 - idx % p.q_tiles; idx /= p.q_tiles;   // longest KV ranges first
    const int g = idx % p.num_kv_heads;
    const int r = idx / p.num_kv_heads;
    const int qs = p.q_start[r];
    const int C = p.q_start[r + 1] - qs;
    const int L = p.seq_lens[r];
    const int i0 = qt * tok_m;                            // first query token of the tile
    if (i0 >= C) return;
    const int i1 = min(C, i0 + tok_m);
    const int n_kv = L - C + i1;                          // tokens visible to the last row of the tile
    const int n_tiles = (n_kv + kPfKv - 1) / kPfKv;
    const int n_pages = (n_kv + kPageSize - 1) / kPageSize;

    // block-table entries (and tags) of the visible range
    for (int lb = tid; lb < n_pages; lb += kPfThreads) {
        const int phys = p.block_table[(int64_t)r * p.max_blocks + lb];
        int tag = 0;
        if (HAS_BASE) tag = p.tags[phys];
        pages[lb] = (phys << 1) | tag;
    }

    // Q fragments of this warp's 16 rows: row m = 16*warp + c (+8); token i0 + m / Gp, head m % Gp.
    uint32_t qa[KS][4];
    int row_pos[2];                                       // causal limit of the two rows of this lane
    {
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            const int m = 16 * warp + c + 8 * hf;
            const int i = i0 + m / Gp, hl = m % Gp;
            const bool ok = i < C && hl < G;
            const int h = g * G + (ok ? hl : 0);
            row_pos[hf] = ok ? (L - C + i) : -1;
            const uint32_t *src = (const uint32_t *)(p.q + ((int64_t)(qs + (ok ? i : 0)) * p.num_q_heads + h) * D);
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                qa[ks][hf] = ok ? src[8 * ks + j] : 0u;              // k = 16ks + 2j, +1
                qa[ks][2 + hf] = ok ? src[8 * ks + 4 + j] : 0u;      // k + 8
            }
        }
    }
    __syncthreads();

    const int64_t slab = (int64_t)g * (kPageSize * D * 2);
    auto issue_tile = [&](int t, int stage) {
        uint8_t *st = smem + stage * SM::kStage;
        const uint32_t ks_ = smem_u32(st), vs_ = smem_u32(st + SM::kTile);
        const uint32_t kraw = smem_u32(st + 2 * SM::kTile), vraw = kraw + SM::kRaw;
#pragma unroll
        for (int pg = 0; pg < kPfKv / kPageSize; ++pg) {
            const int lb = t * (kPfKv / kPageSize) + pg;
            const int valid = min(kPageSize, L - lb * kPageSize);     // rows of this page that exist
            const int e = lb < n_pages ? pages[lb] : 0;
            const int64_t blk = (int64_t)(e >> 1) * p.block_bytes + slab;
            if (HAS_BASE && (e & 1) && lb < n_pages) {
                // packed bytes -> raw staging (16 rows x D bytes), expanded after arrival
                const int64_t mem = blk + (int64_t)(lb & 1) * (kPageSize * D);
                for (int id = tid; id < kPageSize * (D / 16); id += kPfThreads) {
                    const int tok = id / (D / 16), ch = id % (D / 16);
                    const int bytes = tok < valid ? 16 : 0;
                    const uint32_t off = (uint32_t)((pg * kPageSize + tok) * D + ch * 16);
                    cp_async16(kraw + off, p.k_layer + mem + tok * D + ch * 16, bytes);
                    cp_async16(vraw + off, p.v_layer + mem + tok * D + ch * 16, bytes);
                }
            } else {
                for (int id = tid; id < kPageSize * CPR; id += kPfThreads) {
                    const int tok = id / CPR, ch = id % CPR;
                    const int bytes = (lb < n_pages && tok < valid) ? 16 : 0;     // zero-fill what does not exist
                    const int trow = pg * kPageSize + tok;
                    const uint32_t off = (uint32_t)(trow * SM::kRowB + ((ch ^ (trow & 7)) << 4));
                    cp_async16(ks_ + off, p.k_layer + blk + tok * (D * 2) + ch * 16, bytes);
                    cp_async16(vs_ + off, p.v_layer + blk + tok * (D * 2) + ch * 16, bytes);
                }
            }
        }
        cp_async_commit();
    };
    auto expand_tile = [&](int t, int stage) {            // BASE pages: raw bytes -> bf16 tile rows
        uint8_t *st = smem + stage * SM::kStage;
        bool any = false;
#pragma unroll
        for (int pg = 0; pg < kPfKv / kPageSize; ++pg) {
            const int lb = t * (kPfKv / kPageSize) + pg;
            if (!(lb < n_pages && (pages[lb] & 1))) continue;
            any = true;
            for (int id = tid; id < kPageSize * (D / 16); id += kPfThreads) {
                const int tok = id / (D / 16), ch = id % (D / 16);
                const int trow = pg * kPageSize + tok;
#pragma unroll
                for (int tensor = 0; tensor < 2; ++tensor) {
                    const uint4 x = *(const uint4 *)(st + 2 * SM::kTile + tensor * SM::kRaw + trow * D + ch * 16);
                    uint4 lo, hi;
                    lo.x = prmt(x.x, 0u, 0x1404); lo.y = prmt(x.x, 0u, 0x3424);
                    lo.z = prmt(x.y, 0u, 0x1404); lo.w = prmt(x.y, 0u, 0x3424);
                    hi.x = prmt(x.z, 0u, 0x1404); hi.y = prmt(x.z, 0u, 0x3424);
                    hi.z = prmt(x.w, 0u, 0x1404); hi.w = prmt(x.w, 0u, 0x3424);
                    uint8_t *row = st + tensor * SM::kTile + trow * SM::kRowB;
                    *(uint4 *)(row + (((2 * ch) ^ (trow & 7)) << 4)) = lo;
                    *(uint4 *)(row + (((2 * ch + 1) ^ (trow & 7)) << 4)) = hi;
                }
            }
        }
        return any;
    };

    float o[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    const int pos_min = L - C + i0;                       // smallest causal limit in the tile

    if (n_tiles > 0) issue_tile(0, 0);
    for (int t = 0; t < n_tiles; ++t) {
        const int stage = t & 1;
        cp_async_wait<0>();
        __syncthreads();                                  // tile t landed; everyone is done with tile t-1
        if (t + 1 < n_tiles) issue_tile(t + 1, stage ^ 1);
        if (HAS_BASE) {
            if (expand_tile(t, stage)) __syncthreads();   // uniform over the CTA
        }
        const uint32_t ks_ = smem_u32(smem + stage * SM::kStage), vs_ = ks_ + SM::kTile;
        const int kv0 = t * kPfKv;

        // ---- S = Q K^T : 16 rows x 64 tokens ----
        float s[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) { s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                const int mi = lane >> 3, rr = lane & 7;
                const int tok = 16 * np + rr + (mi >> 1) * 8, ch = 2 * ks + (mi & 1);
                uint32_t b0, b1, b2, b3;
                ldsm_x4(ks_ + tok * SM::kRowB + ((ch ^ (tok & 7)) << 4), b0, b1, b2, b3);
                mma_16816<F16>(s[2 * np][0], s[2 * np][1], s[2 * np][2], s[2 * np][3],
                          qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1,
                          s[2 * np][0], s[2 * np][1], s[2 * np][2], s[2 * np][3]);
                mma_16816<F16>(s[2 * np + 1][0], s[2 * np + 1][1], s[2 * np + 1][2], s[2 * np + 1][3],
                          qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b2, b3,
                          s[2 * np + 1][0], s[2 * np + 1][1], s[2 * np + 1][2], s[2 * np + 1][3]);
            }
        }
        // ---- scale, causal mask (only tiles that reach the diagonal), online softmax ----
        const bool need_mask = kv0 + kPfKv - 1 > pos_min;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float v = s[nt][e] * p.scale_log2;
                if (need_mask) {
                    const int tk = kv0 + nt * 8 + 2 * j + (e & 1);
                    if (tk > row_pos[e >> 1]) v = -INFINITY;
                }
                s[nt][e] = v;
            }
        }
        float alpha[2];
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            float mx = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) mx = fmaxf(mx, fmaxf(s[nt][2 * hf], s[nt][2 * hf + 1]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run[hf], mx);
            // a row that has seen nothing yet (padding row, or fully masked so far) keeps m = -inf
            const float m_use = m_new == -INFINITY ? 0.f : m_new;
            alpha[hf] = fast_exp2(m_run[hf] - m_use);
            float sum = 0.f;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                s[nt][2 * hf] = fast_exp2(s[nt][2 * hf] - m_use);
                s[nt][2 * hf + 1] = fast_exp2(s[nt][2 * hf + 1] - m_use);
                sum += s[nt][2 * hf] + s[nt][2 * hf + 1];
            }
            l_run[hf] = l_run[hf] * alpha[hf] + sum;
            m_run[hf] = m_new;
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            o[nt][0] *= alpha[0]; o[nt][1] *= alpha[0]; o[nt][2] *= alpha[1]; o[nt][3] *= alpha[1];
        }
        // ---- O += P V ----
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            // P enters the product as hi + lo, both 16-bit: hi = the rounded probability, lo = its rounding
            // residual (exact in fp32). With the one-term product the residuals of the few probabilities that
            // dominate a row are what is left of the output error (up to 5e-3 absolute with bf16).
            uint32_t a[4], lo[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float p0 = s[2 * kk + (i >> 1)][2 * (i & 1)], p1 = s[2 * kk + (i >> 1)][2 * (i & 1) + 1];
                float h0, h1;
                a[i] = pack_16x2<F16>(p0, p1);
                unpack_16x2<F16>(a[i], h0, h1);
                lo[i] = pack_16x2<F16>(p0 - h0, p1 - h1);
            }
            const uint32_t a0 = a[0], a1 = a[1], a2 = a[2], a3 = a[3];
#pragma unroll
            for (int dp = 0; dp < NT / 2; ++dp) {
                const int mi = lane >> 3, rr = lane & 7;
                const int tok = 16 * kk + rr + (mi & 1) * 8, ch = 2 * dp + (mi >> 1);
                uint32_t b0, b1, b2, b3;
                ldsm_x4_t(vs_ + tok * SM::kRowB + ((ch ^ (tok & 7)) << 4), b0, b1, b2, b3);
                mma_16816<F16>(o[2 * dp][0], o[2 * dp][1], o[2 * dp][2], o[2 * dp][3], a0, a1, a2, a3, b0, b1,
                          o[2 * dp][0], o[2 * dp][1], o[2 * dp][2], o[2 * dp][3]);
                mma_16816<F16>(o[2 * dp + 1][0], o[2 * dp + 1][1], o[2 * dp + 1][2], o[2 * dp + 1][3], a0, a1, a2, a3, b2, b3,
                          o[2 * dp + 1][0], o[2 * dp + 1][1], o[2 * dp + 1][2], o[2 * dp + 1][3]);
                mma_16816<F16>(o[2 * dp][0], o[2 * dp][1], o[2 * dp][2], o[2 * dp][3], lo[0], lo[1], lo[2], lo[3], b0, b1,
                          o[2 * dp][0], o[2 * dp][1], o[2 * dp][2], o[2 * dp][3]);
                mma_16816<F16>(o[2 * dp + 1][0], o[2 * dp + 1][1], o[2 * dp + 1][2], o[2 * dp + 1][3], lo[0], lo[1], lo[2], lo[3], b2, b3,
                          o[2 * dp + 1][0], o[2 * dp + 1][1], o[2 * dp + 1][2], o[2 * dp + 1][3]);
            }
        }
    }

    // ---- normalise and store ----
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
        float l = l_run[hf];
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        const int m = 16 * warp + c + 8 * hf;
        const int i = i0 + m / Gp, hl = m % Gp, h = g * G + hl;
        if (i >= C || hl >= G) continue;
        const float inv = l > 0.f ? 1.f / l : 0.f;
        if (p.out_f32) {
            float2 *dst = (float2 *)((float *)p.out + ((int64_t)(qs + i) * p.num_q_heads + h) * D);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) dst[4 * nt + j] = make_float2(o[nt][2 * hf] * inv, o[nt][2 * hf + 1] * inv);
            continue;
        }
        uint32_t *dst = (uint32_t *)(p.out + ((int64_t)(qs + i) * p.num_q_heads + h) * D);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
            dst[4 * nt + j] = pack_16x2<F16>(o[nt][2 * hf] * inv, o[nt][2 * hf + 1] * inv);
    }
}

// tensor-core (tcgen05) kernel, ekv_prefill_ws.cu
struct PrefillTcParams {
    const uint8_t *k_layer, *v_layer;
    const uint8_t *tags;
    const int32_t *block_table, *seq_lens, *q_start;
    const __nv_bfloat16 *q;
    __nv_bfloat16 *out;
    int64_t block_bytes;
    int batch, num_q_heads, num_kv_heads, group, max_blocks;
    int group_rows;
    int q_tiles;
    float scale_log2;
    int split_first, splits;     // used by the warp-specialised kernel only
    float *part;
    int *part_count;
    int out_f32;
};
int launch_prefill_ws(const PrefillTcParams &p, int64_t ctas, int max_pages, int num_blocks, bool has_base, bool f16,
                      void *workspace, size_t workspace_bytes, cudaStream_t st);
constexpr int kTcMaxPagesHost = 4096;

} // namespace ekv

using namespace ekv;

extern "C" int ekv_attn_prefill_chunk(const ekv_pool *pool, int32_t layer, const ekv_batch *batch,
                                      const int32_t *q_start, const void *q, void *out,
                                      int32_t num_q_heads, float sm_scale,
                                      int32_t total_q, int32_t max_q_len, int32_t max_seq_len,
                                      void *workspace, size_t workspace_bytes, void *stream)
{
    int rc = check_pool(pool);
    if (rc) return rc;
    rc = check_batch(batch);
    if (rc) return rc;
    if (!q_start || !q || !out || layer < 0 || layer >= pool->num_layers) return EKV_ERR_INVALID_ARG;
    if (total_q < 0 || max_q_len < 0 || max_seq_len < 0 || max_q_len > max_seq_len) return EKV_ERR_INVALID_ARG;
    if (((uintptr_t)q & 15) || ((uintptr_t)out & 15)) return EKV_ERR_INVALID_ARG;
    if (num_q_heads <= 0 || num_q_heads % pool->num_kv_heads) return EKV_ERR_INVALID_ARG;
    const int G = num_q_heads / pool->num_kv_heads;
    if (G > 8) return EKV_ERR_UNSUPPORTED;
    const int Gp = G <= 1 ? 1 : G <= 2 ? 2 : G <= 4 ? 4 : 8;       // rows per token in a tile (a power of two divides the tile)
    if (batch->has_base && !pool->tags) return EKV_ERR_INVALID_ARG;
    if ((int64_t)max_seq_len > (int64_t)batch->max_blocks * kPageSize) return EKV_ERR_INVALID_ARG;
    const int max_pages = (max_seq_len + kPageSize - 1) / kPageSize;
    if (max_pages > kPfMaxPages) return EKV_ERR_UNSUPPORTED;
    if (batch->batch == 0 || total_q == 0 || max_q_len == 0) return EKV_OK;

    // head_dim 128: tcgen05 kernel (128-row tiles); otherwise, or on request, the mma.sync kernel
    if (pool->head_dim == 128 && g_prefill_variant != 1 && max_pages <= kTcMaxPagesHost) {
        PrefillTcParams tp{};
        tp.k_layer = (const uint8_t *)pool->k_pool + (int64_t)layer * pool->layer_stride_bytes;
        tp.v_layer = (const uint8_t *)pool->v_pool + (int64_t)layer * pool->layer_stride_bytes;
        tp.tags = pool->tags;
        tp.block_table = batch->block_table;
        tp.seq_lens = batch->seq_lens;
        tp.q_start = q_start;
        tp.q = (const __nv_bfloat16 *)q;
        tp.out = (__nv_bfloat16 *)out;
        tp.block_bytes = (int64_t)pool->num_kv_heads * kPageSize * pool->head_dim * 2;
        tp.batch = batch->batch;
        tp.num_q_heads = num_q_heads;
        tp.num_kv_heads = pool->num_kv_heads;
        tp.group = G;
        tp.group_rows = Gp;
        tp.max_blocks = batch->max_blocks;
        const int tok_tc = 2 * (128 / Gp);                // two row tiles of 128 rows per CTA
        tp.q_tiles = (max_q_len + tok_tc - 1) / tok_tc;
        tp.scale_log2 = sm_scale * 1.4426950408889634f;
        tp.out_f32 = g_attn_out_f32 ? 1 : 0;
        const int64_t n = (int64_t)batch->batch * pool->num_kv_heads * tp.q_tiles;
        if (n > 0x7fffffffLL) return EKV_ERR_UNSUPPORTED;
        return launch_prefill_ws(tp, n, max_pages, pool->num_blocks, batch->has_base != 0, pool->elem_type == EKV_FP16, workspace, workspace_bytes, (cudaStream_t)stream);
    }

    PrefillParams p{};
    p.k_layer = (const uint8_t *)pool->k_pool + (int64_t)layer * pool->layer_stride_bytes;
    p.v_layer = (const uint8_t *)pool->v_pool + (int64_t)layer * pool->layer_stride_bytes;
    p.tags = pool->tags;
    p.block_table = batch->block_table;
    p.seq_lens = batch->seq_lens;
    p.q_start = q_start;
    p.q = (const __nv_bfloat16 *)q;
    p.out = (__nv_bfloat16 *)out;
    p.block_bytes = (int64_t)pool->num_kv_heads * kPageSize * pool->head_dim * 2;
    p.batch = batch->batch;
    p.num_q_heads = num_q_heads;
    p.num_kv_heads = pool->num_kv_heads;
    p.group = G;
    p.group_rows = Gp;
    p.max_blocks = batch->max_blocks;
    const int tok_m = kPfRows / Gp;
    p.q_tiles = (max_q_len + tok_m - 1) / tok_m;
    p.scale_log2 = sm_scale * 1.4426950408889634f;
    p.out_f32 = g_attn_out_f32 ? 1 : 0;
    const int64_t ctas = (int64_t)batch->batch * pool->num_kv_heads * p.q_tiles;
    if (ctas > 0x7fffffffLL) return EKV_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const bool hb = batch->has_base != 0;
    const size_t table_bytes = (size_t)((max_pages + 3) / 4 * 4) * sizeof(int32_t);
    cudaError_t err = cudaSuccess;
#define EKV_LAUNCH_PREFILL_T(DD, HB, FF)                                                                  \
    do {                                                                                                  \
        const size_t sm = PfSmem<DD>::kTotal + table_bytes;                                               \
        err = cudaFuncSetAttribute(prefill_chunk_kernel<DD, HB, FF>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm); \
        if (err == cudaSuccess) {                                                                         \
            MainKernelScope scope(st);                                                                    \
            prefill_chunk_kernel<DD, HB, FF><<<(unsigned)ctas, kPfThreads, sm, st>>>(p);                  \
        }                                                                                                 \
    } while (0)
#define EKV_LAUNCH_PREFILL(DD, HB)                                                                        \
    do {                                                                                                  \
        if (pool->elem_type == EKV_FP16) EKV_LAUNCH_PREFILL_T(DD, HB, true); else EKV_LAUNCH_PREFILL_T(DD, HB, false); \
    } while (0)
    if (pool->head_dim == 128) { if (hb) EKV_LAUNCH_PREFILL(128, true); else EKV_LAUNCH_PREFILL(128, false); }
    else                       { if (hb) EKV_LAUNCH_PREFILL(64, true);  else EKV_LAUNCH_PREFILL(64, false); }
#undef EKV_LAUNCH_PREFILL
#undef EKV_LAUNCH_PREFILL_T
    if (err != cudaSuccess) return EKV_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? EKV_OK : EKV_ERR_CUDA;
}
