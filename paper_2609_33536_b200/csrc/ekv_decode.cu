// Dual-mode paged decode attention (Sec. 3.2; App. B.3), split-K flash-decoding.
//
// Work item = (request, kv head, split of the token range). A CTA has 4 warps; every warp walks
// its own share of the split with its own online-softmax state; the warps are merged through
// shared memory at the end and the CTA writes either the final bf16 rows (single split) or an
// fp32 partial (normalised O and log2-sum-exp) that decode_merge_kernel combines.
//
// Tensor-core mapping:
//   decode_ring_kernel (the product path, native and elastic instantiations)
//     QK^T : S^T = K Q^T, mma.m16n8k16 with M = 16 tokens, N = 8 query heads of the group (columns
//            past the group are zero queries), K = 16 dims, so every MMA row is real work. A dot
//            product does not care in which order the head dimension is visited, so each lane owns
//            contiguous runs of dims and the query fragments are laid out with the same ownership:
//            operands are fetched 16 bytes at a time, never element-wise.
//     PV   : transposed, O^T[d][head] += V^T[d][tok] P^T[tok][head]: M = 16 dims, N = 8 heads,
//            K = 16 tokens. movmatrix turns the packed halves of an S^T accumulator into the B
//            fragment of P^T, so P never leaves registers; the V^T fragments come from ldmatrix
//            (16-bit transposing for TARGET slabs, 8-bit transposing plus one byte-permute per
//            register for BASE slabs).
//     K and V slabs are staged global -> shared memory through a per-warp ring, two steps ahead
//     (cp.async by default, TMA tensor copies as an option).
//     Probabilities enter PV as one 16-bit term, or as two (rounded value + rounding residual) on
//     steps that hold a heavy token: see softmax_step_t.
//   decode_page_kernel: an older design kept for A/B runs (option decode_variant = 1): register-
//     direct, page-stepped (every step is one 16-token page), query heads on the M axis of QK^T
//     (rows 8..15 are zero padding), bf16 pools only.
// BASE blocks: half as many bytes are fetched and expanded byte -> (byte << 8) with byte-permute
// instructions in registers; nothing is materialised in memory.
#include "ekv_common.cuh"
#include <cuda.h>
#include <math.h>
#include <string.h>
#include <atomic>

namespace ekv {

constexpr int kDecodeWarps = 4;
constexpr int kMaxChunkTokens = 4096;
constexpr int kDecodeThreads = kDecodeWarps * 32;

struct DecodeParams {
    const uint8_t *k_layer, *v_layer;   // layer base of the pools
    const uint8_t *tags;
    const int32_t *block_table;
    const int32_t *seq_lens;
    const __nv_bfloat16 *q;
    __nv_bfloat16 *out;
    float *part_o;                      // [batch][Hq][max_splits][D]
    float *part_lse;                    // [batch][Hq][max_splits]
    const int32_t *boundaries;          // structured path: [batch][2] first BASE pair, one past the last
    int64_t block_bytes;
    int batch, num_q_heads, num_kv_heads, group, max_blocks;
    int chunk_tokens, max_splits;
    float scale_log2;                   // sm_scale * log2(e)
    int out_f32;                        // debug: `out` is float [batch][Hq][D] and receives the unrounded result
    int two_term;                       // 0 = two-term probabilities by the mass test, 1 = never, 2 = on every step
};

__device__ __forceinline__ bool m_run_is_empty(float m) { return m == -INFINITY; }

constexpr int kTwoTermRefresh = 8;             // steps between refreshes of the two-term threshold (see softmax_step_t)
constexpr float kTwoTermLog2Share = -3.0f;     // log2 of the probability share from which a token gets a two-term probability

template <int BYTES> struct Loader;
template <> struct Loader<64> { template <int N> static __device__ __forceinline__ void ld(const uint8_t *p, uint32_t (&r)[N], int at) {
    uint32_t a[8], b[8]; ldg32B(p, a); ldg32B(p + 32, b);
#pragma unroll
    for (int i = 0; i < 8; ++i) { r[at + i] = a[i]; r[at + 8 + i] = b[i]; } } };
template <> struct Loader<32> { template <int N> static __device__ __forceinline__ void ld(const uint8_t *p, uint32_t (&r)[N], int at) {
    uint32_t a[8]; ldg32B(p, a);
#pragma unroll
    for (int i = 0; i < 8; ++i) r[at + i] = a[i]; } };
template <> struct Loader<16> { template <int N> static __device__ __forceinline__ void ld(const uint8_t *p, uint32_t (&r)[N], int at) {
    uint32_t a[4]; ldg16B(p, a);
#pragma unroll
    for (int i = 0; i < 4; ++i) r[at + i] = a[i]; } };
template <> struct Loader<8> { template <int N> static __device__ __forceinline__ void ld(const uint8_t *p, uint32_t (&r)[N], int at) {
    uint32_t a[2]; ldg8B(p, a);
    r[at] = a[0]; r[at + 1] = a[1]; } };

// Page-stepped variant: warp w walks pages w, w+4, ...; every step is 16 tokens in either mode.
template <int D, bool HAS_BASE>
__global__ void __launch_bounds__(kDecodeThreads, 3) decode_page_kernel(DecodeParams p)
{
    constexpr int KS = D / 16;            // k-steps of QK^T
    constexpr int MT = D / 16;            // m-tiles of PV
    constexpr int KREG_T = D / 8;         // u32 per token per lane, K TARGET (D/4 dims * 2 B)
    constexpr int KREG_B = D / 16;        // K BASE
    constexpr int VREG_T = D / 16;        // V TARGET (D/8 dims * 2 B)
    constexpr int VREG_B = D / 32;        // V BASE
    constexpr int kSlabT = kPageSize * D * 2;   // one (block, head) slab, TARGET words
    constexpr int kSlabB = kPageSize * D;       // one member of a BASE (block, head) slab

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int c = lane >> 2, j = lane & 3;

    int idx = blockIdx.x;
    const int g = idx % p.num_kv_heads; idx /= p.num_kv_heads;
    const int r = idx % p.batch;
    const int split = idx / p.batch;
    const int L = p.seq_lens[r];
    const int G = p.group;
    const int n_splits = (L + p.chunk_tokens - 1) / p.chunk_tokens;
    if (split >= (n_splits > 0 ? n_splits : 1)) return;
    const int h0 = g * G;                                         // first query head of the group
    if (L <= 0) {                                                 // empty request: zeros
        for (int i = threadIdx.x; i < G * D; i += kDecodeThreads) {
            if (p.out_f32) ((float *)p.out)[((int64_t)r * p.num_q_heads + h0) * D + i] = 0.f;
            else p.out[((int64_t)r * p.num_q_heads + h0) * D + i] = __float2bfloat16(0.f);
        }
        return;
    }
    const int t0 = split * p.chunk_tokens;
    const int t1 = min(L, t0 + p.chunk_tokens);
    const int page0 = t0 / kPageSize;
    const int npages = (t1 - t0 + kPageSize - 1) / kPageSize;
    const int n_it = npages > warp ? (npages - warp + kDecodeWarps - 1) / kDecodeWarps : 0;

    // Query fragments: row c = head h0 + c (zero for c >= G), dims [j*D/4, (j+1)*D/4).
    uint32_t qa[KREG_T];
    if (c < G) {
        const uint8_t *qrow = (const uint8_t *)(p.q + ((int64_t)r * p.num_q_heads + h0 + c) * D) + j * (D / 2);
        Loader<D / 2>::ld(qrow, qa, 0);
    } else {
#pragma unroll
        for (int i = 0; i < KREG_T; ++i) qa[i] = 0u;
    }

    float o[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) { o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f; }
    float m_run = -INFINITY, l_run = 0.f;
    float thr_abs = p.two_term == 1 ? INFINITY : -INFINITY;   // two-term threshold of head c (absolute score units)

    const int32_t *bt_row = p.block_table + (int64_t)r * p.max_blocks;
    int packed = 0;                                    // lane i: (phys << 1 | tag) of iteration base+i
    auto refill = [&](int it_base) {
        const int pi = warp + (it_base + lane) * kDecodeWarps;
        int e = 0;
        if (pi < npages) {
            const int phys = bt_row[page0 + pi];
            int tag = 0;
            if (HAS_BASE) tag = p.tags[phys];
            e = (phys << 1) | tag;
        }
        packed = e;
    };

    uint32_t kr[2 * KREG_T];
    uint32_t vr[4 * VREG_T];

    auto issue_k = [&](int entry, int pi) {
        const int phys = entry >> 1;
        const int lb = page0 + pi;
        if (HAS_BASE && (entry & 1)) {
            const uint8_t *base = p.k_layer + (int64_t)phys * p.block_bytes + (int64_t)(g * 2 + (lb & 1)) * kSlabB
                                  + c * D + j * (D / 4);
            Loader<D / 4>::ld(base, kr, 0);
            Loader<D / 4>::ld(base + 8 * D, kr, KREG_B);
        } else {
            const uint8_t *base = p.k_layer + (int64_t)phys * p.block_bytes + (int64_t)g * kSlabT
                                  + c * (D * 2) + j * (D / 2);
            Loader<D / 2>::ld(base, kr, 0);
            Loader<D / 2>::ld(base + 8 * D * 2, kr, KREG_T);
        }
    };
    auto issue_v = [&](int entry, int pi) {
        const int phys = entry >> 1;
        const int lb = page0 + pi;
        if (HAS_BASE && (entry & 1)) {
            const uint8_t *base = p.v_layer + (int64_t)phys * p.block_bytes + (int64_t)(g * 2 + (lb & 1)) * kSlabB
                                  + (2 * j) * D + c * (D / 8);
            Loader<D / 8>::ld(base, vr, 0);
            Loader<D / 8>::ld(base + D, vr, VREG_B);
            Loader<D / 8>::ld(base + 8 * D, vr, 2 * VREG_B);
            Loader<D / 8>::ld(base + 9 * D, vr, 3 * VREG_B);
        } else {
            const uint8_t *base = p.v_layer + (int64_t)phys * p.block_bytes + (int64_t)g * kSlabT
                                  + (2 * j) * (D * 2) + c * (D / 4);
            Loader<D / 4>::ld(base, vr, 0);
            Loader<D / 4>::ld(base + D * 2, vr, VREG_T);
            Loader<D / 4>::ld(base + 8 * D * 2, vr, 2 * VREG_T);
            Loader<D / 4>::ld(base + 9 * D * 2, vr, 3 * VREG_T);
        }
    };

    int cur = 0;
    if (n_it > 0) {
        refill(0);
        cur = __shfl_sync(0xffffffffu, packed, 0);
        issue_k(cur, warp);
    }

#pragma unroll 1
    for (int it = 0; it < n_it; ++it) {
        const int pi = warp + it * kDecodeWarps;
        issue_v(cur, pi);
        const bool is_base = HAS_BASE && (cur & 1);

        // ---- S = Q K^T for 16 tokens (two n-tiles of 8) ----
        float s[2][2];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f;
            if (is_base) {
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const uint32_t x = kr[nt * KREG_B + ks];
                    mma_16816(c0, c1, c2, c3, qa[2 * ks], 0u, qa[2 * ks + 1], 0u,
                              prmt(x, 0u, 0x1404), prmt(x, 0u, 0x3424), c0, c1, 0.f, 0.f);
                }
            } else {
#pragma unroll
                for (int ks = 0; ks < KS; ++ks)
                    mma_16816(c0, c1, c2, c3, qa[2 * ks], 0u, qa[2 * ks + 1], 0u,
                              kr[nt * KREG_T + 2 * ks], kr[nt * KREG_T + 2 * ks + 1], c0, c1, 0.f, 0.f);
            }
            s[nt][0] = c0 * p.scale_log2;
            s[nt][1] = c1 * p.scale_log2;
        }

        // ---- next page: table entry, then its K loads (kr is free now) ----
        int nxt = 0;
        if (it + 1 < n_it) {
            if (((it + 1) & 31) == 0) refill(it + 1);
            nxt = __shfl_sync(0xffffffffu, packed, (it + 1) & 31);
        }

        // ---- mask the tail, online softmax (log2 domain) ----
        const int valid = t1 - (t0 + pi * kPageSize);          // tokens of this page that exist
        if (valid < kPageSize) {
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e)
                    if (nt * 8 + 2 * j + e >= valid) s[nt][e] = -INFINITY;
        }
        float mx = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);                   // finite: token 0 of a page is valid
        const bool two_term = __any_sync(0xffffffffu, !(mx < thr_abs));   // see softmax_step_t: p = hi + lo for steps with a heavy token
        const float alpha = fast_exp2(m_run - m_new);
        float pr[2][2];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            pr[nt][0] = fast_exp2(s[nt][0] - m_new);
            pr[nt][1] = fast_exp2(s[nt][1] - m_new);
        }
        l_run = l_run * alpha + (pr[0][0] + pr[0][1]) + (pr[1][0] + pr[1][1]);
        m_run = m_new;
        const uint32_t pb0 = pack_bf16x2(pr[0][0], pr[0][1]);
        const uint32_t pb1 = pack_bf16x2(pr[1][0], pr[1][1]);
        uint32_t pl0 = 0u, pl1 = 0u;
        if (two_term) {
            float h0, h1;
            unpack_16x2<false>(pb0, h0, h1);
            pl0 = pack_bf16x2(pr[0][0] - h0, pr[0][1] - h1);
            unpack_16x2<false>(pb1, h0, h1);
            pl1 = pack_bf16x2(pr[1][0] - h0, pr[1][1] - h1);
        }
        // rescale factors of the two heads this lane holds in O^T (columns 2j, 2j+1)
        const float al0 = __shfl_sync(0xffffffffu, alpha, (2 * j) * 4);
        const float al1 = __shfl_sync(0xffffffffu, alpha, (2 * j + 1) * 4);

        if (it + 1 < n_it) issue_k(nxt, pi + kDecodeWarps);

#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            o[mt][0] *= al0; o[mt][1] *= al1; o[mt][2] *= al0; o[mt][3] *= al1;
        }

        // ---- O^T += V^T P^T ----
        if (valid < kPageSize) {          // rows past the end may hold anything: 0 * NaN must not leak
            constexpr int VR = VREG_T;    // clears the BASE sub-ranges too (they are a prefix)
#pragma unroll
            for (int tk = 0; tk < 4; ++tk) {
                const int tok = 2 * j + (tk & 1) + (tk >> 1) * 8;
                if (tok >= valid) {
                    if (is_base) {
#pragma unroll
                        for (int i = 0; i < VREG_B; ++i) vr[tk * VREG_B + i] = 0u;
                    } else {
#pragma unroll
                        for (int i = 0; i < VR; ++i) vr[tk * VR + i] = 0u;
                    }
                }
            }
        }
        if (is_base) {
#pragma unroll
            for (int qd = 0; qd < VREG_B; ++qd) {
                const uint32_t x0 = vr[0 * VREG_B + qd], x1 = vr[1 * VREG_B + qd];
                const uint32_t x2 = vr[2 * VREG_B + qd], x3 = vr[3 * VREG_B + qd];
                // [t0.b1, t0.b0, t1.b1, t1.b0] and the same for bytes 3,2
                const uint32_t ul = prmt(x0, x1, 0x4501), uh = prmt(x0, x1, 0x6723);
                const uint32_t wl = prmt(x2, x3, 0x4501), wh = prmt(x2, x3, 0x6723);
                const uint32_t a0 = ul & 0xFF00FF00u, a1 = prmt(ul, 0u, 0x2404), a2 = wl & 0xFF00FF00u, a3 = prmt(wl, 0u, 0x2404);
                const uint32_t b0 = uh & 0xFF00FF00u, b1 = prmt(uh, 0u, 0x2404), b2 = wh & 0xFF00FF00u, b3 = prmt(wh, 0u, 0x2404);
                mma_16816(o[2 * qd][0], o[2 * qd][1], o[2 * qd][2], o[2 * qd][3], a0, a1, a2, a3,
                          pb0, pb1, o[2 * qd][0], o[2 * qd][1], o[2 * qd][2], o[2 * qd][3]);
                mma_16816(o[2 * qd + 1][0], o[2 * qd + 1][1], o[2 * qd + 1][2], o[2 * qd + 1][3], b0, b1, b2, b3,
                          pb0, pb1, o[2 * qd + 1][0], o[2 * qd + 1][1], o[2 * qd + 1][2], o[2 * qd + 1][3]);
                if (two_term) {
                    mma_16816(o[2 * qd][0], o[2 * qd][1], o[2 * qd][2], o[2 * qd][3], a0, a1, a2, a3,
                              pl0, pl1, o[2 * qd][0], o[2 * qd][1], o[2 * qd][2], o[2 * qd][3]);
                    mma_16816(o[2 * qd + 1][0], o[2 * qd + 1][1], o[2 * qd + 1][2], o[2 * qd + 1][3], b0, b1, b2, b3,
                              pl0, pl1, o[2 * qd + 1][0], o[2 * qd + 1][1], o[2 * qd + 1][2], o[2 * qd + 1][3]);
                }
            }
        } else {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const uint32_t x0 = vr[0 * VREG_T + mt], x1 = vr[1 * VREG_T + mt];
                const uint32_t x2 = vr[2 * VREG_T + mt], x3 = vr[3 * VREG_T + mt];
                const uint32_t a0 = prmt(x0, x1, 0x5410), a1 = prmt(x0, x1, 0x7632), a2 = prmt(x2, x3, 0x5410), a3 = prmt(x2, x3, 0x7632);
                mma_16816(o[mt][0], o[mt][1], o[mt][2], o[mt][3], a0, a1, a2, a3,
                          pb0, pb1, o[mt][0], o[mt][1], o[mt][2], o[mt][3]);
                if (two_term)
                    mma_16816(o[mt][0], o[mt][1], o[mt][2], o[mt][3], a0, a1, a2, a3,
                              pl0, pl1, o[mt][0], o[mt][1], o[mt][2], o[mt][3]);
            }
        }
        cur = nxt;
        if (p.two_term == 0 && ((it & (it + 1)) == 0 || (it & (kTwoTermRefresh - 1)) == kTwoTermRefresh - 1)) {
            float L = l_run;
            L += __shfl_xor_sync(0xffffffffu, L, 1);
            L += __shfl_xor_sync(0xffffffffu, L, 2);
            thr_abs = m_run + __log2f(L) + kTwoTermLog2Share;
        }
    }

    // ---- merge the warps of this CTA ----
    __shared__ float sm_m[kDecodeWarps][8], sm_l[kDecodeWarps][8];
    __shared__ float sm_o[kDecodeWarps][8][D + 4];
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    if (j == 0) { sm_m[warp][c] = m_run; sm_l[warp][c] = l_run; }
    __syncthreads();
    // factor of this warp for heads 2j and 2j+1
    float f[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int h = 2 * j + e;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) M = fmaxf(M, sm_m[w][h]);
        f[e] = (m_run_is_empty(sm_m[warp][h])) ? 0.f : fast_exp2(sm_m[warp][h] - M);
    }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        const int d = c * (D / 8) + 2 * mt;
        sm_o[warp][2 * j][d] = o[mt][0] * f[0];
        sm_o[warp][2 * j + 1][d] = o[mt][1] * f[1];
        sm_o[warp][2 * j][d + 1] = o[mt][2] * f[0];
        sm_o[warp][2 * j + 1][d + 1] = o[mt][3] * f[1];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < G * D; i += kDecodeThreads) {
        const int h = i / D, d = i % D;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) M = fmaxf(M, sm_m[w][h]);
        float lsum = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) {
            const float mw = sm_m[w][h];
            lsum += m_run_is_empty(mw) ? 0.f : sm_l[w][h] * fast_exp2(mw - M);
            acc += sm_o[w][h][d];
        }
        const float val = acc / lsum;
        const int64_t row = (int64_t)r * p.num_q_heads + h0 + h;
        if (n_splits == 1) {
            if (p.out_f32) ((float *)p.out)[row * D + d] = val;
            else p.out[row * D + d] = __float2bfloat16(val);
        } else {
            p.part_o[(row * p.max_splits + split) * D + d] = val;
            if (d == 0) p.part_lse[row * p.max_splits + split] = M + log2f(lsum);
        }
    }
}

// Online-softmax update for one step of the ring kernel, whose QK product has the TOKENS on the M axis
// (S^T = K Q^T: 16 tokens x 8 heads per MMA, so the MMA rows are all real work and the query heads sit
// on the 8-wide N axis). acc[mt] is the accumulator of m-tile mt: {c0, c1} = row g, heads 2t, 2t+1;
// {c2, c3} = row g + 8, same heads (g = lane / 4, t = lane % 4). Row i of m-tile mt stands for token
//   16 mt + i                              (TARGET step, one m-tile), or
//   16 mt + 4 ((i % 8) / 2) + i % 2 + 2 (i / 8)   (BASE step with QUAD_TOKENS: the order in which the
//                                           8-bit transposing ldmatrix delivers V).
// A lane keeps the running maximum and its share of the running sum of TWO heads (2t, 2t+1). On return
// pb[2 mt], pb[2 mt + 1] hold the probabilities of m-tile mt as the B fragment of P^T (k = tokens,
// n = heads) that the transposed PV product wants: the packed accumulator halves are 8 x 8 tiles
// [token row][head pair], and movmatrix transposes them to [head][token pair].
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a)
{
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
// Two-term probabilities. P enters the PV product as a 16-bit float; on a row that a few tokens
// dominate the rounding of those few probabilities (2^-9 relative for bf16) is what remains of the
// output error, up to 5e-3 absolute. When a step holds a token that can end up with an eighth or
// more of a head's probability mass, its probabilities are therefore split as p = hi + lo (both
// 16-bit, lo = the rounding residual, exact in fp32) and PV is taken for both terms. The test must
// not miss such a token, and is cheap: a token's final share is at most p / L, L being any lower
// bound of the head's final probability mass, so "step maximum >= thr_abs" with
// thr_abs = log2(L / 8) in absolute score units (which do not move with the running maximum) is a
// necessary condition. L is the mass this warp has seen so far (a warp's own sums only: the decision
// must not depend on how far other warps have got, or results would differ from run to run),
// refreshed after steps 0, 1, 3, 7 and then every kTwoTermRefresh steps; between refreshes the
// mass only grows, which makes the stale threshold the stricter one. Before the first refresh
// every step takes two terms.
template <int MTILES, bool QUAD_TOKENS, bool F16>
__device__ __forceinline__ void softmax_step_t(float (&s)[MTILES][4], int valid, int g, float (&m_run)[2], float (&l_run)[2],
                                               uint32_t (&pb)[2 * MTILES], float (&alpha)[2],
                                               const float (&thr_abs)[2], bool &two_term, uint32_t save_addr)
{
    if (valid < MTILES * 16) {
#pragma unroll
        for (int mt = 0; mt < MTILES; ++mt)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int tok = QUAD_TOKENS ? 16 * mt + 4 * (g >> 1) + (g & 1) + 2 * half : 16 * mt + g + 8 * half;
                if (tok >= valid) s[mt][2 * half] = s[mt][2 * half + 1] = -INFINITY;
            }
    }
    // the masked scores are parked in this lane's shared-memory slot: the rare two-term pass takes them from there
#pragma unroll
    for (int mt = 0; mt < MTILES; ++mt)
        asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" :: "r"(save_addr + 512 * mt), "f"(s[mt][0]), "f"(s[mt][1]), "f"(s[mt][2]), "f"(s[mt][3]) : "memory");
    float mx[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        mx[e] = fmaxf(s[0][e], s[0][2 + e]);
#pragma unroll
        for (int mt = 1; mt < MTILES; ++mt) mx[e] = fmaxf(mx[e], fmaxf(s[mt][e], s[mt][2 + e]));
    }
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {                // over the eight row groups (lanes with the same t)
        mx[0] = fmaxf(mx[0], __shfl_xor_sync(0xffffffffu, mx[0], o));
        mx[1] = fmaxf(mx[1], __shfl_xor_sync(0xffffffffu, mx[1], o));
    }
    two_term = __any_sync(0xffffffffu, !(mx[0] < thr_abs[0]) || !(mx[1] < thr_abs[1]));
    float sum[2] = {0.f, 0.f};
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const float m_new = fmaxf(m_run[e], mx[e]);  // finite: the first token of a step always exists
        alpha[e] = fast_exp2(m_run[e] - m_new);
        m_run[e] = m_new;
    }
#pragma unroll
    for (int mt = 0; mt < MTILES; ++mt) {
        const float p0 = fast_exp2(s[mt][0] - m_run[0]), p1 = fast_exp2(s[mt][1] - m_run[1]);
        const float p2 = fast_exp2(s[mt][2] - m_run[0]), p3 = fast_exp2(s[mt][3] - m_run[1]);
        sum[0] += p0 + p2;
        sum[1] += p1 + p3;
        pb[2 * mt] = movmatrix_trans(pack_16x2<F16>(p0, p1));
        pb[2 * mt + 1] = movmatrix_trans(pack_16x2<F16>(p2, p3));
    }
    l_run[0] = l_run[0] * alpha[0] + sum[0];
    l_run[1] = l_run[1] * alpha[1] + sum[1];
}

// The low-order terms of a step's probabilities, recomputed from the parked scores with the running
// maxima the step ended on (the same instructions on the same values as in softmax_step_t, so hi is
// bit for bit what the first pass multiplied with): lo = p - hi, in B-fragment order like pb.
template <int MTILES, bool F16>
__device__ __forceinline__ void two_term_residuals(uint32_t save_addr, const float (&m_run)[2], uint32_t (&pl)[2 * MTILES])
{
#pragma unroll
    for (int mt = 0; mt < MTILES; ++mt) {
        float s0, s1, s2, s3, h0, h1, h2, h3;
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(s0), "=f"(s1), "=f"(s2), "=f"(s3) : "r"(save_addr + 512 * mt) : "memory");
        const float p0 = fast_exp2(s0 - m_run[0]), p1 = fast_exp2(s1 - m_run[1]);
        const float p2 = fast_exp2(s2 - m_run[0]), p3 = fast_exp2(s3 - m_run[1]);
        unpack_16x2<F16>(pack_16x2<F16>(p0, p1), h0, h1);
        unpack_16x2<F16>(pack_16x2<F16>(p2, p3), h2, h3);
        pl[2 * mt] = movmatrix_trans(pack_16x2<F16>(p0 - h0, p1 - h1));
        pl[2 * mt + 1] = movmatrix_trans(pack_16x2<F16>(p2 - h2, p3 - h3));
    }
}

// One step of a warp: a run of tokens that is contiguous in one (block, kv head) slab.
struct Step {
    int phys;      // physical block
    int tok0;      // first token, relative to the split start
    int base;      // 1: BASE pair (32 tokens, bytes), 0: one TARGET page (16 tokens, words)
};

// ---- ring-staged variant ---------------------------------------------------------------------
// Warp w walks pairs w, w+4, ... of the split: a TARGET pair is two 16-token steps (one per physical
// block), a BASE pair ONE 32-token step, so a step is 4 KiB of K and 4 KiB of V either way at
// head_dim 128 and both modes keep the same number of bytes in flight. K and V travel
// global -> shared memory with cp.async into a private ring of kRingStages (K slab, V slab)
// slots per warp, issued that many steps ahead. The bytes in flight per SM are then bounded by
// shared memory (about 190 KiB) instead of by landing registers, and a step never waits on a
// load it issued itself. No CTA-wide barrier is needed: each warp owns its ring.
// Slab rows are XOR-swizzled (16-byte chunks) so that every fragment read is conflict free:
//   K TARGET: 16 rows x 16 chunks, chunk' = chunk ^ (row & 1);  lane (c, j) reads row c / c+8,
//             chunks {2j, 2j+1, 8+2j, 9+2j}: dims [16j, 16j+16) and [D/2+16j, D/2+16j+16)
//   K BASE  : 32 rows x  8 chunks, chunk' = chunk ^ ((row & 1) * 4); chunks {j, 4+j}: same dims
//   V (both): chunk' = chunk ^ (row & 7), the layout ldmatrix wants: eight token rows of one chunk
//             column land in eight different bank groups. TARGET tiles are fetched with
//             ldmatrix.x4.trans (16-bit), which delivers the V^T A-fragments as they are; BASE
//             tiles with the 8-bit transposing ldmatrix (16 tokens x 16 dims), which delivers four
//             tokens of one dim per register: two byte-permutes expand them to A-fragments.
//             Output dim of accumulator (m-tile mt, row g / g+8) is 16 mt + g / 16 mt + 8 + g.
template <int STAGES> struct RingCfg { static constexpr int kStages = STAGES; };

// Tensor maps of the TMA-staged instantiation (head_dim 128): one layer of a pool seen as
//   kv_target : [blocks * kv heads * 16 token rows][128 16-bit words], box 64 words x 16 rows, 128-byte swizzle
//               (K and V; a TARGET slab = two boxes, one per half of the head dimension)
//   k_base    : [blocks * kv heads * 32 token rows][128 bytes], box 64 bytes x 32 rows, no swizzle
//               (a BASE K slab = two boxes; rows of 64 bytes alternate between the two halves of the banks)
//   v_base    : the same bytes, box 128 bytes x 32 rows, 128-byte swizzle (the layout ldmatrix wants)
struct DecodeMaps {
    alignas(64) CUtensorMap k_target, v_target, k_base, v_base;
};

__device__ int g_decode_ring_status = 0;           // 0 ok; 1 = a bounded wait for a staged slab expired (results invalid)
constexpr int kRingSpinLimit = 1 << 24;

__device__ __forceinline__ void ring_tma_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 :: "r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
// Bounded wait for a phase of an mbarrier; false when the limit is hit.
__device__ __forceinline__ bool ring_mbar_wait(uint32_t bar, uint32_t parity)
{
    for (int i = 0; i < kRingSpinLimit; ++i) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}

__device__ __forceinline__ void ring_cp16(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void lds16B(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// 16 x 16 bytes, transposed: lane (g = lane / 4, t = lane % 4) receives rows 4t..4t+3 of column g
// (r0) and of column g + 8 (r1); .x2 does that for two matrices (rows given by lanes 0-15, 16-31).
__device__ __forceinline__ void ldsm_b8_x2_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m16n16.x2.trans.shared.b8 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}

template <int D, bool HAS_BASE, int STAGES, int MIN_CTAS, bool BOUNDS = false, bool F16 = false, bool TMA = false>
__global__ void __launch_bounds__(kDecodeThreads, MIN_CTAS) decode_ring_kernel(DecodeParams p, const __grid_constant__ DecodeMaps maps)
{
    static_assert(!TMA || D == 128, "the TMA-staged instantiation is for head_dim 128");
    static_assert(D == 128 || D == 64, "head_dim");
    constexpr int KS = D / 16;
    constexpr int MT = D / 16;
    constexpr int kSlab = kPageSize * D * 2;
    constexpr int kSlot = 2 * kSlab;      // K slab + V slab
    constexpr int CPR_T = D / 8;          // 16-byte chunks per TARGET row
    constexpr int CPR_B = D / 16;         // per BASE row
    extern __shared__ __align__(1024) uint8_t dsm[];
    // Launched with programmatic stream serialisation: nothing in global memory is touched before
    // the previous kernel of the stream (a transition commit, the caller's producer of q) is done.
    cudaGridDependencySynchronize();
    // layout: [ring: 4 warps x STAGES x kSlot] (reused by the epilogue) [sm_q] [sm_m, sm_l]
    uint2 (*sm_q)[32] = (uint2 (*)[32])(dsm + kDecodeWarps * STAGES * kSlot);
    float (*sm_m)[8] = (float (*)[8])((uint8_t *)sm_q + KS * 32 * sizeof(uint2));
    float (*sm_l)[8] = sm_m + kDecodeWarps;
    uint2 *sm_steps = (uint2 *)(sm_l + kDecodeWarps);     // [4 warps][64] step descriptors
    // after them: the parked scores (kDecodeThreads x 32 bytes), then, for the TMA-staged instantiation, the
    // "slab landed" mbarriers [4 warps][K: STAGES, V: STAGES]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int c = lane >> 2, j = lane & 3;
    // parked scores of a step: [warp][m-tile][lane] x 16 bytes, so that a warp's stores fall on consecutive banks
    const uint32_t save_addr = (uint32_t)__cvta_generic_to_shared(sm_steps + kDecodeWarps * 64) + warp * 1024 + lane * 16;

    int idx = blockIdx.x;
    const int g = idx % p.num_kv_heads; idx /= p.num_kv_heads;
    const int r = idx % p.batch;
    const int split = idx / p.batch;
    const int L = p.seq_lens[r];
    // The table entries of this lane's pair (pairs w, w + 4, ... of the split) are read before L is
    // known, so that the two loads are in flight together; an entry past the end of the sequence
    // is inside the table row and is not used.
    const int32_t *bt_row = p.block_table + (int64_t)r * p.max_blocks;
    const int pp = warp + lane * kDecodeWarps;
    int e0 = 0, e1 = -1;
    {
        const int64_t lb0 = ((int64_t)split * p.chunk_tokens / (2 * kPageSize) + pp) * 2;
        if (lb0 < p.max_blocks) e0 = bt_row[lb0];
        if (lb0 + 1 < p.max_blocks) e1 = bt_row[lb0 + 1];
    }
    const int G = p.group;
    const int n_splits = (L + p.chunk_tokens - 1) / p.chunk_tokens;
    if (split >= (n_splits > 0 ? n_splits : 1)) return;
    const int h0 = g * G;
    if (L <= 0) {
        for (int i = threadIdx.x; i < G * D; i += kDecodeThreads) {
            if (p.out_f32) ((float *)p.out)[((int64_t)r * p.num_q_heads + h0) * D + i] = 0.f;
            else ((uint16_t *)p.out)[((int64_t)r * p.num_q_heads + h0) * D + i] = 0;
        }
        return;
    }
    const int t0 = split * p.chunk_tokens;
    const int t1 = min(L, t0 + p.chunk_tokens);
    const int pair0 = t0 / (2 * kPageSize);
    const int npairs = (t1 - t0 + 2 * kPageSize - 1) / (2 * kPageSize);
    const int last_lb = (t1 - 1) / kPageSize;

    float o[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) { o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};     // heads 2j, 2j + 1; sums over this lane's token rows
    float thr_abs[2] = {-INFINITY, -INFINITY};       // two-term threshold of the two heads (absolute score units); -inf = always
    if (p.two_term == 1) thr_abs[0] = thr_abs[1] = INFINITY;

    // Step list of this warp, built once: a TARGET pair is two steps (one per member that exists), a
    // BASE pair one. Lane i looks at the warp's i-th pair (w, w+4, ...): table entries, tag (or
    // the structured path's boundaries), then an exclusive scan over the lanes places its steps.
    // The split is at most kMaxChunkTokens long, so a warp has at most 32 pairs / 64 steps.
    uint2 *steps = sm_steps + warp * 64;
    int n_steps;
    {
        int tag = 0, mine = 0;
        if (pp < npairs) {
            const int lb0 = (pair0 + pp) * 2;
            if (HAS_BASE) {
                // structured path: the mode follows from the sequence's two boundaries, no per-pair lookup
                if (BOUNDS) tag = (pair0 + pp >= p.boundaries[2 * r] && pair0 + pp < p.boundaries[2 * r + 1]) ? 1 : 0;
                else        tag = p.tags[e0];
            }
            if (lb0 + 1 > last_lb) e1 = -1;
            mine = (tag || e1 < 0) ? 1 : 2;
        }
        int pre = mine;                                        // inclusive scan
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, pre, o);
            if (lane >= o) pre += v;
        }
        n_steps = __shfl_sync(0xffffffffu, pre, 31);
        pre -= mine;
        if (mine >= 1) steps[pre] = make_uint2((uint32_t)((e0 << 1) | tag), (uint32_t)(pp * 2 * kPageSize));
        if (mine == 2) steps[pre + 1] = make_uint2((uint32_t)(e1 << 1), (uint32_t)(pp * 2 * kPageSize + kPageSize));
        __syncwarp();
    }
    auto step_at = [&](int k) {
        const uint2 d = steps[k];                              // same address in every lane: a broadcast
        Step st;
        st.base = HAS_BASE ? (int)(d.x & 1u) : 0;
        st.phys = (int)(d.x >> 1);
        st.tok0 = (int)d.y;
        return st;
    };

    const uint32_t ring0 = (uint32_t)__cvta_generic_to_shared(dsm) + warp * (STAGES * kSlot);
    const int64_t head_off = (int64_t)g * kSlab;
    const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(sm_steps + kDecodeWarps * 64) + kDecodeThreads * 32 + warp * (2 * STAGES * 8);
    bool dead = false;                                     // a bounded wait expired: stop waiting, report
    if (TMA) {
        if (lane == 0) {
#pragma unroll
            for (int i = 0; i < 2 * STAGES; ++i)
                asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar0 + 8 * i), "r"(1) : "memory");
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
    }
    // wait until the K (which = 0) or V (which = 1) slab of step k has landed in its slot
    auto landed = [&](int k, int slot, int which) {
        if (TMA) {
            if (!dead && !ring_mbar_wait(bar0 + 8 * (which * STAGES + slot), (uint32_t)((k / STAGES) & 1))) dead = true;
        } else {
            asm volatile("cp.async.wait_group %0;" :: "n"(2 * STAGES - 1) : "memory");
        }
        __syncwarp();
    };

    // producer: copy the K and V slabs of a step into ring slot `slot` (8 + 8 x 16 B per lane at D = 128)
    // producer: copy the K (which = 0) or V (which = 1) slab of a step into ring slot `slot`
    auto issue = [&](const Step &st, int slot, int which) {
        const uint32_t dst = ring0 + slot * kSlot + which * kSlab;
        if (TMA) {
            // one lane posts the byte count and issues the tensor copies of the slab (two boxes, or one for a BASE V slab)
            if (lane == 0) {
                const uint32_t bar = bar0 + 8 * (which * STAGES + slot);
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(kSlab) : "memory");
                const int slab = st.phys * p.num_kv_heads + g;
                if (HAS_BASE && st.base) {
                    if (which) ring_tma_2d(dst, &maps.v_base, 0, slab * 32, bar);
                    else { ring_tma_2d(dst, &maps.k_base, 0, slab * 32, bar); ring_tma_2d(dst + kSlab / 2, &maps.k_base, 64, slab * 32, bar); }
                } else {
                    const CUtensorMap *m = which ? &maps.v_target : &maps.k_target;
                    ring_tma_2d(dst, m, 0, slab * 16, bar);
                    ring_tma_2d(dst + kSlab / 2, m, 64, slab * 16, bar);
                }
            }
            return;
        }
        const uint8_t *src = (which ? p.v_layer : p.k_layer) + (int64_t)st.phys * p.block_bytes + head_off;
        if (HAS_BASE && st.base) {
#pragma unroll
            for (int q = 0; q < kSlab / 512; ++q) {
                const int id = q * 32 + lane;                 // chunk id in the slab
                const int row = id / CPR_B, ch = id % CPR_B;
                const int sw = which ? ((ch ^ (row & 7)) & (CPR_B - 1)) : (ch ^ ((row & 1) * (CPR_B / 2)));
                ring_cp16(dst + row * (CPR_B * 16) + (sw << 4), src + id * 16);
            }
        } else {
#pragma unroll
            for (int q = 0; q < kSlab / 512; ++q) {
                const int id = q * 32 + lane;
                const int row = id / CPR_T, ch = id % CPR_T;
                const int sw = which ? ((ch ^ (row & 7)) & (CPR_T - 1)) : (ch ^ (row & 1));
                ring_cp16(dst + row * (CPR_T * 16) + (sw << 4), src + id * 16);
            }
        }
    };
    auto commit = [&]() { if (!TMA) asm volatile("cp.async.commit_group;" ::: "memory"); };
    auto rescale = [&](const float (&alpha)[2]) {            // O^T accumulators: columns = heads 2j, 2j + 1
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) { o[mt][0] *= alpha[0]; o[mt][1] *= alpha[1]; o[mt][2] *= alpha[0]; o[mt][3] *= alpha[1]; }
    };

#pragma unroll
    for (int s = 0; s < STAGES; ++s) {                       // prologue: fill the ring (K group, V group per step)
        if (s < n_steps) issue(step_at(s), s, 0);
        commit();
        if (s < n_steps) issue(step_at(s), s, 1);
        commit();
    }

    // The first slabs are on their way; now the query fragments, in shared memory as [k-step][lane]: k-step s = 4a + r4 covers dims
    // 16j + (D/2)a + 4*r4 .. +3 of head c (zero rows for c >= G).
    if (warp == 0) {
        const uint8_t *qrow = (const uint8_t *)(p.q + ((int64_t)r * p.num_q_heads + h0 + (c < G ? c : 0)) * D);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            const int dim = 16 * j + (D / 2) * (ks >> 2) + 4 * (ks & 3);
            uint2 v = make_uint2(0u, 0u);
            if (c < G) v = *(const uint2 *)(qrow + dim * 2);
            sm_q[ks][lane] = v;
        }
    }
    __syncthreads();

    // ---- the parts of a step ----
    // S^T = K Q^T of a BASE step: two m-tiles of 16 tokens, heads on the N axis; the K bytes become the A operand
    // (rows c and c + 8 of m-tile mt are the slab rows that the loop below calls nt = 2 mt, 2 mt + 1)
    auto qk_base = [&](uint32_t kslot, float (&s)[2][4]) {
        float acc[2][2][4];                                    // [m-tile][half of the head dimension]: four independent chains
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int a = 0; a < 2; ++a) acc[mt][a][0] = acc[mt][a][1] = acc[mt][a][2] = acc[mt][a][3] = 0.f;
#pragma unroll
        for (int a = 0; a < (KS + 3) / 4; ++a) {               // one 16-byte chunk = 4 k-steps
            uint32_t x[4][4];
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                // row c / c + 8 of m-tile nt / 2 is token 16 (nt / 2) + 4 (c / 2) + c % 2 (+ 2 for the upper rows)
                const int row = 16 * (nt >> 1) + 4 * (c >> 1) + 2 * (nt & 1) + (c & 1);
                if (TMA) lds16B(kslot + a * (kSlab / 2) + row * 64 + (j << 4), x[nt]);     // [half of the head dimension][token][64 bytes]
                else lds16B(kslot + row * (CPR_B * 16) + (((j + (CPR_B / 2) * a) ^ ((row & 1) * (CPR_B / 2))) << 4), x[nt]);
            }
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const uint2 qf = sm_q[4 * a + w][lane];
#pragma unroll
                for (int mt = 0; mt < 2; ++mt)
                    mma_16816<F16>(acc[mt][a & 1][0], acc[mt][a & 1][1], acc[mt][a & 1][2], acc[mt][a & 1][3],
                              prmt(x[2 * mt][w], 0u, 0x1404), prmt(x[2 * mt + 1][w], 0u, 0x1404),
                              prmt(x[2 * mt][w], 0u, 0x3424), prmt(x[2 * mt + 1][w], 0u, 0x3424),
                              qf.x, qf.y,
                              acc[mt][a & 1][0], acc[mt][a & 1][1], acc[mt][a & 1][2], acc[mt][a & 1][3]);
            }
        }
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) s[mt][i] = (acc[mt][0][i] + acc[mt][1][i]) * p.scale_log2;
    };
    // S^T of a TARGET step: one m-tile of 16 tokens (in s[0]); two chains over the k-steps
    auto qk_target = [&](uint32_t kslot, float (&s)[2][4]) {
        float acc[2][4];
#pragma unroll
        for (int a = 0; a < 2; ++a) acc[a][0] = acc[a][1] = acc[a][2] = acc[a][3] = 0.f;
#pragma unroll
        for (int cc = 0; cc < KS / 2; ++cc) {                  // one 16-byte chunk = 2 k-steps
            const int lch = 2 * j + (cc & 1) + (CPR_T / 2) * (cc >> 1);
            uint32_t x[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {                   // rows c and c + 8 of the m-tile
                const int row = nt * 8 + c;
                if (TMA) lds16B(kslot + (lch >> 3) * (kSlab / 2) + row * 128 + (((lch & 7) ^ (row & 7)) << 4), x[nt]);   // [half][token][128 bytes], hardware swizzle
                else lds16B(kslot + row * (CPR_T * 16) + ((lch ^ (row & 1)) << 4), x[nt]);
            }
            const uint2 q0 = sm_q[2 * cc][lane], q1 = sm_q[2 * cc + 1][lane];
            mma_16816<F16>(acc[0][0], acc[0][1], acc[0][2], acc[0][3], x[0][0], x[1][0], x[0][1], x[1][1], q0.x, q0.y,
                      acc[0][0], acc[0][1], acc[0][2], acc[0][3]);
            mma_16816<F16>(acc[1][0], acc[1][1], acc[1][2], acc[1][3], x[0][2], x[1][2], x[0][3], x[1][3], q1.x, q1.y,
                      acc[1][0], acc[1][1], acc[1][2], acc[1][3]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) s[0][i] = (acc[0][i] + acc[1][i]) * p.scale_log2;
    };
    // softmax and PV of a BASE step. V: 16 tokens x 16 dims per 8-bit transposing ldmatrix: r0 = tokens 4j..4j+3 of
    // dim c, r1 = the same tokens of dim c + 8; two matrices (two m-tiles) per instruction
    auto tail_base = [&](float (&s)[2][4], int valid, uint32_t vslot, int k, int slot) {
        uint32_t pb[4];
        float alpha[2];
        bool two_term;
        softmax_step_t<2, true, F16>(s, valid, c, m_run, l_run, pb, alpha, thr_abs, two_term, save_addr);
        landed(k, slot, 1);                                     // V of this step landed
        if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) rescale(alpha);      // the running maxima rarely move
        auto pv_base = [&](const uint32_t (&pf)[4]) {
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                // 0 * NaN must not leak from rows past the end: a token byte past the end is replaced by
                // the zero byte of the permute's second operand (selector nibble 4)
                uint32_t sel_lo = 0x1404u, sel_hi = 0x3424u;   // bytes (0, 1) / (2, 3) become high halves
                if (valid < 32) {
                    const int rem = valid - (16 * hf + 4 * j);
                    if (rem < 1) sel_lo = (sel_lo & 0xff0fu) | 0x0040u;      // token 4j
                    if (rem < 2) sel_lo = (sel_lo & 0x0fffu) | 0x4000u;      // token 4j + 1
                    if (rem < 3) sel_hi = (sel_hi & 0xff0fu) | 0x0040u;      // token 4j + 2
                    if (rem < 4) sel_hi = (sel_hi & 0x0fffu) | 0x4000u;      // token 4j + 3
                }
                const int vrow = 16 * hf + (lane & 15);
                const uint32_t rowp = vslot + vrow * (CPR_B * 16);
#pragma unroll
                for (int mp = 0; mp < MT / 2; ++mp) {
                    const int ch = 2 * mp + (lane >> 4);
                    uint32_t r0, r1, r2, r3;
                    ldsm_b8_x2_trans(rowp + (((ch ^ (vrow & 7)) & (CPR_B - 1)) << 4), r0, r1, r2, r3);
                    mma_16816<F16>(o[2 * mp][0], o[2 * mp][1], o[2 * mp][2], o[2 * mp][3],
                              prmt(r0, 0u, sel_lo), prmt(r1, 0u, sel_lo), prmt(r0, 0u, sel_hi), prmt(r1, 0u, sel_hi),
                              pf[2 * hf], pf[2 * hf + 1], o[2 * mp][0], o[2 * mp][1], o[2 * mp][2], o[2 * mp][3]);
                    mma_16816<F16>(o[2 * mp + 1][0], o[2 * mp + 1][1], o[2 * mp + 1][2], o[2 * mp + 1][3],
                              prmt(r2, 0u, sel_lo), prmt(r3, 0u, sel_lo), prmt(r2, 0u, sel_hi), prmt(r3, 0u, sel_hi),
                              pf[2 * hf], pf[2 * hf + 1],
                              o[2 * mp + 1][0], o[2 * mp + 1][1], o[2 * mp + 1][2], o[2 * mp + 1][3]);
                }
            }
        };
        pv_base(pb);
        if (two_term) {                                        // rare, uniform over the warp: the low-order terms of P
            uint32_t pl[4];
            two_term_residuals<2, F16>(save_addr, m_run, pl);
            pv_base(pl);
        }
    };
    // softmax and PV of a TARGET step. V: ldmatrix.x4.trans delivers the V^T A-fragments of one m-tile (16 dims x 16 tokens)
    auto tail_target = [&](float (&s2)[2][4], int valid, uint32_t vslot, int k, int slot) {
        float (&s)[1][4] = *(float (*)[1][4])&s2[0];
        uint32_t pb[2];
        float alpha[2];
        bool two_term;
        softmax_step_t<1, false, F16>(s, valid, c, m_run, l_run, pb, alpha, thr_abs, two_term, save_addr);
        landed(k, slot, 1);
        if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) rescale(alpha);
        auto pv_target = [&](const uint32_t (&pf)[2]) {
            uint32_t mlo = 0xffffffffu, mhi = 0xffffffffu;     // tokens 2j, 2j+1 | 2j+8, 2j+9
            if (valid < kPageSize) {
                mlo = (2 * j < valid ? 0x0000ffffu : 0u) | (2 * j + 1 < valid ? 0xffff0000u : 0u);
                mhi = (2 * j + 8 < valid ? 0x0000ffffu : 0u) | (2 * j + 9 < valid ? 0xffff0000u : 0u);
            }
            const int vrow = (lane & 7) + 8 * (lane >> 4);
            const uint32_t rowp = vslot + vrow * (TMA ? 128 : CPR_T * 16);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const int ch = 2 * mt + ((lane >> 3) & 1);
                uint32_t a0, a1, a2, a3;
                if (TMA) ldsm_x4_trans(rowp + (ch >> 3) * (kSlab / 2) + (((ch & 7) ^ (vrow & 7)) << 4), a0, a1, a2, a3);
                else ldsm_x4_trans(rowp + (((ch ^ (vrow & 7)) & (CPR_T - 1)) << 4), a0, a1, a2, a3);
                mma_16816<F16>(o[mt][0], o[mt][1], o[mt][2], o[mt][3], a0 & mlo, a1 & mlo, a2 & mhi, a3 & mhi,
                          pf[0], pf[1], o[mt][0], o[mt][1], o[mt][2], o[mt][3]);
            }
        };
        pv_target(pb);
        if (two_term) {
            uint32_t pl[2];
            two_term_residuals<1, F16>(save_addr, m_run, pl);
            pv_target(pl);
        }
    };
    auto refresh_thresholds = [&](int k) {
        if (p.two_term == 0 && ((k & (k + 1)) == 0 || (k & (kTwoTermRefresh - 1)) == kTwoTermRefresh - 1)) {
            // refresh the two-term thresholds (after steps 0, 1, 3, 7, then every 8th) from the warp-wide sums
            float L0 = l_run[0], L1 = l_run[1];
#pragma unroll
            for (int o = 4; o < 32; o <<= 1) {
                L0 += __shfl_xor_sync(0xffffffffu, L0, o);
                L1 += __shfl_xor_sync(0xffffffffu, L1, o);
            }
            thr_abs[0] = m_run[0] + __log2f(L0) + kTwoTermLog2Share;
            thr_abs[1] = m_run[1] + __log2f(L1) + kTwoTermLog2Share;
        }
    };

    int slot = 0;
#pragma unroll 1
    for (int k = 0; k < n_steps; ++k) {
        const Step cur = step_at(k);
        const int valid = (t1 - t0) - cur.tok0;
        landed(k, slot, 0);                                     // K of this step landed
        const uint32_t kslot = ring0 + slot * kSlot, vslot = kslot + kSlab;
        const bool more = k + STAGES < n_steps;
        Step nxt{0, 0, 0};
        if (more) nxt = step_at(k + STAGES);
        float s[2][4];
        if (HAS_BASE && cur.base) qk_base(kslot, s); else qk_target(kslot, s);
        __syncwarp();                                          // every lane has read this K slab: refill it
        if (more) issue(nxt, slot, 0);
        commit();
        if (HAS_BASE && cur.base) tail_base(s, valid, vslot, k, slot); else tail_target(s, valid, vslot, k, slot);
        __syncwarp();                                          // every lane is done with this slot
        if (more) issue(nxt, slot, 1);                        // the V slab of this slot is free now
        commit();
        slot = slot + 1 == STAGES ? 0 : slot + 1;
        refresh_thresholds(k);
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (TMA && dead) atomicExch(&g_decode_ring_status, 1);

    // ---- merge the warps of this CTA (the ring is dead: reuse it for the partial outputs) ----
    __syncthreads();
    float (*sm_o)[8][D + 4] = (float (*)[8][D + 4])dsm;
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {                       // the eight row groups each hold a share of the sums
        l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], o);
        l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], o);
    }
    if (c == 0) {
        sm_m[warp][2 * j] = m_run[0]; sm_l[warp][2 * j] = l_run[0];
        sm_m[warp][2 * j + 1] = m_run[1]; sm_l[warp][2 * j + 1] = l_run[1];
    }
    __syncthreads();
    float f[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int h = 2 * j + e;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) M = fmaxf(M, sm_m[w][h]);
        f[e] = m_run_is_empty(sm_m[warp][h]) ? 0.f : fast_exp2(sm_m[warp][h] - M);
    }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        const int d = 16 * mt + c;
        sm_o[warp][2 * j][d] = o[mt][0] * f[0];
        sm_o[warp][2 * j + 1][d] = o[mt][1] * f[1];
        sm_o[warp][2 * j][d + 8] = o[mt][2] * f[0];
        sm_o[warp][2 * j + 1][d + 8] = o[mt][3] * f[1];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < G * D; i += kDecodeThreads) {
        const int h = i / D, d = i % D;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) M = fmaxf(M, sm_m[w][h]);
        float lsum = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) {
            const float mw = sm_m[w][h];
            lsum += m_run_is_empty(mw) ? 0.f : sm_l[w][h] * fast_exp2(mw - M);
            acc += sm_o[w][h][d];
        }
        const float val = acc / lsum;
        const int64_t row = (int64_t)r * p.num_q_heads + h0 + h;
        if (n_splits == 1) {
            if (p.out_f32) ((float *)p.out)[row * D + d] = val;
            else ((uint16_t *)p.out)[row * D + d] = f32_to_16<F16>(val);
        } else {
            p.part_o[(row * p.max_splits + split) * D + d] = val;
            if (d == 0) p.part_lse[row * p.max_splits + split] = M + log2f(lsum);
        }
    }
}

template <int D, int STAGES>
constexpr size_t ring_smem_bytes()
{
    return (size_t)kDecodeWarps * STAGES * (2 * kPageSize * D * 2) + (D / 16) * 32 * sizeof(uint2)
           + 2 * kDecodeWarps * 8 * sizeof(float) + kDecodeWarps * 64 * sizeof(uint2) + kDecodeThreads * 32 + kDecodeWarps * 2 * STAGES * 8;
}

// Combine the per-split partials of one (request, query head) row: weights 2^(lse_s - max).
// One CTA per row. With SG = 1 a thread per output column walks the splits (up to 8: every load is
// issued before the first use). With SG = 4 or 8 (launches whose longest request has many splits:
// long contexts in small batches) that many slices of threads share the splits of the row, so that
// the chain of dependent round trips is that much shorter; the slices' sums meet in shared memory.
template <int D, bool F16, int SG>
__global__ void __launch_bounds__(D * SG) decode_merge_kernel(DecodeParams p)
{
    const int row = blockIdx.x;
    const int r = row / p.num_q_heads;
    const int L = p.seq_lens[r];
    const int ns = (L + p.chunk_tokens - 1) / p.chunk_tokens;
    // Launched with programmatic stream serialisation: this grid may start while the split kernel
    // is still draining; its partials are only read after this point.
    cudaGridDependencySynchronize();
    if (ns <= 1) return;                       // written directly by the split kernel
    const float *lse = p.part_lse + (int64_t)row * p.max_splits;
    const float *po = p.part_o + (int64_t)row * p.max_splits * D + threadIdx.x;
    float acc = 0.f, wsum = 0.f;
    if (SG == 1 && ns > 8) {
        float M = -INFINITY;
        for (int s = 0; s < ns; ++s) M = fmaxf(M, lse[s]);
#pragma unroll 4
        for (int s = 0; s < ns; ++s) {
            const float w = fast_exp2(lse[s] - M);
            wsum += w;
            acc += w * po[(int64_t)s * D];
        }
    } else if (SG == 1) {
        float l8[8], o8[8];
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            l8[s] = s < ns ? lse[s] : -INFINITY;
            o8[s] = s < ns ? po[(int64_t)s * D] : 0.f;
        }
        float M = l8[0];
#pragma unroll
        for (int s = 1; s < 8; ++s) M = fmaxf(M, l8[s]);
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            const float w = fast_exp2(l8[s] - M);      // 2^(-inf) = 0 for the splits that do not exist
            wsum += w;
            acc += w * o8[s];
        }
    } else {
        constexpr int kWarps = D * SG / 32;
        __shared__ float sm_max[kWarps];
        __shared__ float sm_acc[SG][D];
        __shared__ float sm_w[SG];
        const int sg = threadIdx.y, tid = sg * D + threadIdx.x;
        float M = -INFINITY;                               // maximum over all splits of the row, found by all threads together
        for (int s = tid; s < ns; s += D * SG) M = fmaxf(M, lse[s]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        if ((tid & 31) == 0) sm_max[tid >> 5] = M;
        __syncthreads();
#pragma unroll
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, sm_max[w]);
#pragma unroll 4
        for (int s = sg; s < ns; s += SG) {                // this slice's splits
            const float w = fast_exp2(lse[s] - M);
            wsum += w;
            acc += w * po[(int64_t)s * D];
        }
        sm_acc[sg][threadIdx.x] = acc;
        if (threadIdx.x == 0) sm_w[sg] = wsum;
        __syncthreads();
        if (sg != 0) return;
        acc = 0.f; wsum = 0.f;
#pragma unroll
        for (int g = 0; g < SG; ++g) { acc += sm_acc[g][threadIdx.x]; wsum += sm_w[g]; }
    }
    if (p.out_f32) ((float *)p.out)[(int64_t)row * D + threadIdx.x] = acc / wsum;
    else ((uint16_t *)p.out)[(int64_t)row * D + threadIdx.x] = f32_to_16<F16>(acc / wsum);
}

// Launch the merge kernel so that its launch latency overlaps the tail of the split kernel.
template <int D, bool F16>
static cudaError_t launch_merge(const DecodeParams &p, int rows, cudaStream_t st)
{
    // Slices of threads that share a row's splits: as many (8, 4 or 1) as keep the whole grid within
    // one wave of resident threads, and 1 when no row can have more than 8 splits;
    // "decode_merge_slices" overrides.
    const int64_t wave_threads = (int64_t)device_sm_count() * 2048;
    int sg = (int64_t)rows * D * 8 <= wave_threads ? 8 : ((int64_t)rows * D * 4 <= wave_threads ? 4 : 1);
    if (g_decode_merge_slices > 0) sg = (int)g_decode_merge_slices;
    if (p.max_splits <= 8) sg = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)rows);
    cfg.blockDim = dim3(D, sg);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (sg == 8) return cudaLaunchKernelEx(&cfg, decode_merge_kernel<D, F16, 8>, p);
    if (sg == 4) return cudaLaunchKernelEx(&cfg, decode_merge_kernel<D, F16, 4>, p);
    return cudaLaunchKernelEx(&cfg, decode_merge_kernel<D, F16, 1>, p);
}

// Tokens per split. Automatic choice, from the upper bound max_seq_len of every sequence:
//   - small launches (all units = requests x kv heads fit, with splits of at most 4096 tokens, into two
//     CTAs per SM): as many equal splits per unit as keep the grid within two CTAs per SM, i.e. one
//     balanced wave; more, smaller CTAs only add per-CTA set-up and a merge with more partials;
//   - otherwise: about three waves of 3 CTAs per SM, at most 3200 tokens (large splits pay in the last
//     wave, where an SM left with one CTA cannot draw its share of the bandwidth), at least 256.
// Rounded to 64 tokens so that a pair never straddles splits.
int decode_chunk_tokens(int batch, int num_kv_heads, int max_seq_len)
{
    int64_t chunk = g_decode_chunk_tokens;
    if (chunk <= 0) {
        const int64_t sms = device_sm_count();
        const int64_t units = (int64_t)batch * num_kv_heads;
        const int64_t len = max_seq_len > 0 ? max_seq_len : 1;
        if (units * ((len + kMaxChunkTokens - 1) / kMaxChunkTokens) <= 2 * sms) {
            int64_t splits = 2 * sms / units;
            if (splits > (len + 255) / 256) splits = (len + 255) / 256;
            if (splits < 1) splits = 1;
            chunk = (len + splits - 1) / splits;
        } else {
            const int64_t want_ctas = sms * 3 * 3;
            chunk = (len * units + want_ctas - 1) / want_ctas;
            if (chunk > 3200) chunk = 3200;
        }
        if (chunk < 256) chunk = 256;
    }
    if (chunk > kMaxChunkTokens) chunk = kMaxChunkTokens;      // a warp's step list holds 32 pairs
    chunk = (chunk + 63) / 64 * 64;
    return (int)chunk;
}

size_t decode_workspace_bytes(int batch, int num_q_heads, int num_kv_heads, int head_dim, int max_seq_len)
{
    const int chunk = decode_chunk_tokens(batch, num_kv_heads, max_seq_len);
    const int64_t max_splits = ((int64_t)max_seq_len + chunk - 1) / chunk;
    if (max_splits <= 1) return 0;
    const int64_t rows = (int64_t)batch * num_q_heads * max_splits;
    return (size_t)(rows * head_dim * 4 + (rows * 4 + 255) / 256 * 256);
}

} // namespace ekv

using namespace ekv;

// ---- tensor maps of the TMA-staged decode kernel (host) ----
namespace ekv {

static int encode_2d(CUtensorMap *map, CUtensorMapDataType type, int elem_bytes, const void *base, uint64_t rows,
                     uint32_t box_x, uint32_t box_rows, CUtensorMapSwizzle swizzle)
{
    typedef CUresult (*encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static encode_fn encode = [] {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) fn = nullptr;
        return (encode_fn)fn;
    }();
    if (!encode) return EKV_ERR_CUDA;
    // a row is 128 elements: 256 bytes of 16-bit words (16 rows per slab) or 128 bytes (32 rows per slab)
    const cuuint64_t dims1[2] = {(cuuint64_t)128, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)(128 * elem_bytes)};
    const cuuint32_t box[2] = {box_x, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult rc = encode(map, type, 2, const_cast<void *>(base), dims1, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                               swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS ? EKV_OK : EKV_ERR_CUDA;
}

// The four maps of one (device, layer base pair, pool geometry); the last few are kept, since a serving loop
// calls with the same pool over and over and an encode costs about a microsecond of host time each.
static int decode_maps_for(const uint8_t *k_layer, const uint8_t *v_layer, int num_blocks, int num_kv_heads, bool need_base, DecodeMaps *out)
{
    struct Entry { const uint8_t *k, *v; int nb, hkv, dev; bool base; DecodeMaps maps; };
    constexpr int kKeep = 8;
    static thread_local Entry cache[kKeep];
    static thread_local int next = 0, used = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return EKV_ERR_CUDA;
    for (int i = 0; i < used; ++i) {
        const Entry &e = cache[i];
        if (e.k == k_layer && e.v == v_layer && e.nb == num_blocks && e.hkv == num_kv_heads && e.dev == dev && (e.base || !need_base)) {
            *out = e.maps;
            return EKV_OK;
        }
    }
    Entry &e = cache[next];
    const uint64_t rows16 = (uint64_t)num_blocks * num_kv_heads * kPageSize;     // TARGET view: 16 rows of 128 words per slab
    int rc = encode_2d(&e.maps.k_target, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, k_layer, rows16, 64, 16, CU_TENSOR_MAP_SWIZZLE_128B);
    if (!rc) rc = encode_2d(&e.maps.v_target, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, v_layer, rows16, 64, 16, CU_TENSOR_MAP_SWIZZLE_128B);
    if (!rc) rc = encode_2d(&e.maps.k_base, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, k_layer, 2 * rows16, 64, 32, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (!rc) rc = encode_2d(&e.maps.v_base, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, v_layer, 2 * rows16, 128, 32, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    e.k = k_layer; e.v = v_layer; e.nb = num_blocks; e.hkv = num_kv_heads; e.dev = dev; e.base = true;
    *out = e.maps;
    next = (next + 1) % kKeep;
    if (used < kKeep) ++used;
    return EKV_OK;
}

} // namespace ekv

static int decode_impl(const ekv_pool *pool, int32_t layer, const ekv_batch *batch, const int32_t *boundaries,
                       const void *q, void *out, int32_t num_q_heads, float sm_scale,
                       int32_t max_seq_len, void *workspace, size_t workspace_bytes, void *stream)
{
    int rc = check_pool(pool);
    if (rc) return rc;
    rc = check_batch(batch);
    if (rc) return rc;
    if (!q || !out || layer < 0 || layer >= pool->num_layers || max_seq_len < 0) return EKV_ERR_INVALID_ARG;
    if (((uintptr_t)q & 15) || ((uintptr_t)out & 15)) return EKV_ERR_INVALID_ARG;
    if (num_q_heads <= 0 || num_q_heads % pool->num_kv_heads) return EKV_ERR_INVALID_ARG;
    const int G = num_q_heads / pool->num_kv_heads;
    if (G > 8) return EKV_ERR_UNSUPPORTED;
    if (batch->has_base && !pool->tags) return EKV_ERR_INVALID_ARG;
    if ((int64_t)max_seq_len > (int64_t)batch->max_blocks * kPageSize) return EKV_ERR_INVALID_ARG;
    if (batch->batch == 0) return EKV_OK;

    DecodeParams p{};
    p.k_layer = (const uint8_t *)pool->k_pool + (int64_t)layer * pool->layer_stride_bytes;
    p.v_layer = (const uint8_t *)pool->v_pool + (int64_t)layer * pool->layer_stride_bytes;
    p.tags = pool->tags;
    p.boundaries = boundaries;
    p.block_table = batch->block_table;
    p.seq_lens = batch->seq_lens;
    p.q = (const __nv_bfloat16 *)q;
    p.out = (__nv_bfloat16 *)out;
    p.block_bytes = (int64_t)pool->num_kv_heads * kPageSize * pool->head_dim * 2;
    p.batch = batch->batch;
    p.num_q_heads = num_q_heads;
    p.num_kv_heads = pool->num_kv_heads;
    p.group = G;
    p.max_blocks = batch->max_blocks;
    p.chunk_tokens = decode_chunk_tokens(batch->batch, pool->num_kv_heads, max_seq_len);
    p.max_splits = max_seq_len > 0 ? (max_seq_len + p.chunk_tokens - 1) / p.chunk_tokens : 1;
    p.scale_log2 = sm_scale * 1.4426950408889634f;
    p.out_f32 = g_attn_out_f32 ? 1 : 0;
    p.two_term = (int)g_decode_two_term;
    if (p.max_splits > 1) {
        const size_t need = decode_workspace_bytes(batch->batch, num_q_heads, pool->num_kv_heads, pool->head_dim, max_seq_len);
        if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return EKV_ERR_WORKSPACE;
        const int64_t rows = (int64_t)batch->batch * num_q_heads * p.max_splits;
        p.part_o = (float *)workspace;
        p.part_lse = (float *)((uint8_t *)workspace + rows * pool->head_dim * 4);
    }
    const int64_t ctas = (int64_t)batch->batch * pool->num_kv_heads * p.max_splits;
    if (ctas > 0x7fffffffLL) return EKV_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const bool hb = batch->has_base != 0;
    // Both paths run the ring-staged kernel: the native instantiation (no BASE block in the batch)
    // has every tag load, byte path and pair rule compiled out. Variant 1 selects the simpler
    // page-stepped, register-direct kernel, kept as the plain bf16 paged-decode comparator.
    const int variant = boundaries ? 3 : (g_decode_variant ? (int)g_decode_variant : 3);
    const bool f16 = pool->elem_type == EKV_FP16;
    if (f16 && variant == 1) return EKV_ERR_UNSUPPORTED;      // the comparator kernel is bf16 only
    const unsigned nb = (unsigned)ctas;
    cudaError_t aerr = cudaSuccess;
    // Staging of the K/V slabs: cp.async (16 bytes per lane and instruction) by default; with "decode_staging" = 2,
    // at head_dim 128, tensor copies (TMA: one lane issues two box copies per slab, completion on an mbarrier).
    // Measured 1-2 % slower than cp.async on every decode configuration, so it is kept as an option only.
    const bool tma = pool->head_dim == 128 && variant != 1 && g_decode_staging == 2;
    DecodeMaps maps{};
    if (tma) {
        if ((int64_t)pool->num_blocks * pool->num_kv_heads * 32 > 0x7fffffffLL) return EKV_ERR_UNSUPPORTED;    // row coordinates are 32-bit
        const int mrc = decode_maps_for(p.k_layer, p.v_layer, pool->num_blocks, pool->num_kv_heads, hb, &maps);
        if (mrc) return mrc;
    }
#define EKV_LAUNCH_RING_M(DD, HB, BD, FF, TT)                                                             \
    do {                                                                                                  \
        aerr = cudaFuncSetAttribute(decode_ring_kernel<DD, HB, 2, 3, BD, FF, TT>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                    (int)ring_smem_bytes<DD, 2>());                                       \
        if (aerr == cudaSuccess)                                                                          \
            aerr = launch_pdl(decode_ring_kernel<DD, HB, 2, 3, BD, FF, TT>, nb, kDecodeThreads, ring_smem_bytes<DD, 2>(), st, p, maps); \
    } while (0)
#define EKV_LAUNCH_RING_T(DD, HB, BD, FF)                                                                 \
    do {                                                                                                  \
        if (DD == 128 && tma) EKV_LAUNCH_RING_M(128, HB, BD, FF, true); else EKV_LAUNCH_RING_M(DD, HB, BD, FF, false); \
    } while (0)
#define EKV_LAUNCH_RING_B(DD, HB, BD)                                                                     \
    do {                                                                                                  \
        if (f16) EKV_LAUNCH_RING_T(DD, HB, BD, true); else EKV_LAUNCH_RING_T(DD, HB, BD, false);          \
    } while (0)
#define EKV_LAUNCH_RING(DD, HB)                                                                           \
    do {                                                                                                  \
        if (HB && boundaries) EKV_LAUNCH_RING_B(DD, HB, true); else EKV_LAUNCH_RING_B(DD, HB, false);     \
    } while (0)
    if (pool->head_dim == 128) {
        { MainKernelScope scope(st);
        if (variant == 1) { if (hb) decode_page_kernel<128, true><<<nb, kDecodeThreads, 0, st>>>(p);
                            else    decode_page_kernel<128, false><<<nb, kDecodeThreads, 0, st>>>(p); }
        else              { if (hb) EKV_LAUNCH_RING(128, true); else EKV_LAUNCH_RING(128, false); } }
        if (p.max_splits > 1 && aerr == cudaSuccess)
            aerr = f16 ? launch_merge<128, true>(p, batch->batch * num_q_heads, st) : launch_merge<128, false>(p, batch->batch * num_q_heads, st);
    } else {
        { MainKernelScope scope(st);
        if (variant == 1) { if (hb) decode_page_kernel<64, true><<<nb, kDecodeThreads, 0, st>>>(p);
                            else    decode_page_kernel<64, false><<<nb, kDecodeThreads, 0, st>>>(p); }
        else              { if (hb) EKV_LAUNCH_RING(64, true); else EKV_LAUNCH_RING(64, false); } }
        if (p.max_splits > 1 && aerr == cudaSuccess)
            aerr = f16 ? launch_merge<64, true>(p, batch->batch * num_q_heads, st) : launch_merge<64, false>(p, batch->batch * num_q_heads, st);
    }
#undef EKV_LAUNCH_RING
#undef EKV_LAUNCH_RING_B
#undef EKV_LAUNCH_RING_T
#undef EKV_LAUNCH_RING_M
    if (aerr != cudaSuccess) return EKV_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? EKV_OK : EKV_ERR_CUDA;
}

extern "C" int ekv_attn_decode(const ekv_pool *pool, int32_t layer, const ekv_batch *batch,
                               const void *q, void *out, int32_t num_q_heads, float sm_scale,
                               int32_t max_seq_len, void *workspace, size_t workspace_bytes, void *stream)
{
    return decode_impl(pool, layer, batch, nullptr, q, out, num_q_heads, sm_scale, max_seq_len, workspace,
                       workspace_bytes, stream);
}

extern "C" int ekv_attn_decode_structured(const ekv_pool *pool, int32_t layer, const ekv_batch *batch,
                                          const int32_t *boundaries, const void *q, void *out,
                                          int32_t num_q_heads, float sm_scale, int32_t max_seq_len,
                                          void *workspace, size_t workspace_bytes, void *stream)
{
    if (!boundaries || !batch || !batch->has_base) return EKV_ERR_INVALID_ARG;
    return decode_impl(pool, layer, batch, boundaries, q, out, num_q_heads, sm_scale, max_seq_len, workspace,
                       workspace_bytes, stream);
}

// ---- metadata lowering: per-sequence mode boundaries from the per-block tags -----------------
namespace ekv {

// One warp per request: scan the pair modes, report the first BASE pair, one past the last, and
// whether everything in between is BASE (the TARGET-BASE-TARGET shape with at most two boundaries).
__global__ void lower_metadata_kernel(const int32_t *block_table, const int32_t *seq_lens, const uint8_t *tags,
                                      int batch, int max_blocks, int32_t *boundaries, int32_t *flags)
{
    const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= batch) return;
    const int L = seq_lens[r];
    const int npairs = (L + 2 * kPageSize - 1) / (2 * kPageSize);
    int first = 0x7fffffff, last = -1, count = 0;
    for (int pp = lane; pp < npairs; pp += 32) {
        if (tags[block_table[(int64_t)r * max_blocks + 2 * pp]] == EKV_BASE) {
            first = min(first, pp); last = max(last, pp); ++count;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        first = min(first, __shfl_xor_sync(0xffffffffu, first, o));
        last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
        count += __shfl_xor_sync(0xffffffffu, count, o);
    }
    if (lane == 0) {
        const bool any = count > 0;
        boundaries[2 * r] = any ? first : 0;
        boundaries[2 * r + 1] = any ? last + 1 : 0;
        if (any) atomicOr(&flags[0], 1);
        if (any && count != last + 1 - first) atomicOr(&flags[1], 1);
    }
}

} // namespace ekv

extern "C" int ekv_lower_metadata(const ekv_pool *pool, const ekv_batch *batch, int32_t *boundaries,
                                  int32_t *flags, void *stream)
{
    int rc = check_pool(pool);
    if (rc) return rc;
    rc = check_batch(batch);
    if (rc) return rc;
    if (!pool->tags || !boundaries || !flags) return EKV_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(flags, 0, 2 * sizeof(int32_t), st) != cudaSuccess) return EKV_ERR_CUDA;
    if (batch->batch == 0) return EKV_OK;
    lower_metadata_kernel<<<(batch->batch + 3) / 4, 128, 0, st>>>(batch->block_table, batch->seq_lens, pool->tags,
                                                                 batch->batch, batch->max_blocks, boundaries, flags);
    return cudaGetLastError() == cudaSuccess ? EKV_OK : EKV_ERR_CUDA;
}

// ---- decode attention for callers that cannot allocate --------------------------------------
//
// Same computation as ekv_attn_decode, but the split-K scratch (per-split partial outputs and
// log-sum-exps) lives in a fixed array inside the library image instead of a caller workspace.
namespace ekv {

constexpr size_t kNoAllocScratchBytes = 16u << 20;      // 16 MiB, held by every GPU that loads the library
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

constexpr int kMaxDevices = 64;
static std::atomic<void *> g_noalloc_scratch_ptr[kMaxDevices];   // device address of the array, per device; null = not asked yet

// In host code `g_noalloc_scratch` is only a handle; the device address has to be asked for,
// once per device, with that device current. Host threads that make their first calls at the
// same time each ask and store the same answer (release / acquire on the slot).
static int noalloc_scratch_address(void **ptr)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return EKV_ERR_CUDA;
    void *p = g_noalloc_scratch_ptr[dev].load(std::memory_order_acquire);
    if (!p) {
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) return EKV_ERR_CUDA;
        g_noalloc_scratch_ptr[dev].store(p, std::memory_order_release);
    }
    *ptr = p;
    return EKV_OK;
}

} // namespace ekv

extern "C" size_t ekv_attn_decode_noalloc_max_bytes(void) { return ekv::kNoAllocScratchBytes; }

extern "C" int ekv_attn_decode_noalloc(const ekv_pool *pool, int32_t layer, const ekv_batch *batch,
                                       const void *q, void *out, int32_t num_q_heads, float sm_scale,
                                       int32_t max_seq_len, void *stream)
{
    int rc0 = check_pool(pool);
    if (rc0) return rc0;
    rc0 = check_batch(batch);
    if (rc0) return rc0;
    if (num_q_heads <= 0 || max_seq_len < 0) return EKV_ERR_INVALID_ARG;
    // Refuse, before touching the GPU, any shape whose partials would not fit the fixed array.
    const size_t need = ekv_attn_workspace_bytes(pool, batch->batch, num_q_heads, max_seq_len, 0);
    if (need > ekv::kNoAllocScratchBytes) return EKV_ERR_WORKSPACE;
    void *scratch = nullptr;
    const int rc = ekv::noalloc_scratch_address(&scratch);
    if (rc != EKV_OK) return rc;
    // Every partial that the merge kernel reads is written by the split kernel of the same call,
    // so nothing in the array has to start at zero and nothing is cleared.
    return ekv_attn_decode(pool, layer, batch, q, out, num_q_heads, sm_scale, max_seq_len,
                           scratch, ekv::kNoAllocScratchBytes, stream);
}

// Host-synchronising debug query: status word of the TMA-staged decode kernel since the last call. Resets the word.
extern "C" int ekv_decode_status(void)
{
    int v = -1, zero = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return EKV_ERR_CUDA;
    if (cudaMemcpyFromSymbol(&v, ekv::g_decode_ring_status, sizeof(int)) != cudaSuccess) return EKV_ERR_CUDA;
    if (cudaMemcpyToSymbol(ekv::g_decode_ring_status, &zero, sizeof(int)) != cudaSuccess) return EKV_ERR_CUDA;
    return v;
}
