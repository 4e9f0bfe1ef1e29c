// Chunked-prefill attention over a mixed-fidelity paged prefix on the 5th-generation tensor
// cores, warp-specialised: S = Q K^T and O += P V are tcgen05.mma (kind::f16, fp32 accumulators in
// tensor memory), head_dim 128.
//
// CTA = (request, kv head, 256 query rows) = two row tiles of 128; a row is (query token, query
// head of the group), so every K/V tile fetched serves 256 rows. The KV axis is walked in tiles of
// 128 tokens (8 pages). 24 warps; the first eight (two warpgroups) are utility warps that give
// registers to the sixteen softmax warps (setmaxnreg: 64 and 88 per thread of the 80 launched with):
//   - copy issuer (1 warp, one lane per copy): K and V tiles arrive by TMA into the canonical
//     128-byte-swizzled layout ([dim half][token][64 dims]): a full TARGET page is two tiled tensor
//     copies (16 tokens x 64 dims, hardware swizzle) that complete on the stage's "full" barrier; a
//     BASE page is one 2 KiB bulk copy of its packed bytes, parked in the page's own upper-half
//     rows, that completes on the stage's "raw" barrier. Two K stages and two V stages. What each
//     page needs is read from page words laid down once per CTA.
//   - expander warps (6): wait for the raw bytes and expand them (byte << 8, the load rule of
//     Sec. 3.2 / App. B.3) into the same bf16 rows, a half warp per token row, so the tensor cores
//     see one format; they also fetch Q and the one page per request that may be partly filled
//     (plain cp.async with zero fill), then arrive on "full".
//   - MMA issuer (1 warp, one effective lane): S_w(j) = Q_w K_j^T (both operands from shared
//     memory, K-major) and O_w += P_w(j) V_j with P read from TENSOR MEMORY (the A operand) and V
//     as the MN-major B operand from shared memory. Order in the tensor pipe:
//         S_0(0) S_1(0) | PV_0(0) S_0(1) PV_1(0) S_1(1) | PV_0(1) S_0(2) ...
//     so the softmax of one row tile runs while the tensor cores work on the other.
//   - softmax warps (16): four threads per row (TMEM lane), 32 of the 128 scores each, read once
//     from tensor memory and kept in registers. All sixteen warps work on ONE row tile at a time,
//     in the order S_0(j), S_1(j), S_0(j+1), ...: four warps per scheduler keep the special-function
//     unit busy, and while one row tile is exponentiated the tensor cores run PV and the next S
//     of the other. The exponentials of a tile are taken against the row's reference maximum
//     as it stands; the sum of a thread's 32 exponentials shows whether every score was within
//     2^8 of the reference, and the verdicts of the 128 threads that share 32 rows are OR-ed by
//     the named barrier that also puts every score read before any probability write. Only
//     after a failed test do those four warps take the row maxima (swapped through shared
//     memory), move the references, rescale O in TMEM and redo the tile. Exponentials and the
//     row sum run on packed f32x2 instructions; the probabilities are written as packed 16-bit
//     pairs over the scores (P aliases S).
//   - two-term probabilities (template parameter TWO_TERM; the default for bf16 pools): the softmax
//     thread also forms the rounding residual of every probability (kept negated, hi - p) and writes
//     it, as 16-bit pairs, into the upper 64 columns of the row tile's score region; the MMA issuer
//     follows PV_w(j) with a second pass over the same V tile whose A operand is that region, with
//     the negate-A bit of the instruction descriptor set. One bf16 term alone leaves up to 5e-3 of
//     output error on rows that two or three tokens dominate.
// TMEM columns: S_0/P_0 [0,128) (probabilities in [0,64), their residuals in [64,128)), S_1/P_1
// [128,256) likewise, O_0 [256,384), O_1 [384,512).
// Every wait on an mbarrier is bounded; on expiry the thread records a status word, stops
// waiting (it still arrives where others count on it), and the CTA frees its tensor memory.
#include "ekv_common.cuh"
#include <cuda.h>
#include <math.h>

namespace ekv {

constexpr int kWsRowThreads = 4;                   // softmax threads per row (each takes 128 / kWsRowThreads scores of a KV tile)
constexpr int kWsCols = 128 / kWsRowThreads;       // scores per thread, and output columns per thread
constexpr int kWsSoftmaxThreads = 128 * kWsRowThreads;
constexpr int kWsLoaderThreads = 192;              // expanders: 12 half warps, one token row (16 x 8 packed bytes) each per pass
constexpr int kWsThreads = kWsSoftmaxThreads + kWsLoaderThreads + 64;   // + the MMA-issuing warp + the copy-issuing warp
constexpr int kWsRows = 128;                       // rows per row tile (TMEM lanes)
constexpr int kWsKv = 128;                         // KV tokens per tile
constexpr int kWsRowPasses = (kWsKv + 11) / 12;    // expander passes over the 128 token rows of a tile
constexpr int kWsD = 128;
constexpr int kWsHalf = 128 * 128;                 // 16 KiB: [128 rows or tokens][64 dims]
constexpr int kWsTile = 2 * kWsHalf;               // 32 KiB: a Q row tile, a K tile or a V tile
constexpr int kWsStages = 2;
constexpr int kWsSmemBytes = 2 * kWsTile + 2 * kWsStages * kWsTile;     // 192 KiB
constexpr int kWsSpinLimit = 1 << 22;
constexpr float kWsSafeSum = 256.0f;               // 2^8: a thread whose exponentials of a tile sum to this or less has no score more than 8 (log2 units) above the reference maximum
constexpr float kWsMoveMargin = 3.0f;              // log2 units; 32 columns x 2^3 = kWsSafeSum, so a row left in place cannot fail the sum test
constexpr int kWsPagesPerTile = kWsKv / kPageSize; // 8
constexpr int kWsPartFloats = 2 * kWsRows * (kWsD + 2);   // a piece's unnormalised O [32 column quads][256 rows][4], then (reference maximum, row sum) [256 rows][2]
constexpr int kWsMaxSplits = 4;

// barrier slots
enum { kPgNone = 0, kPgTarget = 1, kPgBase = 2, kPgPartial = 3 };
enum { kBarKFull = 0, kBarVFull = 2, kBarKEmpty = 4, kBarVEmpty = 6, kBarSFull = 8, kBarPFull = 10, kBarODone = 12,
       kBarKRaw = 13, kBarVRaw = 15, kBarCount = 17 };

__device__ int g_prefill_ws_status = 0;            // 0 ok; 1 a bounded wait expired; 2 shared memory misaligned

struct PrefillTcParams {
    const uint8_t *k_layer, *v_layer;
    const uint8_t *tags;
    const int32_t *block_table, *seq_lens, *q_start;
    const __nv_bfloat16 *q;
    __nv_bfloat16 *out;
    int64_t block_bytes;
    int batch, num_q_heads, num_kv_heads, group, max_blocks;
    int group_rows;              // rows a token takes in a tile: the group size rounded up to a power of two
    int q_tiles;
    float scale_log2;
    // balancing of the last wave (warp-specialised kernel only): CTAs from split_first on are pieces,
    // `splits` per unit, each over a share of the unit's KV tiles; the last piece to finish merges
    int split_first, splits;
    float *part;                 // [unit - split_first][piece]: kWsPartFloats floats
    int *part_count;             // [unit - split_first], zero at launch
    int out_f32;                 // debug: `out` is float and receives the unrounded result
};

__device__ __forceinline__ uint32_t ws_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ws_cp16(uint32_t dst, const void *src, int bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void ws_commit_group() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void ws_wait_group() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }
__device__ __forceinline__ void ws_fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void ws_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void ws_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void ws_mbar_init(uint32_t bar, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void ws_mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ void ws_mbar_expect(uint32_t bar, uint32_t bytes)        // one arrival + `bytes` expected
{
    if (bytes) asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
    else ws_mbar_arrive(bar);
}
// Tiled TMA copy of one box at element (x, y) into this CTA's shared memory; completes on `bar`.
__device__ __forceinline__ void ws_tma_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 :: "r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
// Untiled bulk copy of `bytes` (multiple of 16, both addresses 16-byte aligned); completes on `bar`.
__device__ __forceinline__ void ws_bulk(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Bounded wait: false when the limit is hit. HINT_NS is the time the hardware may keep the thread
// suspended inside one try_wait before it reports "not yet"; with a long hint fewer polls are
// allowed, so that the bound stays about a second either way.
template <int HINT_NS>
__device__ __forceinline__ bool ws_mbar_wait(uint32_t bar, uint32_t parity)
{
    constexpr int kPolls = HINT_NS >= 1000 ? (1 << 16) : kWsSpinLimit;
    for (int i = 0; i < kPolls; ++i) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity), "r"(HINT_NS > 0 ? (uint32_t)HINT_NS : 1u) : "memory");
        if (ok) return true;
    }
    return false;
}
// The issuing warp runs its loop with all lanes (so that addresses and descriptors stay in the uniform
// datapath); `leader` is true in the one lane whose instruction takes effect.
// One non-blocking look at a barrier phase.
__device__ __forceinline__ bool ws_mbar_test(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void ws_commit_mma(uint32_t bar, uint32_t leader)
{
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
                 "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" :: "r"(bar), "r"(leader) : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, version 1.
__device__ __forceinline__ uint64_t ws_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    return (uint64_t)((addr >> 4) & 0x3FFF) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16)
           | ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) | (1ull << 46) | (2ull << 61);
}
// D[tmem] (+)= A[smem] * B[smem], K = 16, bf16 -> fp32.
__device__ __forceinline__ void ws_mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate, uint32_t leader)
{
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %4, 0;\n\tsetp.ne.b32 q, %5, 0;\n\t"
                 "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(leader) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem], K = 16: A is 128 lanes x 8 columns of packed bf16 pairs.
__device__ __forceinline__ void ws_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate, uint32_t leader)
{
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %4, 0;\n\tsetp.ne.b32 q, %5, 0;\n\t"
                 "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 :: "r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(leader) : "memory");
}
__device__ __forceinline__ void ws_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void ws_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void ws_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void ws_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void ws_st16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
                 "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 :: "r"(taddr),
                    "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                    "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
                 : "memory");
}

// Packed pairs of fp32 (sm_100): one instruction for two lanes of the softmax arithmetic.
__device__ __forceinline__ uint64_t ws_pack2(float lo, float hi)
{
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ void ws_unpack2(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t ws_fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t ws_add2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// lo += bf16 low half of pw, hi += bf16 high half, both exact conversions, sums rounded to nearest in fp32
__device__ __forceinline__ void ws_add_bf16x2(float &lo, float &hi, uint32_t pw)
{
    asm("{\n\t.reg .b16 hl, hh;\n\tmov.b32 {hl, hh}, %2;\n\t"
        "add.rn.f32.bf16 %0, hl, %0;\n\tadd.rn.f32.bf16 %1, hh, %1;\n\t}"
        : "+f"(lo), "+f"(hi) : "r"(pw));
}
// d0 = (low 16-bit half of pw) - c0, d1 = (high half) - c1: the halves widen exactly, the differences round to nearest in fp32
template <bool F16>
__device__ __forceinline__ void ws_sub_16x2(float &d0, float &d1, uint32_t pw, float c0, float c1)
{
    if (F16)
        asm("{\n\t.reg .b16 hl, hh;\n\tmov.b32 {hl, hh}, %2;\n\t"
            "sub.rn.f32.f16 %0, hl, %3;\n\tsub.rn.f32.f16 %1, hh, %4;\n\t}"
            : "=f"(d0), "=f"(d1) : "r"(pw), "f"(c0), "f"(c1));
    else
        asm("{\n\t.reg .b16 hl, hh;\n\tmov.b32 {hl, hh}, %2;\n\t"
            "sub.rn.f32.bf16 %0, hl, %3;\n\tsub.rn.f32.bf16 %1, hh, %4;\n\t}"
            : "=f"(d0), "=f"(d1) : "r"(pw), "f"(c0), "f"(c1));
}
__device__ __forceinline__ float ws_max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Byte offset of 16-byte chunk `ch16` (0..15 along the 128 dims) of row `row` in a two-half tile;
// rows are 128 bytes, chunks XOR-swizzled with the row.
__device__ __forceinline__ uint32_t ws_tile_off(int row, int ch16)
{
    return (uint32_t)((ch16 >> 3) * kWsHalf + row * 128 + (((ch16 & 7) ^ (row & 7)) << 4));
}

template <bool HAS_BASE, bool F16, bool TWO_TERM, bool OUT_F32 = false>
__global__ void __launch_bounds__(kWsThreads, 1) prefill_ws_kernel(PrefillTcParams p, const __grid_constant__ CUtensorMap map_k,
                                                                   const __grid_constant__ CUtensorMap map_v)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t *q_s = smem;                                  // 2 row tiles
    uint8_t *k_s = smem + 2 * kWsTile;                    // 2 stages
    uint8_t *v_s = k_s + kWsStages * kWsTile;             // 2 stages
    uint64_t *bars = (uint64_t *)(smem + kWsSmemBytes);
    uint32_t *tmem_slot = (uint32_t *)(bars + kBarCount + 1);
    float *xch = (float *)(tmem_slot + 4);                // mailboxes of the row halves: maxima [2 parities][256], sums [2 row tiles][256]
    int32_t *pages = (int32_t *)(xch + 4 * kWsSoftmaxThreads);        // [n_tiles * 8], then tinfo [n_tiles]

    // Roles are laid out by a rotated thread index: the four utility warps are the first warps of the CTA.
    const int tid = (int)((threadIdx.x + kWsSoftmaxThreads) % kWsThreads), warp = tid >> 5;
    // A token's query heads of this kv head take group_rows consecutive rows (the group size rounded up
    // to a power of two, so that it divides the tile); rows past the real group are dead: zero queries, no store.
    const int G = p.group, Gp = p.group_rows;
    const int tok_m = kWsRows / Gp;                       // query tokens per row tile

    int unit = blockIdx.x, piece = 0, n_pieces = 1;
    if (unit >= p.split_first) {
        const int k = unit - p.split_first;
        unit = p.split_first + k / p.splits;
        piece = k % p.splits;
        n_pieces = p.splits;
    }
    int idx = unit;
    const int qt = p.q_tiles - 1 - idx % p.q_tiles; idx /= p.q_tiles;   // longest KV ranges first
    const int g = idx % p.num_kv_heads;
    const int r = idx / p.num_kv_heads;
    const int qs = p.q_start[r];
    const int C = p.q_start[r + 1] - qs;
    const int L = p.seq_lens[r];
    const int i0 = qt * 2 * tok_m;
    if (i0 >= C) return;                                  // uniform over the CTA, before any allocation
    const int i1 = min(C, i0 + 2 * tok_m);
    const int n_kv = L - C + i1;
    const int n_tiles_all = (n_kv + kWsKv - 1) / kWsKv;   // >= 1
    const int tile0 = piece * n_tiles_all / n_pieces;     // this CTA's share of the KV tiles (all of them unless it is a piece)
    const int n_tiles = (piece + 1) * n_tiles_all / n_pieces - tile0;
    const int n_pages = (n_kv + kPageSize - 1) / kPageSize;

    uint32_t *tinfo = (uint32_t *)(pages + n_tiles * kWsPagesPerTile);

    if (ws_smem_u32(smem) & 1023u) {                      // the swizzle atoms need 1024-byte alignment
        if (tid == 0) atomicExch(&g_prefill_ws_status, 2);
        return;
    }
    // ---- set-up: tensor memory, barriers, block-table entries ----
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(ws_smem_u32(tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 32) {
        for (int i = 0; i < 4; ++i) ws_mbar_init(ws_smem_u32(&bars[kBarKFull + i]), kWsLoaderThreads + 1);   // K full, V full: expanders + copy issuer
        for (int i = 0; i < 4; ++i) ws_mbar_init(ws_smem_u32(&bars[kBarKRaw + i]), 1);                       // K raw, V raw
        for (int i = 0; i < 4; ++i) ws_mbar_init(ws_smem_u32(&bars[kBarKEmpty + i]), 1);                 // K empty, V empty
        for (int i = 0; i < 2; ++i) ws_mbar_init(ws_smem_u32(&bars[kBarSFull + i]), 1);
        for (int i = 0; i < 2; ++i) ws_mbar_init(ws_smem_u32(&bars[kBarPFull + i]), kWsSoftmaxThreads);
        ws_mbar_init(ws_smem_u32(&bars[kBarODone]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // Page words for the copy issuer and the expanders, padded to whole tiles: kind in bits 0-1 (kPgNone,
    // kPgTarget = full TARGET page, kPgBase, kPgPartial = TARGET page that ends the request), and above it
    // the page's slab index (phys * num_kv_heads + g), for a BASE page doubled plus the member.
    for (int lbl = tid; lbl < n_tiles * kWsPagesPerTile; lbl += kWsThreads) {
        const int lb = tile0 * kWsPagesPerTile + lbl;
        int word = kPgNone;
        if (lb < n_pages) {
            const int phys = p.block_table[(int64_t)r * p.max_blocks + lb];
            int tag = 0;
            if (HAS_BASE) tag = p.tags[phys];
            const int slab_idx = phys * p.num_kv_heads + g;
            if (tag) word = kPgBase | ((2 * slab_idx + (lb & 1)) << 2);
            else word = (L - lb * kPageSize >= kPageSize ? kPgTarget : kPgPartial) | (slab_idx << 2);
        }
        pages[lbl] = word;
    }
    __syncthreads();
    // per tile: BASE pages (bits 0-7), partly filled pages (8-15), number of full TARGET pages (16-23), of BASE pages (24-31)
    for (int j = tid; j < n_tiles; j += kWsThreads) {
        uint32_t info = 0;
        for (int pg = 0; pg < kWsPagesPerTile; ++pg) {
            const int kind = pages[j * kWsPagesPerTile + pg] & 3;
            if (kind == kPgBase) info += (1u << pg) + (1u << 24);
            else if (kind == kPgPartial) info += 1u << (8 + pg);
            else if (kind == kPgTarget) info += 1u << 16;
        }
        tinfo[j] = info;
    }
    // K/V stages start as zeros: rows that no copy ever fills (beyond the last page) must hold finite values
    for (int i = tid; i < 2 * kWsStages * kWsTile / 16; i += kWsThreads) *(uint4 *)(k_s + (size_t)i * 16) = make_uint4(0u, 0u, 0u, 0u);
    ws_fence_async_proxy();
    ws_fence_before();
    __syncthreads();
    ws_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t bar0 = ws_smem_u32(bars);
    auto bar = [&](int slot) { return bar0 + (uint32_t)slot * 8u; };
    bool dead = false;                                    // a bounded wait expired: stop waiting
    auto wait = [&](int slot, uint32_t parity) {          // the MMA issuer: polls without pause
        if (!dead && !ws_mbar_test(bar(slot), parity) && !ws_mbar_wait<0>(bar(slot), parity)) dead = true;
    };
    auto wait_idle = [&](int slot, uint32_t parity) {     // copy issuer, expanders: long waits off the critical path
        if (!dead && !ws_mbar_wait<20000>(bar(slot), parity)) dead = true;
    };
    auto wait_warp = [&](int slot, uint32_t parity) {     // softmax warps, which go on to warp-wide tensor-memory accesses
        // the phase has usually completed already: one plain test first (a try_wait costs a few hundred cycles even then)
        if (!dead && !ws_mbar_test(bar(slot), parity) && !ws_mbar_wait<20000>(bar(slot), parity)) dead = true;
        __syncwarp();
    };

    // Registers move from the utility warps (two warpgroups: expanders and the two issuers) to the softmax warps.
    // The pool is what the launch allocated (threads x registers per thread) and a request beyond it faults:
    // 768 threads x 80 = 512 x 88 + 256 x 64.
    static_assert(kWsRowThreads == 4 && kWsThreads == 768, "the register split below is for sixteen softmax warps of 24");
    if (warp < 16) asm volatile("setmaxnreg.inc.sync.aligned.u32 88;" ::: "memory");
    else asm volatile("setmaxnreg.dec.sync.aligned.u32 64;" ::: "memory");

    if (warp < 4 * kWsRowThreads) {
        // =========================== softmax: all softmax warps on one row tile at a time ===========================
        // kWsRowThreads threads per row (TMEM lane): warp -> lanes 32 * (warp & 3), column part hf = warp >> 2
        // (kWsCols of the 128 scores of a KV tile); partner warps = same warp & 3. The warps work through
        // S_0(j), S_1(j), S_0(j+1), ...: while they exponentiate one row tile, the tensor cores run PV and the
        // next S of the other.
        const int hf = warp >> 2, row = tid & 127;
        const uint32_t tmem_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        const int pair_bar = 1 + (warp & 3);              // named barrier of the warps that share these 32 rows
        int row_i[2], row_pos[2], pos_min[2];
        float m_ref[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};      // l over this thread's columns only
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            row_i[w] = i0 + w * tok_m + row / Gp;
            row_pos[w] = row_i[w] < C ? (L - C + row_i[w]) : -1;
            pos_min[w] = L - C + i0 + w * tok_m;          // smallest position of the row tile
        }
        int n_xch = 0;                                    // exchanges done so far (double-buffered mailbox)

#pragma unroll 1
        for (int j = 0; j < n_tiles; ++j) {
#pragma unroll
            for (int w = 0; w < 2; ++w) {
                const uint32_t tmem_s = tmem_lane + (uint32_t)(w * kWsKv + hf * kWsCols);             // this thread's 64 scores
                const uint32_t tmem_p = tmem_lane + (uint32_t)(w * kWsKv + hf * (kWsCols / 2));             // their probabilities (P aliases S)
                const uint32_t tmem_o = tmem_lane + (uint32_t)(2 * kWsKv + w * kWsD + hf * kWsCols);  // this thread's 64 output columns
                wait_warp(kBarSFull + w, (uint32_t)(j & 1));   // S_w(j) is in tensor memory; PV_w(j-1) has completed
                ws_fence_after();
                const int kv0 = (tile0 + j) * kWsKv + hf * kWsCols;
                const bool need_mask = kv0 + kWsCols - 1 > pos_min[w];
                uint32_t sc[kWsCols / 32][32];
#pragma unroll
                for (int c = 0; c < kWsCols / 32; ++c) ws_ld32(tmem_s + 32 * c, sc[c]);
                ws_wait_ld();
                if (need_mask) {
#pragma unroll
                    for (int c = 0; c < kWsCols / 32; ++c)
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (kv0 + 32 * c + i > row_pos[w]) sc[c][i] = 0xff800000u;        // -inf
                }
                // The exponentials are taken against the reference maximum as it stands, and their sum tells
                // whether that was safe: a sum of at most kWsSafeSum over this thread's columns
                // means that no score of them stands more than the threshold above the reference. Only when
                // some row of the 32 fails that test (or has no reference yet) do the warps of these rows
                // take the row maxima, move the references and redo the tile. The named barrier that carries
                // the vote is needed in any case: it puts every score read of a row before any probability
                // write (P of one part lands on S of another).
                static_assert(kWsCols == 32, "one 32-column tensor-memory load per thread and tile");
                const uint64_t scale2 = ws_pack2(p.scale_log2, p.scale_log2);
                uint32_t pw[16];
                uint32_t pl[TWO_TERM ? 16 : 1];           // two-term mode: the rounding residuals p - hi, as 16-bit pairs like pw
                float tile_sum;
                // P = 2^(s * scale - m) as packed 16-bit pairs over the scores. One-term mode: the row sum uses the
                // rounded values (bf16) or the fp32 ones (fp16). Two-term mode: P enters the PV product as hi + lo,
                // hi = the rounded probability, lo = its rounding residual (exact in fp32, then rounded to 16 bits
                // itself: 2^-17 relative to p), and the sum takes the fp32 values.
                auto exponentials = [&](float m) {
                    const float neg_m = m == -INFINITY ? 0.f : -m;
                    const uint64_t neg_m2 = ws_pack2(neg_m, neg_m);
                    uint64_t sum2[2] = {0ull, 0ull};      // {even columns, odd columns} x 2 chains (fp32 sums)
                    float sum1[2][2] = {{0.f, 0.f}, {0.f, 0.f}};              // the same four chains (sums of the rounded bf16 values)
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float s0 = __uint_as_float(sc[0][2 * i]), s1 = __uint_as_float(sc[0][2 * i + 1]);
                        float x0, x1;
                        ws_unpack2(ws_fma2(ws_pack2(s0, s1), scale2, neg_m2), x0, x1);
                        const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                        pw[i] = pack_16x2<F16>(p0, p1);
                        if (TWO_TERM) {
                            // pl holds hi - p, the NEGATED residual: one mixed-precision subtract per element, no
                            // unpacking; the instruction descriptor of the residual MMA negates A to match
                            float n0, n1;
                            ws_sub_16x2<F16>(n0, n1, pw[i], p0, p1);
                            pl[i] = pack_16x2<F16>(n0, n1);
                            sum2[i & 1] = ws_add2(sum2[i & 1], ws_pack2(p0, p1));
                        } else if (F16) {
                            // fp16 rounds eight times finer than bf16 and takes the fp32 values as they are
                            sum2[i & 1] = ws_add2(sum2[i & 1], ws_pack2(p0, p1));
                        } else {
                            // bf16, one term: the sum has to see the rounding that P enters the PV product with; the
                            // bf16 halves go into the fp32 sums as they are (mixed-precision add): no unpacking
                            ws_add_bf16x2(sum1[i & 1][0], sum1[i & 1][1], pw[i]);
                        }
                    }
                    float e0 = sum1[0][0], o0 = sum1[0][1], e1 = sum1[1][0], o1 = sum1[1][1];
                    if (F16 || TWO_TERM) {
                        ws_unpack2(sum2[0], e0, o0);
                        ws_unpack2(sum2[1], e1, o1);
                    }
                    tile_sum = (e0 + o0) + (e1 + o1);
                };
                exponentials(m_ref[w]);
                // not (sum <= bound) also catches an overflowed or undefined sum
                const bool want = (m_ref[w] == -INFINITY) ? (kv0 <= row_pos[w]) : !(tile_sum <= kWsSafeSum);
                uint32_t any_want;
                asm volatile("{\n\t.reg .pred pin, pout;\n\tsetp.ne.u32 pin, %1, 0;\n\t"
                             "bar.red.or.pred pout, %2, %3, pin;\n\tselp.u32 %0, 1, 0, pout;\n\t}"
                             : "=r"(any_want) : "r"((uint32_t)want), "r"(pair_bar), "n"(32 * kWsRowThreads) : "memory");
                if (any_want) {                               // the same answer in all four warps of these rows
                    ws_ld32(tmem_s, sc[0]);                   // S is still whole: no P has been written
                    ws_wait_ld();
                    if (need_mask) {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (kv0 + i > row_pos[w]) sc[0][i] = 0xff800000u;
                    }
                    float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int i = 0; i < 32; i += 8)
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            m4[k] = ws_max3(m4[k], __uint_as_float(sc[0][i + k]), __uint_as_float(sc[0][i + 4 + k]));
                    const float m_loc = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
                    float *box = xch + (n_xch & 1) * kWsSoftmaxThreads;
                    ++n_xch;
                    box[tid] = m_loc;
                    asm volatile("bar.sync %0, %1;" :: "r"(pair_bar), "n"(32 * kWsRowThreads) : "memory");
                    float m_row = m_loc;
#pragma unroll
                    for (int k = 1; k < kWsRowThreads; ++k) m_row = fmaxf(m_row, box[(tid + 128 * k) % kWsSoftmaxThreads]);
                    const float mx = m_row * p.scale_log2;                               // scale > 0 commutes with max
                    // A reference moves when the row maximum stands more than kWsMoveMargin above it; a row
                    // that stays has every score within that margin, so its sums pass the test from now on.
                    float alpha = 1.f;
                    if (mx > m_ref[w] + kWsMoveMargin || m_ref[w] == -INFINITY) {
                        const float m_new = fmaxf(m_ref[w], mx);
                        if (m_new != -INFINITY) {
                            alpha = (m_ref[w] == -INFINITY) ? 0.f : fast_exp2(m_ref[w] - m_new);
                            m_ref[w] = m_new;
                            l_run[w] *= alpha;
                        }
                    }
                    if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {  // the partner warps take the same decision
#pragma unroll 1
                        for (int q = 0; q < kWsCols / 16; ++q) {
                            uint32_t v[16];
                            ws_ld16(tmem_o + q * 16, v);
                            ws_wait_ld();
#pragma unroll
                            for (int i = 0; i < 16; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
                            ws_st16(tmem_o + q * 16, v);
                        }
                    }
                    exponentials(m_ref[w]);
                }
                ws_st16(tmem_p, pw);
                if (TWO_TERM) ws_st16(tmem_p + 64, (const uint32_t (&)[16])pl);     // the upper half of the score columns is free by now
                l_run[w] += tile_sum;
                ws_wait_st();
                ws_fence_before();
                ws_mbar_arrive(bar(kBarPFull + w));
            }
        }

        // ---- epilogue: the halves of a row add up their sums; all PV done -> (pieces: hand over or merge) -> store ----
        float l_tot[2];
        {
            float *box = xch + 2 * kWsSoftmaxThreads;     // [2 row tiles][256]
            box[tid] = l_run[0];
            box[kWsSoftmaxThreads + tid] = l_run[1];
            asm volatile("bar.sync %0, %1;" :: "r"(pair_bar), "n"(32 * kWsRowThreads) : "memory");
            l_tot[0] = l_run[0];
            l_tot[1] = l_run[1];
#pragma unroll
            for (int k = 1; k < kWsRowThreads; ++k) {
                l_tot[0] += box[(tid + 128 * k) % kWsSoftmaxThreads];
                l_tot[1] += box[kWsSoftmaxThreads + (tid + 128 * k) % kWsSoftmaxThreads];
            }
        }
        wait_warp(kBarODone, 0u);
        ws_fence_after();
        if (n_pieces == 1) {
#pragma unroll
            for (int w = 0; w < 2; ++w) {
                const uint32_t tmem_o = tmem_lane + (uint32_t)(2 * kWsKv + w * kWsD + hf * kWsCols);
                const bool row_ok = row_i[w] < C && row % Gp < G;
                uint8_t *dst = (uint8_t *)(p.out + ((int64_t)(qs + (row_ok ? row_i[w] : 0)) * p.num_q_heads + (g * G + (row_ok ? row % Gp : 0))) * kWsD) + hf * (kWsCols * 2);
                const float inv = l_tot[w] > 0.f ? 1.f / l_tot[w] : 0.f;
#pragma unroll 1
                for (int q = 0; q < kWsCols / 32; ++q) {  // every lane takes part in the warp-wide loads; only real rows are stored
                    uint32_t v[32];
                    ws_ld32(tmem_o + q * 32, v);
                    ws_wait_ld();
                    if (OUT_F32 && row_ok) {
                        float *dstf = (float *)p.out + ((int64_t)(qs + row_i[w]) * p.num_q_heads + (g * G + row % Gp)) * kWsD + hf * kWsCols + q * 32;
#pragma unroll
                        for (int c4 = 0; c4 < 8; ++c4) {
                            uint32_t ow[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) ow[i] = __float_as_uint(__uint_as_float(v[4 * c4 + i]) * inv);
                            st16B(dstf + 4 * c4, ow);
                        }
                    } else if (row_ok) {
#pragma unroll
                        for (int c4 = 0; c4 < 4; ++c4) {
                            uint32_t ow[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                ow[i] = pack_16x2<F16>(__uint_as_float(v[8 * c4 + 2 * i]) * inv, __uint_as_float(v[8 * c4 + 2 * i + 1]) * inv);
                            st16B(dst + q * 64 + c4 * 16, ow);
                        }
                    }
                }
            }
        } else {
            // A piece: publish (reference maximum, row sum, unnormalised O); the piece that finds all the
            // others published merges them with its own accumulators and stores the rows.
            const int su = unit - p.split_first;
            float *mine = p.part + ((int64_t)su * n_pieces + piece) * kWsPartFloats;
#pragma unroll
            for (int w = 0; w < 2; ++w) {
                const uint32_t tmem_o = tmem_lane + (uint32_t)(2 * kWsKv + w * kWsD + hf * kWsCols);
                const int rowidx = w * kWsRows + row;
                const bool have = m_ref[w] != -INFINITY;  // a row (or a piece) that saw no token has nothing in O
                if (hf == 0) *(float2 *)(mine + 2 * kWsRows * kWsD + 2 * rowidx) = make_float2(m_ref[w], l_tot[w]);
#pragma unroll 1
                for (int q = 0; q < kWsCols / 32; ++q) {
                    uint32_t v[32];
                    ws_ld32(tmem_o + q * 32, v);
                    ws_wait_ld();
#pragma unroll
                    for (int c4 = 0; c4 < 8; ++c4) {
                        float4 o = make_float4(__uint_as_float(v[4 * c4]), __uint_as_float(v[4 * c4 + 1]), __uint_as_float(v[4 * c4 + 2]), __uint_as_float(v[4 * c4 + 3]));
                        if (!have) o = make_float4(0.f, 0.f, 0.f, 0.f);
                        *(float4 *)(mine + ((hf * (kWsCols / 4) + q * 8 + c4) * 2 * kWsRows + rowidx) * 4) = o;
                    }
                }
            }
            __threadfence();
            asm volatile("bar.sync 5, %0;" :: "n"(kWsSoftmaxThreads) : "memory");
            if (tid == 0) *(volatile int *)(tmem_slot + 1) = atomicAdd(p.part_count + su, 1);
            asm volatile("bar.sync 5, %0;" :: "n"(kWsSoftmaxThreads) : "memory");
            const int arrived_before = *(volatile int *)(tmem_slot + 1);
            if (arrived_before == n_pieces - 1) {
                __threadfence();
                if (tid == 0) p.part_count[su] = 0;       // left at zero for the next launch
#pragma unroll
                for (int w = 0; w < 2; ++w) {
                    const uint32_t tmem_o = tmem_lane + (uint32_t)(2 * kWsKv + w * kWsD + hf * kWsCols);
                    const int rowidx = w * kWsRows + row;
                    const bool have = m_ref[w] != -INFINITY;
                    const bool row_ok = row_i[w] < C && row % Gp < G;
                    uint8_t *dst = (uint8_t *)(p.out + ((int64_t)(qs + (row_ok ? row_i[w] : 0)) * p.num_q_heads + (g * G + (row_ok ? row % Gp : 0))) * kWsD) + hf * (kWsCols * 2);
                    float m_all = m_ref[w];
                    float m_o[kWsMaxSplits], l_o[kWsMaxSplits];
#pragma unroll
                    for (int k = 0; k < kWsMaxSplits; ++k) {
                        m_o[k] = -INFINITY; l_o[k] = 0.f;
                        if (k < n_pieces && k != piece) {
                            const float2 ml = __ldcg((const float2 *)(p.part + ((int64_t)su * n_pieces + k) * kWsPartFloats + 2 * kWsRows * kWsD + 2 * rowidx));
                            m_o[k] = ml.x; l_o[k] = ml.y;
                            m_all = fmaxf(m_all, ml.x);
                        }
                    }
                    const float w_mine = have ? fast_exp2(m_ref[w] - m_all) : 0.f;
                    float l_all = l_tot[w] * w_mine, w_o[kWsMaxSplits];
#pragma unroll
                    for (int k = 0; k < kWsMaxSplits; ++k) {
                        w_o[k] = m_o[k] != -INFINITY ? fast_exp2(m_o[k] - m_all) : 0.f;
                        l_all += l_o[k] * w_o[k];
                    }
                    const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
#pragma unroll 1
                    for (int q = 0; q < kWsCols / 32; ++q) {
                        uint32_t v[32];
                        ws_ld32(tmem_o + q * 32, v);
                        ws_wait_ld();
                        float acc[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) acc[i] = have ? __uint_as_float(v[i]) * w_mine : 0.f;
#pragma unroll
                        for (int k = 0; k < kWsMaxSplits; ++k) {
                            if (k < n_pieces && k != piece) {
                                const float *other = p.part + ((int64_t)su * n_pieces + k) * kWsPartFloats;
#pragma unroll
                                for (int c4 = 0; c4 < 8; ++c4) {
                                    const float4 o = __ldcg((const float4 *)(other + ((hf * (kWsCols / 4) + q * 8 + c4) * 2 * kWsRows + rowidx) * 4));
                                    acc[4 * c4] = fmaf(o.x, w_o[k], acc[4 * c4]);
                                    acc[4 * c4 + 1] = fmaf(o.y, w_o[k], acc[4 * c4 + 1]);
                                    acc[4 * c4 + 2] = fmaf(o.z, w_o[k], acc[4 * c4 + 2]);
                                    acc[4 * c4 + 3] = fmaf(o.w, w_o[k], acc[4 * c4 + 3]);
                                }
                            }
                        }
                        if (OUT_F32 && row_ok) {
                            float *dstf = (float *)p.out + ((int64_t)(qs + row_i[w]) * p.num_q_heads + (g * G + row % Gp)) * kWsD + hf * kWsCols + q * 32;
#pragma unroll
                            for (int c4 = 0; c4 < 8; ++c4) {
                                uint32_t ow[4];
#pragma unroll
                                for (int i = 0; i < 4; ++i) ow[i] = __float_as_uint(acc[4 * c4 + i] * inv);
                                st16B(dstf + 4 * c4, ow);
                            }
                        } else if (row_ok) {
#pragma unroll
                            for (int c4 = 0; c4 < 4; ++c4) {
                                uint32_t ow[4];
#pragma unroll
                                for (int i = 0; i < 4; ++i) ow[i] = pack_16x2<F16>(acc[8 * c4 + 2 * i] * inv, acc[8 * c4 + 2 * i + 1] * inv);
                                st16B(dst + q * 64 + c4 * 16, ow);
                            }
                        }
                    }
                }
            }
        }
    } else if (warp < (kWsSoftmaxThreads + kWsLoaderThreads) / 32) {
        // =========================== expanders ===========================
        const int lt = tid - kWsSoftmaxThreads;
        const int hw = lt >> 4, ch = lt & 15;             // half warp hw takes token rows hw, hw + 12, ... of the tile; lane chunk ch
        // Q: 256 rows x 16 chunks; published with the first arrival on K full[0]
        {
            const uint32_t dst = ws_smem_u32(q_s);
            for (int id = lt; id < 2 * kWsRows * 16; id += kWsLoaderThreads) {
                const int rr = id >> 4, c16 = id & 15;
                const int w = rr >> 7, m = rr & 127;
                const int i = i0 + w * tok_m + m / Gp, hl = m % Gp;
                const bool ok = i < C && hl < G;
                const int h = g * G + (ok ? hl : 0);
                const uint8_t *src = (const uint8_t *)(p.q + ((int64_t)(qs + (ok ? i : 0)) * p.num_q_heads + h) * kWsD) + c16 * 16;
                ws_cp16(dst + w * kWsTile + ws_tile_off(m, c16), src, ok ? 16 : 0);
            }
            ws_commit_group();
        }
        const int n_items = 2 * n_tiles;                  // item i: K(i/2) for even i, V(i/2) for odd i; stage (i/2) & 1
#pragma unroll 1
        for (int item = 0; item < n_items; ++item) {
            const int j = item >> 1, is_v = item & 1, stage = j & 1;
            uint8_t *st = (is_v ? v_s : k_s) + stage * kWsTile;
            const uint32_t info = tinfo[j];
            const uint32_t base_mask = HAS_BASE ? (info & 0xFFu) : 0u, part_mask = (info >> 8) & 0xFFu;
            // the previous use of the stage has been consumed, so its "full" phase is over
            if (j >= kWsStages) wait_idle((is_v ? kBarVEmpty : kBarKEmpty) + stage, (uint32_t)(((j >> 1) - 1) & 1));
            bool wrote = item == 0;                       // Q
            if (part_mask) {                              // at most the last page of the request: plain copies, zero fill behind the last token
                const uint8_t *layer = is_v ? p.v_layer : p.k_layer;
#pragma unroll 1
                for (int trow = hw; trow < kWsKv; trow += 12) {
                    const int pg = trow >> 4, tok = trow & 15;
                    if (!((part_mask >> pg) & 1)) continue;
                    const int valid = L - ((tile0 + j) * kWsPagesPerTile + pg) * kPageSize;
                    const uint8_t *blk = layer + (int64_t)(pages[j * kWsPagesPerTile + pg] >> 2) * (kPageSize * kWsD * 2);
                    ws_cp16(ws_smem_u32(st) + ws_tile_off(trow, ch), blk + tok * (kWsD * 2) + ch * 16, tok < valid ? 16 : 0);
                }
                ws_commit_group();
                wrote = true;
            }
            if (wrote) ws_wait_group<0>();
            if (base_mask) {
                wait_idle((is_v ? kBarVRaw : kBarKRaw) + stage, (uint32_t)((j >> 1) & 1));    // the packed bytes have landed
                __syncwarp();
                // all reads of a token row (its 16 lanes sit in one warp), then all its writes
                uint2 x[kWsRowPasses];
#pragma unroll
                for (int q = 0; q < kWsRowPasses; ++q) {
                    const int trow = hw + 12 * q;
                    if (trow < kWsKv && ((base_mask >> (trow >> 4)) & 1)) x[q] = *(const uint2 *)(st + kWsHalf + trow * 128 + ch * 8);
                }
                __syncwarp();
#pragma unroll
                for (int q = 0; q < kWsRowPasses; ++q) {
                    const int trow = hw + 12 * q;
                    if (trow < kWsKv && ((base_mask >> (trow >> 4)) & 1)) {
                        uint4 w;
                        w.x = prmt(x[q].x, 0u, 0x1404); w.y = prmt(x[q].x, 0u, 0x3424);
                        w.z = prmt(x[q].y, 0u, 0x1404); w.w = prmt(x[q].y, 0u, 0x3424);
                        *(uint4 *)(st + ws_tile_off(trow, ch)) = w;
                    }
                }
                wrote = true;
            }
            if (wrote) ws_fence_async_proxy();            // generic-proxy writes -> visible to the tensor cores
            ws_mbar_arrive(bar((is_v ? kBarVFull : kBarKFull) + stage));
        }
        ws_wait_group<0>();                               // (a piece without tiles never published its copy of Q)
    } else if (warp == (kWsSoftmaxThreads + kWsLoaderThreads) / 32 + 1) {
        // =========================== copy issue (one warp: a lane per copy) ===========================
        // lane -> page lane >> 1 of the tile and dim half lane & 1; lanes 16..31 only keep the warp together
        const int lane = tid & 31, pg = (lane >> 1) & 7, half = lane & 1;
        const int n_items = 2 * n_tiles;
        int word = n_tiles > 0 ? pages[pg] : 0;
#pragma unroll 1
        for (int item = 0; item < n_items; ++item) {
            const int j = item >> 1, is_v = item & 1, stage = j & 1;
            const uint32_t info = tinfo[j];
            const uint32_t full = bar((is_v ? kBarVFull : kBarKFull) + stage), raw = bar((is_v ? kBarVRaw : kBarKRaw) + stage);
            const uint32_t dst = ws_smem_u32((is_v ? v_s : k_s) + stage * kWsTile) + (uint32_t)(pg * (kPageSize * 128));
            if (j >= kWsStages) wait_idle((is_v ? kBarVEmpty : kBarKEmpty) + stage, (uint32_t)(((j >> 1) - 1) & 1));
            __syncwarp();
            if (lane == 0) {
                ws_mbar_expect(full, ((info >> 16) & 0xFFu) * (uint32_t)(kPageSize * kWsD * 2));
                ws_mbar_expect(raw, (info >> 24) * (uint32_t)(kPageSize * kWsD));
            }
            __syncwarp();                                 // the byte counts are posted before any copy can complete
            const int kind = word & 3, idx = word >> 2;
            if (lane < 16) {
                if (kind == kPgTarget)
                    ws_tma_2d(dst + half * kWsHalf, is_v ? &map_v : &map_k, half * 64, idx * kPageSize, full);
                else if (HAS_BASE && kind == kPgBase && half == 0)
                    ws_bulk(dst + kWsHalf, (is_v ? p.v_layer : p.k_layer) + (int64_t)idx * (kPageSize * kWsD), kPageSize * kWsD, raw);
            }
            if (is_v && j + 1 < n_tiles) word = pages[(j + 1) * kWsPagesPerTile + pg];       // K and V of a tile share the page words
        }
    } else if (warp == (kWsSoftmaxThreads + kWsLoaderThreads) / 32) {
        // =========================== MMA issue (one warp, one effective lane) ===========================
        const uint32_t leader = (tid & 31) == 0;
        // instruction descriptor: fp32 accumulator (bits 4-5 = 1), A and B format (bits 7-9, 10-12: 0 = fp16, 1 = bf16), N >> 3, M >> 4
        constexpr uint32_t kFmt = F16 ? 0u : ((1u << 7) | (1u << 10));
        constexpr uint32_t kIdescQK = (1u << 4) | kFmt | ((uint32_t)(kWsKv >> 3) << 17) | ((uint32_t)(kWsRows >> 4) << 24);
        constexpr uint32_t kIdescPV = (1u << 4) | kFmt | (1u << 16) | ((uint32_t)(kWsD >> 3) << 17) | ((uint32_t)(kWsRows >> 4) << 24);
        const uint64_t q_desc[2] = {ws_desc(ws_smem_u32(q_s), 16, 1024), ws_desc(ws_smem_u32(q_s + kWsTile), 16, 1024)};
        const uint64_t k_desc0 = ws_desc(ws_smem_u32(k_s), 16, 1024);
        const uint64_t v_desc0 = ws_desc(ws_smem_u32(v_s), kWsHalf, 1024);
        auto issue_s = [&](int w, int j) {                // S_w = Q_w K_j^T
            const uint64_t kb = k_desc0 + (uint64_t)(((j & 1) * kWsTile) >> 4);
            const uint32_t d = tmem_base + (uint32_t)(w * kWsKv);
#pragma unroll
            for (int k16 = 0; k16 < kWsD / 16; ++k16) {
                const uint32_t off = (uint32_t)((k16 >> 2) * kWsHalf + (k16 & 3) * 32) >> 4;
                ws_mma_ss(d, q_desc[w] + off, kb + off, kIdescQK, k16 > 0, leader);
            }
            ws_commit_mma(bar(kBarSFull + w), leader);
        };
        auto issue_pv = [&](int w, int j) {               // O_w (+)= P_w V_j, P from tensor memory
            const uint64_t vb = v_desc0 + (uint64_t)(((j & 1) * kWsTile) >> 4);
            const uint32_t d = tmem_base + (uint32_t)(2 * kWsKv + w * kWsD);
            const uint32_t a = tmem_base + (uint32_t)(w * kWsKv);
#pragma unroll
            for (int k16 = 0; k16 < kWsKv / 16; ++k16)
                ws_mma_ts(d, a + (uint32_t)(8 * k16), vb + (uint32_t)((k16 * 2048) >> 4), kIdescPV, (j > 0) || (k16 > 0), leader);
            if (TWO_TERM) {                               // the residual terms of P (stored negated), 64 columns further on
#pragma unroll
                for (int k16 = 0; k16 < kWsKv / 16; ++k16)
                    ws_mma_ts(d, a + (uint32_t)(64 + 8 * k16), vb + (uint32_t)((k16 * 2048) >> 4), kIdescPV | (1u << 13), 1u, leader);   // bit 13: negate A
            }
        };
        if (n_tiles > 0) {
            wait(kBarKFull + 0, 0u);                      // Q and K(0)
            ws_fence_after();
            issue_s(0, 0);
            issue_s(1, 0);
            ws_commit_mma(bar(kBarKEmpty + 0), leader);
        }
#pragma unroll 1
        for (int j = 0; j < n_tiles; ++j) {
            const int st = j & 1, ph = (j >> 1) & 1;
            const bool more = j + 1 < n_tiles;
            wait(kBarVFull + st, (uint32_t)ph);
            // K(j+1) has usually landed by now: look once here, so that nothing stands between PV_0 and S_0
            const bool k_ready = more && ws_mbar_test(bar(kBarKFull + (st ^ 1)), (uint32_t)(((j + 1) >> 1) & 1));
            wait(kBarPFull + 0, (uint32_t)(j & 1));
            ws_fence_after();
            issue_pv(0, j);
            if (more) {
                if (!k_ready) {
                    wait(kBarKFull + (st ^ 1), (uint32_t)(((j + 1) >> 1) & 1));
                    ws_fence_after();
                }
                issue_s(0, j + 1);
            }
            wait(kBarPFull + 1, (uint32_t)(j & 1));
            ws_fence_after();
            issue_pv(1, j);
            ws_commit_mma(bar(kBarVEmpty + st), leader);
            if (more) {
                issue_s(1, j + 1);
                ws_commit_mma(bar(kBarKEmpty + (st ^ 1)), leader);
            }
        }
        ws_commit_mma(bar(kBarODone), leader);
    }

    if (dead) atomicExch(&g_prefill_ws_status, 1);
    ws_fence_before();
    __syncthreads();
    if (warp == 0) {
        ws_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(512) : "memory");
    }
}

// Tensor map over one layer of a KV pool seen as [num_blocks * num_kv_heads * 16 tokens][128 dims] bf16,
// box = 16 tokens x 64 dims, 128-byte swizzle: one copy lands as 16 rows of the canonical K/V tile.
static int make_page_map(CUtensorMap *map, const void *layer_base, int num_blocks, int num_kv_heads)
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
    const cuuint64_t dims[2] = {(cuuint64_t)kWsD, (cuuint64_t)num_blocks * (cuuint64_t)num_kv_heads * kPageSize};
    const cuuint64_t strides[1] = {(cuuint64_t)kWsD * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kPageSize};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult rc = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(layer_base), dims, strides, box, estr,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS ? EKV_OK : EKV_ERR_CUDA;
}

static int sm_count() { return device_sm_count(); }

// Workspace that lets the kernel balance its last wave: at most one piece per SM.
size_t prefill_ws_workspace_bytes()
{
    const int sms = sm_count();
    return sms > 0 ? (size_t)sms * kWsPartFloats * sizeof(float) + 256 + (size_t)sms * sizeof(int) : 0;
}

int launch_prefill_ws(const PrefillTcParams &p_in, int64_t ctas, int max_pages, int num_blocks, bool has_base, bool f16,
                      void *workspace, size_t workspace_bytes, cudaStream_t st)
{
    PrefillTcParams p = p_in;
    const size_t sm = (size_t)kWsSmemBytes + 8 * (kBarCount + 1) + 16 + 4 * kWsSoftmaxThreads * sizeof(float)
                      + (size_t)((max_pages + kWsPagesPerTile - 1) / kWsPagesPerTile) * (kWsPagesPerTile + 1) * sizeof(int32_t);
    if ((int64_t)num_blocks * p.num_kv_heads >= (1LL << 28)) return EKV_ERR_UNSUPPORTED;      // page words hold 2 * slab index + 2 bits
    CUtensorMap map_k, map_v;
    if (make_page_map(&map_k, p.k_layer, num_blocks, p.num_kv_heads) || make_page_map(&map_v, p.v_layer, num_blocks, p.num_kv_heads))
        return EKV_ERR_CUDA;
    // One CTA per SM at a time: `ctas` units run in waves of sm_count(). When the last wave would fill
    // at most half the SMs, its units are cut along the KV axis into pieces that fill it (the last piece
    // of a unit to finish merges the others' partial results from the workspace).
    p.split_first = (int)ctas;
    p.splits = 1;
    p.part = nullptr;
    p.part_count = nullptr;
    int64_t grid = ctas;
    const int sms = sm_count();
    const int rem = sms > 0 ? (int)(ctas % sms) : 0;
    const int max_tiles = (max_pages + kWsPagesPerTile - 1) / kWsPagesPerTile;
    if (rem > 0 && 2 * rem <= sms && workspace && !((uintptr_t)workspace & 255) && workspace_bytes >= prefill_ws_workspace_bytes()) {
        int splits = sms / rem;
        if (splits > kWsMaxSplits) splits = kWsMaxSplits;
        if (splits > max_tiles / 4) splits = max_tiles / 4;          // a piece is worth at least four KV tiles
        if (splits >= 2) {
            p.split_first = (int)(ctas - rem);
            p.splits = splits;
            p.part = (float *)workspace;
            p.part_count = (int *)((uint8_t *)workspace + (((size_t)sms * kWsPartFloats * sizeof(float) + 255) & ~(size_t)255));
            grid = ctas - rem + (int64_t)rem * splits;
            if (cudaMemsetAsync(p.part_count, 0, (size_t)rem * sizeof(int), st) != cudaSuccess) return EKV_ERR_CUDA;
        }
    }
    // Probabilities enter the PV product as one 16-bit term, or as two (rounded value + rounding residual).
    // Default: two for bf16 pools (one bf16 term leaves up to 5e-3 of output error on rows that a few tokens
    // dominate), one for fp16 pools (eight times finer); "prefill_p_terms" overrides.
    const bool two = g_prefill_p_terms == 0 ? !f16 : g_prefill_p_terms == 2;
    cudaError_t err = cudaSuccess;
#define EKV_LAUNCH_WS(HB, FF, TT)                                                                          \
    do {                                                                                                  \
        err = cudaFuncSetAttribute(prefill_ws_kernel<HB, FF, TT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm); \
        if (err == cudaSuccess) {                                                                         \
            MainKernelScope scope(st);                                                                    \
            prefill_ws_kernel<HB, FF, TT><<<(unsigned)grid, kWsThreads, sm, st>>>(p, map_k, map_v);       \
        }                                                                                                 \
    } while (0)
    if (p.out_f32) {
        // debug output in fp32: its own instantiations, so that the production kernels carry no trace of it
#define EKV_LAUNCH_WS_F32(HB, FF, TT)                                                                      \
    do {                                                                                                  \
        err = cudaFuncSetAttribute(prefill_ws_kernel<HB, FF, TT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm); \
        if (err == cudaSuccess) {                                                                         \
            MainKernelScope scope(st);                                                                    \
            prefill_ws_kernel<HB, FF, TT, true><<<(unsigned)grid, kWsThreads, sm, st>>>(p, map_k, map_v); \
        }                                                                                                 \
    } while (0)
        if (has_base) {
            if (f16) { if (two) EKV_LAUNCH_WS_F32(true, true, true); else EKV_LAUNCH_WS_F32(true, true, false); }
            else     { if (two) EKV_LAUNCH_WS_F32(true, false, true); else EKV_LAUNCH_WS_F32(true, false, false); }
        } else {
            if (f16) { if (two) EKV_LAUNCH_WS_F32(false, true, true); else EKV_LAUNCH_WS_F32(false, true, false); }
            else     { if (two) EKV_LAUNCH_WS_F32(false, false, true); else EKV_LAUNCH_WS_F32(false, false, false); }
        }
#undef EKV_LAUNCH_WS_F32
    } else if (has_base) {
        if (f16) { if (two) EKV_LAUNCH_WS(true, true, true); else EKV_LAUNCH_WS(true, true, false); }
        else     { if (two) EKV_LAUNCH_WS(true, false, true); else EKV_LAUNCH_WS(true, false, false); }
    } else {
        if (f16) { if (two) EKV_LAUNCH_WS(false, true, true); else EKV_LAUNCH_WS(false, true, false); }
        else     { if (two) EKV_LAUNCH_WS(false, false, true); else EKV_LAUNCH_WS(false, false, false); }
    }
#undef EKV_LAUNCH_WS
    if (err != cudaSuccess) return EKV_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? EKV_OK : EKV_ERR_CUDA;
}

} // namespace ekv

using namespace ekv;

// Host-synchronising debug query: status word of the tensor-core prefill kernel since the last
// call (0 = no bounded wait ever expired). Resets the word.
extern "C" int ekv_prefill_status(void)
{
    int v = -1, zero = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return EKV_ERR_CUDA;
    if (cudaMemcpyFromSymbol(&v, g_prefill_ws_status, sizeof(int)) != cudaSuccess) return EKV_ERR_CUDA;
    if (cudaMemcpyToSymbol(g_prefill_ws_status, &zero, sizeof(int)) != cudaSuccess) return EKV_ERR_CUDA;
    return v;
}
