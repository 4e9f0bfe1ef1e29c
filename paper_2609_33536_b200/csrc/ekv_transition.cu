// TARGET <-> BASE pair transitions (Sec. 3.1 pair layout; App. B.2 transition protocols).
//
// Both directions are pure byte movement and HBM-bound. One CTA owns up to four consecutive (kv head)
// slabs of one (pair, layer, tensor): a slab is 16*D*2 bytes both as one member's
// TARGET words and as the pair's packed BASE bytes, so every in-place hazard (the kept block is
// source and destination) stays inside the CTA: all loads, one barrier, all stores.
// The block table and tags are only read by the data CTAs; the new mapping is published after all
// of them are done -- by the CTA that finishes last when the batch is small (one launch per
// transition), by a second, tiny kernel when it is large -- so a partially written state is never
// visible to later work.
#include "ekv_common.cuh"
#include <atomic>

namespace ekv {

struct TransParams {
    uint8_t *k_pool, *v_pool;
    int64_t layer_stride, block_bytes;
    int32_t *block_table;
    uint8_t *tags;
    const int32_t *pair_req, *pair_idx, *resid_slot, *new_blocks;
    uint8_t *k_resid, *v_resid;
    int32_t *freed_out;
    int n_pairs, num_layers, max_blocks, groups_per_block;
    unsigned *done;              // this launch's counter of finished CTAs (zero at rest)
};

// Counters for "the CTA that finishes last publishes": one slot per launch, taken round robin on
// the host, so launches that overlap on the GPU (other streams) do not share one; a slot is back
// at zero when its launch ends.
constexpr int kTransCounters = 4096;
__device__ unsigned g_trans_done[kTransCounters];

// Publication of a demoted pair (App. B.2: the released page is returned only after the packed
// block is complete): tags, the table entry of member 1, the released id.
__device__ __forceinline__ void downgrade_commit_one(const TransParams &p, int i)
{
    int32_t *row = p.block_table + (int64_t)p.pair_req[i] * p.max_blocks + 2 * p.pair_idx[i];
    const int kept = row[0], released = row[1];
    p.tags[kept] = EKV_BASE;
    p.tags[released] = EKV_TARGET;
    row[1] = kept;
    p.freed_out[i] = released;
}
// Publication of a promoted pair (the mapping is published only after full materialisation).
__device__ __forceinline__ void refine_commit_one(const TransParams &p, int i)
{
    int32_t *row = p.block_table + (int64_t)p.pair_req[i] * p.max_blocks + 2 * p.pair_idx[i];
    const int kept = row[0], fresh = p.new_blocks[i];
    p.tags[kept] = EKV_TARGET;
    p.tags[fresh] = EKV_TARGET;
    row[1] = fresh;
}
// True in every thread of the CTA that finishes last: all other CTAs' stores are then visible.
__device__ __forceinline__ bool last_cta_done(const TransParams &p)
{
    __shared__ int is_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = atomicAdd(p.done, 1u) == gridDim.x - 1;
    __syncthreads();
    if (is_last) __threadfence();
    return is_last != 0;
}

// One CTA per (pair, layer, tensor, kv head) slab: 2 * D threads, 16 packed bytes each.
constexpr int trans_threads(int D) { return kPageSize * D * 2 / 16; }

// Decompose the CTA index into (pair, layer, tensor, group of slabs).
__device__ __forceinline__ void trans_decode(const TransParams &p, int &pair, int &layer, int &tensor, int &group)
{
    int idx = blockIdx.x;
    group = idx % p.groups_per_block; idx /= p.groups_per_block;
    tensor = idx & 1; idx >>= 1;
    layer = idx % p.num_layers;
    pair = idx / p.num_layers;
}

// NS consecutive kv-head slabs per CTA: every thread issues NS 32-byte loads before the barrier,
// so NS times as many bytes are in flight per SM.
template <int D, int NS>
__global__ void __launch_bounds__(trans_threads(D)) downgrade_pack_kernel(TransParams p)
{
    constexpr int kSlab = kPageSize * D * 2;          // bytes: one member's words == packed pair bytes
    constexpr int kTasksPerSlab = kSlab / 16;         // 32 source bytes per task, two members
    cudaGridDependencySynchronize();                    // (launched with programmatic stream serialisation)
    int pair, layer, tensor, group;
    trans_decode(p, pair, layer, tensor, group);
    const int32_t *row = p.block_table + (int64_t)p.pair_req[pair] * p.max_blocks + 2 * p.pair_idx[pair];
    const int kept = row[0], released = row[1];
    uint8_t *pool = (tensor ? p.v_pool : p.k_pool) + (int64_t)layer * p.layer_stride;
    uint8_t *resid = tensor ? p.v_resid : p.k_resid;

    const int u = threadIdx.x;
    const int m = u / (kTasksPerSlab / 2), o = (u % (kTasksPerSlab / 2)) * 32;
    const uint8_t *src = pool + (int64_t)(m ? released : kept) * p.block_bytes + (int64_t)group * NS * kSlab + o;
    const int64_t packed_off = (int64_t)group * NS * kSlab + m * (kSlab / 2) + o / 2;

    uint32_t w[NS][8];
#pragma unroll
    for (int s = 0; s < NS; ++s) ld32B(src + s * kSlab, w[s]);
    uint32_t hi[NS][4], lo[NS][4];
#pragma unroll
    for (int s = 0; s < NS; ++s)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            hi[s][i] = prmt(w[s][2 * i], w[s][2 * i + 1], 0x7531);   // bytes 1,3 of each word pair: high bytes
            lo[s][i] = prmt(w[s][2 * i], w[s][2 * i + 1], 0x6420);   // bytes 0,2: low bytes
        }
    __syncthreads();                                    // every word of these slabs is in registers
    uint8_t *dst = pool + (int64_t)kept * p.block_bytes + packed_off;
#pragma unroll
    for (int s = 0; s < NS; ++s) st16B(dst + s * kSlab, hi[s]);
    if (resid) {
        uint8_t *rd = resid + ((int64_t)p.resid_slot[pair] * p.num_layers + layer) * p.block_bytes + packed_off;
#pragma unroll
        for (int s = 0; s < NS; ++s) st16B(rd + s * kSlab, lo[s]);
    }
    if (p.done && last_cta_done(p)) {                   // small batch: every pair is packed, publish them all
        for (int i = threadIdx.x; i < p.n_pairs; i += blockDim.x) downgrade_commit_one(p, i);
        if (threadIdx.x == 0) *p.done = 0;
    }
}

template <int D, int NS>
__global__ void __launch_bounds__(trans_threads(D)) refine_expand_kernel(TransParams p)
{
    constexpr int kSlab = kPageSize * D * 2;
    constexpr int kTasksPerSlab = kSlab / 16;
    cudaGridDependencySynchronize();
    int pair, layer, tensor, group;
    trans_decode(p, pair, layer, tensor, group);
    const int kept = p.block_table[(int64_t)p.pair_req[pair] * p.max_blocks + 2 * p.pair_idx[pair]];
    const int fresh = p.new_blocks[pair];
    uint8_t *pool = (tensor ? p.v_pool : p.k_pool) + (int64_t)layer * p.layer_stride;
    const uint8_t *resid = tensor ? p.v_resid : p.k_resid;

    const int u = threadIdx.x;
    const int m = u / (kTasksPerSlab / 2), o = (u % (kTasksPerSlab / 2)) * 16;
    const int64_t slab_off = (int64_t)group * NS * kSlab;
    const int64_t packed_off = slab_off + m * (kSlab / 2) + o;
    const uint8_t *hsrc = pool + (int64_t)kept * p.block_bytes + packed_off;
    const uint8_t *lsrc = resid + ((int64_t)p.resid_slot[pair] * p.num_layers + layer) * p.block_bytes + packed_off;

    uint32_t hi[NS][4], lo[NS][4];
#pragma unroll
    for (int s = 0; s < NS; ++s) { ld16B(hsrc + s * kSlab, hi[s]); ldg16B(lsrc + s * kSlab, lo[s]); }
    uint32_t w[NS][8];
#pragma unroll
    for (int s = 0; s < NS; ++s)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            w[s][2 * i]     = prmt(lo[s][i], hi[s][i], 0x5140);      // [lo0, hi0, lo1, hi1]
            w[s][2 * i + 1] = prmt(lo[s][i], hi[s][i], 0x7362);      // [lo2, hi2, lo3, hi3]
        }
    __syncthreads();                                    // member 0 expands over its own source
    uint8_t *dst = pool + (int64_t)(m ? fresh : kept) * p.block_bytes + slab_off + 2 * o;
#pragma unroll
    for (int s = 0; s < NS; ++s) st32B(dst + s * kSlab, w[s]);
    if (p.done && last_cta_done(p)) {                   // small batch: every pair is materialised, publish them all
        for (int i = threadIdx.x; i < p.n_pairs; i += blockDim.x) refine_commit_one(p, i);
        if (threadIdx.x == 0) *p.done = 0;
    }
}

// Large batches publish with a kernel of their own (one thread per pair): there the per-CTA fence
// and the counter cost more than a launch.
constexpr int kFusedCommitMaxPairs = 64;
__global__ void downgrade_commit_kernel(TransParams p)
{
    cudaGridDependencySynchronize();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < p.n_pairs) downgrade_commit_one(p, i);
}
__global__ void refine_commit_kernel(TransParams p)
{
    cudaGridDependencySynchronize();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < p.n_pairs) refine_commit_one(p, i);
}

// KV append (Sec. 3.2: newly appended KV is written in TARGET form into the recent region).
// One thread per 16 bytes of one new token's K or V row; rows of a token go to the (block, head)
// slabs of the logical block that holds its position.
struct AppendParams {
    uint8_t *k_layer, *v_layer;
    const uint8_t *tags;
    const int32_t *block_table, *seq_lens, *q_start;
    const uint8_t *k_new, *v_new;
    int32_t *dev_status;
    int64_t block_bytes;
    int batch, num_kv_heads, head_dim, max_blocks, total;
};

__global__ void append_kernel(AppendParams p)
{
    const int chunks_per_row = p.head_dim / 8;                       // 16-byte chunks per (token, head) row
    const int64_t per_tok = (int64_t)p.num_kv_heads * chunks_per_row;
    const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= (int64_t)p.total * per_tok * 2) return;
    const int tensor = (int)(gid & 1);
    const int64_t id = gid >> 1;
    const int tok = (int)(id / per_tok);
    const int rem = (int)(id % per_tok);
    const int g = rem / chunks_per_row, ch = rem % chunks_per_row;
    // request of this token: binary search in q_start
    int lo = 0, hi = p.batch;
    while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (p.q_start[mid] <= tok) lo = mid; else hi = mid; }
    const int r = lo;
    const int c = p.q_start[r + 1] - p.q_start[r];
    const int pos = p.seq_lens[r] - c + (tok - p.q_start[r]);
    const int phys = p.block_table[(int64_t)r * p.max_blocks + pos / kPageSize];
    if (p.tags && p.tags[phys] != EKV_TARGET) {                      // never write words into a BASE block
        if (p.dev_status) atomicCAS(p.dev_status, 0, tok + 1);
        return;
    }
    const uint8_t *src = (tensor ? p.v_new : p.k_new) + ((int64_t)tok * p.num_kv_heads + g) * p.head_dim * 2 + ch * 16;
    uint8_t *dst = (tensor ? p.v_layer : p.k_layer) + (int64_t)phys * p.block_bytes
                   + ((int64_t)g * kPageSize + pos % kPageSize) * p.head_dim * 2 + ch * 16;
    uint32_t w[4];
    ldg16B(src, w);
    st16B(dst, w);
}

static int slabs_per_cta(int num_kv_heads) { return num_kv_heads % 4 == 0 ? 4 : (num_kv_heads % 2 == 0 ? 2 : 1); }

// Counter slot for one launch on the current device (the array's address is looked up once per device).
static unsigned *trans_counter_slot()
{
    constexpr int kMaxDevices = 64;
    static std::atomic<unsigned *> base[kMaxDevices];
    static std::atomic<unsigned> next{0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    unsigned *b = base[dev].load(std::memory_order_acquire);
    if (!b) {
        void *sym = nullptr;
        if (cudaGetSymbolAddress(&sym, g_trans_done) != cudaSuccess || !sym) return nullptr;
        b = (unsigned *)sym;
        base[dev].store(b, std::memory_order_release);
    }
    return b + next.fetch_add(1, std::memory_order_relaxed) % kTransCounters;
}

static int fill_params(TransParams &tp, const ekv_pool *pool, const ekv_batch *batch, int n_pairs,
                       const int32_t *pair_req, const int32_t *pair_idx)
{
    int rc = check_pool(pool);
    if (rc) return rc;
    rc = check_batch(batch);
    if (rc) return rc;
    if (!pool->tags || n_pairs < 0) return EKV_ERR_INVALID_ARG;
    if (n_pairs > 0 && (!pair_req || !pair_idx)) return EKV_ERR_INVALID_ARG;
    tp.k_pool = (uint8_t *)pool->k_pool;
    tp.v_pool = (uint8_t *)pool->v_pool;
    tp.layer_stride = pool->layer_stride_bytes;
    tp.block_bytes = (int64_t)pool->num_kv_heads * kPageSize * pool->head_dim * 2;
    tp.block_table = batch->block_table;
    tp.tags = pool->tags;
    tp.pair_req = pair_req;
    tp.pair_idx = pair_idx;
    tp.n_pairs = n_pairs;
    tp.num_layers = pool->num_layers;
    tp.max_blocks = batch->max_blocks;
    tp.groups_per_block = pool->num_kv_heads;   // divided by the slabs per CTA at launch
    return EKV_OK;
}

} // namespace ekv

using namespace ekv;

extern "C" int ekv_downgrade(const ekv_pool *pool, const ekv_batch *batch, int32_t n_pairs,
                             const int32_t *pair_req, const int32_t *pair_idx,
                             void *k_resid, void *v_resid, const int32_t *resid_slot,
                             int32_t *freed_blocks_out, void *stream)
{
    TransParams tp{};
    int rc = fill_params(tp, pool, batch, n_pairs, pair_req, pair_idx);
    if (rc) return rc;
    if ((k_resid == nullptr) != (v_resid == nullptr)) return EKV_ERR_INVALID_ARG;
    if (k_resid && !resid_slot && n_pairs > 0) return EKV_ERR_INVALID_ARG;
    if (((uintptr_t)k_resid & 15) || ((uintptr_t)v_resid & 15)) return EKV_ERR_INVALID_ARG;
    if (n_pairs > 0 && !freed_blocks_out) return EKV_ERR_INVALID_ARG;
    if (n_pairs == 0) return EKV_OK;
    tp.k_resid = (uint8_t *)k_resid;
    tp.v_resid = (uint8_t *)v_resid;
    tp.resid_slot = resid_slot;
    tp.freed_out = freed_blocks_out;
    const int ns = slabs_per_cta(pool->num_kv_heads);
    tp.groups_per_block = pool->num_kv_heads / ns;
    int64_t ctas = (int64_t)n_pairs * tp.num_layers * 2 * tp.groups_per_block;
    if (ctas > 0x7fffffffLL) return EKV_ERR_UNSUPPORTED;
    if (n_pairs <= kFusedCommitMaxPairs) {
        tp.done = trans_counter_slot();                 // after every argument check: needs the device
        if (!tp.done) return EKV_ERR_CUDA;
    }
    cudaStream_t st = (cudaStream_t)stream;
    {
        MainKernelScope scope(st);
        const unsigned nb = (unsigned)ctas;
        if (pool->head_dim == 128) {
            if (ns == 4)      launch_pdl(downgrade_pack_kernel<128, 4>, nb, trans_threads(128), 0, st, tp);
            else if (ns == 2) launch_pdl(downgrade_pack_kernel<128, 2>, nb, trans_threads(128), 0, st, tp);
            else              launch_pdl(downgrade_pack_kernel<128, 1>, nb, trans_threads(128), 0, st, tp);
        } else {
            if (ns == 4)      launch_pdl(downgrade_pack_kernel<64, 4>, nb, trans_threads(64), 0, st, tp);
            else if (ns == 2) launch_pdl(downgrade_pack_kernel<64, 2>, nb, trans_threads(64), 0, st, tp);
            else              launch_pdl(downgrade_pack_kernel<64, 1>, nb, trans_threads(64), 0, st, tp);
        }
    }
    if (!tp.done) launch_pdl(downgrade_commit_kernel, (unsigned)((n_pairs + 127) / 128), 128, 0, st, tp);
    return cudaGetLastError() == cudaSuccess ? EKV_OK : EKV_ERR_CUDA;
}

extern "C" int ekv_kv_append(const ekv_pool *pool, int32_t layer, const ekv_batch *batch, const int32_t *q_start,
                             const void *k_new, const void *v_new, int32_t total_new, int32_t *dev_status,
                             void *stream)
{
    int rc = check_pool(pool);
    if (rc) return rc;
    rc = check_batch(batch);
    if (rc) return rc;
    if (!q_start || !k_new || !v_new || total_new < 0 || layer < 0 || layer >= pool->num_layers) return EKV_ERR_INVALID_ARG;
    if (((uintptr_t)k_new & 15) || ((uintptr_t)v_new & 15)) return EKV_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (dev_status && cudaMemsetAsync(dev_status, 0, sizeof(int32_t), st) != cudaSuccess) return EKV_ERR_CUDA;
    if (total_new == 0 || batch->batch == 0) return EKV_OK;
    AppendParams ap{};
    ap.k_layer = (uint8_t *)pool->k_pool + (int64_t)layer * pool->layer_stride_bytes;
    ap.v_layer = (uint8_t *)pool->v_pool + (int64_t)layer * pool->layer_stride_bytes;
    ap.tags = pool->tags;
    ap.block_table = batch->block_table;
    ap.seq_lens = batch->seq_lens;
    ap.q_start = q_start;
    ap.k_new = (const uint8_t *)k_new;
    ap.v_new = (const uint8_t *)v_new;
    ap.dev_status = dev_status;
    ap.block_bytes = (int64_t)pool->num_kv_heads * kPageSize * pool->head_dim * 2;
    ap.batch = batch->batch;
    ap.num_kv_heads = pool->num_kv_heads;
    ap.head_dim = pool->head_dim;
    ap.max_blocks = batch->max_blocks;
    ap.total = total_new;
    const int64_t threads = (int64_t)total_new * pool->num_kv_heads * (pool->head_dim / 8) * 2;
    const int64_t ctas = (threads + 255) / 256;
    if (ctas > 0x7fffffffLL) return EKV_ERR_UNSUPPORTED;
    {
        MainKernelScope scope(st);
        append_kernel<<<(unsigned)ctas, 256, 0, st>>>(ap);
    }
    return cudaGetLastError() == cudaSuccess ? EKV_OK : EKV_ERR_CUDA;
}

extern "C" int ekv_refine(const ekv_pool *pool, const ekv_batch *batch, int32_t n_pairs,
                          const int32_t *pair_req, const int32_t *pair_idx, const int32_t *new_blocks,
                          const void *k_resid, const void *v_resid, const int32_t *resid_slot, void *stream)
{
    TransParams tp{};
    int rc = fill_params(tp, pool, batch, n_pairs, pair_req, pair_idx);
    if (rc) return rc;
    if (n_pairs == 0) return EKV_OK;
    if (!new_blocks || !k_resid || !v_resid || !resid_slot) return EKV_ERR_INVALID_ARG;
    if (((uintptr_t)k_resid & 15) || ((uintptr_t)v_resid & 15)) return EKV_ERR_INVALID_ARG;
    tp.k_resid = (uint8_t *)k_resid;
    tp.v_resid = (uint8_t *)v_resid;
    tp.resid_slot = resid_slot;
    tp.new_blocks = new_blocks;
    const int ns = slabs_per_cta(pool->num_kv_heads);
    tp.groups_per_block = pool->num_kv_heads / ns;
    int64_t ctas = (int64_t)n_pairs * tp.num_layers * 2 * tp.groups_per_block;
    if (ctas > 0x7fffffffLL) return EKV_ERR_UNSUPPORTED;
    if (n_pairs <= kFusedCommitMaxPairs) {
        tp.done = trans_counter_slot();                 // after every argument check: needs the device
        if (!tp.done) return EKV_ERR_CUDA;
    }
    cudaStream_t st = (cudaStream_t)stream;
    {
        MainKernelScope scope(st);
        const unsigned nb = (unsigned)ctas;
        if (pool->head_dim == 128) {
            if (ns == 4)      launch_pdl(refine_expand_kernel<128, 4>, nb, trans_threads(128), 0, st, tp);
            else if (ns == 2) launch_pdl(refine_expand_kernel<128, 2>, nb, trans_threads(128), 0, st, tp);
            else              launch_pdl(refine_expand_kernel<128, 1>, nb, trans_threads(128), 0, st, tp);
        } else {
            if (ns == 4)      launch_pdl(refine_expand_kernel<64, 4>, nb, trans_threads(64), 0, st, tp);
            else if (ns == 2) launch_pdl(refine_expand_kernel<64, 2>, nb, trans_threads(64), 0, st, tp);
            else              launch_pdl(refine_expand_kernel<64, 1>, nb, trans_threads(64), 0, st, tp);
        }
    }
    if (!tp.done) launch_pdl(refine_commit_kernel, (unsigned)((n_pairs + 127) / 128), 128, 0, st, tp);
    return cudaGetLastError() == cudaSuccess ? EKV_OK : EKV_ERR_CUDA;
}
