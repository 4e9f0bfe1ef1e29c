// Worker-side lowering of the scheduler's per-step metadata (Sec. 3.4; App. B.3): the scheduler
// describes a request by its logical -> physical block list and a SPARSE list of BASE pair ranges;
// the attention kernels read dense device tensors (block-table rows, sequence lengths, the two
// mode boundaries of the structured path, the batch-level flags). One launch turns the former into
// the latter and checks the sparse description against the per-block tags on the way.
#include "ekv_common.cuh"

namespace ekv {

struct LowerParams {
    const int32_t *row_of, *lens, *blk_start, *blk_ids, *range_start, *ranges;
    const uint8_t *tags;
    int32_t *block_table, *seq_lens, *boundaries, *flags;
    int n_req, max_blocks, num_blocks;
};

// One CTA per scheduled request. Threads walk the request's blocks (copy into its table row) and
// its pairs (mode by binary search in the request's sorted ranges, compared with the tag).
constexpr int kLowerThreads = 128;
__global__ void __launch_bounds__(kLowerThreads) lower_sparse_kernel(LowerParams p)
{
    const int i = blockIdx.x;
    const int tid = threadIdx.x;
    const int row = p.row_of ? p.row_of[i] : i;
    const int L = p.lens[i];
    const int b0 = p.blk_start[i], nb = p.blk_start[i + 1] - b0;
    const int r0 = p.range_start[i], nr = p.range_start[i + 1] - r0;
    const int32_t *ids = p.blk_ids + b0;
    const int32_t *rg = p.ranges + 2 * (int64_t)r0;
    int32_t *dst = p.block_table + (int64_t)row * p.max_blocks;
    for (int lb = tid; lb < nb && lb < p.max_blocks; lb += kLowerThreads) dst[lb] = ids[lb];

    // ranges -> the regular / irregular verdict (sorted, disjoint; two ranges that touch count as one)
    int gaps = 0;
    for (int k = tid + 1; k < nr; k += kLowerThreads) gaps += rg[2 * k] > rg[2 * k - 1] ? 1 : 0;

    // cross-check against the tags: a pair is BASE exactly when it lies in a range, and then both of
    // its table entries name the one block that stores it
    const int npairs = (nb + 1) / 2;
    int bad = 0;
    for (int pp = tid; pp < npairs; pp += kLowerThreads) {
        int lo = 0, hi = nr;                               // first range whose end is beyond pp
        while (lo < hi) { const int mid = (lo + hi) >> 1; if (rg[2 * mid + 1] > pp) hi = mid; else lo = mid + 1; }
        const bool in_range = lo < nr && rg[2 * lo] <= pp;
        const int id0 = ids[2 * pp];
        const int id1 = 2 * pp + 1 < nb ? ids[2 * pp + 1] : -1;
        bool ok = id0 >= 0 && id0 < p.num_blocks && (id1 < p.num_blocks);
        if (ok) {
            const bool tag_base = p.tags[id0] == EKV_BASE;
            ok = tag_base == in_range && (!in_range || id1 == id0) && (in_range || id1 != id0);
        }
        bad += ok ? 0 : 1;
    }
    const int any_gap = __syncthreads_or(gaps);
    __shared__ int sm_bad;
    if (tid == 0) sm_bad = 0;
    __syncthreads();
    if (bad) atomicAdd(&sm_bad, bad);
    __syncthreads();
    if (tid == 0) {
        p.seq_lens[row] = L;
        p.boundaries[2 * row] = nr > 0 ? rg[0] : 0;
        p.boundaries[2 * row + 1] = nr > 0 ? rg[2 * nr - 1] : 0;
        if (nr > 0) atomicOr(&p.flags[0], 1);
        if (any_gap) atomicOr(&p.flags[1], 1);
        if (sm_bad > 0) {
            atomicAdd(&p.flags[2], sm_bad);
            atomicMax(&p.flags[3], p.n_req - i);           // largest for the first request; 0 = none
        }
    }
}

__global__ void reset_tags_kernel(uint8_t *tags, const int32_t *ids, int n, int num_blocks)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n && ids[i] >= 0 && ids[i] < num_blocks) tags[ids[i]] = EKV_TARGET;
}

} // namespace ekv

using namespace ekv;

extern "C" int ekv_lower_sparse_metadata(const ekv_pool *pool, const ekv_batch *batch, int32_t *seq_lens_out,
                                         int32_t n_req, const int32_t *row_of, const int32_t *lens,
                                         const int32_t *blk_start, const int32_t *blk_ids,
                                         const int32_t *range_start, const int32_t *ranges,
                                         int32_t *boundaries, int32_t *flags, void *stream)
{
    int rc = check_pool(pool);
    if (rc) return rc;
    if (!batch || !batch->block_table || batch->max_blocks <= 0 || batch->batch < 0) return EKV_ERR_INVALID_ARG;
    if (!pool->tags || !seq_lens_out || !boundaries || !flags || n_req < 0) return EKV_ERR_INVALID_ARG;
    if (n_req > 0 && (!lens || !blk_start || !blk_ids || !range_start)) return EKV_ERR_INVALID_ARG;
    if (!row_of && n_req > batch->batch) return EKV_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(flags, 0, 4 * sizeof(int32_t), st) != cudaSuccess) return EKV_ERR_CUDA;
    if (n_req > 0) {
        LowerParams p{};
        p.row_of = row_of; p.lens = lens; p.blk_start = blk_start; p.blk_ids = blk_ids;
        p.range_start = range_start; p.ranges = ranges;
        p.tags = pool->tags;
        p.block_table = batch->block_table; p.seq_lens = seq_lens_out;
        p.boundaries = boundaries; p.flags = flags;
        p.n_req = n_req; p.max_blocks = batch->max_blocks; p.num_blocks = pool->num_blocks;
        lower_sparse_kernel<<<n_req, kLowerThreads, 0, st>>>(p);
    }
    return cudaGetLastError() == cudaSuccess ? EKV_OK : EKV_ERR_CUDA;
}

extern "C" int ekv_reset_tags(const ekv_pool *pool, const int32_t *block_ids, int32_t n, void *stream)
{
    int rc = check_pool(pool);
    if (rc) return rc;
    if (!pool->tags || n < 0 || (n > 0 && !block_ids)) return EKV_ERR_INVALID_ARG;
    if (n == 0) return EKV_OK;
    reset_tags_kernel<<<(n + 127) / 128, 128, 0, (cudaStream_t)stream>>>(pool->tags, block_ids, n, pool->num_blocks);
    return cudaGetLastError() == cudaSuccess ? EKV_OK : EKV_ERR_CUDA;
}
