// Entry points that launch nothing heavy: version, status text, options, workspace sizing and
// the device-side batch checker.
#include "ekv_common.cuh"
#include <string.h>
#include <atomic>

namespace ekv {

int64_t g_decode_chunk_tokens = 0;
int64_t g_decode_variant = 0;
int64_t g_decode_merge_slices = 0;
int64_t g_prefill_variant = 0;
int64_t g_attn_out_f32 = 0;
int64_t g_decode_two_term = 0;
int64_t g_decode_staging = 0;
int64_t g_prefill_p_terms = 0;
void *g_profile_ev[2] = {nullptr, nullptr};

int device_sm_count()
{
    constexpr int kMaxDevices = 64;
    static std::atomic<int> cache[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return kSmCountB200;
    int v = cache[dev].load(std::memory_order_relaxed);
    if (v == 0) {
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return kSmCountB200;
        cache[dev].store(v, std::memory_order_relaxed);
    }
    return v;
}

__global__ void validate_batch_kernel(const int32_t *block_table, const int32_t *seq_lens, const uint8_t *tags,
                                      int batch, int max_blocks, int num_blocks, int has_base, int32_t *status)
{
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= batch) return;
    int err = 0;
    const int L = seq_lens[r];
    if (L < 0 || (int64_t)L > (int64_t)max_blocks * kPageSize) err = 5;
    const int nb = err ? 0 : (L + kPageSize - 1) / kPageSize;
    const int32_t *row = block_table + (int64_t)r * max_blocks;
    for (int lb = 0; lb < nb && !err; ++lb) {
        const int b = row[lb];
        if (b < 0 || b >= num_blocks) { err = 1; break; }
        const int tag = tags ? tags[b] : EKV_TARGET;
        if (tag == EKV_BASE && !has_base) { err = 2; break; }
        if ((lb & 1) == 0 && lb + 1 < nb) {
            const int b1 = row[lb + 1];
            if (tag == EKV_BASE && b1 != b) { err = 3; break; }
            if (tag != EKV_BASE && b1 == b) { err = 4; break; }
        }
        if ((lb & 1) == 0 && lb + 1 >= nb && tag == EKV_BASE) { err = 3; break; }   // unpaired block must be TARGET
    }
    if (err && atomicCAS(status, 0, err) == 0) status[1] = r;
}

} // namespace ekv

using namespace ekv;

extern "C" int ekv_version(void) { return 100; }

extern "C" const char *ekv_status_string(int status)
{
    switch (status) {
    case EKV_OK: return "ok";
    case EKV_ERR_INVALID_ARG: return "invalid argument";
    case EKV_ERR_UNSUPPORTED: return "unsupported shape";
    case EKV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case EKV_ERR_CUDA: return "CUDA launch or runtime error";
    default: return "unknown status";
    }
}

extern "C" int ekv_set_option(const char *name, int64_t value)
{
    if (!name) return EKV_ERR_INVALID_ARG;
    if (!strcmp(name, "decode_chunk_tokens")) {
        if (value < 0 || value > (1 << 20)) return EKV_ERR_INVALID_ARG;
        g_decode_chunk_tokens = value;
        return EKV_OK;
    }
    if (!strcmp(name, "prefill_variant")) {
        if (value < 0 || value > 1) return EKV_ERR_INVALID_ARG;
        g_prefill_variant = value;
        return EKV_OK;
    }
    if (!strcmp(name, "decode_merge_slices")) {
        if (value != 0 && value != 1 && value != 4 && value != 8) return EKV_ERR_INVALID_ARG;
        g_decode_merge_slices = value;
        return EKV_OK;
    }
    if (!strcmp(name, "attn_out_f32")) {
        if (value != 0 && value != 1) return EKV_ERR_INVALID_ARG;
        g_attn_out_f32 = value;
        return EKV_OK;
    }
    if (!strcmp(name, "prefill_p_terms")) {
        if (value < 0 || value > 2) return EKV_ERR_INVALID_ARG;
        g_prefill_p_terms = value;
        return EKV_OK;
    }
    if (!strcmp(name, "decode_staging")) {
        if (value < 0 || value > 2) return EKV_ERR_INVALID_ARG;
        g_decode_staging = value;
        return EKV_OK;
    }
    if (!strcmp(name, "decode_two_term")) {
        if (value < 0 || value > 2) return EKV_ERR_INVALID_ARG;
        g_decode_two_term = value;
        return EKV_OK;
    }
    if (!strcmp(name, "decode_variant")) {
        if (value != 0 && value != 1 && value != 3) return EKV_ERR_INVALID_ARG;
        g_decode_variant = value;
        return EKV_OK;
    }
    return EKV_ERR_INVALID_ARG;
}

extern "C" int ekv_set_profile_events(void *ev_begin, void *ev_end)
{
    g_profile_ev[0] = ev_begin;
    g_profile_ev[1] = ev_end;
    return EKV_OK;
}

extern "C" size_t ekv_attn_workspace_bytes(const ekv_pool *pool, int32_t batch, int32_t num_q_heads,
                                           int32_t max_seq_len, int32_t total_q)
{
    if (!pool || batch <= 0 || num_q_heads <= 0 || max_seq_len <= 0) return 0;
    size_t dec = decode_workspace_bytes(batch, num_q_heads, pool->num_kv_heads, pool->head_dim, max_seq_len);
    if (total_q > 0 && pool->head_dim == 128) {           // prefill: room for the pieces of the last wave (a device-wide constant)
        const size_t pf = prefill_ws_workspace_bytes();
        if (pf > dec) dec = pf;
    }
    return dec;
}

extern "C" int ekv_validate_batch(const ekv_pool *pool, const ekv_batch *batch, int32_t *dev_status, void *stream)
{
    int rc = check_pool(pool);
    if (rc) return rc;
    rc = check_batch(batch);
    if (rc) return rc;
    if (!dev_status) return EKV_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(dev_status, 0, 2 * sizeof(int32_t), st) != cudaSuccess) return EKV_ERR_CUDA;
    if (batch->batch == 0) return EKV_OK;
    validate_batch_kernel<<<(batch->batch + 127) / 128, 128, 0, st>>>(
        batch->block_table, batch->seq_lens, pool->tags, batch->batch, batch->max_blocks, pool->num_blocks,
        batch->has_base, dev_status);
    return cudaGetLastError() == cudaSuccess ? EKV_OK : EKV_ERR_CUDA;
}
