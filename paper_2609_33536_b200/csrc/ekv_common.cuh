// Shared device helpers for the libekv kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include "../../include/ekv.h"

namespace ekv {

constexpr int kPageSize = 16;
constexpr int kSmCountB200 = 148;        // fallback when the device cannot be queried
int device_sm_count();                   // SMs of the current device (cached per device)

extern int64_t g_decode_chunk_tokens;   // option "decode_chunk_tokens"; 0 = automatic
extern int64_t g_prefill_variant;       // option "prefill_variant"; 0 = automatic (tcgen05 kernel at head_dim 128), 1 = mma.sync kernel
extern void *g_profile_ev[2];           // ekv_set_profile_events: recorded around the main kernel of a call
extern int64_t g_decode_merge_slices;   // option "decode_merge_slices"; 0 = automatic, else 1, 4 or 8
extern int64_t g_attn_out_f32;          // option "attn_out_f32"; 1 = attention entry points store fp32 outputs (debug)
extern int64_t g_prefill_p_terms;       // option "prefill_p_terms"; 0 = automatic, 1 = one 16-bit term, 2 = two
extern int64_t g_decode_staging;        // option "decode_staging"; 0 / 1 = cp.async ring (default), 2 = TMA tensor copies (head_dim 128)
extern int64_t g_decode_two_term;       // option "decode_two_term"; 0 = by the mass test (default), 1 = never, 2 = every step
extern int64_t g_decode_variant;        // option "decode_variant"; 0 / 3 = ring-staged kernel, 1 = page-stepped comparator
int decode_chunk_tokens(int batch, int num_kv_heads, int max_seq_len);
size_t decode_workspace_bytes(int batch, int num_q_heads, int num_kv_heads, int head_dim, int max_seq_len);
size_t prefill_ws_workspace_bytes();    // workspace with which the tcgen05 prefill kernel balances its last wave

// Record the caller's profiling events (if any) around a main-kernel launch.
struct MainKernelScope {
    cudaStream_t st;
    explicit MainKernelScope(cudaStream_t s) : st(s) { if (g_profile_ev[0]) cudaEventRecord((cudaEvent_t)g_profile_ev[0], st); }
    ~MainKernelScope() { if (g_profile_ev[1]) cudaEventRecord((cudaEvent_t)g_profile_ev[1], st); }
};

// Launch with programmatic stream serialisation: the grid may be scheduled while the previous
// kernel of the stream drains, which hides its launch latency. Every kernel launched this way
// calls cudaGridDependencySynchronize() before it touches memory (that call returns once the
// previous kernel has completed and its writes are visible).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

struct PoolView {
    uint8_t *k;            // layer base of the K pool (bytes)
    uint8_t *v;            // layer base of the V pool
    const uint8_t *tags;
    int64_t block_bytes;   // Hkv * 16 * D * 2
    int num_kv_heads;
    int head_dim;
};

// ---- argument checks shared by the entry points (host) ----
inline int check_pool(const ekv_pool *p)
{
    if (!p || !p->k_pool || !p->v_pool) return EKV_ERR_INVALID_ARG;
    if (p->num_blocks <= 0 || p->num_kv_heads <= 0 || p->num_layers <= 0) return EKV_ERR_INVALID_ARG;
    if (p->head_dim != 64 && p->head_dim != 128) return EKV_ERR_UNSUPPORTED;
    if (p->elem_type != EKV_BF16 && p->elem_type != EKV_FP16) return EKV_ERR_INVALID_ARG;
    if (p->page_size != kPageSize) return EKV_ERR_UNSUPPORTED;
    int64_t bb = (int64_t)p->num_kv_heads * kPageSize * p->head_dim * 2;
    if (p->layer_stride_bytes < bb * p->num_blocks || (p->layer_stride_bytes & 31)) return EKV_ERR_INVALID_ARG;
    if (((uintptr_t)p->k_pool & 31) || ((uintptr_t)p->v_pool & 31)) return EKV_ERR_INVALID_ARG;
    return EKV_OK;
}

inline int check_batch(const ekv_batch *b)
{
    if (!b || !b->block_table || !b->seq_lens) return EKV_ERR_INVALID_ARG;
    if (b->batch < 0 || b->max_blocks <= 0) return EKV_ERR_INVALID_ARG;
    return EKV_OK;
}

// ---- loads: streamed once, so keep them out of L1 ----
__device__ __forceinline__ void ldg32B(const void *p, uint32_t (&r)[8])
{
    asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "l"(p));
}
__device__ __forceinline__ void ldg16B(const void *p, uint32_t (&r)[4])
{
    asm volatile("ld.global.nc.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "l"(p));
}
__device__ __forceinline__ void ldg8B(const void *p, uint32_t (&r)[2])
{
    asm volatile("ld.global.nc.L1::no_allocate.v2.b32 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "l"(p));
}
// Plain (coherent) variants for data another launch on the stream may have rewritten in place.
__device__ __forceinline__ void ld32B(const void *p, uint32_t (&r)[8])
{
    asm volatile("ld.global.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "l"(p) : "memory");
}
__device__ __forceinline__ void ld16B(const void *p, uint32_t (&r)[4])
{
    asm volatile("ld.global.v4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "l"(p) : "memory");
}
__device__ __forceinline__ void st32B(void *p, const uint32_t (&r)[8])
{
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void st16B(void *p, const uint32_t (&r)[4])
{
    asm volatile("st.global.v4.b32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// D(16x8, f32) = A(16x16, row) * B(16x8, col) + C; operands bf16 (default) or, with F16, fp16
template <bool F16 = false>
__device__ __forceinline__ void mma_16816(float &d0, float &d1, float &d2, float &d3,
                                          uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1,
                                          float c0, float c1, float c2, float c3)
{
    if (F16)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 "
                     "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
                     : "=f"(d0), "=f"(d1), "=f"(d2), "=f"(d3)
                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1),
                       "f"(c0), "f"(c1), "f"(c2), "f"(c3));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 "
                     "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
                     : "=f"(d0), "=f"(d1), "=f"(d2), "=f"(d3)
                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1),
                       "f"(c0), "f"(c1), "f"(c2), "f"(c3));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
// Two floats -> a pair of the pool's 16-bit elements (round to nearest even), lo in the low half.
template <bool F16>
__device__ __forceinline__ uint32_t pack_16x2(float lo, float hi) { return F16 ? pack_f16x2(lo, hi) : pack_bf16x2(lo, hi); }
// The two elements of such a pair widened back to fp32.
template <bool F16>
__device__ __forceinline__ void unpack_16x2(uint32_t w, float &lo, float &hi)
{
    if (F16) {
        asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tcvt.f32.f16 %0, l;\n\tcvt.f32.f16 %1, h;\n\t}" : "=f"(lo), "=f"(hi) : "r"(w));
    } else {
        lo = __uint_as_float(w << 16);
        hi = __uint_as_float(w & 0xFFFF0000u);
    }
}
// One float -> the pool's 16-bit element, as bits.
template <bool F16>
__device__ __forceinline__ uint16_t f32_to_16(float v)
{
    return F16 ? __half_as_ushort(__float2half_rn(v)) : __bfloat16_as_ushort(__float2bfloat16(v));
}

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

} // namespace ekv
