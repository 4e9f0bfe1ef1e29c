/*
 * ekv.h -- C ABI of the mixed-fidelity paged attention library (libekv.so).
 *
 * The library implements, for one B200 GPU, the GPU execution plane of the
 * ElasticKV paper ("Does Execution Require Target KV Fidelity? A Mixed-Fidelity
 * KV Runtime for LLM Serving"): paged attention over a KV pool whose physical
 * blocks are either TARGET (16-bit elements: bf16, or fp16 when ekv_pool.elem_type says so) or BASE (the high-order
 * byte of every element, two logical blocks packed into one physical block),
 * plus the TARGET->BASE and BASE->TARGET transition kernels.
 *
 * General rules for every entry point
 *   - Pointers are DEVICE pointers unless the comment says "host". The structs
 *     themselves are read on the host at call time.
 *   - The caller owns every buffer. Nothing is allocated, nothing is freed and
 *     the host is never synchronised: all work is enqueued on `stream`
 *     (a cudaStream_t passed as void*; NULL is the legacy default stream).
 *     For the same reason a sequence of calls may be recorded by CUDA stream
 *     capture and replayed as a graph, once each kernel has been launched
 *     at least one time outside a capture (its first launch sets function
 *     attributes). Exceptions: ekv_set_profile_events records events, and a
 *     replayed graph reuses the buffers it was captured with.
 *   - Return value: EKV_OK, or a negative ekv_status. Errors that can be seen
 *     from the host arguments (null pointer, unsupported shape, workspace too
 *     small) are returned before anything is enqueued. Contents of device
 *     arrays (block ids, tags, pair lists) are trusted, except by
 *     ekv_validate_batch.
 *   - Supported shapes: head_dim 64 or 128, page_size 16, query heads a
 *     multiple of kv heads with at most 8 query heads per kv head.
 *
 * Memory layout (the paper states the representation, Sec. 3 opening and
 * Sec. 3.1; the byte order inside a block is this library's convention)
 *   k_pool, v_pool : one pool per tensor; layer l starts at
 *                    pool + l * layer_stride_bytes; inside a layer, physical
 *                    block b starts at b * block_bytes,
 *                    block_bytes = num_kv_heads * page_size * head_dim * 2.
 *   TARGET block   : [num_kv_heads][page_size][head_dim] 16-bit words
 *                    (little-endian 16-bit floats): the native paged layout.
 *   BASE block     : [num_kv_heads][2 members][page_size][head_dim] bytes, the
 *                    high-order byte of each word of the pair's two logical
 *                    blocks (member 0 = logical block 2p, member 1 = 2p+1).
 *   tags           : one byte per physical block id, EKV_TARGET or EKV_BASE,
 *                    shared by K, V and all layers.
 *   block_table    : int32 [batch][max_blocks], logical block -> physical block
 *                    id. For a BASE pair p both entries 2p and 2p+1 hold the one
 *                    physical block that stores the pair.
 *   residual slot  : low-order bytes of one pair, one tensor:
 *                    [num_layers][num_kv_heads][2][page_size][head_dim] bytes;
 *                    slot s of a residual buffer starts at
 *                    s * num_layers * block_bytes.
 */
#ifndef EKV_H_
#define EKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum ekv_status {
    EKV_OK = 0,
    EKV_ERR_INVALID_ARG = -1,   /* null pointer, negative size, inconsistent sizes */
    EKV_ERR_UNSUPPORTED = -2,   /* shape outside the supported set */
    EKV_ERR_WORKSPACE = -3,     /* workspace missing, misaligned or too small */
    EKV_ERR_CUDA = -4           /* a launch or runtime call failed */
} ekv_status;

enum { EKV_TARGET = 0, EKV_BASE = 1 };
enum { EKV_BF16 = 0, EKV_FP16 = 1 };      /* ekv_pool.elem_type */

typedef struct ekv_pool {
    void    *k_pool;              /* device, 16-byte aligned */
    void    *v_pool;              /* device, 16-byte aligned */
    uint8_t *tags;                /* device, [num_blocks] */
    int32_t  num_blocks;
    int32_t  num_kv_heads;
    int32_t  head_dim;            /* 64 or 128 */
    int32_t  page_size;           /* 16 */
    int32_t  num_layers;
    int32_t  elem_type;           /* EKV_BF16 (0) or EKV_FP16 (1): the 16-bit float the words of the
                                     pool, of q and of out are. The codec (downgrade, refine, append)
                                     moves bytes and does not look at it; attention reads a BASE byte
                                     as (byte << 8) in this type, which for fp16 is an E5M2 number */
    int64_t  layer_stride_bytes;  /* >= num_blocks * block_bytes, multiple of 32 */
} ekv_pool;

typedef struct ekv_batch {
    int32_t       *block_table;   /* device, [batch][max_blocks] */
    const int32_t *seq_lens;      /* device, [batch]: tokens visible to attention */
    int32_t        batch;
    int32_t        max_blocks;
    int32_t        has_base;      /* host flag: 0 = no block of this batch is BASE; tags are
                                     then not read at all (native path) */
    int32_t        reserved_;     /* set to 0 */
} ekv_batch;

/* Library version (major * 10000 + minor * 100 + patch). No paper counterpart. */
int ekv_version(void);

/* Static text for a status code. */
const char *ekv_status_string(int status);

/* Tuning knobs, process-wide, read at call time by later calls. Names:
 *   "decode_chunk_tokens" : tokens per split of ekv_attn_decode; 0 = automatic.
 *                           Rounded up to a multiple of 64, at most 4096.
 *   "decode_merge_slices" : how many slices of threads share the splits of one output row in the
 *                           merge kernel: 0 = automatic (by the largest possible number of
 *                           splits), or 1, 4, 8.
 *   "decode_variant"      : 0 (default) or 3 = the ring-staged decode kernel; 1 = the simpler
 *                           page-stepped register-direct kernel (plain paged-decode comparator
 *                           used by the benchmark; bf16 pools only, EKV_ERR_UNSUPPORTED for fp16).
 *   "prefill_variant"     : 0 (default) = warp-specialised tcgen05 tensor-core kernel at
 *                           head_dim 128, mma.sync kernel otherwise; 1 = always the mma.sync
 *                           kernel (comparator).
 *   "prefill_p_terms"     : how many 16-bit terms a probability enters the PV product of the tcgen05 prefill
 *                           kernel with: 0 (default) = two for bf16 pools (the rounded value and its rounding
 *                           residual; the residual costs a second pass of PV MMAs), one for fp16 pools;
 *                           1 = one (faster; with bf16 the output's error before its final rounding can
 *                           reach 5e-3 on rows that two or three tokens dominate); 2 = two.
 *   "decode_staging"      : how the ring-staged decode kernel brings K/V slabs into shared memory: 0 or 1
 *                           (default) = cp.async, 16 bytes per lane and instruction; 2 = TMA tensor copies
 *                           (head_dim 128 only; one lane issues two box copies per slab, completion on an
 *                           mbarrier). Same results; measured 1-2 % slower, kept for measurements.
 *   "decode_two_term"     : how the decode kernels treat the 16-bit rounding of the probabilities that
 *                           enter the PV product: 0 (default) = a step that holds a token with an eighth
 *                           or more of the probability mass its warp has seen so far takes PV a second
 *                           time with the rounding residuals; 1 = never (one-term product: the output's
 *                           error before its final rounding can then reach 5e-3 on rows that two or
 *                           three tokens dominate); 2 = every step. For measurements.
 *   "attn_out_f32"        : debug aid, 0 (default) or 1: the attention entry points (decode, its
 *                           structured and no-workspace forms, prefill) then treat `out` as a float32
 *                           array of the same shape and store the result as it stands before the
 *                           rounding to the 16-bit output type.
 * Returns EKV_OK or EKV_ERR_INVALID_ARG for an unknown name / bad value. */
int ekv_set_option(const char *name, int64_t value);

/* Profiling hook (no paper counterpart): while both handles are non-NULL, every later call of
 * ekv_attn_decode / ekv_attn_prefill_chunk / ekv_downgrade / ekv_refine records ev_begin
 * (a cudaEvent_t) on the caller's stream immediately before the launch of its main kernel (the
 * split kernel, the attention kernel, the pack / expand kernel) and ev_end immediately after
 * it, so that kernel can be timed inside a longer stream of work. Pass NULLs to switch off.
 * Process-wide; the caller must read or replace the events before the next call. */
int ekv_set_profile_events(void *ev_begin, void *ev_end);

/* Bytes of workspace ekv_attn_decode / ekv_attn_prefill_chunk need for a batch of
 * `batch` requests with `num_q_heads` query heads and no sequence longer than
 * `max_seq_len` (and, for prefill, `total_q` query tokens; pass 0 for decode).
 * The workspace holds the per-split softmax partials of the split-K scheme. It must be
 * 256-byte aligned. */
size_t ekv_attn_workspace_bytes(const ekv_pool *pool, int32_t batch, int32_t num_q_heads,
                                int32_t max_seq_len, int32_t total_q);

/* Decode attention, one query token per request (Sec. 3.2 "Dual-mode Elastic Attention
 * Backend"; App. B.3): out[r][h] = softmax_t(sm_scale * q[r][h] . K[r][t][h / G]) V[r][t][h / G]
 * over t < seq_lens[r], G = num_q_heads / num_kv_heads, where an element of a BASE block
 * enters as (high byte << 8) read in the pool's element type (bf16, or fp16: then an E5M2
 * number) and an element of a TARGET block as stored.
 * batch->has_base == 0 selects the native path (no tag is read); otherwise each block's tag
 * decides its load path. A request with seq_lens[r] == 0 gets zeros.
 *   q, out       : pool->elem_type [batch][num_q_heads][head_dim], 16-byte aligned
 *   max_seq_len  : host upper bound of seq_lens (sizes the launch grid)
 *   workspace    : at least ekv_attn_workspace_bytes(...) bytes
 * Launches the split kernel and, when a sequence spans more than one split, the merge
 * kernel. */
int ekv_attn_decode(const ekv_pool *pool, int32_t layer, const ekv_batch *batch,
                    const void *q, void *out, int32_t num_q_heads, float sm_scale,
                    int32_t max_seq_len, void *workspace, size_t workspace_bytes, void *stream);

/* Mode boundaries from the tags (Sec. 3.2, structured path; App. B.3). A "regular" sequence has
 * all its BASE pairs in one contiguous run of pair indices, so two integers describe its modes.
 * From the per-block tags of a batch this call writes, for every request, that run:
 * boundaries[2r] = first BASE pair, boundaries[2r+1] = one past the last BASE pair (0, 0 when the
 * request has none), and two batch flags: flags[0] = 1 if any request has a BASE pair (the
 * batch-level indicator), flags[1] = 1 if any request is irregular (a TARGET pair between two BASE
 * pairs), in which case the boundaries do not describe that request and the general path must be
 * used.
 *   boundaries : device int32 [batch][2];  flags : device int32 [2] (cleared by this call) */
int ekv_lower_metadata(const ekv_pool *pool, const ekv_batch *batch, int32_t *boundaries,
                       int32_t *flags, void *stream);

/* Lowering of the scheduler's sparse per-request metadata (Sec. 3.4; App. B.3: the scheduler emits
 * sparse BASE metadata per request and the worker lowers it into device tensors). The scheduler
 * describes scheduled request i by its sequence length, its logical -> physical block list (for a
 * BASE pair both entries name the block that stores the pair) and a short, sorted list of disjoint
 * pair-index ranges [first, one past last) that are BASE. One kernel launch writes what the
 * attention entry points read:
 *   block_table row row_of[i] : entries [0, n_blocks_i) = the block list (later entries untouched)
 *   seq_lens_out[row_of[i]]   : lens[i]
 *   boundaries[row_of[i]]     : first BASE pair, one past the last BASE pair (0, 0 without ranges)
 *   flags[0] : 1 if any request has a range;  flags[1] : 1 if any request has two ranges with a gap
 *              between them (irregular: use the general path, not ekv_attn_decode_structured)
 * and cross-checks the description against the tags, which the transition kernels own:
 *   flags[2] : number of pairs whose tag disagrees with the ranges (BASE tag outside every range,
 *              TARGET tag inside one, a BASE pair whose two entries differ, a TARGET pair whose
 *              entries coincide, a block id out of range)
 *   flags[3] : 0 if flags[2] == 0, else n_req minus the index i of the first such request
 * Nothing else is read or written; tags are never modified.
 *   batch       : block_table and max_blocks are used (seq_lens is not; pass the output separately)
 *   row_of      : device int32 [n_req] table row of each scheduled request, or NULL for row i = i
 *   lens        : device int32 [n_req]
 *   blk_start   : device int32 [n_req+1] offsets into blk_ids;  blk_ids : device int32 [blk_start[n_req]]
 *   range_start : device int32 [n_req+1] offsets into ranges;   ranges  : device int32 [..][2]
 *   boundaries  : device int32 [batch][2];  flags : device int32 [4] (cleared by this call)
 * The inputs can be views of one buffer, so a step's metadata travels in one host-to-device copy. */
int ekv_lower_sparse_metadata(const ekv_pool *pool, const ekv_batch *batch, int32_t *seq_lens_out,
                              int32_t n_req, const int32_t *row_of, const int32_t *lens,
                              const int32_t *blk_start, const int32_t *blk_ids,
                              const int32_t *range_start, const int32_t *ranges,
                              int32_t *boundaries, int32_t *flags, void *stream);

/* Tags of released blocks (Sec. 3.1: a released physical block carries no fidelity): sets
 * tags[block_ids[i]] = EKV_TARGET for i < n, e.g. for the blocks of a finished request that stored
 * BASE pairs, before the allocator hands them out again.
 *   block_ids : device int32 [n] */
int ekv_reset_tags(const ekv_pool *pool, const int32_t *block_ids, int32_t n, void *stream);

/* Structured elastic decode path (Sec. 3.2; App. B.3): same computation and arguments as
 * ekv_attn_decode for a batch with has_base != 0 whose sequences all have the regular
 * TARGET-BASE-TARGET shape; a pair's mode is taken from the request's two boundaries
 * (as written by ekv_lower_metadata) and no per-block tag is read. The result is undefined when
 * the boundaries do not match the pool (an irregular request): dispatch on flags[1]. */
int ekv_attn_decode_structured(const ekv_pool *pool, int32_t layer, const ekv_batch *batch,
                               const int32_t *boundaries, const void *q, void *out,
                               int32_t num_q_heads, float sm_scale, int32_t max_seq_len,
                               void *workspace, size_t workspace_bytes, void *stream);

/* Decode attention without a caller workspace (the paper has no counterpart: this is a
 * convenience of this library). Computes exactly what ekv_attn_decode computes, with the same
 * arguments minus the workspace: the split-K partials go to a fixed 16 MiB array that is part of
 * the library image (every GPU that loads the library holds those 16 MiB until the process
 * exits; ekv_attn_decode_noalloc_max_bytes() returns the figure). It exists for callers that
 * must not, or cannot, obtain device memory at the point of the call: an inference engine that
 * has handed all free HBM to its KV pool, a plugin running inside someone else's memory budget,
 * code on a latency path where an allocator call may synchronise the device. The call itself
 * allocates and frees nothing, on the host or the device.
 *   - A shape whose partials need more than the array (ekv_attn_workspace_bytes(...) >
 *     ekv_attn_decode_noalloc_max_bytes()) is refused with EKV_ERR_WORKSPACE before any launch:
 *     use ekv_attn_decode with a workspace, or a larger "decode_chunk_tokens".
 *   - The first call on each device looks up the array's device address (one runtime query, with
 *     that device current). Make that first call outside any CUDA stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left.
 *     Nothing in it needs to start at zero, so nothing is cleared; but two calls that run on the
 *     GPU at the same time (different streams, or different host threads) overwrite each other's
 *     partials. Issue these calls on one stream, or order them with events. */
int ekv_attn_decode_noalloc(const ekv_pool *pool, int32_t layer, const ekv_batch *batch,
                            const void *q, void *out, int32_t num_q_heads, float sm_scale,
                            int32_t max_seq_len, void *stream);
size_t ekv_attn_decode_noalloc_max_bytes(void);

/* Chunked-prefill attention against a mixed-fidelity prefix (same load semantics, Sec. 3.2;
 * the prefill/decode split is the one of App. A). Request r contributes
 * C_r = q_start[r+1] - q_start[r] query tokens; they are the last C_r of its seq_lens[r]
 * tokens and their K/V are already in the pool (TARGET, as newly written KV always is).
 * Query i of the chunk sits at position seq_lens[r] - C_r + i and attends causally to
 * tokens 0 .. position.
 *   q_start      : device int32 [batch+1], q_start[0] = 0, non-decreasing
 *   q, out       : pool->elem_type [total_q][num_q_heads][head_dim]
 *   total_q, max_q_len, max_seq_len : host values (sum and maximum of C_r; bound of seq_lens)
 *   workspace    : optional (NULL / 0 is valid). With at least
 *                  ekv_attn_workspace_bytes(pool, batch, num_q_heads, max_seq_len, total_q) bytes,
 *                  256-byte aligned, the head_dim-128 kernel may cut the work units of its last
 *                  wave into pieces along the KV axis so that the wave fills the GPU; the pieces'
 *                  partial results and counters live in the workspace for the duration of the
 *                  call (contents on entry are irrelevant; one memset node precedes the kernel).
 *                  Results differ from the workspace-free call only by fp32 re-association. */
int ekv_attn_prefill_chunk(const ekv_pool *pool, int32_t layer, const ekv_batch *batch,
                           const int32_t *q_start, const void *q, void *out,
                           int32_t num_q_heads, float sm_scale,
                           int32_t total_q, int32_t max_q_len, int32_t max_seq_len,
                           void *workspace, size_t workspace_bytes, void *stream);

/* KV append (Sec. 3.2 / App. B.3): new tokens always enter the pool as full 16-bit words, in
 * TARGET blocks; demotion only ever touches older pairs. Request r contributes
 * C_r = q_start[r+1] - q_start[r] new tokens, the last C_r of its seq_lens[r] tokens; token i of
 * the chunk is written at position seq_lens[r] - C_r + i, i.e. into slot position % 16 of the
 * physical block that block_table maps logical block position / 16 to (TARGET layout). One
 * layer per call. A destination block tagged BASE is never written: the token is skipped and,
 * when dev_status is given, dev_status[0] receives (first such token index + 1); 0 = all written.
 *   q_start : device int32 [batch+1];  k_new, v_new : 16-bit words [total_new][num_kv_heads][head_dim]
 *   dev_status : device int32 [1] or NULL (cleared by this call) */
int ekv_kv_append(const ekv_pool *pool, int32_t layer, const ekv_batch *batch, const int32_t *q_start,
                  const void *k_new, const void *v_new, int32_t total_new, int32_t *dev_status,
                  void *stream);

/* Debug query for the TMA-staged decode kernel (no paper counterpart): synchronises the device, returns the
 * kernel's status word and clears it: 0 = ok, 1 = a bounded wait for a staged slab expired (results are
 * invalid); negative = ekv_status. */
int ekv_decode_status(void);

/* Debug query for the tensor-core prefill kernel (no paper counterpart). Synchronises the
 * device, returns the kernel's status word and clears it: 0 = ok, 1 = a bounded wait inside the
 * kernel expired (results are invalid), 2 = shared memory was not 1024-byte aligned (nothing
 * was computed); negative = ekv_status. */
int ekv_prefill_status(void);

/* TARGET -> BASE demotion of n_pairs pairs, in place (Sec. 3.1 "Pair-Structured Elastic KV
 * Layout"; App. B.2 "Transition Protocols"). Item i names pair pair_idx[i] of request
 * pair_req[i]: logical blocks 2p and 2p+1, both TARGET, distinct physical blocks. For every
 * layer, K and V: the high bytes of both members are packed into member 0's physical block
 * (BASE layout) and, when the residual buffers are given, the low bytes go to residual slot
 * resid_slot[i]. Then tags[kept] = EKV_BASE, tags[released] = EKV_TARGET, block_table entry
 * 2p+1 is pointed at the kept block, and freed_blocks_out[i] receives the released physical
 * id (input order). The released block's bytes are left unchanged. The released id may be
 * reused by work enqueued later on `stream`.
 *   pair_req, pair_idx, resid_slot : device int32 [n_pairs]; pairs must be distinct
 *   k_resid, v_resid : device byte buffers, or both NULL (low bytes are dropped; resid_slot
 *                      may then be NULL too)
 *   freed_blocks_out : device int32 [n_pairs] */
int ekv_downgrade(const ekv_pool *pool, const ekv_batch *batch, int32_t n_pairs,
                  const int32_t *pair_req, const int32_t *pair_idx,
                  void *k_resid, void *v_resid, const int32_t *resid_slot,
                  int32_t *freed_blocks_out, void *stream);

/* BASE -> TARGET exact refinement of n_pairs pairs (Sec. 3 opening: the low-order 8 bits refine
 * BASE back to the original TARGET; App. B.2: one step from 8 to 16 bits, mapping published
 * after materialisation). For every layer, K and V: word = (high byte << 8) | low byte;
 * member 0 is expanded in place in the kept block, member 1 into new_blocks[i]. Then both
 * tags become EKV_TARGET and block_table entry 2p+1 points at new_blocks[i]. Work enqueued
 * earlier on `stream` still sees the intact BASE pair; work enqueued later sees TARGET.
 *   new_blocks : device int32 [n_pairs], distinct free physical ids supplied by the caller
 *   k_resid, v_resid, resid_slot : as written by ekv_downgrade (required) */
int ekv_refine(const ekv_pool *pool, const ekv_batch *batch, int32_t n_pairs,
               const int32_t *pair_req, const int32_t *pair_idx, const int32_t *new_blocks,
               const void *k_resid, const void *v_resid, const int32_t *resid_slot, void *stream);

/* Device-side consistency check of a batch (no paper counterpart; stands in for a memory
 * checker). Writes to dev_status[0] the first problem found, 0 if none:
 *   1 block id out of range, 2 BASE tag while has_base == 0, 3 the two entries of a BASE pair
 *   differ, 4 a TARGET block referenced twice inside one request's pair, 5 negative seq_len or
 *   seq_len beyond max_blocks * page_size.
 * dev_status[1] receives the request index of that problem. Never traps. */
int ekv_validate_batch(const ekv_pool *pool, const ekv_batch *batch, int32_t *dev_status, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* EKV_H_ */
