/*
 * ekv_controller.h -- C ABI of the host-side pressure-aware fidelity controller.
 *
 * A host library (no GPU work, no allocation on the device): it owns the logical -> physical
 * block mapping of the requests, the free list, the pair state table and the reserve of the
 * paper's Algorithm 1 ("Pressure-aware fidelity control", Sec. 3.3), and tells the caller WHICH
 * pairs to hand to ekv_downgrade / ekv_refine (ekv.h) and which block ids to use. The caller
 * enqueues the kernels and reports completion; the controller never exposes a half-made state:
 * released blocks re-enter the free list only at ekv_ctrl_commit_demotion, and a promoted pair
 * counts as TARGET only at ekv_ctrl_commit_promotion (App. B.2 "Transition Protocols").
 *
 * Algorithm 1, per scheduling step t (symbols as in the paper):
 *   Delta_t = max(0, D_t - F_t)                     shortage of the step's block demand D_t
 *   if Delta_t > 0:  n_d = min(|P_d|, max(Delta_t, B_min_d)) pairs are demoted,
 *                    E_t = max(0, n_d - Delta_t)    surplus released beyond the shortage
 *   R_t = max(0, R_{t-1} - lambda) + E_t            decaying demotion reserve
 *   P_t = max(0, F_t_post - R_t)                    promotion budget after required scheduling
 * Eligibility (Sec. 3.3; App. B.1): only pairs whose two blocks are full, outside the first
 * sink_pairs and the last recent_pairs pairs of their request, and for which a residual slot
 * (the recoverable backing) is available; ranked least-recently-used request first, oldest pair
 * first. Promotion candidates are ranked most-recently-used request first.
 *
 * All functions return 0 on success or a negative EKV_CTRL_* code; none of them blocks.
 * The controller is not thread-safe: call it from the scheduling thread.
 */
#ifndef EKV_CONTROLLER_H_
#define EKV_CONTROLLER_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ekv_ctrl ekv_ctrl;   /* opaque */

enum {
    EKV_CTRL_OK = 0,
    EKV_CTRL_ERR_ARG = -1,          /* null pointer, unknown request, bad size */
    EKV_CTRL_ERR_NO_BLOCKS = -2,    /* not enough free physical blocks */
    EKV_CTRL_ERR_STATE = -3,        /* call out of order (e.g. commit without a plan) */
    EKV_CTRL_ERR_CAPACITY = -4      /* output array too small */
};

typedef struct ekv_ctrl_config {
    int32_t num_blocks;          /* physical blocks of the pool; ids 0 .. num_blocks-1 */
    int32_t page_size;           /* tokens per block (16) */
    int32_t min_demote_pairs;    /* B_min^d; the paper's default is 16 */
    int32_t reserve_decay;       /* lambda, blocks per step; the paper's default is 2 */
    int32_t sink_pairs;          /* leading pairs of every request that are never demoted */
    int32_t recent_pairs;        /* trailing pairs of every request that are never demoted */
    int32_t resid_slots;         /* residual slots = pairs that can be BASE at the same time */
    int32_t reserved_;           /* set to 0 */
} ekv_ctrl_config;

ekv_ctrl *ekv_ctrl_create(const ekv_ctrl_config *cfg);      /* NULL on bad arguments */
void ekv_ctrl_destroy(ekv_ctrl *c);

/* Requests. add allocates ceil(n_tokens / page_size) blocks from the free list (lowest ids
 * first); grow extends to new_n_tokens (new blocks are TARGET: appended KV is written in TARGET
 * form, Sec. 3.2); remove returns every block and residual slot. touch marks the request as
 * used in the current step (ranking signal). */
int ekv_ctrl_add_request(ekv_ctrl *c, int32_t req, int32_t n_tokens);
int ekv_ctrl_grow_request(ekv_ctrl *c, int32_t req, int32_t new_n_tokens);
int ekv_ctrl_remove_request(ekv_ctrl *c, int32_t req);
int ekv_ctrl_touch(ekv_ctrl *c, int32_t req);

/* Blocks a step would need: demand for growing `req` to new_n_tokens (side-effect free). */
int32_t ekv_ctrl_demand_for(const ekv_ctrl *c, int32_t req, int32_t new_n_tokens);

/* Step t, before required scheduling: given the step's demand D_t, choose the demotion batch
 * (possibly empty). Writes n_out items: request, pair index, residual slot for each. The batch
 * is "in flight" until ekv_ctrl_commit_demotion. */
int ekv_ctrl_plan_demotion(ekv_ctrl *c, int32_t demand, int32_t *pair_req, int32_t *pair_idx,
                           int32_t *resid_slot, int32_t cap, int32_t *n_out);
/* After the GPU transition completed: freed_blocks[i] as written by ekv_downgrade (checked
 * against the controller's own table; a mismatch is EKV_CTRL_ERR_STATE). Pairs become BASE, the
 * released blocks join the free list, E_t is recorded. */
int ekv_ctrl_commit_demotion(ekv_ctrl *c, int32_t n, const int32_t *freed_blocks);

/* Step t, after required scheduling and allocation: advances the reserve (R_t; once per step,
 * however often this is called; a step in which it is not called at all has its update applied
 * when the next ekv_ctrl_plan_demotion opens the following step), computes the promotion budget
 * P_t from the current free count and picks min(P_t, transfer_slack) BASE pairs. Each reserves
 * one free block now (new_blocks[i]). In flight until commit. */
int ekv_ctrl_plan_promotion(ekv_ctrl *c, int32_t transfer_slack, int32_t *pair_req, int32_t *pair_idx,
                            int32_t *new_blocks, int32_t *resid_slot, int32_t cap, int32_t *n_out);
/* After ekv_refine completed (or was enqueued on the stream all consumers use): the first n
 * in-flight promotions become TARGET and their residual slots are released. */
int ekv_ctrl_commit_promotion(ekv_ctrl *c, int32_t n);

/* Queries. */
int32_t ekv_ctrl_free_blocks(const ekv_ctrl *c);
int32_t ekv_ctrl_reserve(const ekv_ctrl *c);              /* R_t after the last plan_promotion */
int32_t ekv_ctrl_last_shortage(const ekv_ctrl *c);        /* Delta_t of the last plan_demotion */
int32_t ekv_ctrl_last_surplus(const ekv_ctrl *c);         /* E_t of the last committed demotion */
int32_t ekv_ctrl_last_budget(const ekv_ctrl *c);          /* P_t of the last plan_promotion */
int32_t ekv_ctrl_base_pairs(const ekv_ctrl *c);           /* pairs currently BASE (published) */
int32_t ekv_ctrl_request_blocks(const ekv_ctrl *c, int32_t req);     /* logical blocks of req, <0 if unknown */
/* Block-table row of a request as the GPU sees it (both entries of a BASE pair hold the kept
 * block); returns the number of entries written or a negative code. */
int ekv_ctrl_block_table(const ekv_ctrl *c, int32_t req, int32_t *out, int32_t cap);
/* Mode (0 TARGET, 1 BASE, 2 demotion in flight, 3 promotion in flight) of pair p of req. */
int ekv_ctrl_pair_mode(const ekv_ctrl *c, int32_t req, int32_t pair);

#ifdef __cplusplus
}
#endif
#endif /* EKV_CONTROLLER_H_ */
