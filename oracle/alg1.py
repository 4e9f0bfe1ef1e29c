"""TEST INFRASTRUCTURE. The five scalar quantities that Algorithm 1 (Sec. 3.3) fixes for one
scheduling step (shortage, demotion count, surplus, reserve, promotion budget), as one function
over counts, for checking the host controller on random traces. Which pairs are picked is a
ranking choice the paper leaves to the runtime; only how many is fixed. The function is pinned by
hand-computed steps and by the properties the section states (tests/test_controller.py: bounds of
the demotion count, reserve at least the surplus, decay to zero in ceil(R / lambda) idle steps,
budget = free blocks beyond the reserve)."""


def step(D_t, F_t, eligible_target_pairs, R_prev, B_min_d, lam, blocks_allocated, eligible_base_pairs,
         transfer_slack):
    """One scheduling step. Returns dict(Delta, n_d, E, R, F_post, P, n_p).
    D_t: block demand of the step; F_t: free blocks before it; blocks_allocated: blocks the
    required scheduling actually takes (<= D_t when everything fits after demotion)."""
    Delta = max(0, D_t - F_t)
    E = 0
    n_d = 0
    if Delta > 0:
        n_d = min(eligible_target_pairs, max(Delta, B_min_d))
        E = max(0, n_d - Delta)
    F_post = F_t + n_d - blocks_allocated          # one block released per demoted pair (Sec. 3.1)
    R = max(0, R_prev - lam) + E
    P = max(0, F_post - R)
    n_p = min(P, transfer_slack, eligible_base_pairs) if P > 0 else 0
    return dict(Delta=Delta, n_d=n_d, E=E, R=R, F_post=F_post, P=P, n_p=n_p)
