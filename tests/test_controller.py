"""Host-side fidelity controller against the paper's Algorithm 1 (Sec. 3.3) and its state rules
(Sec. 3.1: exactly one block per pair either way; App. B.1: sink / recent / backing eligibility;
App. B.2: released blocks and new mappings appear only at commit). CPU only."""
import numpy as np
import pytest

from oracle import alg1
from paper_2609_33536_b200 import build as ekv_build, controller


@pytest.fixture(scope="module", autouse=True)
def _built():
    ekv_build.build()


def test_worked_numbers_of_the_recurrences():
    """Hand-computed from the formulas: B_min = 16, lambda = 2."""
    s = alg1.step(D_t=8, F_t=5, eligible_target_pairs=20, R_prev=0, B_min_d=16, lam=2, blocks_allocated=8,
                  eligible_base_pairs=0, transfer_slack=4)
    assert s == dict(Delta=3, n_d=16, E=13, R=13, F_post=13, P=0, n_p=0)
    s = alg1.step(D_t=1, F_t=13, eligible_target_pairs=4, R_prev=13, B_min_d=16, lam=2, blocks_allocated=1,
                  eligible_base_pairs=16, transfer_slack=4)
    assert s == dict(Delta=0, n_d=0, E=0, R=11, F_post=12, P=1, n_p=1)
    s = alg1.step(D_t=30, F_t=2, eligible_target_pairs=10, R_prev=0, B_min_d=16, lam=2, blocks_allocated=12,
                  eligible_base_pairs=0, transfer_slack=4)
    assert s["Delta"] == 28 and s["n_d"] == 10 and s["E"] == 0 and s["P"] == 0      # capped by |P_d|


def _total_blocks_in_use(c, reqs):
    used = []
    for r in reqs:
        t = c.block_table(r)
        for p in range((len(t) + 1) // 2):
            mode = c.pair_mode(r, p)
            used.append(int(t[2 * p]))
            if 2 * p + 1 < len(t) and t[2 * p + 1] != t[2 * p]:
                used.append(int(t[2 * p + 1]))
            elif 2 * p + 1 < len(t):
                assert mode in (1, 3)           # both entries equal only for a BASE pair (or one being promoted)
    return used


def test_controller_follows_algorithm_1():
    rs = np.random.default_rng(0)
    num_blocks, B_min, lam = 400, 16, 2
    c = controller.Controller(num_blocks, min_demote_pairs=B_min, reserve_decay=lam, sink_pairs=1, recent_pairs=1,
                              resid_slots=128)
    reqs = list(range(10))
    lens = {}
    for r in reqs:
        lens[r] = int(rs.integers(300, 600))
        c.add_request(r, lens[r])
    R_prev = 0
    in_flight_new = 0
    for t in range(60):
        grow = {r: int(rs.integers(0, 40)) for r in rs.choice(reqs, 4, replace=False)}
        D = sum(c.demand_for(r, lens[r] + g) for r, g in grow.items())
        F = c.free_blocks
        # what the paper's eligibility leaves: full pairs minus sink and recent pairs, TARGET, slot available
        elig = 0
        for r in reqs:
            n_pairs = (c.block_table(r).size + 1) // 2
            for p in range(n_pairs):
                full = p < lens[r] // 32
                if full and 1 <= p < n_pairs - 1 and c.pair_mode(r, p) == 0:
                    elig += 1
        slots_free = 128 - c.base_pairs - in_flight_new
        base_before = c.base_pairs
        pr, pi, sl = c.plan_demotion(D)
        exp = alg1.step(D, F, min(elig, slots_free), R_prev, B_min, lam, blocks_allocated=0,
                        eligible_base_pairs=0, transfer_slack=0)
        assert c.last_shortage == exp["Delta"] and len(pr) == exp["n_d"]
        # never a protected pair, never twice the same pair, distinct residual slots
        assert len({(a, b) for a, b in zip(pr, pi)}) == len(pr) == len(set(sl.tolist()))
        for r, p in zip(pr, pi):
            n_pairs = (c.block_table(r).size + 1) // 2
            assert 1 <= p < n_pairs - 1 and p < lens[r] // 32 and c.pair_mode(r, p) == 2
        # the GPU would report the second member's block as released
        freed = [int(c.block_table(r)[2 * p + 1]) for r, p in zip(pr, pi)]
        free_mid = c.free_blocks
        assert free_mid == F                                   # nothing is released before the commit
        c.commit_demotion(freed)
        assert c.free_blocks == F + len(pr) and c.last_surplus == exp["E"] and c.base_pairs == base_before + len(pr)
        # required scheduling: grow what fits
        allocated = 0
        for r, g in grow.items():
            need = c.demand_for(r, lens[r] + g)
            if need <= c.free_blocks:
                c.grow_request(r, lens[r] + g); lens[r] += g; allocated += need
            c.touch(r)
        F_post = c.free_blocks
        slack = int(rs.integers(0, 6))
        qr, qi, nb, qs = c.plan_promotion(slack)
        exp2 = alg1.step(D, F, min(elig, slots_free), R_prev, B_min, lam, blocks_allocated=allocated,
                         eligible_base_pairs=c.base_pairs, transfer_slack=slack)
        assert exp2["F_post"] == F_post
        assert c.reserve == exp2["R"] and c.last_budget == exp2["P"] and len(qr) == exp2["n_p"]
        assert c.free_blocks == F_post - len(qr)               # one block reserved per promoted pair, up front
        for r, p in zip(qr, qi):
            assert c.pair_mode(r, p) == 3
            assert c.block_table(r)[2 * p] == c.block_table(r)[2 * p + 1]     # mapping not published yet
        c.commit_promotion(len(qr))
        for r, p, b in zip(qr, qi, nb):
            assert c.pair_mode(r, p) == 0 and c.block_table(r)[2 * p + 1] == b
        R_prev = exp2["R"]
        # conservation: every physical block is free or used exactly once
        used = _total_blocks_in_use(c, reqs)
        assert len(used) == len(set(used)) and len(used) + c.free_blocks == num_blocks
    assert c.base_pairs > 0
    for r in reqs:
        c.remove_request(r)
    assert c.free_blocks == num_blocks and c.base_pairs == 0


def test_commit_rules_and_errors():
    c = controller.Controller(64, min_demote_pairs=2, reserve_decay=1, sink_pairs=0, recent_pairs=0, resid_slots=8)
    c.add_request(7, 16 * 10)
    with pytest.raises(controller.ControllerError):
        c.add_request(8, 16 * 100)                            # not enough blocks
    pr, pi, sl = c.plan_demotion(c.free_blocks + 1)           # shortage 1 -> B_min = 2 pairs
    assert len(pr) == 2 and c.last_shortage == 1
    with pytest.raises(controller.ControllerError):
        c.plan_promotion(1)                                   # demotion still in flight
    with pytest.raises(controller.ControllerError):
        c.commit_demotion([0, 0])                             # not the blocks the table says
    with pytest.raises(controller.ControllerError):
        c.remove_request(7)                                   # transition in flight
    freed = [int(c.block_table(7)[2 * p + 1]) for p in pi]
    c.commit_demotion(freed)
    assert c.last_surplus == 1


def test_reserve_bounds_decay_and_budget():
    """Properties Alg. 1 / Sec. 3.3 fix, checked on the controller alone with hand-computed numbers
    (B_min = 6, lambda = 2, 40 blocks, one request of 30 blocks -> 10 free):
      step 1: demand 12 -> Delta = 2, n_d = max(2, 6) = 6 <= eligible, E = 4, R_1 = 0 + 4 >= E, F_post = 16
      then idle steps: R decays 4 -> 2 -> 0 in ceil(4 / 2) = 2 steps and stays 0;
      the promotion budget is P_t = max(0, F_post - R_t) at every step (no transfer slack is granted,
      so nothing is promoted and F_post stays 16)."""
    c = controller.Controller(40, min_demote_pairs=6, reserve_decay=2, sink_pairs=0, recent_pairs=0, resid_slots=16)
    c.add_request(1, 16 * 30)
    assert c.free_blocks == 10
    pr, pi, sl = c.plan_demotion(12)
    assert c.last_shortage == 2 and len(pr) == 6           # Delta <= n_d <= |P_d|, n_d >= min(B_min, |P_d|)
    c.commit_demotion([int(c.block_table(1)[2 * p + 1]) for p in pi])
    assert c.last_surplus == 4 and c.free_blocks == 16
    expected = [(4, 12), (2, 14), (0, 16), (0, 16)]        # (R_t, P_t) for steps 1..4
    for t, (R, P) in enumerate(expected):
        if t > 0:
            assert len(c.plan_demotion(0)[0]) == 0
        got = c.plan_promotion(0)
        assert len(got[0]) == 0
        assert (c.reserve, c.last_budget) == (R, P), f"step {t + 1}"
        assert c.reserve >= (4 if t == 0 else 0)           # R_t >= E_t


def test_a_step_without_a_promotion_plan_still_updates_the_reserve_once():
    """lambda = 1, B_min = 4. Step 1 demotes with E_1 = 3 and never asks for a promotion plan; its
    update R_1 = max(0, 0 - 1) + 3 = 3 is applied when step 2 opens. Step 2 (no shortage) asks
    twice: R_2 = max(0, 3 - 1) + 0 = 2 both times. Step 3 has neither a shortage nor a promotion
    plan; step 4 then sees R_3 = 1 applied and computes R_4 = 0."""
    c = controller.Controller(40, min_demote_pairs=4, reserve_decay=1, sink_pairs=0, recent_pairs=0, resid_slots=16)
    c.add_request(1, 16 * 30)
    pr, pi, sl = c.plan_demotion(c.free_blocks + 1)
    assert len(pr) == 4
    c.commit_demotion([int(c.block_table(1)[2 * p + 1]) for p in pi])
    assert c.last_surplus == 3
    c.plan_demotion(0)                                     # step 2 opens
    c.plan_promotion(0)
    assert c.reserve == 2
    c.plan_promotion(0)
    assert c.reserve == 2                                  # once per step
    c.plan_demotion(0)                                     # step 3: no promotion plan at all
    c.plan_demotion(0)                                     # step 4
    c.plan_promotion(0)
    assert c.reserve == 0
