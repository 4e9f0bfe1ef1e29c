"""Controller-driven step loop on the GPU (Algorithm 1 around the transition kernels, App. B.2):
shortage -> synchronous demotion -> allocation -> attention -> reserve-aware promotion whose
residuals come back from the pinned host backing. Pool state is compared bit for bit with the
oracle driven by the same decisions, and attention within tolerance, at every step."""
import numpy as np
import pytest
import torch

from paper_2609_33536_b200 import synth
from gpu_util import require_gpu, words, assert_attn_close

pytestmark = pytest.mark.gpu


def test_pressure_loop_with_controller(oracle):
    b = require_gpu()
    from paper_2609_33536_b200.runtime import ElasticRuntime
    H, Hq, D, PS = 2, 8, 128, 16
    num_blocks, n_req, max_blocks = 176, 6, 64
    rs = np.random.default_rng(42)
    kw = synth.normal_bf16(5, 1, (1, num_blocks, H * PS * D))
    vw = synth.normal_bf16(5, 2, (1, num_blocks, H * PS * D))
    k = torch.from_numpy(kw.view(np.int16)).cuda(); v = torch.from_numpy(vw.view(np.int16)).cuda()
    tags = torch.zeros(num_blocks, dtype=torch.uint8, device="cuda")
    pool = b.Pool(k, v, tags, H, D, PS)
    rt = ElasticRuntime(pool, n_req, max_blocks, resid_slots=48, min_demote_pairs=4, reserve_decay=2,
                        sink_pairs=1, recent_pairs=1)
    lens = [int(x) for x in rs.integers(300, 520, n_req)]
    for r, L in enumerate(lens):
        rt.add_request(r, L)
    # oracle mirror of the same pool
    def mirror():
        return oracle.OraclePool(kw, vw, np.zeros(num_blocks, np.uint8), rt.block_table.cpu().numpy(),
                                 rt.seq_lens.cpu().numpy(), num_kv_heads=H, head_dim=D)
    op = mirror()
    okres, ovres = op.new_resid(48), op.new_resid(48)
    q_bits = synth.normal_bf16(5, 3, (n_req, Hq, D))
    q = torch.from_numpy(q_bits.view(np.int16)).cuda().view(torch.bfloat16)
    out = torch.empty_like(q)
    saw_demotion = saw_promotion = False
    paths = set()
    released_pairs = 0
    for step in range(14):
        # pressure for the first steps, then calm: the reserve decays and promotion gets a budget
        grow = {int(r): int(rs.integers(8, 60)) for r in rs.choice(n_req - 1, 3, replace=False)} if step < 8 else {}
        if step == 9:                                     # a request finishes: its blocks come back
            released_base = rt.finish_request(5)
            released_pairs = len(released_base)
            op.tags[released_base] = 0
            op.block_table[5] = -1
            op.seq_lens[5] = 0
            lens[5] = 0
        demand = sum(rt.ctrl.demand_for(r, lens[r] + g) for r, g in grow.items())
        rows, pi, sl = rt.relieve(demand)
        if len(rows):
            saw_demotion = True
            oracle.downgrade(op, rows, pi, okres, ovres, sl)
            rt.k_resid.zero_(); rt.v_resid.zero_()        # device slots are volatile: backing must restore them
        for r, g in grow.items():
            if rt.ctrl.demand_for(r, lens[r] + g) <= rt.ctrl.free_blocks:
                lens[r] += g
                rt.grow_request(r, lens[r])
            rt.ctrl.touch(r)
        # mirror the growth (new blocks are TARGET; their content is whatever the pool holds)
        op.block_table[:] = np.where(op.block_table >= 0, op.block_table, -1)
        bt_now = rt.block_table.cpu().numpy()
        grown = (op.block_table < 0) & (bt_now >= 0)
        op.block_table[grown] = bt_now[grown]
        op.seq_lens[:] = rt.seq_lens.cpu().numpy()
        msl = int(max(lens))
        ws = b.new_workspace(pool, n_req, Hq, msl)
        b.ekv_attn_decode(pool, 0, rt.batch, q, out, Hq, D ** -0.5, msl, ws)
        out2 = torch.empty_like(out)                                    # the runtime's own dispatch: native / structured / general
        path = rt.decode(q, out2, Hq, D ** -0.5, ws)
        paths.add(path)
        assert torch.equal(out2.view(torch.int16), out.view(torch.int16)), f"step {step}: {path} path differs from the general one"
        prow, ppi, pnb, psl = rt.restore(transfer_slack=3)
        torch.cuda.synchronize()
        exp = oracle.attn_decode(op, 0, q_bits, Hq, D ** -0.5)          # attention ran before the promotion
        assert_attn_close(out.to(torch.float64).cpu().numpy(), exp, f"step {step}")
        if len(prow):
            saw_promotion = True
            oracle.refine(op, prow, ppi, pnb, okres, ovres, psl)
        assert np.array_equal(pool.tags.cpu().numpy(), op.tags), f"step {step}: tags"
        assert np.array_equal(rt.block_table.cpu().numpy(), op.block_table), f"step {step}: table"
        assert np.array_equal(words(pool.k_pool), op.k_pool), f"step {step}: k_pool"
        assert np.array_equal(words(pool.v_pool), op.v_pool), f"step {step}: v_pool"
        fl = rt.lower().cpu().tolist()                                  # re-lowering the controller's view changes nothing
        assert fl[2] == 0 and fl[0] == int(rt.ctrl.base_pairs > 0), f"step {step}: sparse metadata vs tags {fl}"
        assert np.array_equal(rt.block_table.cpu().numpy(), op.block_table), f"step {step}: table after lowering"
        for r in range(n_req):                                          # controller and device agree
            if lens[r] == 0:
                continue
            t = rt.ctrl.block_table(r)
            assert np.array_equal(t, rt.block_table[r, : len(t)].cpu().numpy())
    assert saw_demotion and saw_promotion
    assert "native" in paths and len(paths) >= 2, paths
    assert rt.stats["demoted"] - rt.stats["promoted"] - released_pairs == rt.ctrl.base_pairs == int(pool.tags.sum().item())


def test_table_rows_are_reused():
    """A finished request gives its table row back: more requests than rows can pass through."""
    b = require_gpu()
    from paper_2609_33536_b200.runtime import ElasticRuntime
    H, D = 2, 64
    k = torch.zeros((1, 64, H * 16 * D), dtype=torch.int16, device="cuda")
    pool = b.Pool(k, k.clone(), torch.zeros(64, dtype=torch.uint8, device="cuda"), H, D)
    rt = ElasticRuntime(pool, max_batch=3, max_blocks=8, resid_slots=4)
    for req in range(3):
        rt.add_request(req, 40 + req)
    for req in range(3, 9):
        rt.finish_request(req - 3)
        rt.add_request(req, 17 + req)
        row = rt.rows[req]
        assert 0 <= row < 3 and int(rt.seq_lens[row].item()) == 17 + req
        t = rt.ctrl.block_table(req)
        assert np.array_equal(rt.block_table[row, : len(t)].cpu().numpy(), t)
    assert sorted(rt.rows.values()) == [0, 1, 2]
