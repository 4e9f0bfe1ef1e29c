"""ekv_attn_prefill_chunk against the oracle: causal chunk queries over a mixed-fidelity paged
prefix (load rule of Sec. 3.2 / App. B.3; prefill phase as in App. A)."""
import numpy as np
import pytest
import torch

from paper_2609_33536_b200 import synth
from gpu_util import require_gpu, upload_state, mixed_oracle_pool, assert_attn_close, gpu_prefill

pytestmark = pytest.mark.gpu


def _check(oracle, wl, what="", with_workspace=False):
    b = require_gpu()
    op, *_ = mixed_oracle_pool(oracle, wl)
    exp = oracle.attn_prefill_chunk(op, 0, wl.q_start, wl.q, wl.num_q_heads, wl.sm_scale)
    pool, batch, q = upload_state(b, op, wl.q)
    got = gpu_prefill(b, pool, batch, q, wl, with_workspace=with_workspace)
    return assert_attn_close(got, exp, what or wl.name)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("G", [1, 2, 3, 4, 5, 6, 7, 8])     # 3, 5, 6, 7: a token's rows are padded to the next power of two
def test_ragged_chunks_mixed_prefix(oracle, D, G):
    lens = [300, 77, 64, 17, 129, 1]
    chunks = [100, 77, 1, 16, 65, 1]
    wl = synth.make_workload("pf", seed=900 + D + G, seq_lens=lens, num_q_heads=2 * G, num_kv_heads=2, head_dim=D,
                             chunk_lens=chunks, base_fraction=0.5)
    assert len(wl.base_pair_req) > 0
    _check(oracle, wl, f"D{D} G{G}")


@pytest.mark.parametrize("frac", [0.0, 1.0])
def test_all_target_and_all_base_prefix(oracle, frac):
    wl = synth.make_workload("pf2", seed=77, seq_lens=[520, 260], num_q_heads=8, num_kv_heads=2, head_dim=128,
                             chunk_lens=[130, 68], base_fraction=frac)
    _check(oracle, wl)


@pytest.mark.parametrize("variant", [0, 1])
def test_both_prefill_kernels(oracle, variant):
    """head_dim 128: the tcgen05 kernel (default) and the mma.sync kernel agree with the oracle."""
    b = require_gpu()
    wl = synth.make_workload("pfv", seed=991, seq_lens=[700, 300, 129, 1], num_q_heads=8, num_kv_heads=2, head_dim=128,
                             chunk_lens=[300, 33, 129, 1], base_fraction=0.5)
    b.ekv_set_option("prefill_variant", variant)
    try:
        _check(oracle, wl, f"prefill variant {variant}")
    finally:
        b.ekv_set_option("prefill_variant", 0)


@pytest.mark.parametrize("lens,chunks", [
    ([1100], [64]),                        # 2 units -> 2 pieces each
    ([2100, 130, 40], [64, 64, 8]),        # 4 pieces each; the short requests leave pieces without a KV tile
    ([3000, 2500, 2049, 1999, 777], [200, 130, 64, 31, 5]),
])
def test_last_wave_cut_into_pieces(oracle, lens, chunks):
    """With a workspace, a last wave that fills at most half the SMs is cut into pieces along the KV
    axis; the merged rows must meet the same bound. Run twice on one workspace: the piece counters
    have to be back at zero after a call."""
    b = require_gpu()
    wl = synth.make_workload("pfs", seed=4242 + len(lens), seq_lens=lens, num_q_heads=8, num_kv_heads=2, head_dim=128,
                             chunk_lens=chunks, base_fraction=0.5)
    op, *_ = mixed_oracle_pool(oracle, wl)
    exp = oracle.attn_prefill_chunk(op, 0, wl.q_start, wl.q, wl.num_q_heads, wl.sm_scale)
    pool, batch, q = upload_state(b, op, wl.q)
    assert_attn_close(gpu_prefill(b, pool, batch, q, wl, with_workspace=True), exp, "pieces")
    qs = torch.from_numpy(wl.q_start).cuda()
    ws = b.new_workspace(pool, len(lens), wl.num_q_heads, max(lens), int(wl.q_start[-1]))
    outs = []
    for _ in range(2):
        out = torch.full(q.shape, float("nan"), dtype=q.dtype, device="cuda")
        b.ekv_attn_prefill_chunk(pool, 0, batch, qs, q, out, wl.num_q_heads, wl.sm_scale, int(wl.q_start[-1]),
                                 max(chunks), max(lens), ws)
        outs.append(out.to(torch.float64).cpu().numpy())
    assert b.ekv_prefill_status() == 0
    assert_attn_close(outs[1], exp, "pieces, second call on the same workspace")


def test_prefill_matches_decode_on_last_row(oracle):
    """The last query of a chunk sees the whole sequence: same row as a decode step."""
    from gpu_util import gpu_decode
    b = require_gpu()
    wl = synth.make_workload("pf3", seed=78, seq_lens=[333, 200], num_q_heads=8, num_kv_heads=2, head_dim=128,
                             chunk_lens=[50, 200], base_fraction=0.5)
    op, *_ = mixed_oracle_pool(oracle, wl)
    pool, batch, q = upload_state(b, op, wl.q)
    pf = gpu_prefill(b, pool, batch, q, wl)
    last = wl.q_start[1:] - 1
    qd = q[torch.from_numpy(last.astype(np.int64)).cuda()].contiguous()
    dec = gpu_decode(b, pool, batch, qd, wl.num_q_heads, wl.sm_scale)
    assert np.max(np.abs(dec - pf[last])) <= 1e-2


@pytest.mark.parametrize("n_req,with_workspace", [(2, False), (1, True), (8, True)])
def test_prefill_config_shape_sampled(oracle, n_req, with_workspace):
    """The chunked-prefill configuration at reduced batch (8192-token prefix with 50 % BASE pairs +
    512-token chunk, 32/8 heads, D=128): all rows of 2 query heads of one request plus 64 seeded
    rows elsewhere are compared with the oracle. With one request and a workspace the 64 units are
    cut into two pieces each; with eight requests and a workspace it is the launch the benchmark
    times (444 whole units and 68 units in two pieces on 148 SMs)."""
    b = require_gpu()
    wl = synth.cfg_prefill(batch=n_req)
    op, *_ = mixed_oracle_pool(oracle, wl)
    pool, batch, q = upload_state(b, op, wl.q)
    got = gpu_prefill(b, pool, batch, q, wl, with_workspace=with_workspace)
    assert np.all(np.isfinite(got))
    rs = np.random.default_rng(5)
    C = 512
    rows = [(0, i, h) for i in range(C) for h in (3, 17)]
    rows += [(int(rs.integers(0, n_req)), int(rs.integers(0, C)), int(rs.integers(0, 32))) for _ in range(64)]
    rr = np.array([r for r, _, _ in rows], np.int32)
    hh = np.array([h for _, _, h in rows], np.int32)
    ii = np.array([i for _, i, _ in rows], np.int32)
    nv = wl.seq_lens[rr] - C + ii + 1
    qrows = wl.q[wl.q_start[rr] + ii, hh]
    exp = oracle.attend_rows(op, 0, rr, hh, nv, qrows, wl.num_q_heads, wl.sm_scale)
    assert_attn_close(got[wl.q_start[rr] + ii, hh], exp, "cfg5 sample")


@pytest.mark.parametrize("with_workspace", [False, True])
def test_growing_scores_force_rescales(oracle, with_workspace):
    """Scores that grow by about 13 (log2 units) per 128-token KV tile: the lazily kept reference
    maximum has to move, and O has to be rescaled in tensor memory, at every tile of every row."""
    b = require_gpu()
    wl = synth.make_workload("pfr", seed=5150, seq_lens=[2100, 700], num_q_heads=8, num_kv_heads=2, head_dim=128,
                             chunk_lens=[200, 64], base_fraction=0.5)
    ps, D, Hkv = wl.page_size, wl.head_dim, wl.num_kv_heads
    k5 = wl.k_pool[0].reshape(wl.num_blocks, Hkv, ps, D)
    for r, L in enumerate(wl.seq_lens):
        t = np.arange(int(L))
        ramp = synth.f32_to_bf16_bits((0.2 * t).astype(np.float32))
        phys = wl.block_table[r, t // ps]
        for g in range(Hkv):
            k5[phys, g, t % ps, 0] = ramp                 # channel 0 of K grows with the position
    wl.q[:, :, 0] = synth.f32_to_bf16_bits(np.full(wl.q.shape[:2], 4.0, np.float32))
    op, *_ = mixed_oracle_pool(oracle, wl)
    exp = oracle.attn_prefill_chunk(op, 0, wl.q_start, wl.q, wl.num_q_heads, wl.sm_scale)
    pool, batch, q = upload_state(b, op, wl.q)
    assert_attn_close(gpu_prefill(b, pool, batch, q, wl, with_workspace=with_workspace), exp, "growing scores")


@pytest.mark.parametrize("D", [64, 128])
def test_requests_without_query_tokens(oracle, D):
    """Requests whose chunk is empty contribute no rows and must not disturb their neighbours."""
    wl = synth.make_workload("pfz", seed=5160 + D, seq_lens=[130, 90, 257, 16], num_q_heads=8, num_kv_heads=2, head_dim=D,
                             chunk_lens=[0, 33, 0, 16], base_fraction=0.5)
    _check(oracle, wl, f"empty chunks D{D}")
    _check(oracle, wl, f"empty chunks D{D}, workspace", with_workspace=True)


def test_long_prefix_sampled(oracle):
    """A 32768-token prefix (2048 pages, 256 KV tiles per unit, cut into pieces with a workspace):
    sampled rows against the oracle."""
    b = require_gpu()
    wl = synth.make_workload("pfl", seed=5170, seq_lens=[32768 + 96], num_q_heads=8, num_kv_heads=2, head_dim=128,
                             chunk_lens=[96], base_fraction=0.5, base_pattern="runs", run_blocks=64)
    op, *_ = mixed_oracle_pool(oracle, wl)
    pool, batch, q = upload_state(b, op, wl.q)
    rs = np.random.default_rng(11)
    ii = np.concatenate([[0, 95], rs.integers(0, 96, size=30)]).astype(np.int32)
    hh = rs.integers(0, 8, size=len(ii)).astype(np.int32)
    rr = np.zeros(len(ii), np.int32)
    nv = (int(wl.seq_lens[0]) - 96 + ii + 1).astype(np.int32)
    exp = oracle.attend_rows(op, 0, rr, hh, nv, wl.q[ii, hh], wl.num_q_heads, wl.sm_scale)
    for ws in (False, True):
        got = gpu_prefill(b, pool, batch, q, wl, with_workspace=ws)
        assert np.all(np.isfinite(got))
        assert_attn_close(got[ii, hh], exp, f"long prefix, workspace {ws}")
