"""ekv_attn_decode against the oracle on the same seeded inputs and the same dequantised KV
(Sec. 3.2; App. B.3). Tolerance: max-abs <= 1e-2 and relative L2 <= 5e-3 on the bf16 output."""
import numpy as np
import pytest
import torch

from paper_2609_33536_b200 import synth
from helpers import oracle_pool
from gpu_util import require_gpu, upload_state, mixed_oracle_pool, gpu_decode, assert_attn_close

pytestmark = pytest.mark.gpu


def _check(oracle, wl, chunk=0, has_base=None, what=""):
    b = require_gpu()
    op, *_ = mixed_oracle_pool(oracle, wl)
    exp = oracle.attn_decode(op, 0, wl.q, wl.num_q_heads, wl.sm_scale)
    pool, batch, q = upload_state(b, op, wl.q, has_base)
    b.ekv_set_option("decode_chunk_tokens", chunk)
    try:
        got = gpu_decode(b, pool, batch, q, wl.num_q_heads, wl.sm_scale)
    finally:
        b.ekv_set_option("decode_chunk_tokens", 0)
    return assert_attn_close(got, exp, what or wl.name)


@pytest.mark.parametrize("frac", [0.0, 0.5, 1.0])
@pytest.mark.parametrize("chunk", [0, 64, 128])
def test_tiny_config(oracle, frac, chunk):
    _check(oracle, synth.cfg_tiny(base_fraction=frac), chunk)


def test_tiny_all_target_through_elastic_path(oracle):
    """has_base = 1 although no block is BASE: tags are read and all say TARGET."""
    _check(oracle, synth.cfg_tiny(base_fraction=0.0), has_base=True)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("G", [1, 2, 4, 8, 3])
def test_group_sizes_and_ragged_lengths(oracle, D, G):
    lens = [1, 15, 16, 17, 31, 32, 33, 63, 64, 65, 100, 257, 700, 1029]
    wl = synth.make_workload("ragged", seed=300 + D + G, seq_lens=lens, num_q_heads=2 * G, num_kv_heads=2,
                             head_dim=D, base_fraction=0.5)
    for chunk in (0, 64, 256):
        _check(oracle, wl, chunk, what=f"D{D} G{G} chunk{chunk}")


@pytest.mark.parametrize("variant", [1, 3])
@pytest.mark.parametrize("D,G", [(128, 4), (128, 8), (64, 4), (64, 1)])
def test_every_kernel_variant(oracle, variant, D, G):
    """The ring-staged kernel and the page-stepped comparator both serve any batch."""
    b = require_gpu()
    lens = [1, 16, 17, 33, 64, 95, 129, 700, 1029, 2500]
    for frac in (0.0, 0.5, 1.0):
        wl = synth.make_workload("var", seed=400 + D + G, seq_lens=lens, num_q_heads=2 * G, num_kv_heads=2,
                                 head_dim=D, base_fraction=frac)
        b.ekv_set_option("decode_variant", variant)
        try:
            for chunk in (0, 128):
                _check(oracle, wl, chunk, what=f"variant{variant} D{D} G{G} f{frac} chunk{chunk}")
            if frac == 0.0:
                _check(oracle, wl, 0, has_base=False, what=f"variant{variant} native")
        finally:
            b.ekv_set_option("decode_variant", 0)


def test_many_splits_long_sequence(oracle):
    wl = synth.make_workload("long", seed=77, seq_lens=[5000, 4097, 64], num_q_heads=8, num_kv_heads=2,
                             head_dim=128, base_fraction=0.5, base_pattern="runs", run_blocks=8)
    for chunk in (64, 512, 1024, 0):
        _check(oracle, wl, chunk, what=f"chunk{chunk}")


@pytest.mark.parametrize("slices", [1, 4, 8])
def test_merge_slices(oracle, slices):
    """The merge kernel with 1, 4 or 8 slices of threads sharing a row's splits (79 and 3 splits here)."""
    b = require_gpu()
    wl = synth.make_workload("slices", seed=78, seq_lens=[5000, 130, 0, 640], num_q_heads=8, num_kv_heads=2,
                             head_dim=128, base_fraction=0.5)
    b.ekv_set_option("decode_merge_slices", slices)
    try:
        for chunk in (64, 256):
            _check(oracle, wl, chunk, what=f"slices{slices} chunk{chunk}")
    finally:
        b.ekv_set_option("decode_merge_slices", 0)


def test_empty_request_and_padded_table(oracle):
    b = require_gpu()
    wl = synth.make_workload("empty", seed=9, seq_lens=[0, 40, 0, 16], num_q_heads=4, num_kv_heads=2, head_dim=64)
    op = oracle_pool(oracle, wl)
    exp = oracle.attn_decode(op, 0, wl.q, 4, wl.sm_scale)
    pool, batch, q = upload_state(b, op, wl.q)
    got = gpu_decode(b, pool, batch, q, 4, wl.sm_scale)
    assert not got[0].any() and not got[2].any()
    assert_attn_close(got, exp)
    got = gpu_decode(b, pool, batch, q, 4, wl.sm_scale, max_seq_len=wl.max_blocks * 16)   # loose bound
    assert_attn_close(got, exp)


def test_partially_filled_base_pair_and_garbage_tail(oracle):
    """Second member of a BASE pair half filled; the unused slots of tail pages hold NaN / Inf bit
    patterns, which must not leak into the result in either mode."""
    b = require_gpu()
    wl = synth.make_workload("part", seed=8, seq_lens=[56, 40], num_q_heads=8, num_kv_heads=2, head_dim=128)
    H, D = 2, 128
    for r, L in enumerate(wl.seq_lens):
        last = wl.block_table[r, (L - 1) // 16]
        for pool_arr in (wl.k_pool, wl.v_pool):
            blk = pool_arr[0, last].reshape(H, 16, D)
            blk[:, L % 16:, :] = 0x7FC0                      # bf16 NaN (its high byte reads as +2^127 in BASE)
            blk[:, L % 16:, ::2] = 0xFF80                    # -Inf
    op = oracle_pool(oracle, wl)
    oracle.downgrade(op, [0], [1])
    exp = oracle.attn_decode(op, 0, wl.q, 8, wl.sm_scale)
    pool, batch, q = upload_state(b, op, wl.q)
    got = gpu_decode(b, pool, batch, q, 8, wl.sm_scale)
    assert_attn_close(got, exp)


def test_layers_are_addressed_separately(oracle):
    b = require_gpu()
    wl = synth.make_workload("layers", seed=31, seq_lens=[200, 90], num_q_heads=4, num_kv_heads=2, head_dim=128,
                             num_layers=3, base_fraction=0.5)
    op, *_ = mixed_oracle_pool(oracle, wl)
    pool, batch, q = upload_state(b, op, wl.q)
    for layer in range(3):
        exp = oracle.attn_decode(op, layer, wl.q, 4, wl.sm_scale)
        assert_attn_close(gpu_decode(b, pool, batch, q, 4, wl.sm_scale, layer=layer), exp, f"layer {layer}")


def test_attention_around_gpu_transitions(oracle):
    """Same stream: attend (TARGET) -> ekv_downgrade -> attend (mixed) -> ekv_refine -> attend; each
    result matches the oracle in the corresponding state, and the last equals the first bit for bit."""
    from gpu_util import dev_i32
    b = require_gpu()
    wl = synth.cfg_tiny()
    op = oracle_pool(oracle, wl)
    pool, batch, q = b.upload(wl)
    n = len(wl.base_pair_req)
    kres, vres = pool.new_resid(n), pool.new_resid(n)
    okres, ovres = op.new_resid(n), op.new_resid(n)
    slots = np.arange(n, dtype=np.int32)
    ws = b.new_workspace(pool, wl.batch, wl.num_q_heads, 256)
    outs = [torch.empty_like(q) for _ in range(3)]
    freed = torch.empty(n, dtype=torch.int32, device="cuda")
    pr, pi, sl = dev_i32(wl.base_pair_req), dev_i32(wl.base_pair_idx), dev_i32(slots)
    b.ekv_attn_decode(pool, 0, batch, q, outs[0], wl.num_q_heads, wl.sm_scale, 256, ws)
    b.ekv_downgrade(pool, batch, pr, pi, kres, vres, sl, freed)
    batch.has_base = True
    b.ekv_attn_decode(pool, 0, batch, q, outs[1], wl.num_q_heads, wl.sm_scale, 256, ws)
    b.ekv_refine(pool, batch, pr, pi, freed, kres, vres, sl)      # released ids handed straight back
    batch.has_base = False
    b.ekv_attn_decode(pool, 0, batch, q, outs[2], wl.num_q_heads, wl.sm_scale, 256, ws)
    torch.cuda.synchronize()
    e0 = oracle.attn_decode(op, 0, wl.q, wl.num_q_heads, wl.sm_scale)
    oracle.downgrade(op, wl.base_pair_req, wl.base_pair_idx, okres, ovres, slots)
    e1 = oracle.attn_decode(op, 0, wl.q, wl.num_q_heads, wl.sm_scale)
    g = [o.to(torch.float64).cpu().numpy() for o in outs]
    assert_attn_close(g[0], e0, "before")
    assert_attn_close(g[1], e1, "mixed")
    assert np.array_equal(g[0], g[2])
    assert np.max(np.abs(g[0] - g[1])) > 1e-3


def test_growing_scores_across_splits(oracle):
    """Scores that grow steeply with the position: every step moves the running maximum and the last
    split dominates the merge by hundreds of log2 units."""
    wl = synth.make_workload("dgr", seed=5151, seq_lens=[2100, 700, 33], num_q_heads=8, num_kv_heads=2, head_dim=128,
                             base_fraction=0.5)
    ps, D, Hkv = wl.page_size, wl.head_dim, wl.num_kv_heads
    k5 = wl.k_pool[0].reshape(wl.num_blocks, Hkv, ps, D)
    for r, L in enumerate(wl.seq_lens):
        t = np.arange(int(L))
        ramp = synth.f32_to_bf16_bits((0.2 * t).astype(np.float32))
        phys = wl.block_table[r, t // ps]
        for g in range(Hkv):
            k5[phys, g, t % ps, 0] = ramp
    wl.q[:, :, 0] = synth.f32_to_bf16_bits(np.full(wl.q.shape[:2], 4.0, np.float32))
    for chunk in (0, 256):
        _check(oracle, wl, chunk, what=f"growing scores chunk{chunk}")


@pytest.mark.parametrize("frac", [0.0, 0.5, 1.0])
def test_tma_staging_matches_cp_async(oracle, frac):
    """Option decode_staging = 2 (tensor copies into the ring, head_dim 128) changes how the slabs travel,
    not what is computed: outputs equal the default path's bit for bit, and no bounded wait expires."""
    b = require_gpu()
    wl = synth.make_workload("tma", seed=808, seq_lens=[1500, 257, 64, 33, 1, 900], num_q_heads=8, num_kv_heads=2, head_dim=128,
                             base_fraction=frac)
    op, *_ = mixed_oracle_pool(oracle, wl)
    pool, batch, q = upload_state(b, op, wl.q)
    ref = gpu_decode(b, pool, batch, q, wl.num_q_heads, wl.sm_scale)
    b.ekv_set_option("decode_staging", 2)
    try:
        got = gpu_decode(b, pool, batch, q, wl.num_q_heads, wl.sm_scale)
    finally:
        b.ekv_set_option("decode_staging", 0)
    assert b.ekv_decode_status() == 0
    assert np.array_equal(got, ref)
    assert_attn_close(got, oracle.attn_decode(op, 0, wl.q, wl.num_q_heads, wl.sm_scale), f"tma f={frac}")
