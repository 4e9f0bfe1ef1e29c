"""The CUDA path on an fp16 pool (ekv_pool.elem_type = EKV_FP16; the 16-bit format the paper
names for its baselines in Sec. 4.1) against the oracle reading the same words as fp16: decode
(ring kernel, split and merge, structured path), chunked prefill (tcgen05 kernel at head_dim 128
with and without last-wave pieces, mma.sync kernel at head_dim 64) and the byte-level transitions.
Same bound as for bf16: max-abs <= 1e-2 and relative L2 <= 5e-3 on the 16-bit output."""
import numpy as np
import pytest
import torch

from paper_2609_33536_b200 import synth
from gpu_util import require_gpu, upload_state, mixed_oracle_pool, gpu_decode, gpu_prefill, assert_attn_close, dev_i32, words

pytestmark = pytest.mark.gpu


def _decode_check(oracle, wl, chunk=0, what=""):
    b = require_gpu()
    op, *_ = mixed_oracle_pool(oracle, wl)
    assert op.elem_type == oracle.FP16
    exp = oracle.attn_decode(op, 0, wl.q, wl.num_q_heads, wl.sm_scale)
    pool, batch, q = upload_state(b, op, wl.q)
    assert q.dtype == torch.float16 and pool.c.elem_type == b.EKV_FP16
    b.ekv_set_option("decode_chunk_tokens", chunk)
    try:
        got = gpu_decode(b, pool, batch, q, wl.num_q_heads, wl.sm_scale)
    finally:
        b.ekv_set_option("decode_chunk_tokens", 0)
    return assert_attn_close(got, exp, what or wl.name, elem_type="fp16")


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("G", [1, 4, 8, 3])
def test_decode_ragged_mixed(oracle, D, G):
    lens = [1, 15, 16, 17, 31, 32, 33, 63, 64, 65, 100, 257, 700, 1029]
    for frac in (0.0, 0.5, 1.0):
        wl = synth.make_workload("h16", seed=1300 + D + G, seq_lens=lens, num_q_heads=2 * G, num_kv_heads=2,
                                 head_dim=D, base_fraction=frac, elem_type="fp16")
        for chunk in (0, 64, 256):
            _decode_check(oracle, wl, chunk, what=f"fp16 D{D} G{G} f{frac} chunk{chunk}")


def test_decode_differs_from_bf16_reading(oracle):
    """The same bits on a pool declared bf16 give a different result: the element type reaches the kernel."""
    b = require_gpu()
    wl = synth.make_workload("h16b", seed=77, seq_lens=[300, 64], num_q_heads=8, num_kv_heads=2, head_dim=128,
                             base_fraction=0.5, elem_type="fp16")
    op, *_ = mixed_oracle_pool(oracle, wl)
    pool, batch, q = upload_state(b, op, wl.q)
    got16 = gpu_decode(b, pool, batch, q, wl.num_q_heads, wl.sm_scale)
    pool_b = b.Pool(pool.k_pool, pool.v_pool, pool.tags, pool.num_kv_heads, pool.head_dim, pool.page_size, elem_type=b.EKV_BF16)
    got_b = gpu_decode(b, pool_b, batch, q.view(torch.bfloat16), wl.num_q_heads, wl.sm_scale)
    assert np.max(np.abs(got16 - got_b)) > 1e-2


def test_comparator_kernel_refuses_fp16(oracle):
    b = require_gpu()
    wl = synth.make_workload("h16c", seed=78, seq_lens=[64], num_q_heads=4, num_kv_heads=2, head_dim=128, elem_type="fp16")
    op, *_ = mixed_oracle_pool(oracle, wl)
    pool, batch, q = upload_state(b, op, wl.q)
    b.ekv_set_option("decode_variant", 1)
    try:
        with pytest.raises(b.EkvError):
            gpu_decode(b, pool, batch, q, wl.num_q_heads, wl.sm_scale)
    finally:
        b.ekv_set_option("decode_variant", 0)


def test_structured_path_fp16(oracle):
    b = require_gpu()
    wl = synth.make_workload("h16s", seed=79, seq_lens=[900, 300, 64, 33], num_q_heads=8, num_kv_heads=2, head_dim=128,
                             base_fraction=0.5, base_pattern="middle", elem_type="fp16")
    op, *_ = mixed_oracle_pool(oracle, wl)
    exp = oracle.attn_decode(op, 0, wl.q, wl.num_q_heads, wl.sm_scale)
    pool, batch, q = upload_state(b, op, wl.q)
    bounds = torch.empty((batch.batch, 2), dtype=torch.int32, device="cuda")
    flags = torch.empty(2, dtype=torch.int32, device="cuda")
    b.ekv_lower_metadata(pool, batch, bounds, flags)
    f = flags.cpu().numpy()
    if f[0] == 1 and f[1] == 0:
        ws = b.new_workspace(pool, batch.batch, wl.num_q_heads, int(wl.seq_lens.max()))
        out = torch.full(q.shape, float("nan"), dtype=q.dtype, device="cuda")
        b.ekv_attn_decode_structured(pool, 0, batch, bounds, q, out, wl.num_q_heads, wl.sm_scale, int(wl.seq_lens.max()), ws)
        torch.cuda.synchronize()
        assert_attn_close(out.to(torch.float64).cpu().numpy(), exp, "fp16 structured", elem_type="fp16")
    else:
        pytest.skip("generator did not produce a T-B-T batch")


@pytest.mark.parametrize("D,G", [(128, 4), (128, 1), (128, 8), (64, 4)])
def test_prefill_ragged_mixed(oracle, D, G):
    b = require_gpu()
    lens = [300, 77, 64, 17, 129, 1]
    chunks = [100, 77, 1, 16, 65, 1]
    wl = synth.make_workload("h16p", seed=1900 + D + G, seq_lens=lens, num_q_heads=2 * G, num_kv_heads=2, head_dim=D,
                             chunk_lens=chunks, base_fraction=0.5, elem_type="fp16")
    op, *_ = mixed_oracle_pool(oracle, wl)
    exp = oracle.attn_prefill_chunk(op, 0, wl.q_start, wl.q, wl.num_q_heads, wl.sm_scale)
    pool, batch, q = upload_state(b, op, wl.q)
    assert_attn_close(gpu_prefill(b, pool, batch, q, wl), exp, f"fp16 prefill D{D} G{G}", elem_type="fp16")


def test_prefill_pieces_fp16(oracle):
    b = require_gpu()
    wl = synth.make_workload("h16q", seed=1950, seq_lens=[2100, 130, 40], num_q_heads=8, num_kv_heads=2, head_dim=128,
                             chunk_lens=[64, 64, 8], base_fraction=0.5, elem_type="fp16")
    op, *_ = mixed_oracle_pool(oracle, wl)
    exp = oracle.attn_prefill_chunk(op, 0, wl.q_start, wl.q, wl.num_q_heads, wl.sm_scale)
    pool, batch, q = upload_state(b, op, wl.q)
    assert_attn_close(gpu_prefill(b, pool, batch, q, wl, with_workspace=True), exp, "fp16 prefill pieces", elem_type="fp16")


def test_transitions_bit_exact_on_fp16_pool(oracle):
    """Downgrade and refine move bytes whatever the element type: packed bytes, residuals, tags and the
    restored words equal the oracle's."""
    b = require_gpu()
    wl = synth.make_workload("h16t", seed=1960, seq_lens=[200, 96, 64], num_q_heads=4, num_kv_heads=2, head_dim=128,
                             base_fraction=0.6, elem_type="fp16", min_free_blocks=16)
    from helpers import oracle_pool
    op = oracle_pool(oracle, wl)
    pool, batch, q = upload_state(b, op, wl.q)
    n = len(wl.base_pair_req)
    assert n > 0
    kr, vr = op.new_resid(n), op.new_resid(n)
    freed = oracle.downgrade(op, wl.base_pair_req, wl.base_pair_idx, kr, vr, np.arange(n))
    dkr, dvr = pool.new_resid(n), pool.new_resid(n)
    dfreed = torch.empty(n, dtype=torch.int32, device="cuda")
    b.ekv_downgrade(pool, batch, dev_i32(wl.base_pair_req), dev_i32(wl.base_pair_idx), dkr, dvr, dev_i32(np.arange(n)), dfreed)
    torch.cuda.synchronize()
    assert np.array_equal(dfreed.cpu().numpy(), freed)
    assert np.array_equal(pool.tags.cpu().numpy(), op.tags)
    assert np.array_equal(dkr.cpu().numpy(), kr) and np.array_equal(dvr.cpu().numpy(), vr)
    kept = np.unique(op.block_table[op.block_table >= 0])
    assert np.array_equal(words(pool.k_pool)[:, kept], op.k_pool[:, kept])
    b.ekv_refine(pool, batch, dev_i32(wl.base_pair_req), dev_i32(wl.base_pair_idx), dfreed, dkr, dvr, dev_i32(np.arange(n)))
    torch.cuda.synchronize()
    assert np.array_equal(words(pool.k_pool), wl.k_pool) and np.array_equal(words(pool.v_pool), wl.v_pool)


def test_prefill_two_terms_forced_on_fp16(oracle):
    """fp16 pools take one probability term by default; with prefill_p_terms = 2 the residual pass runs for
    them too and the fp32 result comes within 1e-4 of the oracle (one term: about 1.5e-3)."""
    from gpu_util import assert_attn_close_f32
    b = require_gpu()
    wl = synth.make_workload("pf16two", seed=515, seq_lens=[300, 129, 40], num_q_heads=8, num_kv_heads=2, head_dim=128,
                             chunk_lens=[300, 60, 40], base_fraction=0.5, elem_type="fp16")
    op, *_ = mixed_oracle_pool(oracle, wl)
    exp = oracle.attn_prefill_chunk(op, 0, wl.q_start, wl.q, wl.num_q_heads, wl.sm_scale)
    pool, batch, q = upload_state(b, op, wl.q)
    b.ekv_set_option("prefill_p_terms", 2)
    try:
        got32 = gpu_prefill(b, pool, batch, q, wl, f32=True)
        got = gpu_prefill(b, pool, batch, q, wl)
    finally:
        b.ekv_set_option("prefill_p_terms", 0)
    assert np.abs(got32 - exp).max() < 1e-4
    assert_attn_close_f32(got32, exp, "fp16, two terms")
    assert_attn_close(got, exp, "fp16, two terms", elem_type="fp16")
