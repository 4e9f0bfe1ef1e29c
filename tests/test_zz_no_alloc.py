"""ekv_attn_decode_noalloc: the decode entry point for callers that cannot allocate device
memory (its split-K partials live in a fixed array inside the library instead of a workspace
the caller would have to obtain). Checked through the C ABI against ekv_attn_decode on the
same inputs, on two calls in a row: the second call finds the first call's partials in the
shared array and must not be disturbed by them. The two entry points launch the same kernels
with the same split size, so their outputs must be equal bit for bit; and the call must leave
the device's free memory and torch's allocator figures as it found them. Collected last on
purpose."""
import numpy as np
import pytest
import torch

from paper_2609_33536_b200 import synth
from gpu_util import require_gpu, upload_state, mixed_oracle_pool, assert_attn_close

pytestmark = pytest.mark.gpu


def _both_entry_points(b, oracle, wl, chunk):
    """Workspace call and no-alloc call on the same inputs; returns (max splits, outputs equal?)."""
    op, *_ = mixed_oracle_pool(oracle, wl)
    pool, batch, q = upload_state(b, op, wl.q)
    msl = int(wl.seq_lens.max())
    need = b.ekv_attn_workspace_bytes(pool, wl.batch, wl.num_q_heads, msl)
    assert need <= b.ekv_attn_decode_noalloc_max_bytes()
    ws = b.new_workspace(pool, wl.batch, wl.num_q_heads, msl)
    ref = torch.full(q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    got = torch.full(q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    b.ekv_attn_decode(pool, 0, batch, q, ref, wl.num_q_heads, wl.sm_scale, msl, ws)
    torch.cuda.synchronize()
    free0, alloc0, resv0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    b.ekv_attn_decode_noalloc(pool, 0, batch, q, got, wl.num_q_heads, wl.sm_scale, msl)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0, "free device memory changed across the no-alloc call"
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == resv0
    assert torch.equal(got.view(torch.int16), ref.view(torch.int16)), f"{wl.name}: no-alloc and workspace entry points differ"
    assert_attn_close(got.to(torch.float64).cpu().numpy(), oracle.attn_decode(op, 0, wl.q, wl.num_q_heads, wl.sm_scale),
                      f"{wl.name}: vs oracle")
    return need


def test_noalloc_matches_workspace_entry_point_twice(oracle):
    b = require_gpu()
    # two different batches, several splits each (chunk 64), so the shared array is really used
    wls = [synth.make_workload("na1", seed=501, seq_lens=[700, 64, 1029, 33], num_q_heads=8, num_kv_heads=2,
                               head_dim=128, base_fraction=0.5),
           synth.make_workload("na2", seed=502, seq_lens=[257, 900], num_q_heads=8, num_kv_heads=2,
                               head_dim=128, base_fraction=1.0)]
    # the first call on a device looks up the array's address: make it before the memory figures are read
    b.ekv_set_option("decode_chunk_tokens", 64)
    try:
        for wl in wls:
            assert _both_entry_points(b, oracle, wl, 64) > 0
    finally:
        b.ekv_set_option("decode_chunk_tokens", 0)


def test_noalloc_single_split_leaves_the_array_alone(oracle):
    """No sequence longer than one split: nothing is written to the shared array, the rows come
    straight from the split kernel, and the result is still that of the workspace call."""
    b = require_gpu()
    wl = synth.make_workload("na3", seed=503, seq_lens=[200, 1, 256, 17], num_q_heads=8, num_kv_heads=2,
                             head_dim=128, base_fraction=0.5)
    b.ekv_set_option("decode_chunk_tokens", 256)
    try:
        assert _both_entry_points(b, oracle, wl, 256) == 0      # a single split needs no partials
    finally:
        b.ekv_set_option("decode_chunk_tokens", 0)


def test_noalloc_refuses_shapes_beyond_its_array(oracle):
    b = require_gpu()
    wl = synth.cfg_tiny()
    op, *_ = mixed_oracle_pool(oracle, wl)
    pool, batch, q = upload_state(b, op, wl.q)
    out = torch.empty_like(q)
    b.ekv_set_option("decode_chunk_tokens", 64)
    try:
        # claim a far longer maximum length than the table allows for: refused on the host
        with pytest.raises(b.EkvError):
            b.ekv_attn_decode_noalloc(pool, 0, batch, q, out, wl.num_q_heads, wl.sm_scale, 1 << 28)
    finally:
        b.ekv_set_option("decode_chunk_tokens", 0)
