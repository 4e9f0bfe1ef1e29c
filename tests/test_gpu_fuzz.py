"""Seeded fuzz of the attention entry points against the oracle: random shapes over the supported
space (head_dim 64 / 128, 1-8 query heads per kv head, 1-3 kv heads, 1-5 requests whose lengths
over-sample the page and tile boundaries, BASE fraction 0 / 0.3 / 0.5 / 1 in three patterns, both
element types, every kernel variant, split sizes 64-1024, chunk lengths 0..L). Every case is
checked twice: the 16-bit output under the comparison rule of the task (max-abs 1e-2, relative L2
5e-3), and the library's unrounded fp32 result (option "attn_out_f32") under the tighter
pre-rounding bound, which separates kernel error from the error of the output grid.

The case lists are fixed by the seeds below; the three prefill cases that an earlier unseeded run
recorded as outside 1e-2 (rows that two or three tokens dominate) are listed explicitly."""
import numpy as np
import pytest

from paper_2609_33536_b200 import synth
from gpu_util import (require_gpu, upload_state, mixed_oracle_pool, gpu_decode, gpu_prefill,
                      assert_attn_close, assert_attn_close_f32)

pytestmark = pytest.mark.gpu

SPECIAL_LENS = [1, 15, 16, 17, 31, 32, 33, 47, 48, 63, 64, 65, 127, 128, 129, 255, 256, 257]
CASES_PER_GROUP = 32
DECODE_GROUPS = 10          # 320 decode cases
PREFILL_GROUPS = 10         # 320 prefill cases
WORK_CAP = 2.5e8            # oracle multiply-adds per case (rows x tokens x head_dim)


def draw_case(rs, kind):
    """One random case description (a dict of plain values, so that a failure can be replayed)."""
    while True:
        c = dict(kind=kind, D=int(rs.choice([64, 128])), G=int(rs.choice([1, 2, 3, 4, 5, 8])), H=int(rs.choice([1, 2, 3])),
                 et=str(rs.choice(["bf16", "bf16", "fp16"])), f=float(rs.choice([0.0, 0.3, 0.5, 1.0])),
                 pat=str(rs.choice(["random", "middle", "oldest"])), seed=int(rs.integers(1, 1 << 30)))
        n = int(rs.integers(1, 6))
        c["lens"] = [int(rs.choice(SPECIAL_LENS)) if rs.random() < 0.4 else int(rs.integers(1, 2000)) for _ in range(n)]
        if kind == "decode":
            c["chunk"] = int(rs.choice([0, 64, 128, 256, 1024]))
            c["v"] = int(rs.choice([0, 0, 0, 1])) if c["et"] == "bf16" else 0
            c["hb"] = bool(rs.random() < 0.3)             # has_base forced on although the pool may hold no BASE block
            work = sum(c["lens"]) * c["G"] * c["H"] * c["D"]
        else:
            c["chunks"] = [int(rs.integers(0, L + 1)) if rs.random() < 0.8 else L for L in c["lens"]]
            if sum(c["chunks"]) == 0:
                c["chunks"][0] = 1
            c["v"] = int(rs.choice([0, 0, 1]))
            c["ws"] = bool(rs.random() < 0.5)
            work = sum(ch * L for ch, L in zip(c["chunks"], c["lens"])) * c["G"] * c["H"] * c["D"]
        if work <= WORK_CAP:
            return c


def run_case(b, oracle, c):
    """Returns (max-abs of the 16-bit output, relative L2, max-abs of the fp32 result)."""
    kw = dict(seed=c["seed"], seq_lens=c["lens"], num_q_heads=c["G"] * c["H"], num_kv_heads=c["H"], head_dim=c["D"],
              base_fraction=c["f"], base_pattern=c["pat"], elem_type=c["et"])
    what = " ".join(f"{k}={v}" for k, v in c.items())
    if c["kind"] == "decode":
        wl = synth.make_workload("fz", **kw)
        op, *_ = mixed_oracle_pool(oracle, wl)
        exp = oracle.attn_decode(op, 0, wl.q, wl.num_q_heads, wl.sm_scale)
        pool, batch, q = upload_state(b, op, wl.q, True if c["hb"] else None)
        b.ekv_set_option("decode_chunk_tokens", c["chunk"])
        b.ekv_set_option("decode_variant", c["v"])
        try:
            got = gpu_decode(b, pool, batch, q, wl.num_q_heads, wl.sm_scale)
            got32 = gpu_decode(b, pool, batch, q, wl.num_q_heads, wl.sm_scale, f32=True)
        finally:
            b.ekv_set_option("decode_chunk_tokens", 0)
            b.ekv_set_option("decode_variant", 0)
    else:
        wl = synth.make_workload("fz", chunk_lens=c["chunks"], **kw)
        op, *_ = mixed_oracle_pool(oracle, wl)
        exp = oracle.attn_prefill_chunk(op, 0, wl.q_start, wl.q, wl.num_q_heads, wl.sm_scale)
        pool, batch, q = upload_state(b, op, wl.q)
        b.ekv_set_option("prefill_variant", c["v"])
        try:
            got = gpu_prefill(b, pool, batch, q, wl, with_workspace=c["ws"])
            got32 = gpu_prefill(b, pool, batch, q, wl, with_workspace=c["ws"], f32=True)
        finally:
            b.ekv_set_option("prefill_variant", 0)
    pre = assert_attn_close_f32(got32, exp, "fp32 result, " + what)
    err, rel = assert_attn_close(got, exp, what, elem_type=c["et"])
    return err, rel, pre


@pytest.mark.parametrize("group", range(DECODE_GROUPS))
def test_fuzz_decode(oracle, group):
    b = require_gpu()
    rs = np.random.default_rng(7_100 + group)
    for _ in range(CASES_PER_GROUP):
        run_case(b, oracle, draw_case(rs, "decode"))


@pytest.mark.parametrize("group", range(PREFILL_GROUPS))
def test_fuzz_prefill(oracle, group):
    b = require_gpu()
    rs = np.random.default_rng(9_200 + group)
    for _ in range(CASES_PER_GROUP):
        run_case(b, oracle, draw_case(rs, "prefill"))


RECORDED = [
    dict(kind="prefill", D=128, G=8, H=2, et="bf16", f=0.3, pat="middle", seed=210266793,
         lens=[63, 245, 17, 581], chunks=[63, 55, 7, 302], v=0, ws=True),
    dict(kind="prefill", D=64, G=1, H=3, et="bf16", f=0.0, pat="oldest", seed=51312497,
         lens=[2347, 17, 1282, 1477, 129], chunks=[2347, 7, 711, 1477, 27], v=0, ws=False),
    dict(kind="prefill", D=64, G=8, H=3, et="bf16", f=0.0, pat="oldest", seed=266995072,
         lens=[144, 257], chunks=[128, 103], v=1, ws=True),
]


@pytest.mark.parametrize("case", RECORDED, ids=lambda c: f"seed{c['seed']}")
def test_recorded_prefill_offenders(oracle, case):
    """Cases an earlier run found between 1.0e-2 and 1.55e-2 (probabilities rounded to bf16 on rows
    that a few tokens dominate)."""
    b = require_gpu()
    run_case(b, oracle, case)


def test_one_term_options_stay_close_to_the_default(oracle):
    """The measurement options that switch the second probability term off (decode_two_term = 1,
    prefill_p_terms = 1) or force it on (2) change results only at the level the second term is
    there to remove: within 6e-3 of the oracle before the output rounding (one term), within the
    pre-rounding bound (two terms)."""
    b = require_gpu()
    rs = np.random.default_rng(31)
    for kind, opt, one, two in (("decode", "decode_two_term", 1, 2), ("prefill", "prefill_p_terms", 1, 2)):
        for _ in range(12):
            c = draw_case(rs, kind)
            c["et"], c["v"] = "bf16", 0
            kw = dict(seed=c["seed"], seq_lens=c["lens"], num_q_heads=c["G"] * c["H"], num_kv_heads=c["H"], head_dim=c["D"],
                      base_fraction=c["f"], base_pattern=c["pat"], elem_type="bf16")
            if kind == "decode":
                wl = synth.make_workload("fz", **kw)
                op, *_ = mixed_oracle_pool(oracle, wl)
                exp = oracle.attn_decode(op, 0, wl.q, wl.num_q_heads, wl.sm_scale)
                pool, batch, q = upload_state(b, op, wl.q)
                run = lambda: gpu_decode(b, pool, batch, q, wl.num_q_heads, wl.sm_scale, f32=True)
            else:
                wl = synth.make_workload("fz", chunk_lens=c["chunks"], **kw)
                op, *_ = mixed_oracle_pool(oracle, wl)
                exp = oracle.attn_prefill_chunk(op, 0, wl.q_start, wl.q, wl.num_q_heads, wl.sm_scale)
                pool, batch, q = upload_state(b, op, wl.q)
                run = lambda: gpu_prefill(b, pool, batch, q, wl, f32=True)
            try:
                b.ekv_set_option(opt, one)
                got1 = run()
                b.ekv_set_option(opt, two)
                got2 = run()
            finally:
                b.ekv_set_option(opt, 0)
            assert np.abs(got1 - exp).max() <= 6e-3 * max(1.0, np.abs(exp).max() / 4), (kind, c)
            assert_attn_close_f32(got2, exp, f"{opt} = {two}: {c}")
