#!/usr/bin/env python
"""Benchmark of the mixed-fidelity paged attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extras]

One step = one pass of the whole hot path over one batch of the Llama-3-8B-shaped decode
workload (batch 64, contexts U[1024, 8192], 32/8 heads, head_dim 128, page 16, 50 % of the
eligible pairs in BASE, random physical placement):
    ekv_downgrade (16 TARGET pairs, residual kept)  ->  ekv_attn_decode (mixed fidelity)
    ->  ekv_refine (the same 16 pairs, released blocks handed back)
so the pool is bit-identical at the start of every step. `value` is the bytes the path must
move per step (K/V bytes of the visible tokens at their stored width + the transition bytes)
divided by the device time per step, summed over ranks (independent replicas).

Rank 0 prints ONE JSON line. With --impl reference the same step is run by the CPU oracle on
the host cores (a bounded sample of the requests), rank 0 only.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_33536_b200 import synth  # noqa: E402

METRIC = "decode_attn_kv_GBps"
UNIT = "GB/s"
TRANSITION_PAIRS = 16          # the paper's minimum demotion batch B_min^d (App. B.1)
# dram__bytes_read.sum + dram__bytes_write.sum divided by the algorithmic K/V bytes, from the ncu
# capture summarised in profiles/decode_ring_kernel_llama8b_decode_f05.md
NCU_TRAFFIC_PER_KV_BYTE = 1.0173
WORKLOAD = ("llama3-8b-shaped decode: batch 64, ctx U[1024,8192], Hq 32 / Hkv 8, D 128, page 16, "
            "BASE fraction 0.5 (random pairs), random physical placement; per step: downgrade 16 pairs "
            "-> mixed-fidelity decode attention -> refine 16 pairs")


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy read+write)"
        except Exception:
            pass
    return 6650.0, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled in the background (read-only query)."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc, self.t0, self.t1 = [], None, None, None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100", "-i", str(index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def mark_begin(self):
        self.t0 = time.time()

    def mark_end(self):
        self.t1 = time.time()

    def stop(self):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()
        rows = [r for t, r in self.rows if self.t0 is not None and self.t0 <= t <= (self.t1 or t) + 0.1]
        scope = "timed region"
        if not rows:
            rows, scope = [r for _, r in self.rows], "whole run (timed region shorter than the sampling period)"
        sm, mx, reasons = [], [], set()
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "scope": scope}


def _dist():
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return world, rank, local


def aggregate_over_ranks(ms: float, step_bytes: float, device=None):
    """Replicas only: the job's time is the slowest rank's device time, its work the sum of what
    all ranks moved. Works on any initialised process group (NCCL on GPUs, gloo on CPU)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms, step_bytes
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    b = torch.tensor([float(step_bytes)], dtype=torch.float64, device=device)
    dist.all_reduce(b, op=dist.ReduceOp.SUM)
    return float(t.item()), float(b.item())


def transition_bytes(wl, n_pairs, with_resid=True):
    """Downgrade: read 2 blocks, write 1 packed block (+1 block of low bytes) per tensor per layer.
    Refine: read packed + residual, write 2 blocks."""
    bb = wl.block_words * 2
    down = n_pairs * wl.num_layers * 2 * (2 * bb + bb + (bb if with_resid else 0))
    up = n_pairs * wl.num_layers * 2 * (bb + bb + 2 * bb)
    return down, up


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------

def run_ours(args):
    import torch
    from paper_2609_33536_b200 import binding as b

    world, rank, local = _dist()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    b.load()
    dev = torch.device("cuda", local)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)

    sampler = ClockSampler(local) if rank == 0 else None
    seed = synth.BASE_SEED + 2 + 1000 * rank            # replicas: same shape, rank-specific draw
    wl = synth.cfg_llama8b_decode(seed=seed, base_fraction=0.5, batch=args.batch)
    pool, batch, q = b.upload(wl, dev)
    nb = len(wl.base_pair_req)
    freed0 = torch.empty(nb, dtype=torch.int32, device=dev)
    b.ekv_downgrade(pool, batch, i32(wl.base_pair_req), i32(wl.base_pair_idx), None, None, None, freed0)
    batch.has_base = True

    # the per-step transition batch: 16 pairs that are TARGET in the resident state
    is_base = set(zip(wl.base_pair_req.tolist(), wl.base_pair_idx.tolist()))
    cand = [(r, p) for r in range(wl.batch) for p in range(wl.eligible_pairs(r)) if (r, p) not in is_base]
    sel = synth.rng(seed, 7).permutation(len(cand))[:TRANSITION_PAIRS]
    tp_req = np.array([cand[i][0] for i in sel], np.int32)
    tp_idx = np.array([cand[i][1] for i in sel], np.int32)
    n_tp = len(tp_req)
    d_req, d_idx, d_slot = i32(tp_req), i32(tp_idx), i32(np.arange(n_tp))
    kres, vres = pool.new_resid(n_tp), pool.new_resid(n_tp)
    freed = torch.empty(n_tp, dtype=torch.int32, device=dev)
    msl = int(wl.seq_lens.max())
    ws = b.new_workspace(pool, wl.batch, wl.num_q_heads, msl)
    out = torch.empty_like(q)

    kv_bytes = wl.kv_bytes() - n_tp * 2 * wl.page_size * wl.num_kv_heads * 2 * wl.head_dim   # 16 more pairs are BASE in-step
    down_b, up_b = transition_bytes(wl, n_tp)
    step_bytes = kv_bytes + down_b + up_b

    def step():
        b.ekv_downgrade(pool, batch, d_req, d_idx, kres, vres, d_slot, freed)
        b.ekv_attn_decode(pool, 0, batch, q, out, wl.num_q_heads, wl.sm_scale, msl, ws)
        b.ekv_refine(pool, batch, d_req, d_idx, freed, kres, vres, d_slot)

    k0 = pool.k_pool.clone()
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()

    # ---- timed region: K steps, device time by CUDA events on the launching stream ----
    K = args.steps
    # The decode split kernel is timed inside the timed region, in a spread-out subset of the steps: the two
    # event records around it keep its launch from overlapping the neighbouring kernels' tails, which slows
    # such a step by a few per cent, so only about one step in eight carries them.
    n_prof = min(64, max(1, (K + 7) // 8))
    prof_every = max(1, K // n_prof)
    prof = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_prof)]
    for e0, e1 in prof:
        e0.record(); e1.record()                           # create the handles
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.mark_begin()
    ev0.record()
    for i in range(K):
        if i % prof_every == 0 and i // prof_every < n_prof:
            b.ekv_downgrade(pool, batch, d_req, d_idx, kres, vres, d_slot, freed)
            b.ekv_set_profile_events(*prof[i // prof_every])
            b.ekv_attn_decode(pool, 0, batch, q, out, wl.num_q_heads, wl.sm_scale, msl, ws)
            b.ekv_set_profile_events(None, None)
            b.ekv_refine(pool, batch, d_req, d_idx, freed, kres, vres, d_slot)
        else:
            step()
    ev1.record()
    torch.cuda.synchronize()
    if sampler:
        sampler.mark_end()
    ms = ev0.elapsed_time(ev1)
    ms, total_bytes = aggregate_over_ranks(ms, float(step_bytes), dev)
    if world > 1:
        dist.barrier()
    ms_per_step = ms / K
    value = total_bytes / (ms_per_step * 1e-3) / 1e9
    main_ms = float(np.mean([e0.elapsed_time(e1) for e0, e1 in prof]))

    result = None
    # every rank from here on: the end-to-end leg is measured on all of them
    assert torch.equal(pool.k_pool, k0), "pool state drifted across steps"
    clocks = sampler.stop() if sampler else None
    peak, peak_src = _peaks()
    achieved = kv_bytes / (main_ms * 1e-3) / 1e9
    result = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD if args.batch == 64 else WORKLOAD.replace("batch 64", f"batch {args.batch}"), "seed": seed, "l2": "inputs larger than L2 (0.9 GB of KV per step vs 126 MB)",
                   "tokens": int(wl.seq_lens.sum()), "realised_base_fraction": round(wl.realised_base_fraction(), 4),
                   "bytes_per_step": int(step_bytes), "kv_bytes_per_step": int(kv_bytes),
                   "multi_gpu": "replicas only (no exchange step on this path)"},
        "clocks": clocks,
        "gpu_launches": 4 * K,          # per step: downgrade pack, decode split, decode merge, refine expand
        "roofline": {"bound": "hbm", "kernel": "decode_ring_kernel<128,true> (split kernel of ekv_attn_decode)",
                     "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s", "frac": round(achieved / peak, 4),
                     "frac_of_8000_nominal": round(achieved / 8000.0, 4), "peak_source": peak_src,
                     "us_per_launch": round(main_ms * 1e3, 2), "launches_timed": n_prof,
                     "traffic": round(kv_bytes * NCU_TRAFFIC_PER_KV_BYTE) if NCU_TRAFFIC_PER_KV_BYTE else None,
                     "traffic_note": "dram read+write bytes of one ncu capture of this kernel on a smaller batch "
                                     "of the same workload, scaled by the K/V bytes of a full launch"},
        "tokens_per_s": round(wl.batch / (ms_per_step * 1e-3), 1),
    }
    if args.profile_only:
        result["config"]["note"] = "profiling run: reduced batch, no e2e / cpu_baseline / extras"
        return result if rank == 0 else None
    # ---- end to end: host buffers, H2D of the step's inputs and D2H of its result, every step ----
    # The step's inputs (queries, block table, sequence lengths, the transition batch) sit in ONE pinned
    # host arena and travel in one copy to a device arena the calls read through views; the result comes
    # back into pinned memory. Copy in, the three library calls and copy out are captured once as a CUDA
    # graph on the caller's side (the library allocates nothing and orders everything on the stream it is
    # given, so its calls can be captured as they are) and replayed once per step.
    parts = [("q", wl.q.view(np.int16)), ("bt", batch.block_table.cpu().numpy()), ("sl", wl.seq_lens),
             ("req", tp_req), ("idx", tp_idx), ("slot", np.arange(n_tp, dtype=np.int32))]
    offs, total = {}, 0
    for name, a in parts:
        offs[name] = total
        total += (a.nbytes + 255) // 256 * 256
    arena_h = torch.empty(total, dtype=torch.uint8).pin_memory()
    arena_d = torch.empty(total, dtype=torch.uint8, device=dev)
    for name, a in parts:
        arena_h[offs[name]:offs[name] + a.nbytes].copy_(torch.from_numpy(np.ascontiguousarray(a)).view(torch.uint8).reshape(-1))

    def dview(name, a, dtype):
        return arena_d[offs[name]:offs[name] + a.nbytes].view(dtype).reshape(a.shape)
    q2 = dview("q", wl.q, q.dtype)
    batch2 = b.Batch(dview("bt", wl.block_table, torch.int32), dview("sl", wl.seq_lens, torch.int32), True)
    req2, idx2, slot2 = (dview(n, tp_req, torch.int32) for n in ("req", "idx", "slot"))
    outh = torch.empty(out.shape, dtype=out.dtype).pin_memory()
    h2d, d2h = int(sum(a.nbytes for _, a in parts)), outh.numel() * 2

    def e2e_body():
        arena_d.copy_(arena_h, non_blocking=True)
        b.ekv_downgrade(pool, batch2, req2, idx2, kres, vres, slot2, freed)
        b.ekv_attn_decode(pool, 0, batch2, q2, out, wl.num_q_heads, wl.sm_scale, msl, ws)
        b.ekv_refine(pool, batch2, req2, idx2, freed, kres, vres, slot2)
        outh.copy_(out, non_blocking=True)

    def timed_e2e(fn, n):
        for _ in range(3):
            fn()
        t0 = time.perf_counter()
        for _ in range(n):
            fn()
        return (time.perf_counter() - t0) / n

    def eager_step():
        e2e_body()
        torch.cuda.synchronize()

    Ke = min(K, 500)
    dt_eager = timed_e2e(eager_step, Ke)
    out_eager = outh.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        e2e_body()                                       # warm the side stream before capture
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            e2e_body()
    torch.cuda.synchronize()
    outh.zero_()

    def graph_step():
        graph.replay()
        torch.cuda.synchronize()

    dt = timed_e2e(graph_step, Ke)
    assert torch.equal(outh.view(torch.int16), out_eager.view(torch.int16)), "graph replay and eager step disagree"
    assert torch.equal(pool.k_pool, k0), "pool state drifted across end-to-end steps"
    # every rank measured its own replica: the job's time is the slowest rank's, its work the sum
    dt, e2e_bytes = aggregate_over_ranks(dt * 1e3, float(step_bytes), dev)
    dt *= 1e-3
    dt_eager = aggregate_over_ranks(dt_eager * 1e3, 0.0, dev)[0] * 1e-3
    result["e2e"] = {"value": round(e2e_bytes / dt / 1e9, 1), "unit": UNIT, "h2d_bytes_per_step": h2d * world,
                     "d2h_bytes_per_step": int(d2h) * world, "ms_per_step": round(dt * 1e3, 5), "steps": Ke,
                     "eager_ms_per_step": round(dt_eager * 1e3, 5),
                     "note": "host wall clock, one stream sync per step; per step: one pinned-host -> device copy of the "
                             "inputs, the three library calls, one device -> pinned-host copy of the output, replayed "
                             "as one CUDA graph (eager_ms_per_step: the same sequence issued call by call); the KV pool "
                             "is resident cache state"}
    # Two steps in flight: step i + 1's inputs go up on a copy stream and step i - 1's output comes down on
    # another while step i's kernels run. Every step still uploads its own inputs from pinned memory and has
    # its result read back to pinned memory; only the waiting is overlapped. Reported beside the serial figure.
    arenas = [arena_d, torch.empty_like(arena_d)]
    outs_d = [out, torch.empty_like(out)]
    outs_h = [outh, torch.empty(out.shape, dtype=out.dtype).pin_memory()]
    views = []
    for a in arenas:
        dv = lambda name, arr, dtype, a=a: a[offs[name]:offs[name] + arr.nbytes].view(dtype).reshape(arr.shape)
        views.append((dv("q", wl.q, q.dtype), b.Batch(dv("bt", wl.block_table, torch.int32), dv("sl", wl.seq_lens, torch.int32), True),
                      dv("req", tp_req, torch.int32), dv("idx", tp_idx, torch.int32), dv("slot", tp_req, torch.int32)))
    s_in, s_out, s_main = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_done = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def pipelined(n):
        for i in range(n):
            par = i & 1
            if i >= 2:
                ev_out[par].synchronize()              # the host has step i - 2's result; its buffers are free again
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_done[par])          # step i - 2 no longer reads this arena
                arenas[par].copy_(arena_h, non_blocking=True)
                ev_in[par].record()
            s_main.wait_event(ev_in[par])
            s_main.wait_event(ev_out[par])             # step i - 2's output has left outs_d[par]
            q_v, batch_v, req_v, idx_v, slot_v = views[par]
            b.ekv_downgrade(pool, batch_v, req_v, idx_v, kres, vres, slot_v, freed)
            b.ekv_attn_decode(pool, 0, batch_v, q_v, outs_d[par], wl.num_q_heads, wl.sm_scale, msl, ws)
            b.ekv_refine(pool, batch_v, req_v, idx_v, freed, kres, vres, slot_v)
            ev_done[par].record()
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[par])
                outs_h[par].copy_(outs_d[par], non_blocking=True)
                ev_out[par].record()
        torch.cuda.synchronize()

    pipelined(8)
    t0 = time.perf_counter()
    pipelined(Ke)
    dt_p = (time.perf_counter() - t0) / Ke
    assert torch.equal(outs_h[0].view(torch.int16), out_eager.view(torch.int16)), "pipelined step and eager step disagree"
    assert torch.equal(outs_h[1].view(torch.int16), out_eager.view(torch.int16)), "pipelined step and eager step disagree"
    assert torch.equal(pool.k_pool, k0), "pool state drifted across pipelined steps"
    dt_p, p_bytes = aggregate_over_ranks(dt_p * 1e3, float(step_bytes), dev)
    dt_p *= 1e-3
    result["e2e"]["two_steps_in_flight"] = {
        "value": round(p_bytes / dt_p / 1e9, 1), "ms_per_step": round(dt_p * 1e3, 5), "steps": Ke,
        "note": "same copies every step, on copy streams: step i + 1's upload and step i - 1's read-back overlap step i's "
                "kernels; the host waits for a step's result two steps later"}
    if rank == 0 and world == 1:                       # the oracle on the host cores: rank 0 at N = 1 only
        result["cpu_baseline"] = cpu_baseline(wl, tp_req, tp_idx, outs_d[0].to(torch.float64).cpu().numpy(), budget_s=20.0)
    if rank == 0 and world == 1 and not args.no_extras:
        result["extras"] = extras(b, torch, dev, args)
        result["roofline"]["others"] = roofline_others(result["extras"], peak)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return result if rank == 0 else None


def cpu_baseline(wl, tp_req, tp_idx, gpu_out, budget_s):
    """The oracle as it stands on this machine's host cores: the same step (downgrade 16 pairs, mixed
    decode attention, refine) on a bounded sample of the requests. Also reports GPU-vs-oracle
    parity on the sampled rows, since the oracle's output is at hand."""
    import oracle
    tags = np.zeros(wl.num_blocks, dtype=np.uint8)
    op = oracle.OraclePool(wl.k_pool, wl.v_pool, tags, wl.block_table, wl.seq_lens,
                           num_kv_heads=wl.num_kv_heads, head_dim=wl.head_dim)
    oracle.downgrade(op, wl.base_pair_req, wl.base_pair_idx)
    n_tp = len(tp_req)
    kres, vres = op.new_resid(n_tp), op.new_resid(n_tp)
    slots = np.arange(n_tp, dtype=np.int32)
    # calibrate on one request, then size the sample to the budget
    t0 = time.perf_counter()
    oracle.attend_rows(op, 0, [0] * wl.num_q_heads, list(range(wl.num_q_heads)), [int(wl.seq_lens[0])] * wl.num_q_heads,
                       wl.q[0], wl.num_q_heads, wl.sm_scale)
    per_tok = (time.perf_counter() - t0) / max(1, int(wl.seq_lens[0]))
    n_req, tok = 0, 0
    while n_req < wl.batch and (tok + int(wl.seq_lens[n_req])) * per_tok <= budget_s:
        tok += int(wl.seq_lens[n_req]); n_req += 1
    n_req = max(1, n_req)
    rows_r = np.repeat(np.arange(n_req, dtype=np.int32), wl.num_q_heads)
    rows_h = np.tile(np.arange(wl.num_q_heads, dtype=np.int32), n_req)
    rows_n = wl.seq_lens[rows_r]
    t0 = time.perf_counter()
    freed = oracle.downgrade(op, tp_req, tp_idx, kres, vres, slots)
    exp = oracle.attend_rows(op, 0, rows_r, rows_h, rows_n, wl.q[:n_req].reshape(-1, wl.head_dim), wl.num_q_heads, wl.sm_scale)
    oracle.refine(op, tp_req, tp_idx, freed, kres, vres, slots)
    dt = time.perf_counter() - t0
    sel = np.isin(tp_req, np.arange(n_req))
    per_tok_t = wl.num_kv_heads * 2 * wl.head_dim * 2
    base_tok = sum(2 * wl.page_size for r in wl.base_pair_req if r < n_req) + int(sel.sum()) * 2 * wl.page_size
    kvb = int(wl.seq_lens[:n_req].sum()) * per_tok_t - base_tok * (per_tok_t // 2)
    down_b, up_b = transition_bytes(wl, n_tp)
    got = gpu_out[:n_req].reshape(-1, wl.head_dim)
    err = float(np.max(np.abs(got - exp)))
    rel = float(np.linalg.norm(got - exp) / np.linalg.norm(exp))
    return {"value": round((kvb + down_b + up_b) / dt / 1e9, 4), "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": f"first {n_req} of {wl.batch} requests ({int(wl.seq_lens[:n_req].sum())} tokens, all {wl.num_q_heads} heads) "
                      f"+ the 16-pair downgrade/refine, one pass, {dt:.2f} s",
            "parity_vs_gpu": {"rows": int(len(rows_r)), "max_abs": err, "rel_l2": rel,
                              "pass": bool(err <= 1e-2 and rel <= 5e-3)}}



class L2Flush:
    """Flush L2 before a timed launch: write a 256 MB buffer (twice the 126 MB L2), then read a second
    256 MB buffer, so that the written lines are back in DRAM before the timed launch starts and it
    meets a cold L2 with nothing of its own in it and no write-backs owed."""

    def __init__(self, torch, dev):
        self.w = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        self.r = torch.zeros(64 << 20, dtype=torch.int32, device=dev)
        self.sink = torch.zeros(1, dtype=torch.int64, device=dev)

    def __call__(self):
        self.w.zero_()
        self.sink.copy_(self.r.sum())



def pressure_step_loop(b, torch, dev, i32, flush, steady_steps=6):
    """High-concurrency configuration as a loop of steps on one stream: demote every TARGET pair among
    the oldest 40 % of blocks of a seeded 60 % of requests -> decode attention -> refine a seeded 10 %
    of the BASE pairs (into the blocks the demotion just released). Step 0 demotes all of them (cold);
    a steady-state step demotes what the step before refined. Each phase is timed by CUDA events."""
    wl = synth.cfg_pressure()
    pool, batch, q = b.upload(wl, dev)
    batch.has_base = True
    n_all = len(wl.base_pair_req)
    n_pick = max(1, n_all // 10)
    kres, vres = pool.new_resid(n_all), pool.new_resid(n_all)
    msl = int(wl.seq_lens.max())
    ws = b.new_workspace(pool, wl.batch, wl.num_q_heads, msl)
    out = torch.empty_like(q)
    rs = synth.rng(wl.seed, 11)
    slots_all = np.arange(n_all, dtype=np.int32)           # pair i of the list keeps residual slot i
    picks = [np.sort(rs.permutation(n_all)[:n_pick]) for _ in range(steady_steps + 1)]
    kvb = wl.kv_bytes()
    rows = []
    todo = np.arange(n_all)
    for step in range(steady_steps + 1):
        pick = picks[step]
        d_req, d_idx, d_slot = i32(wl.base_pair_req[todo]), i32(wl.base_pair_idx[todo]), i32(slots_all[todo])
        r_req, r_idx, r_slot = i32(wl.base_pair_req[pick]), i32(wl.base_pair_idx[pick]), i32(slots_all[pick])
        freed = torch.empty(len(todo), dtype=torch.int32, device=dev)
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        flush()
        e[0].record(); b.ekv_downgrade(pool, batch, d_req, d_idx, kres, vres, d_slot, freed)
        e[1].record(); b.ekv_attn_decode(pool, 0, batch, q, out, wl.num_q_heads, wl.sm_scale, msl, ws)
        e[2].record(); b.ekv_refine(pool, batch, r_req, r_idx, freed[:len(pick)], kres, vres, r_slot)
        e[3].record(); torch.cuda.synchronize()
        down_b, _ = transition_bytes(wl, len(todo))
        _, up_b = transition_bytes(wl, len(pick))
        t = [e[i].elapsed_time(e[i + 1]) for i in range(3)]
        rows.append({"downgrade_pairs": int(len(todo)), "downgrade_us": t[0] * 1e3, "downgrade_GBps": down_b / t[0] / 1e6,
                     "decode_us": t[1] * 1e3, "decode_GBps": kvb / t[1] / 1e6,
                     "refine_pairs": int(len(pick)), "refine_us": t[2] * 1e3, "refine_GBps": up_b / t[2] / 1e6,
                     "step_us": sum(t) * 1e3})
        todo = pick                                        # the next step demotes these again
    med = lambda k: float(np.median([r[k] for r in rows[1:]]))
    rnd = lambda d: {k: (round(v, 1) if isinstance(v, float) else v) for k, v in d.items()}
    steady = {k: (rows[1][k] if k.endswith("_pairs") else med(k)) for k in rows[0]}
    del pool, batch, q, ws, out, kres, vres
    torch.cuda.empty_cache()
    return {"workload": "batch 256, lognormal contexts (median 2048, clipped to [128, 16384]), 32/8 heads, D 128, 1 layer; "
                        "L2 flushed before each step",
            "tokens": int(wl.seq_lens.sum()), "step0": rnd(rows[0]), "steady_state_median": rnd(steady)}


def transitions_multi_layer(b, torch, dev, i32, flush, num_layers):
    """Downgrade / refine GB/s when a transition covers several layers (one tag per block for all layers)."""
    wl = synth.cfg_llama8b_decode(base_fraction=0.0, batch=16, num_layers=num_layers)
    pool, batch, q = b.upload(wl, dev)
    pr = np.concatenate([np.full(wl.eligible_pairs(r), r, np.int32) for r in range(wl.batch)])
    pi = np.concatenate([np.arange(wl.eligible_pairs(r), dtype=np.int32) for r in range(wl.batch)])
    n = len(pr)
    kres, vres = pool.new_resid(n), pool.new_resid(n)
    fr = torch.empty(n, dtype=torch.int32, device=dev)
    dpr, dpi, dsl = i32(pr), i32(pi), i32(np.arange(n))
    down_b, up_b = transition_bytes(wl, n)
    e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    td, tu = [], []
    for _ in range(6):
        flush()
        e[0].record(); b.ekv_downgrade(pool, batch, dpr, dpi, kres, vres, dsl, fr)
        e[1].record(); b.ekv_refine(pool, batch, dpr, dpi, fr, kres, vres, dsl)
        e[2].record(); torch.cuda.synchronize()
        td.append(e[0].elapsed_time(e[1])); tu.append(e[1].elapsed_time(e[2]))
    del pool, batch, q, kres, vres
    torch.cuda.empty_cache()
    return {"layers": num_layers, "pairs": n,
            "downgrade": {"us": round(float(np.median(td)) * 1e3, 1), "GBps": round(down_b / np.median(td) / 1e6, 1)},
            "refine": {"us": round(float(np.median(tu)) * 1e3, 1), "GBps": round(up_b / np.median(tu) / 1e6, 1)}}

def metadata_lowering(b, torch, dev, batch=256):
    """Worker-side metadata lowering for one step of the high-concurrency configuration: the scheduler's
    sparse description (lengths, block lists, BASE pair ranges of all 256 requests) goes up in ONE pinned
    host-to-device copy and ekv_lower_sparse_metadata writes table rows, lengths, boundaries and flags in
    one launch; beside it, the same update done request by request with torch copies (one table-row copy
    and one length write per request). Host wall clock per step, device synchronised at the end."""
    wl = synth.cfg_pressure()
    pool, bt, q = b.upload(wl, dev)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    fr = torch.empty(len(wl.base_pair_req), dtype=torch.int32, device=dev)
    b.ekv_downgrade(pool, bt, i32(wl.base_pair_req), i32(wl.base_pair_idx), None, None, None, fr)
    torch.cuda.synchronize()
    table = bt.block_table.cpu().numpy()
    tags = pool.tags.cpu().numpy()
    lists, ranges = [], []
    for r in range(wl.batch):
        nb = -(-int(wl.seq_lens[r]) // wl.page_size)
        ids = table[r, :nb]
        lists.append(ids)
        base = tags[ids[0::2]] == 1
        rr, start = [], None
        for pidx, flag in enumerate(list(base) + [False]):
            if flag and start is None:
                start = pidx
            if not flag and start is not None:
                rr += [start, pidx]; start = None
        ranges.append(rr)
    parts = [np.arange(wl.batch, dtype=np.int32), wl.seq_lens.astype(np.int32),
             np.concatenate([[0], np.cumsum([len(x) for x in lists])]).astype(np.int32), np.concatenate(lists).astype(np.int32),
             np.concatenate([[0], np.cumsum([len(x) // 2 for x in ranges])]).astype(np.int32),
             np.array([v for x in ranges for v in x], np.int32)]
    offs = np.concatenate([[0], np.cumsum([len(x) for x in parts])])
    arena_h = torch.from_numpy(np.concatenate(parts).astype(np.int32)).pin_memory()
    arena_d = torch.empty_like(arena_h, device=dev)
    v = [arena_d[offs[k]:offs[k + 1]] for k in range(6)]
    out_table = torch.full_like(bt.block_table, -1)
    out_sl = torch.zeros_like(bt.seq_lens)
    out_batch = b.Batch(out_table, out_sl, True)
    bounds = torch.zeros((wl.batch, 2), dtype=torch.int32, device=dev)
    flags = torch.zeros(4, dtype=torch.int32, device=dev)

    def lowered():
        arena_d.copy_(arena_h, non_blocking=True)
        b.ekv_lower_sparse_metadata(pool, out_batch, out_sl, v[0], v[1], v[2], v[3], v[4], v[5] if len(v[5]) else None, bounds, flags)
        torch.cuda.synchronize()

    host_rows = [torch.from_numpy(np.ascontiguousarray(x)).pin_memory() for x in lists]
    lens_h = wl.seq_lens.tolist()

    def per_request():
        for r in range(wl.batch):
            out_table[r, : len(lists[r])].copy_(host_rows[r], non_blocking=True)
            out_sl[r] = lens_h[r]
        torch.cuda.synchronize()

    def wall(fn, n=20):
        for _ in range(3):
            fn()
        t0 = time.perf_counter()
        for _ in range(n):
            fn()
        return (time.perf_counter() - t0) / n
    t_low = wall(lowered)
    assert torch.equal(out_table[:, :1], bt.block_table[:, :1]) and flags.cpu().tolist()[2] == 0
    t_py = wall(per_request, n=5)
    return {"workload": f"batch {wl.batch} of the high-concurrency configuration, {int(offs[-1]) * 4} bytes of sparse description",
            "lowered_us_per_step": round(t_low * 1e6, 1),
            "per_request_copies_us_per_step": round(t_py * 1e6, 1), "flags": flags.cpu().tolist(),
            "note": "host wall clock per step, device synchronised: one pinned copy + one launch, against one table-row copy "
                    "and one length write per request"}


def extras(b, torch, dev, args):
    """Context numbers (not part of the timed step): decode GB/s over the BASE-fraction sweep,
    the native / elastic-idle comparison on the all-TARGET pool, and transition GB/s."""
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    res = {"decode_sweep": {}, "note": "median of 20 launches of ekv_attn_decode (split + merge) timed from outside, "
                                       "L2 flushed between launches (256 MB written, then 256 MB read so no write-backs are owed); split_kernel_* = the split "
                                       "kernel alone, timed by the library's profile events around that one launch"}
    flush = L2Flush(torch, dev)

    def timed(fn, iters=20, warm=5):
        ts = []
        for i in range(warm + iters):
            flush()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record(); torch.cuda.synchronize()
            if i >= warm:
                ts.append(e0.elapsed_time(e1))
        return float(np.median(ts))

    for f in (0.0, 0.25, 0.5, 1.0):
        wl = synth.cfg_llama8b_decode(base_fraction=f)
        pool, batch, q = b.upload(wl, dev)
        n = len(wl.base_pair_req)
        if n:
            fr = torch.empty(n, dtype=torch.int32, device=dev)
            b.ekv_downgrade(pool, batch, i32(wl.base_pair_req), i32(wl.base_pair_idx), None, None, None, fr)
        msl = int(wl.seq_lens.max())
        ws = b.new_workspace(pool, wl.batch, wl.num_q_heads, msl)
        out = torch.empty_like(q)
        kvb = wl.kv_bytes()
        modes = [("native", False, 0), ("plain_comparator", False, 1), ("elastic_idle", True, 0)] if f == 0.0 \
            else [("elastic", True, 0)]
        for name, hb, variant in modes:
            batch.has_base = hb
            b.ekv_set_option("decode_variant", variant)     # 1 = the page-stepped plain paged-decode kernel
            ms = timed(lambda: b.ekv_attn_decode(pool, 0, batch, q, out, wl.num_q_heads, wl.sm_scale, msl, ws))
            # the split kernel alone (the library records the two events around that one launch), L2 flushed
            pe0, pe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            pe0.record(); pe1.record(); torch.cuda.synchronize()
            ks = []
            for _ in range(12):
                flush()
                b.ekv_set_profile_events(pe0, pe1)
                b.ekv_attn_decode(pool, 0, batch, q, out, wl.num_q_heads, wl.sm_scale, msl, ws)
                b.ekv_set_profile_events(None, None)
                torch.cuda.synchronize()
                ks.append(pe0.elapsed_time(pe1))
            kms = float(np.median(ks[2:]))
            b.ekv_set_option("decode_variant", 0)
            res["decode_sweep"][f"f={f}:{name}"] = {"us": round(ms * 1e3, 1), "GBps": round(kvb / ms / 1e6, 1),
                                                    "frac_of_8000": round(kvb / ms / 1e6 / 8000, 4),
                                                    "tokens_per_s": round(wl.batch / ms * 1e3, 1),
                                                    "split_kernel_us": round(kms * 1e3, 1),
                                                    "split_kernel_GBps": round(kvb / kms / 1e6, 1),
                                                    "split_kernel_frac_of_8000": round(kvb / kms / 1e6 / 8000, 4)}
        if f == 0.0:
            # transitions on a large batch of pairs (every eligible pair of the first 32 requests)
            pr = np.concatenate([np.full(wl.eligible_pairs(r), r, np.int32) for r in range(32)])
            pi = np.concatenate([np.arange(wl.eligible_pairs(r), dtype=np.int32) for r in range(32)])
            n = len(pr)
            kres, vres = pool.new_resid(n), pool.new_resid(n)
            fr = torch.empty(n, dtype=torch.int32, device=dev)
            dpr, dpi, dsl = i32(pr), i32(pi), i32(np.arange(n))
            down_b, up_b = transition_bytes(wl, n)
            e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            td, tu = [], []
            for _ in range(6):
                flush()
                e[0].record(); b.ekv_downgrade(pool, batch, dpr, dpi, kres, vres, dsl, fr)
                e[1].record(); b.ekv_refine(pool, batch, dpr, dpi, fr, kres, vres, dsl)
                e[2].record(); torch.cuda.synchronize()
                td.append(e[0].elapsed_time(e[1])); tu.append(e[1].elapsed_time(e[2]))
            res["downgrade"] = {"pairs": n, "us": round(float(np.median(td)) * 1e3, 1), "GBps": round(down_b / np.median(td) / 1e6, 1)}
            res["refine"] = {"pairs": n, "us": round(float(np.median(tu)) * 1e3, 1), "GBps": round(up_b / np.median(tu) / 1e6, 1)}
        del pool, batch, q, ws, out
        torch.cuda.empty_cache()
    # structured (T-B-T boundaries) vs general (per-block tags) elastic path on a regular layout
    wl = synth.make_workload("llama8b_decode_tbt", seed=synth.BASE_SEED + 2,
                             seq_lens=synth.draw_lengths(synth.BASE_SEED + 2, 64, "uniform", lo=1024, hi=8192),
                             num_q_heads=32, num_kv_heads=8, head_dim=128, base_fraction=0.5, base_pattern="middle")
    pool, batch, q = b.upload(wl, dev)
    fr = torch.empty(len(wl.base_pair_req), dtype=torch.int32, device=dev)
    b.ekv_downgrade(pool, batch, i32(wl.base_pair_req), i32(wl.base_pair_idx), None, None, None, fr)
    batch.has_base = True
    bounds = torch.zeros((wl.batch, 2), dtype=torch.int32, device=dev)
    flags = torch.zeros(2, dtype=torch.int32, device=dev)
    b.ekv_lower_metadata(pool, batch, bounds, flags)
    msl = int(wl.seq_lens.max())
    ws = b.new_workspace(pool, wl.batch, wl.num_q_heads, msl)
    out = torch.empty_like(q)
    kvb = wl.kv_bytes()
    ms_g = timed(lambda: b.ekv_attn_decode(pool, 0, batch, q, out, wl.num_q_heads, wl.sm_scale, msl, ws))
    ms_s = timed(lambda: b.ekv_attn_decode_structured(pool, 0, batch, bounds, q, out, wl.num_q_heads, wl.sm_scale, msl, ws))
    res["structured_vs_general"] = {"workload": "same shape, BASE pairs as one middle run per sequence (T-B-T), f=0.5",
                                    "flags": flags.cpu().tolist(),
                                    "general": {"us": round(ms_g * 1e3, 1), "GBps": round(kvb / ms_g / 1e6, 1)},
                                    "structured": {"us": round(ms_s * 1e3, 1), "GBps": round(kvb / ms_s / 1e6, 1)}}
    del pool, batch, q, ws, out
    torch.cuda.empty_cache()
    # the other two decode configurations (long context with GQA 8:1 and runs of BASE blocks; high concurrency)
    res["other_decode_configs"] = {}
    for cname, mk in (("long70b_ctx32768_batch16", lambda: synth.cfg_long70b()), ("pressure_batch256", lambda: synth.cfg_pressure())):
        wl = mk()
        pool, batch, q = b.upload(wl, dev)
        n = len(wl.base_pair_req)
        if n:
            fr = torch.empty(n, dtype=torch.int32, device=dev)
            b.ekv_downgrade(pool, batch, i32(wl.base_pair_req), i32(wl.base_pair_idx), None, None, None, fr)
            batch.has_base = True
        msl = int(wl.seq_lens.max())
        ws = b.new_workspace(pool, wl.batch, wl.num_q_heads, msl)
        out = torch.empty_like(q)
        ms = timed(lambda: b.ekv_attn_decode(pool, 0, batch, q, out, wl.num_q_heads, wl.sm_scale, msl, ws), iters=10, warm=3)
        res["other_decode_configs"][cname] = {"tokens": int(wl.seq_lens.sum()), "realised_base_fraction": round(wl.realised_base_fraction(), 3),
                                              "us": round(ms * 1e3, 1), "GBps": round(wl.kv_bytes() / ms / 1e6, 1),
                                              "frac_of_8000": round(wl.kv_bytes() / ms / 1e6 / 8000, 4)}
        del pool, batch, q, ws, out
        torch.cuda.empty_cache()
    # batch x context sweep (fixed lengths, f = 0.5, 32/8 heads, D 128): latency, bandwidth and tokens per second
    res["batch_ctx_sweep"] = {}
    for nb_, ctx in ((1, 8192), (8, 8192), (64, 8192), (256, 2048), (4, 32768), (1, 131072)):
        wl = synth.make_workload(f"sweep_b{nb_}_c{ctx}", seed=synth.BASE_SEED + 60 + nb_, seq_lens=[ctx] * nb_, num_q_heads=32,
                                 num_kv_heads=8, head_dim=128, base_fraction=0.5)
        pool, batch, q = b.upload(wl, dev)
        fr = torch.empty(len(wl.base_pair_req), dtype=torch.int32, device=dev)
        b.ekv_downgrade(pool, batch, i32(wl.base_pair_req), i32(wl.base_pair_idx), None, None, None, fr)
        batch.has_base = True
        ws = b.new_workspace(pool, wl.batch, wl.num_q_heads, ctx)
        out = torch.empty_like(q)
        ms = timed(lambda: b.ekv_attn_decode(pool, 0, batch, q, out, wl.num_q_heads, wl.sm_scale, ctx, ws), iters=12, warm=3)
        res["batch_ctx_sweep"][f"batch{nb_}_ctx{ctx}"] = {"us": round(ms * 1e3, 1), "GBps": round(wl.kv_bytes() / ms / 1e6, 1),
                                                         "frac_of_8000": round(wl.kv_bytes() / ms / 1e6 / 8000, 4),
                                                         "tokens_per_s": round(nb_ / ms * 1e3, 1)}
        del pool, batch, q, ws, out, fr
        torch.cuda.empty_cache()
    res["pressure_step_loop"] = pressure_step_loop(b, torch, dev, i32, flush)
    res["transitions_4_layers"] = transitions_multi_layer(b, torch, dev, i32, flush, num_layers=4)
    # the fp16 element type (BASE byte = E5M2): decode at f = 0.5 and the prefill configuration
    wl = synth.cfg_llama8b_decode(base_fraction=0.5, elem_type="fp16")
    pool, batch, q = b.upload(wl, dev)
    fr = torch.empty(len(wl.base_pair_req), dtype=torch.int32, device=dev)
    b.ekv_downgrade(pool, batch, i32(wl.base_pair_req), i32(wl.base_pair_idx), None, None, None, fr)
    batch.has_base = True
    msl = int(wl.seq_lens.max())
    ws = b.new_workspace(pool, wl.batch, wl.num_q_heads, msl)
    out = torch.empty_like(q)
    ms = timed(lambda: b.ekv_attn_decode(pool, 0, batch, q, out, wl.num_q_heads, wl.sm_scale, msl, ws))
    res["fp16_elements"] = {"decode_f=0.5": {"us": round(ms * 1e3, 1), "GBps": round(wl.kv_bytes() / ms / 1e6, 1)}}
    del pool, batch, q, ws, out
    torch.cuda.empty_cache()
    wl = synth.cfg_prefill(elem_type="fp16")
    pool, batch, q = b.upload(wl, dev)
    fr = torch.empty(len(wl.base_pair_req), dtype=torch.int32, device=dev)
    b.ekv_downgrade(pool, batch, i32(wl.base_pair_req), i32(wl.base_pair_idx), None, None, None, fr)
    batch.has_base = True
    qs = torch.from_numpy(wl.q_start).to(dev)
    out = torch.empty_like(q)
    C, L = int(wl.q_start[1]), int(wl.seq_lens[0])
    flops = 4.0 * wl.head_dim * wl.num_q_heads * sum(L - C + i + 1 for i in range(C)) * wl.batch
    pf_ws = b.new_workspace(pool, wl.batch, wl.num_q_heads, L, int(wl.q_start[-1]))
    ms = timed(lambda: b.ekv_attn_prefill_chunk(pool, 0, batch, qs, q, out, wl.num_q_heads, wl.sm_scale,
                                                int(wl.q_start[-1]), C, L, pf_ws), iters=10, warm=3)
    res["fp16_elements"]["prefill_chunk"] = {"ms": round(ms, 4), "TFLOPs": round(flops / ms / 1e9, 1)}
    del pool, batch, q, out, pf_ws
    torch.cuda.empty_cache()
    # chunked prefill against a mixed prefix (configuration 5): dense contraction, tensor-bound
    wl = synth.cfg_prefill()
    pool, batch, q = b.upload(wl, dev)
    n = len(wl.base_pair_req)
    fr = torch.empty(n, dtype=torch.int32, device=dev)
    b.ekv_downgrade(pool, batch, i32(wl.base_pair_req), i32(wl.base_pair_idx), None, None, None, fr)
    batch.has_base = True
    qs = torch.from_numpy(wl.q_start).to(dev)
    out = torch.empty_like(q)
    C, L = int(wl.q_start[1]), int(wl.seq_lens[0])
    flops = 4.0 * wl.head_dim * wl.num_q_heads * sum(L - C + i + 1 for i in range(C)) * wl.batch
    pf_ws = b.new_workspace(pool, wl.batch, wl.num_q_heads, L, int(wl.q_start[-1]))
    run_pf = lambda: b.ekv_attn_prefill_chunk(pool, 0, batch, qs, q, out, wl.num_q_heads, wl.sm_scale,
                                              int(wl.q_start[-1]), C, L, pf_ws)
    ms = timed(run_pf, iters=10, warm=3)
    b.ekv_set_option("prefill_p_terms", 1)                  # one bf16 term per probability: faster, outside the error bound on some rows
    ms_one = timed(run_pf, iters=10, warm=3)
    b.ekv_set_option("prefill_p_terms", 0)
    peak = 1609.8
    try:
        peak = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops"])
    except Exception:
        pass
    res["prefill_chunk"] = {"workload": "batch 8, 512-token chunk over an 8192-token prefix (50 % BASE), 32/8 heads, D 128",
                            "ms": round(ms, 4), "TFLOPs": round(flops / ms / 1e9, 1), "peak_TFLOPs": peak,
                            "frac": round(flops / ms / 1e9 / peak, 4), "bound": "tensor",
                            "p_terms": "two 16-bit terms per probability (default for bf16 pools)",
                            "one_term": {"ms": round(ms_one, 4), "TFLOPs": round(flops / ms_one / 1e9, 1),
                                         "frac": round(flops / ms_one / 1e9 / peak, 4),
                                         "note": "option prefill_p_terms = 1: the output's error before its final rounding "
                                                 "reaches 5e-3 on rows that two or three tokens dominate"}}
    del pool, batch, q, out, pf_ws
    torch.cuda.empty_cache()
    res["metadata_lowering"] = metadata_lowering(b, torch, dev)
    return res


def roofline_others(ex, hbm_peak):
    """The other measured kernels of the path, in the shape of the `roofline` object: one entry per
    (kernel, workload), taken from the `extras` measurements (L2 flushed before every launch)."""
    tf_burst, tf_sust = 1609.8, 1365.0
    try:
        d = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        tf_burst, tf_sust = float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"])
    except Exception:
        pass
    out = []

    def hbm(kernel, workload, us, gbps, **kw):
        out.append({"kernel": kernel, "bound": "hbm", "achieved": gbps, "peak": hbm_peak, "unit": "GB/s",
                    "frac": round(gbps / hbm_peak, 4), "frac_of_8000_nominal": round(gbps / 8000.0, 4), "us": us,
                    "workload": workload, **kw})
    sw = ex.get("decode_sweep", {})
    names = {"f=0.0:native": "decode_ring_kernel<128,false> (native path)", "f=0.0:elastic_idle": "decode_ring_kernel<128,true> on an all-TARGET pool",
             "f=0.25:elastic": "decode_ring_kernel<128,true>", "f=0.5:elastic": "decode_ring_kernel<128,true>", "f=1.0:elastic": "decode_ring_kernel<128,true>"}
    for key, kname in names.items():
        if key in sw:
            hbm(kname, f"llama3-8b-shaped decode, batch 64, BASE fraction {key.split(':')[0][2:]}; split kernel alone",
                sw[key]["split_kernel_us"], sw[key]["split_kernel_GBps"], call_us=sw[key]["us"], call_GBps=sw[key]["GBps"])
    for key, e in ex.get("other_decode_configs", {}).items():
        hbm("ekv_attn_decode (split + merge kernels)", key, e["us"], e["GBps"])
    for key, e in ex.get("batch_ctx_sweep", {}).items():
        hbm("ekv_attn_decode (split + merge kernels)", f"fixed lengths, f = 0.5: {key}", e["us"], e["GBps"])
    for key, kname in (("downgrade", "downgrade_pack_kernel + commit"), ("refine", "refine_expand_kernel + commit")):
        if key in ex:
            hbm(kname, f"{ex[key]['pairs']} pairs, 1 layer", ex[key]["us"], ex[key]["GBps"])
        t4 = ex.get("transitions_4_layers", {})
        if key in t4:
            hbm(kname, f"{t4['pairs']} pairs, {t4['layers']} layers", t4[key]["us"], t4[key]["GBps"])
    pl = ex.get("pressure_step_loop", {}).get("steady_state_median")
    if pl:
        hbm("downgrade_pack_kernel (last CTA publishes)", f"pressure step loop, {pl['downgrade_pairs']} pairs per step", pl["downgrade_us"], pl["downgrade_GBps"])
        hbm("ekv_attn_decode (split + merge kernels)", "pressure step loop, batch 256", pl["decode_us"], pl["decode_GBps"])
        hbm("refine_expand_kernel (last CTA publishes)", f"pressure step loop, {pl['refine_pairs']} pairs per step", pl["refine_us"], pl["refine_GBps"])
    for key, label in (("prefill_chunk", "bf16"), ("prefill_chunk_fp16", "fp16")):
        pf = ex.get(key) if key == "prefill_chunk" else ex.get("fp16_elements", {}).get("prefill_chunk")
        if pf:
            out.append({"kernel": f"prefill_ws_kernel ({label} elements)", "bound": "tensor", "achieved": pf["TFLOPs"], "peak": tf_burst,
                        "unit": "TFLOP/s", "frac": round(pf["TFLOPs"] / tf_burst, 4), "peak_sustained": tf_sust,
                        "frac_of_sustained": round(pf["TFLOPs"] / tf_sust, 4), "us": round(pf["ms"] * 1e3, 1),
                        "workload": "chunked prefill: batch 8, 512-token chunk over an 8192-token prefix (50 % BASE), 32/8 heads, D 128; "
                                    "L2 flushed before every launch"})
    pf1 = ex.get("prefill_chunk", {}).get("one_term")
    if pf1:
        out.append({"kernel": "prefill_ws_kernel (bf16, option prefill_p_terms = 1: one term per probability)", "bound": "tensor",
                    "achieved": pf1["TFLOPs"], "peak": tf_burst, "unit": "TFLOP/s", "frac": round(pf1["TFLOPs"] / tf_burst, 4),
                    "peak_sustained": tf_sust, "frac_of_sustained": round(pf1["TFLOPs"] / tf_sust, 4), "us": round(pf1["ms"] * 1e3, 1),
                    "workload": "the same chunked-prefill configuration"})
    return out


def run_prefill_only(args):
    """Chunked prefill against a mixed prefix (configuration 5) alone, for profiling captures."""
    import torch
    from paper_2609_33536_b200 import binding as b
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    nreq = args.batch if args.batch != 64 else 8
    wl = synth.cfg_prefill(batch=nreq, elem_type=args.elem_type)
    pool, batch, q = b.upload(wl, dev)
    fr = torch.empty(len(wl.base_pair_req), dtype=torch.int32, device=dev)
    b.ekv_downgrade(pool, batch, i32(wl.base_pair_req), i32(wl.base_pair_idx), None, None, None, fr)
    batch.has_base = True
    qs = torch.from_numpy(wl.q_start).to(dev)
    out = torch.empty_like(q)
    C, L = int(wl.q_start[1]), int(wl.seq_lens[0])
    flops = 4.0 * wl.head_dim * wl.num_q_heads * sum(L - C + i + 1 for i in range(C)) * wl.batch
    pf_ws = b.new_workspace(pool, wl.batch, wl.num_q_heads, L, int(wl.q_start[-1]))
    run = lambda: b.ekv_attn_prefill_chunk(pool, 0, batch, qs, q, out, wl.num_q_heads, wl.sm_scale, int(wl.q_start[-1]), C, L, pf_ws)
    for _ in range(max(1, args.warmup if args.warmup < 10 else 2)):
        run()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps if args.steps != 2000 else 5):
        run()
    e1.record()
    torch.cuda.synchronize()
    n = args.steps if args.steps != 2000 else 5
    ms = e0.elapsed_time(e1) / n
    return {"metric": "prefill_chunk_TFLOPs", "value": round(flops / ms / 1e9, 1), "unit": "TFLOP/s", "ms": round(ms, 4),
            "config": {"workload": f"chunked prefill: batch {nreq}, 512-token chunk over an 8192-token prefix (50 % BASE), 32/8 heads, D 128"},
            "status_word": b.ekv_prefill_status()}


def run_decode_only(args):
    """ekv_attn_decode alone on the decode workload at BASE fraction --profile-decode (0 = the native
    path), --batch requests, --steps launches with an L2 flush between them; for profiling captures."""
    import torch
    from paper_2609_33536_b200 import binding as b
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    f = float(args.profile_decode)
    wl = synth.cfg_llama8b_decode(base_fraction=f, batch=args.batch, elem_type=args.elem_type)
    pool, batch, q = b.upload(wl, dev)
    n = len(wl.base_pair_req)
    if n:
        fr = torch.empty(n, dtype=torch.int32, device=dev)
        b.ekv_downgrade(pool, batch, i32(wl.base_pair_req), i32(wl.base_pair_idx), None, None, None, fr)
        batch.has_base = True
    msl = int(wl.seq_lens.max())
    ws = b.new_workspace(pool, wl.batch, wl.num_q_heads, msl)
    out = torch.empty_like(q)
    flush = L2Flush(torch, dev)
    pe0, pe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    pe0.record(); pe1.record(); torch.cuda.synchronize()
    ks = []
    for _ in range(args.steps if args.steps != 2000 else 8):
        flush()
        b.ekv_set_profile_events(pe0, pe1)
        b.ekv_attn_decode(pool, 0, batch, q, out, wl.num_q_heads, wl.sm_scale, msl, ws)
        b.ekv_set_profile_events(None, None)
        torch.cuda.synchronize()
        ks.append(pe0.elapsed_time(pe1))
    kms = float(np.median(ks[1:])) if len(ks) > 1 else ks[0]
    return {"metric": "decode_split_kernel_GBps", "unit": "GB/s", "base_fraction": f, "batch": wl.batch,
            "kv_bytes": int(wl.kv_bytes()), "split_kernel_us": round(kms * 1e3, 1),
            "split_kernel_us_mean": round(float(np.mean(ks[2:])) * 1e3, 2) if len(ks) > 3 else None,
            "value": round(wl.kv_bytes() / kms / 1e6, 1)}


def run_transitions_only(args):
    """ekv_downgrade / ekv_refine on every eligible pair of the first --batch requests (default 32) of
    the decode workload, alone, for profiling captures; prints GB/s of each."""
    import torch
    from paper_2609_33536_b200 import binding as b
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    wl = synth.cfg_llama8b_decode(base_fraction=0.0)
    pool, batch, q = b.upload(wl, dev)
    nreq = args.batch if args.batch != 64 else 32
    pr = np.concatenate([np.full(wl.eligible_pairs(r), r, np.int32) for r in range(nreq)])
    pi = np.concatenate([np.arange(wl.eligible_pairs(r), dtype=np.int32) for r in range(nreq)])
    n = len(pr)
    kres, vres = pool.new_resid(n), pool.new_resid(n)
    fr = torch.empty(n, dtype=torch.int32, device=dev)
    dpr, dpi, dsl = i32(pr), i32(pi), i32(np.arange(n))
    down_b, up_b = transition_bytes(wl, n)
    flush = L2Flush(torch, dev)
    e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    td, tu = [], []
    for _ in range(args.steps if args.steps != 2000 else 6):
        flush()
        e[0].record(); b.ekv_downgrade(pool, batch, dpr, dpi, kres, vres, dsl, fr)
        e[1].record(); b.ekv_refine(pool, batch, dpr, dpi, fr, kres, vres, dsl)
        e[2].record(); torch.cuda.synchronize()
        td.append(e[0].elapsed_time(e[1])); tu.append(e[1].elapsed_time(e[2]))
    return {"metric": "transition_GBps", "unit": "GB/s", "pairs": n,
            "downgrade": {"us": round(float(np.median(td)) * 1e3, 1), "GBps": round(down_b / np.median(td) / 1e6, 1), "bytes": int(down_b)},
            "refine": {"us": round(float(np.median(tu)) * 1e3, 1), "GBps": round(up_b / np.median(tu) / 1e6, 1), "bytes": int(up_b)}}


# ------------------------------------------------------------------------------------------------
# reference arm: the oracle on the host cores
# ------------------------------------------------------------------------------------------------

def run_reference(args):
    world, rank, _ = _dist()
    if rank != 0:
        return None
    import oracle
    seed = synth.BASE_SEED + 2
    wl = synth.cfg_llama8b_decode(seed=seed, base_fraction=0.5)
    tags = np.zeros(wl.num_blocks, dtype=np.uint8)
    op = oracle.OraclePool(wl.k_pool, wl.v_pool, tags, wl.block_table, wl.seq_lens,
                           num_kv_heads=wl.num_kv_heads, head_dim=wl.head_dim)
    oracle.downgrade(op, wl.base_pair_req, wl.base_pair_idx)
    is_base = set(zip(wl.base_pair_req.tolist(), wl.base_pair_idx.tolist()))
    cand = [(r, p) for r in range(wl.batch) for p in range(wl.eligible_pairs(r)) if (r, p) not in is_base]
    sel = synth.rng(seed, 7).permutation(len(cand))[:TRANSITION_PAIRS]
    tp_req = np.array([cand[i][0] for i in sel], np.int32)
    tp_idx = np.array([cand[i][1] for i in sel], np.int32)
    n_tp = len(tp_req)
    kres, vres = op.new_resid(n_tp), op.new_resid(n_tp)
    slots = np.arange(n_tp, dtype=np.int32)
    K, W = args.steps, max(args.warmup, 1)
    # bounded sample: rows (request, head) of the first requests, sized so K + W steps take ~2 minutes
    H = wl.num_q_heads
    t0 = time.perf_counter()
    oracle.attend_rows(op, 0, [0] * H, list(range(H)), [int(wl.seq_lens[0])] * H, wl.q[0], H, wl.sm_scale)
    per_row_tok = (time.perf_counter() - t0) / (H * max(1, int(wl.seq_lens[0])))
    budget = 120.0 / (K + W)
    rows_r, rows_h, tok = [], [], 0
    for r in range(wl.batch):
        for h in range(H):
            if rows_r and (tok + int(wl.seq_lens[r])) * per_row_tok > budget:
                break
            rows_r.append(r); rows_h.append(h); tok += int(wl.seq_lens[r])
        else:
            continue
        break
    rows_r, rows_h = np.array(rows_r, np.int32), np.array(rows_h, np.int32)
    rows_n = wl.seq_lens[rows_r]
    qrows = wl.q[rows_r, rows_h]
    # bytes of the sample: K/V of the sampled (request, head) rows count once per kv head touched
    G = H // wl.num_kv_heads
    kvh = {(int(r), int(h) // G) for r, h in zip(rows_r, rows_h)}
    base_tok = {r: 0 for r in range(wl.batch)}
    for r in wl.base_pair_req.tolist() + tp_req.tolist():
        base_tok[r] += 2 * wl.page_size
    kvb = sum((int(wl.seq_lens[r]) * 2 - base_tok[r]) * 2 * wl.head_dim for r, _ in kvh)   # per kv head: K+V, 2 B or 1 B
    down_b, up_b = transition_bytes(wl, n_tp)
    step_bytes = kvb + down_b + up_b

    def step():
        freed = oracle.downgrade(op, tp_req, tp_idx, kres, vres, slots)
        oracle.attend_rows(op, 0, rows_r, rows_h, rows_n, qrows, H, wl.sm_scale)
        oracle.refine(op, tp_req, tp_idx, freed, kres, vres, slots)

    for _ in range(W):
        step()
    t0 = time.perf_counter()
    for _ in range(K):
        step()
    dt = (time.perf_counter() - t0) / K
    val = step_bytes / dt / 1e9
    sample = (f"{len(rows_r)} (request, query head) rows of the first {int(rows_r.max()) + 1} requests "
              f"({tok} row-tokens) + the 16-pair downgrade/refine per step")
    return {"impl": "reference", "metric": METRIC, "value": round(val, 4), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": W, "ms_per_step": round(dt * 1e3, 4), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD if args.batch == 64 else WORKLOAD.replace("batch 64", f"batch {args.batch}"), "seed": seed, "reference": "CPU float64 oracle (oracle/), host cores only"},
            "cpu_baseline": {"value": round(val, 4), "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": round(val, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def run_plumbing_check(args):
    """What every rank of a multi-GPU run does around its kernels, with the kernels left out and the
    gloo backend on CPU: rendezvous from the launcher's environment, rank-specific workload draw,
    barrier, max over ranks of the (here: made-up, rank-dependent) step time, sum of the bytes."""
    import torch.distributed as dist
    world, rank, _ = _dist()
    if world > 1:
        dist.init_process_group("gloo")
    wl = synth.cfg_llama8b_decode(seed=synth.BASE_SEED + 2 + 1000 * rank, base_fraction=0.5, batch=2)
    step_bytes = float(wl.kv_bytes())
    if world > 1:
        dist.barrier()
    ms, total = aggregate_over_ranks(1.0 + rank, step_bytes)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return {"plumbing_check": True, "n_gpus": world, "ms_per_step": ms, "bytes_all_ranks": total, "bytes_rank0": step_bytes,
            "scaling": "weak", "backend": "gloo"}


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true")
    ap.add_argument("--batch", type=int, default=64, help="requests in the batch (64 = the named workload)")
    ap.add_argument("--profile-only", action="store_true",
                    help="timed steps only (for ncu captures on a reduced --batch)")
    ap.add_argument("--profile-prefill", action="store_true",
                    help="run only the chunked-prefill configuration (--batch requests, --steps launches) and print its line")
    ap.add_argument("--profile-decode", default=None, metavar="F",
                    help="run only ekv_attn_decode at BASE fraction F on --batch requests (--steps launches, L2 flushed)")
    ap.add_argument("--elem-type", default="bf16", choices=["bf16", "fp16"],
                    help="16-bit element type of the pool in the --profile-prefill / --profile-decode modes")
    ap.add_argument("--profile-transitions", action="store_true",
                    help="run only ekv_downgrade / ekv_refine on all eligible pairs of --batch requests (default 32)")
    ap.add_argument("--plumbing-check", action="store_true",
                    help="multi-rank plumbing only, on CPU with the gloo backend: launch, rendezvous, barrier, "
                         "max-over-ranks time, summed bytes, one JSON line from rank 0; no kernel runs")
    args = ap.parse_args(argv)
    world, rank, _ = _dist()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # Launched plainly with --gpus N: start the N ranks (one process per GPU) under torch's launcher
        # and hand them the same arguments.
        import socket
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(sys.argv[1:] if argv is None else argv)
        raise SystemExit(subprocess.call(cmd))
    if args.plumbing_check:
        res = run_plumbing_check(args)
        if rank == 0:
            print(json.dumps(res), flush=True)
        return
    if args.profile_prefill:
        res = run_prefill_only(args)
    elif args.profile_transitions:
        res = run_transitions_only(args)
    elif args.profile_decode is not None:
        res = run_decode_only(args)
    else:
        res = run_reference(args) if args.impl == "reference" else run_ours(args)
    if rank == 0 and res is not None:
        print(json.dumps(res), flush=True)


if __name__ == "__main__":
    main()
