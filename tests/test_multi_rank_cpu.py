"""The N > 1 path of the benchmark is 'replicas only' (no exchange step on this path): ranks draw
rank-specific workloads of the same shape, and rank 0 reports sum(bytes) / max(time). Checked
here with two gloo ranks on CPU; nothing in it needs a GPU."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2609_33536_b200 import synth
    # replicas: same shape, rank-specific draw (the seed rule run_ours uses)
    wl = synth.cfg_llama8b_decode(seed=synth.BASE_SEED + 2 + 1000 * rank, base_fraction=0.5, batch=2)
    ms = 1.0 + rank                      # rank 1 is the slow one
    step_bytes = float(wl.kv_bytes())
    got_ms, got_bytes = bench.aggregate_over_ranks(ms, step_bytes)
    np.save(os.path.join(out_dir, f"r{rank}.npy"), np.array([got_ms, got_bytes, step_bytes, float(wl.seq_lens.sum())]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_gloo(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r = [np.load(tmp_path / f"r{k}.npy") for k in range(world)]
    assert r[0][0] == r[1][0] == 2.0                             # max over ranks
    assert r[0][1] == r[1][1] == r[0][2] + r[1][2]               # sum of both replicas' bytes
    assert r[0][3] != r[1][3]                                    # the replicas drew different workloads


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(3.5, 7.0) == (3.5, 7.0)


def test_bench_main_launches_its_own_ranks():
    """`python bench.py --gpus 2` without a launcher around it starts its two ranks itself; driven
    here through main() on CPU (gloo) with the kernels left out. Rank 0 alone prints the line."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    code = "import sys; sys.path.insert(0, %r); import bench; bench.main(['--gpus', '2', '--plumbing-check'])" % ROOT
    out = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout
    res = json.loads(lines[0])
    assert res["n_gpus"] == 2 and res["ms_per_step"] == 2.0          # the slower rank's time
    assert res["bytes_all_ranks"] > res["bytes_rank0"] > 0           # both replicas' bytes
