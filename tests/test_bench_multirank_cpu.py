"""Host-side logic of bench.py's multi-rank mode (independent replicas), on two gloo ranks."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2011_13635_b200 import inputs as I
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    cfg = I.scaled(I.CONFIGS["base_stage"], batch=4)
    tok = I.make_batch(cfg, seed=bench.rank_seed(cfg, rank))[0]
    ms_local = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    ms, value = bench.aggregate(ms_local, cfg.batch, 20, world, dist, "cpu")
    out.put((rank, ms, value, int(tok.astype(np.int64).sum())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_aggregate_as_max_time_and_summed_sequences():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, ms0, v0, sum0), (_, ms1, v1, sum1) = res
    assert ms0 == ms1 == 15.0                           # the slowest rank sets the time
    assert v0 == v1 == 4 * 2 * 20 / 15e-3               # both replicas' sequences count
    assert sum0 != sum1                                 # replicas draw different batches


def test_reference_arm_prints_the_contract_line():
    import json
    import subprocess
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-500:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "sequences/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_gpus_flag_starts_its_own_replicas():
    """`python bench.py --gpus 2` without a launcher starts two processes itself; here they meet over
    gloo with pretended timings (10 and 20 ms), so the slowest rank sets the time and both count."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--selftest-cpu", "--steps", "20"],
                       capture_output=True, text=True, timeout=300, cwd=ROOT, env=env)
    assert r.returncode == 0, r.stderr[-500:]
    lines = [l for l in r.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1                                # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["ms_per_step"] == 1.0
    assert line["value"] == 128 * 2 * 20 / 20e-3
