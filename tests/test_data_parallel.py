"""Data-parallel form of the stage step (Section 3.1 last paragraph, Section 4.1): only the gradients
of the trainable slice are exchanged, and with the slot count taken over all workers the summed
gradients are exactly those of the concatenated batch.

GPU part (one GPU): two workers are two contexts that run one after the other; their buckets are
summed by hand where NCCL would sum them.  CPU part: two gloo ranks reduce the oracle's gradients
through the same helper.
"""
import os
import socket
import sys

import numpy as np
import pytest

from oracle import mslt_oracle as O
from paper_2011_13635_b200 import inputs as I
from tests import parity as PT

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CFG = I.StageConfig("dp", hidden=128, heads=2, ffn=256, vocab=515, max_pos=64, layers=3, trainable=2, batch=6,
                    seq=32, pred=5, dtype="fp32", varlen=(9, 32), seed_index=31)


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,top_k", [("fp32", 2), ("bf16", 2), ("fp32", 3)])
def test_two_workers_equal_one_worker_on_the_concatenated_batch(dtype, top_k):
    import torch
    cfg = I.scaled(CFG, dtype=dtype, trainable=top_k)
    lr = 1e-3 if dtype == "fp32" else 1e-4
    tok, lens, pos, lab = I.make_batch(cfg)
    halves = (slice(0, 2), slice(2, 6))                   # uneven shares, different slot counts
    n_total = int(((pos >= 0) & (lab >= 0)).sum())
    workers = [PT.build_pair(cfg, lr=lr) for _ in halves]
    oracle = workers[0][1]
    total = torch.tensor([n_total], dtype=torch.int32, device="cuda")
    order = []
    comm = torch.cuda.Stream()
    workers[0][0].mslt_set_bucket_hook(comm, order.append)
    losses = []
    for (m, _), h in zip(workers, halves):
        d = PT.to_cuda(torch, tok[h], lens[h], pos[h], lab[h])
        losses.append(m.mslt_step_backward(d[0], d[1], d[2], d[3], total_valid=total))
    # every bucket was announced once, in the order in which the backward pass finishes them
    n_b = 1 + top_k + (1 if top_k == cfg.layers else 0)
    assert order == list(range(n_b))
    b0, b1 = workers[0][0].grad_buckets(), workers[1][0].grad_buckets()
    assert len(b0) == n_b
    # frozen layers have no bucket: the exchanged volume is the trainable slice only
    names = oracle.trainable_names()
    assert sum(b.numel() for b in b0) >= sum(oracle.p[n].size for n in names)
    assert sum(b.numel() for b in b0) < 1.02 * sum(oracle.p[n].size for n in names) + 64 * len(names)
    with pytest.raises(Exception) as ei:                   # no new step before the update is applied
        workers[0][0].mslt_step(*PT.to_cuda(torch, tok, lens, pos, lab))
    assert ei.value.code == -3
    for x, y in zip(b0, b1):                              # what the all-reduce does
        x += y
        y.copy_(x)
    for m, _ in workers:
        m.mslt_step_apply()
    loss_o = oracle.step(tok, lens, pos, lab)             # one worker, whole batch
    tol = PT.TOL[dtype]
    assert abs(sum(losses) - loss_o) / loss_o < tol["loss"]
    for n in names:
        g = workers[0][0].mslt_get_grad(n)
        assert PT.max_rel(g, oracle.grads[n]) < tol["grad"], n
        assert PT.max_rel(workers[0][0].mslt_get_param(n), oracle.p[n]) < tol["weight"], n
        assert np.array_equal(workers[0][0].mslt_get_param(n), workers[1][0].mslt_get_param(n)), n
    for m, _ in workers:
        m.close()


@pytest.mark.gpu
def test_single_worker_data_parallel_step_is_the_plain_step():
    import torch
    from paper_2011_13635_b200.data_parallel import DataParallelStep
    cfg = I.scaled(CFG, dtype="bf16")
    batch = I.make_batch(cfg)
    (m1, _), (m2, _) = PT.build_pair(cfg, lr=1e-4), PT.build_pair(cfg, lr=1e-4)
    d = PT.to_cuda(torch, *batch)
    dp = DataParallelStep(m2)
    for _ in range(2):
        l1 = m1.mslt_step(*d)
        l2 = dp.step(*d)
        assert abs(l1 - l2) <= 1e-6 * abs(l1)
    for n in m1.tensors():
        # bias sums use atomics: two runs of the same step differ in the last bits
        np.testing.assert_allclose(m1.mslt_get_param(n), m2.mslt_get_param(n), rtol=1e-5, atol=1e-7, err_msg=n)
    assert dp.bytes_exchanged == 0
    m1.close(); m2.close()


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist
    from paper_2011_13635_b200.data_parallel import reduce_buckets
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    cfg = I.scaled(CFG, dtype="fp32")
    tok, lens, pos, lab = I.make_batch(cfg)
    share = (slice(0, 2), slice(2, 6))[rank]
    w = I.make_weights(cfg, variant="parity")
    m = O.MsltOracle(w, cfg.heads)
    m.set_trainable(cfg.trainable)
    loss, g = m.loss_and_grads(tok[share], lens[share], pos[share], lab[share])
    n_local = torch.tensor([int(((pos[share] >= 0) & (lab[share] >= 0)).sum())], dtype=torch.float64)
    n_total = n_local.clone()
    dist.all_reduce(n_total)
    # the library divides by the global count; the oracle divided by the local one: rescale, then sum
    names = m.trainable_names()
    buckets = [torch.from_numpy(g[n] * float(n_local / n_total)) for n in names]
    reduce_buckets(buckets, dist)
    lsum = torch.tensor([loss * float(n_local / n_total)], dtype=torch.float64)
    dist.all_reduce(lsum)
    out.put((rank, float(lsum), {n: b.numpy().copy() for n, b in zip(names, buckets)}))
    dist.barrier()
    dist.destroy_process_group()


def test_reduced_gradients_of_two_ranks_equal_the_concatenated_batch_in_the_oracle():
    import torch.multiprocessing as mp
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted((out.get(timeout=180) for _ in range(2)), key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg = I.scaled(CFG, dtype="fp32")
    w = I.make_weights(cfg, variant="parity")
    m = O.MsltOracle(w, cfg.heads)
    m.set_trainable(cfg.trainable)
    loss, g = m.loss_and_grads(*I.make_batch(cfg))
    for rank, lsum, red in res:
        assert abs(lsum - loss) < 1e-12
        assert set(red) == set(m.trainable_names())         # nothing of the frozen layers travels
        for n in red:
            np.testing.assert_allclose(red[n], g[n], atol=1e-14, rtol=0)
    frozen = sum(v.size for k, v in m.p.items() if k not in res[0][2])
    assert frozen > 0
