"""Micro-benchmark of the contraction kernel through mslt_op_gemm.

    python -m paper_2011_13635_b200.gemm_bench --m 16384 --n 3072 --k 768 [--layout kk|kmn|mnmn]
        [--dtype bf16|fp32] [--epilogue none|bias|gelu|dgelu|residual|accum|f32out|gelu_noaux] [--iters 20]

Times back-to-back launches with CUDA events on the launching stream and prints one JSON line.
"""
from __future__ import annotations

import argparse
import json


def main():
    import torch
    from . import binding as Bd
    ap = argparse.ArgumentParser()
    ap.add_argument("--m", type=int, default=16384)
    ap.add_argument("--n", type=int, default=3072)
    ap.add_argument("--k", type=int, default=768)
    ap.add_argument("--layout", default="kk", choices=["kk", "kmn", "mnmn"])
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp32"])
    ap.add_argument("--epilogue", default="none",
                    choices=["none", "bias", "gelu", "dgelu", "residual", "accum", "f32out", "gelu_noaux"])
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    a = ap.parse_args()
    tdt = torch.bfloat16 if a.dtype == "bf16" else torch.float32
    M, N, K = a.m, a.n, a.k
    g = torch.Generator(device="cuda").manual_seed(1)
    A = (torch.randn((M, K) if a.layout[0] == "k" else (K, M), device="cuda", generator=g) * 0.05).to(tdt)
    B = (torch.randn((N, K) if a.layout == "kk" else (K, N), device="cuda", generator=g) * 0.05).to(tdt)
    d = Bd.GemmDesc()
    d.dtype, d.M, d.N, d.K, d.batch, d.hdiv, d.alpha = (1 if a.dtype == "bf16" else 0), M, N, K, 1, 1, 1.0
    d.A = A.data_ptr()
    d.a_rs, d.a_ks = (K, 1) if a.layout[0] == "k" else (1, M)
    d.B = B.data_ptr()
    d.b_rs, d.b_ks = (K, 1) if a.layout == "kk" else (1, N)
    accum = a.epilogue == "accum"
    f32 = accum or a.epilogue == "f32out"
    ldd = (N + 7) // 8 * 8
    D = torch.zeros((M, ldd), device="cuda", dtype=torch.float32 if f32 else tdt)
    d.D, d.ldd, d.d_fp32, d.accumulate = D.data_ptr(), ldd, int(f32), int(accum)
    keep = []
    if a.epilogue in ("bias", "gelu", "gelu_noaux"):
        bias = torch.randn(N, device="cuda"); keep.append(bias); d.bias = bias.data_ptr()
    if a.epilogue == "gelu":
        aux = torch.empty((M, ldd), device="cuda", dtype=tdt); keep.append(aux)
        d.act, d.aux = 1, aux.data_ptr()
    if a.epilogue == "gelu_noaux":
        d.act = 1
    if a.epilogue == "dgelu":
        aux = torch.randn((M, ldd), device="cuda").to(tdt); keep.append(aux)
        d.act, d.aux = 2, aux.data_ptr()
    if a.epilogue == "residual":
        r = torch.randn((M, ldd), device="cuda").to(tdt); keep.append(r); d.residual = r.data_ptr()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    for _ in range(a.warmup):
        Bd.mslt_op_gemm(d, stream, status)
    # back-to-back launches between two events: kernel time without host round trips
    times = []
    for _ in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(a.iters):
            Bd.mslt_op_gemm_enqueue(d, stream, status)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / a.iters)
    if int(status.item()) != 0:
        raise RuntimeError("the kernel reported a wait that ran out")
    times.sort()
    med = times[len(times) // 2]
    print(json.dumps(dict(M=M, N=N, K=K, layout=a.layout, dtype=a.dtype, epilogue=a.epilogue,
                          us_median=1e3 * med, us_min=1e3 * times[0],
                          tflops_median=2.0 * M * N * K / (med * 1e-3) / 1e12,
                          tflops_best=2.0 * M * N * K / (times[0] * 1e-3) / 1e12)))


if __name__ == "__main__":
    main()
