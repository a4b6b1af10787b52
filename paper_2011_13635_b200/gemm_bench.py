"""Micro-benchmark of the contraction kernel through mslt_op_gemm.

    python -m paper_2011_13635_b200.gemm_bench --m 16384 --n 3072 --k 768 [--layout kk|kmn|mnmn]
        [--dtype bf16|fp32] [--epilogue none|bias|gelu|dgelu|residual|accum|f32out|gelu_noaux] [--iters 20]
    python -m paper_2011_13635_b200.gemm_bench --table [--seconds 1.0]

Times back-to-back launches with CUDA events on the launching stream and prints one JSON line.
--table: every product shape of the BERT-Base and BERT-Large stage steps (forward, input gradient,
weight gradient, logits), this kernel beside the library GEMM behind torch.matmul on the same
operands (cuBLAS, no epilogue: a yardstick, not part of the step), each as a short burst of launches
and as a loop of --seconds (the power-capped regime a step runs in); one JSON line per shape.
"""
from __future__ import annotations

import argparse
import json

# (name, M, N, K, layout, epilogue) of the products of one layer and the head; T = 16384 rows
# (BERT-Base, 128 x 128) or 8192 rows (BERT-Large), 2560 masked slots
TABLE = [
    ("base qkv", 16384, 2304, 768, "kk", "bias"), ("base out-proj", 16384, 768, 768, "kk", "residual"),
    ("base ffn-up", 16384, 3072, 768, "kk", "gelu_noaux"), ("base ffn-up + pre-activation", 16384, 3072, 768, "kk", "gelu"),
    ("base ffn-down", 16384, 768, 3072, "kk", "residual"),
    ("base d ffn-down x gelu'", 16384, 3072, 768, "kmn", "dgelu"), ("base d ffn-up", 16384, 768, 3072, "kmn", "residual"),
    ("base d out-proj", 16384, 768, 768, "kmn", "none"), ("base d qkv", 16384, 768, 2304, "kmn", "residual"),
    ("base w ffn-up", 3072, 768, 16384, "mnmn", "accum"), ("base w ffn-down", 768, 3072, 16384, "mnmn", "accum"),
    ("base w out-proj", 768, 768, 16384, "mnmn", "accum"), ("base w qkv", 2304, 768, 16384, "mnmn", "accum"),
    ("logits", 2560, 30522, 768, "kk", "f32out"),
    ("large qkv", 8192, 3072, 1024, "kk", "bias"), ("large out-proj", 8192, 1024, 1024, "kk", "residual"),
    ("large ffn-up", 8192, 4096, 1024, "kk", "gelu_noaux"), ("large ffn-down", 8192, 1024, 4096, "kk", "residual"),
    ("8192^3", 8192, 8192, 8192, "kk", "none"),
]


def _time(fn, iters):
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters   # ms


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
    ap.add_argument("--table", action="store_true", help="all step shapes beside the library GEMM")
    ap.add_argument("--seconds", type=float, default=1.0, help="--table: length of the sustained loop")
    a = ap.parse_args()
    if a.table:
        return table(a)
    one_case(a.m, a.n, a.k, a.layout, a.dtype, a.epilogue, a.iters, a.warmup)


def one_case(M, N, K, layout, dtype, epilogue, iters, warmup, seconds=0.0, quiet=False):
    """Times one shape; returns (median ms of the short bursts, ms per launch of the long loop or
    None, the operands for a library run)."""
    import torch
    from . import binding as Bd

    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    g = torch.Generator(device="cuda").manual_seed(1)
    A = (torch.randn((M, K) if layout[0] == "k" else (K, M), device="cuda", generator=g) * 0.05).to(tdt)
    B = (torch.randn((N, K) if layout == "kk" else (K, N), device="cuda", generator=g) * 0.05).to(tdt)
    d = Bd.GemmDesc()
    d.dtype, d.M, d.N, d.K, d.batch, d.hdiv, d.alpha = (1 if dtype == "bf16" else 0), M, N, K, 1, 1, 1.0
    d.A = A.data_ptr()
    d.a_rs, d.a_ks = (K, 1) if layout[0] == "k" else (1, M)
    d.B = B.data_ptr()
    d.b_rs, d.b_ks = (K, 1) if layout == "kk" else (1, N)
    accum = epilogue == "accum"
    f32 = accum or epilogue == "f32out"
    ldd = (N + 7) // 8 * 8
    D = torch.zeros((M, ldd), device="cuda", dtype=torch.float32 if f32 else tdt)
    d.D, d.ldd, d.d_fp32, d.accumulate = D.data_ptr(), ldd, int(f32), int(accum)
    keep = []
    if epilogue in ("bias", "gelu", "gelu_noaux"):
        bias = torch.randn(N, device="cuda"); keep.append(bias); d.bias = bias.data_ptr()
    if epilogue == "gelu":
        aux = torch.empty((M, ldd), device="cuda", dtype=tdt); keep.append(aux)
        d.act, d.aux = 1, aux.data_ptr()
    if epilogue == "gelu_noaux":
        d.act = 1
    if epilogue == "dgelu":
        aux = torch.randn((M, ldd), device="cuda").to(tdt); keep.append(aux)
        d.act, d.aux = 2, aux.data_ptr()
    if epilogue == "residual":
        r = torch.randn((M, ldd), device="cuda").to(tdt); keep.append(r); d.residual = r.data_ptr()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    for _ in range(warmup):
        Bd.mslt_op_gemm(d, stream, status)
    # back-to-back launches between two events: kernel time without host round trips
    times = []
    for _ in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            Bd.mslt_op_gemm_enqueue(d, stream, status)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / iters)
    if int(status.item()) != 0:
        raise RuntimeError("the kernel reported a wait that ran out")
    times.sort()
    med = times[len(times) // 2]
    long_ms = None
    if seconds > 0:
        n = max(20, int(seconds / (med * 1e-3)))
        long_ms = _time(lambda: Bd.mslt_op_gemm_enqueue(d, stream, status), n)
    if quiet:
        return med, long_ms, (A, B)
    print(json.dumps(dict(M=M, N=N, K=K, layout=layout, dtype=dtype, epilogue=epilogue,
                          us_median=1e3 * med, us_min=1e3 * times[0],
                          tflops_median=2.0 * M * N * K / (med * 1e-3) / 1e12,
                          tflops_best=2.0 * M * N * K / (times[0] * 1e-3) / 1e12)))
    return med, long_ms, (A, B)


def table(a):
    import torch
    for name, M, N, K, layout, epi in TABLE:
        med, long_ms, (A, B) = one_case(M, N, K, layout, "bf16", epi, 20, 3, seconds=a.seconds, quiet=True)
        # the same contraction through torch.matmul (operands as stored: no copies in the timed part)
        if layout == "kk":
            lib = lambda: torch.matmul(A, B.t())
        elif layout == "kmn":
            lib = lambda: torch.matmul(A, B)
        else:
            lib = lambda: torch.matmul(A.t(), B)
        for _ in range(3):
            lib()
        torch.cuda.synchronize()
        lib_ms = sorted(_time(lib, 20) for _ in range(3))[1]
        lib_long = _time(lib, max(20, int(a.seconds / (lib_ms * 1e-3)))) if a.seconds > 0 else None
        tf = lambda ms: None if ms is None else round(2.0 * M * N * K / (ms * 1e-3) / 1e12, 1)
        print(json.dumps(dict(shape=name, M=M, N=N, K=K, layout=layout, epilogue=epi,
                              us=round(1e3 * med, 1), tflops=tf(med), tflops_sustained=tf(long_ms),
                              library_us=round(1e3 * lib_ms, 1), library_tflops=tf(lib_ms),
                              library_tflops_sustained=tf(lib_long))), flush=True)


if __name__ == "__main__":
    main()
