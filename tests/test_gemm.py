"""The dense contraction kernel alone (mslt_op_gemm) against numpy float64, for every operand
layout the step uses (forward: k contiguous; input gradient and weight gradient: row index
contiguous), batched attention addressing, ragged edges and each fused epilogue."""
import math

import numpy as np
import pytest
from scipy.special import erf

from tests import parity as PT

pytestmark = pytest.mark.gpu


def _gelu(u):
    return 0.5 * u * (1 + erf(u / math.sqrt(2)))


def _dgelu(u):
    return 0.5 * (1 + erf(u / math.sqrt(2))) + u * np.exp(-0.5 * u * u) / math.sqrt(2 * math.pi)


def _run(dtype, M, N, K, a_major, b_major, *, bias=False, act=0, residual=False, aux_out=False,
         d_fp32=False, accumulate=False, alpha=1.0, split_k=0, seed=0):
    import torch
    from paper_2011_13635_b200 import binding as Bd
    tdt = torch.float32 if dtype == 0 else torch.bfloat16
    rng = np.random.default_rng(seed)
    A = rng.standard_normal((M, K)).astype(np.float32)
    B = rng.standard_normal((N, K)).astype(np.float32)
    tA = torch.from_numpy(A).cuda().to(tdt)
    tB = torch.from_numpy(B).cuda().to(tdt)
    A64, B64 = tA.double().cpu().numpy(), tB.double().cpu().numpy()
    # K-major: stored [rows, K]; MN-major: stored [K, rows] (leading dimension padded to 8)
    def store(t, major):
        if major == "k":
            return t.contiguous(), t.shape[1], 1
        ld = (t.shape[0] + 7) // 8 * 8
        buf = torch.zeros((t.shape[1], ld), dtype=t.dtype, device="cuda")
        buf[:, : t.shape[0]] = t.t()
        return buf, 1, ld
    sA, a_rs, a_ks = store(tA, a_major)
    sB, b_rs, b_ks = store(tB, b_major)
    ldd = (N + 7) // 8 * 8
    D0 = rng.standard_normal((M, ldd)).astype(np.float32)
    tD = torch.from_numpy(D0).cuda().to(torch.float32 if d_fp32 else tdt)
    ref = alpha * (A64 @ B64.T)
    d = Bd.GemmDesc()
    d.dtype, d.M, d.N, d.K, d.batch, d.hdiv = dtype, M, N, K, 1, 1
    d.A, d.a_rs, d.a_ks = sA.data_ptr(), a_rs, a_ks
    d.B, d.b_rs, d.b_ks = sB.data_ptr(), b_rs, b_ks
    d.D, d.ldd = tD.data_ptr(), ldd
    d.d_fp32, d.accumulate, d.alpha, d.act, d.split_k = int(d_fp32), int(accumulate), alpha, act, split_k
    keep = [sA, sB, tD]
    if bias:
        bv = rng.standard_normal(N).astype(np.float32)
        tb = torch.from_numpy(bv).cuda()
        d.bias = tb.data_ptr()
        ref = ref + bv.astype(np.float64)
        keep.append(tb)
    taux = None
    if act == 1:
        if aux_out:
            taux = torch.zeros((M, ldd), dtype=tdt, device="cuda")
            d.aux = taux.data_ptr()
        pre = ref
        ref = _gelu(ref)
    elif act == 2:
        U = rng.standard_normal((M, ldd)).astype(np.float32)
        taux = torch.from_numpy(U).cuda().to(tdt)
        d.aux = taux.data_ptr()
        ref = ref * _dgelu(taux.double().cpu().numpy()[:, :N])
    if residual:
        Rm = rng.standard_normal((M, ldd)).astype(np.float32)
        tr = torch.from_numpy(Rm).cuda().to(tdt)
        d.residual = tr.data_ptr()
        ref = ref + tr.double().cpu().numpy()[:, :N]
        keep.append(tr)
    if accumulate:
        ref = ref + D0[:, :N].astype(np.float64)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Bd.mslt_op_gemm(d, torch.cuda.current_stream().cuda_stream, status)
    out = tD.double().cpu().numpy()
    tol = 2e-5 if dtype == 0 else (1e-5 if d_fp32 else 6e-3)
    scale = np.abs(ref).max()
    assert np.abs(out[:, :N] - ref).max() / scale < tol, (M, N, K, a_major, b_major)
    # columns past N (padding of the leading dimension) are never written
    if ldd > N:
        init = torch.from_numpy(D0).cuda().to(tD.dtype).double().cpu().numpy()
        assert np.array_equal(out[:, N:], init[:, N:])
    if act == 1 and aux_out:
        assert np.abs(taux.double().cpu().numpy()[:, :N] - pre).max() / np.abs(pre).max() < (2e-5 if dtype == 0 else 6e-3)


SHAPES = [(128, 128, 64), (256, 256, 128), (200, 136, 72), (130, 1037, 192), (517, 64, 520),
          (64, 72, 8), (1, 8, 16)]


@pytest.mark.parametrize("dtype", [0, 1], ids=["fp32", "bf16"])
@pytest.mark.parametrize("majors", [("k", "k"), ("k", "mn"), ("mn", "mn"), ("mn", "k")])
@pytest.mark.parametrize("shape", SHAPES)
def test_layouts_and_ragged_edges(dtype, majors, shape):
    _run(dtype, *shape, majors[0], majors[1], seed=hash(shape) % 1000)


@pytest.mark.parametrize("dtype", [0, 1], ids=["fp32", "bf16"])
def test_epilogues(dtype):
    _run(dtype, 200, 136, 72, "k", "k", bias=True)
    _run(dtype, 200, 136, 72, "k", "k", bias=True, act=1, aux_out=True)
    _run(dtype, 200, 136, 72, "k", "k", bias=True, act=1)
    _run(dtype, 200, 136, 72, "k", "mn", act=2)
    _run(dtype, 200, 136, 72, "k", "mn", residual=True, alpha=0.125)
    _run(dtype, 200, 136, 72, "k", "k", bias=True, residual=True)
    _run(dtype, 200, 136, 72, "k", "k", bias=True, d_fp32=True)
    _run(dtype, 136, 200, 1000, "mn", "mn", d_fp32=True, accumulate=True)


@pytest.mark.parametrize("variant", [0, 1, 2, 4, 6], ids=["auto", "single", "pair", "auto-rowstores", "pair-rowstores"])
def test_bf16_epilogues_over_several_wide_tiles(variant):
    """Every bf16 epilogue flavour on outputs of several 256-wide tiles with ragged last tiles, in
    each tiling form and with both ways of storing the output (through shared memory and the copy
    engine, or row segments from registers)."""
    from paper_2011_13635_b200 import binding as Bd
    assert Bd.lib.mslt_debug_set_gemm_variant(variant) == 0
    try:
        _run(1, 700, 840, 200, "k", "k", bias=True)
        _run(1, 700, 840, 200, "k", "k", bias=True, act=1, aux_out=True)
        _run(1, 700, 832, 136, "k", "k", bias=True, act=1)
        _run(1, 520, 800, 72, "k", "mn", act=2)
        _run(1, 520, 800, 72, "k", "mn", bias=True, residual=True, alpha=0.125)
        _run(1, 300, 1037, 192, "k", "k", bias=True)           # row pitch 1040: columns end inside a chunk
        _run(1, 33, 168, 64, "mn", "k", bias=True, act=1)      # one 128-wide tile and a ragged second one
    finally:
        Bd.lib.mslt_debug_set_gemm_variant(0)


def test_bf16_long_contraction_split_k():
    """Weight-gradient shape: small output, long contraction, partial sums added in fp32."""
    _run(1, 768, 256, 4096, "mn", "mn", d_fp32=True, accumulate=True)
    _run(1, 768, 256, 4096, "mn", "mn", d_fp32=True, accumulate=True, split_k=7)
    _run(1, 300, 264, 2500, "mn", "mn", d_fp32=True, accumulate=True, split_k=3)


@pytest.mark.parametrize("dtype", [0, 1], ids=["fp32", "bf16"])
def test_batched_attention_addressing(dtype):
    """Scores and context of multi-head attention read straight from the fused [T, 3H] buffer."""
    import torch
    from paper_2011_13635_b200 import binding as Bd
    Bn, A, S, dh = 3, 2, 72, 64
    H = A * dh
    tdt = torch.float32 if dtype == 0 else torch.bfloat16
    rng = np.random.default_rng(3)
    qkv = torch.from_numpy(rng.standard_normal((Bn * S, 3 * H)).astype(np.float32)).cuda().to(tdt)
    q64 = qkv.double().cpu().numpy().reshape(Bn, S, 3, A, dh)
    sc = torch.zeros((Bn * A, S, S), dtype=tdt, device="cuda")
    d = Bd.GemmDesc()
    d.dtype, d.M, d.N, d.K, d.batch, d.hdiv, d.alpha = dtype, S, S, dh, Bn * A, A, 0.125
    d.A, d.a_rs, d.a_ks, d.a_bo, d.a_bi = qkv.data_ptr(), 3 * H, 1, S * 3 * H, dh
    d.B, d.b_rs, d.b_ks, d.b_bo, d.b_bi = qkv.data_ptr() + H * qkv.element_size(), 3 * H, 1, S * 3 * H, dh
    d.D, d.ldd, d.d_bo, d.d_bi = sc.data_ptr(), S, A * S * S, S * S
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Bd.mslt_op_gemm(d, torch.cuda.current_stream().cuda_stream, status)
    ref = 0.125 * np.einsum("bihd,bjhd->bhij", q64[:, :, 0], q64[:, :, 1]).reshape(Bn * A, S, S)
    tol = 2e-5 if dtype == 0 else 6e-3
    assert np.abs(sc.double().cpu().numpy() - ref).max() / np.abs(ref).max() < tol
    # context = P V with V read row-contiguous (its k index strided)
    p = torch.from_numpy(rng.random((Bn * A, S, S)).astype(np.float32)).cuda().to(tdt)
    ctx = torch.zeros((Bn * S, H), dtype=tdt, device="cuda")
    d = Bd.GemmDesc()
    d.dtype, d.M, d.N, d.K, d.batch, d.hdiv, d.alpha = dtype, S, dh, S, Bn * A, A, 1.0
    d.A, d.a_rs, d.a_ks, d.a_bo, d.a_bi = p.data_ptr(), S, 1, A * S * S, S * S
    d.B, d.b_rs, d.b_ks, d.b_bo, d.b_bi = qkv.data_ptr() + 2 * H * qkv.element_size(), 1, 3 * H, S * 3 * H, dh
    d.D, d.ldd, d.d_bo, d.d_bi = ctx.data_ptr(), H, S * H, dh
    Bd.mslt_op_gemm(d, torch.cuda.current_stream().cuda_stream, status)
    p64 = p.double().cpu().numpy().reshape(Bn, A, S, S)
    ref = np.einsum("bhij,bjhd->bihd", p64, q64[:, :, 2]).reshape(Bn * S, H)
    assert np.abs(ctx.double().cpu().numpy() - ref).max() / np.abs(ref).max() < tol


@pytest.mark.parametrize("S", [128, 72, 64, 8])
def test_bf16_softmax_epilogue(S):
    """Attention scores with the scaled masked softmax applied in the kernel's epilogue."""
    import torch
    from paper_2011_13635_b200 import binding as Bd
    Bn, A, dh = 3, 2, 64
    H = A * dh
    rng = np.random.default_rng(S)
    qkv = torch.from_numpy(rng.standard_normal((Bn * S, 3 * H)).astype(np.float32) * 2).cuda().to(torch.bfloat16)
    lens = np.array([S, max(1, S // 3), 1], dtype=np.int32)
    d_lens = torch.from_numpy(lens).cuda()
    prob = torch.full((Bn * A, S, S), 7.0, dtype=torch.bfloat16, device="cuda")
    d = Bd.GemmDesc()
    d.dtype, d.M, d.N, d.K, d.batch, d.hdiv, d.alpha = 1, S, S, dh, Bn * A, A, 0.125
    d.A, d.a_rs, d.a_ks, d.a_bo, d.a_bi = qkv.data_ptr(), 3 * H, 1, S * 3 * H, dh
    d.B, d.b_rs, d.b_ks, d.b_bo, d.b_bi = qkv.data_ptr() + H * 2, 3 * H, 1, S * 3 * H, dh
    d.D, d.ldd, d.d_bo, d.d_bi = prob.data_ptr(), S, A * S * S, S * S
    d.act, d.seq_lens = 3, d_lens.data_ptr()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Bd.mslt_op_gemm(d, torch.cuda.current_stream().cuda_stream, status)
    q64 = qkv.double().cpu().numpy().reshape(Bn, S, 3, A, dh)
    sc = 0.125 * np.einsum("bihd,bjhd->bhij", q64[:, :, 0], q64[:, :, 1])
    valid = (np.arange(S)[None, :] < lens[:, None])[:, None, None, :]
    sc = np.where(valid, sc, -np.inf)
    e = np.exp(sc - sc.max(-1, keepdims=True))
    ref = (e / e.sum(-1, keepdims=True)).reshape(Bn * A, S, S)
    got = prob.double().cpu().numpy()
    assert np.abs(got - ref).max() < 6e-3
    assert np.all(got[ref == 0] == 0)                  # masked keys are exactly zero
    np.testing.assert_allclose(got.sum(-1), 1.0, atol=2e-2)


def test_wait_that_runs_out_is_reported_and_leaves_the_device_usable():
    """Failure path without a fault: the producer of one launch issues no copies, the first wait
    runs out after ~20 ms, the kernel drains and returns, and the call reports MSLT_ERR_DEVICE."""
    import torch
    from paper_2011_13635_b200 import binding as Bd
    M = N = 128
    K = 64
    a = torch.randn((M, K), device="cuda").to(torch.bfloat16)
    b = torch.randn((N, K), device="cuda").to(torch.bfloat16)
    out = torch.zeros((M, N), device="cuda", dtype=torch.bfloat16)
    d = Bd.GemmDesc()
    d.dtype, d.M, d.N, d.K, d.batch, d.hdiv, d.alpha = 1, M, N, K, 1, 1, 1.0
    d.A, d.a_rs, d.a_ks = a.data_ptr(), K, 1
    d.B, d.b_rs, d.b_ks = b.data_ptr(), K, 1
    d.D, d.ldd = out.data_ptr(), N
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    Bd.lib.mslt_debug_starve_next_gemm(1)
    with pytest.raises(Bd.MsltError) as ei:
        Bd.mslt_op_gemm(d, stream, status)
    assert ei.value.code == -5
    assert int(status.item()) & 1
    # the hook disarms itself: the same call now succeeds and is correct
    status.zero_()
    Bd.mslt_op_gemm(d, stream, status)
    ref = a.double() @ b.double().t()
    assert (out.double() - ref).abs().max() / ref.abs().max() < 6e-3
    assert int(status.item()) == 0
