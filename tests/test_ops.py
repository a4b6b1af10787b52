"""Single-kernel entry points against the oracle's per-operation functions."""
import numpy as np
import pytest

from oracle import mslt_oracle as O

pytestmark = pytest.mark.gpu


def run_cross_entropy(fn, dtype, logits, labels, V, want_grad=True, **kw):
    import torch
    R = logits.shape[0]
    ldl = (V + 7) // 8 * 8
    buf = torch.zeros((R, ldl), dtype=torch.float32, device="cuda")
    buf[:, :V] = torch.from_numpy(logits).cuda()
    d_lab = torch.from_numpy(labels.astype(np.int32)).cuda()
    dl = torch.full((R, ldl), 3.0, device="cuda", dtype=torch.float32 if dtype == 0 else torch.bfloat16) \
        if want_grad else None
    loss = torch.zeros(1, device="cuda")
    fn(dtype, buf, d_lab, V, dl, loss, stream=torch.cuda.current_stream().cuda_stream, **kw)
    return float(loss.item()), None if dl is None else dl.float().cpu().numpy()


@pytest.mark.parametrize("dtype", [0, 1], ids=["fp32", "bf16"])
@pytest.mark.parametrize("R,V", [(7, 11), (64, 1037), (300, 30522)])
def test_cross_entropy_matches_oracle(dtype, R, V):
    import torch
    from paper_2011_13635_b200 import binding as Bd
    rng = np.random.default_rng(R + V)
    logits = (rng.standard_normal((R, V)) * 3).astype(np.float32)
    labels = rng.integers(0, V, size=R)
    labels[::5] = -1
    n_valid = int((labels >= 0).sum())
    scratch = torch.empty(Bd.lib.mslt_op_cross_entropy_scratch_bytes(R), dtype=torch.uint8, device="cuda")
    loss, dl = run_cross_entropy(Bd.mslt_op_cross_entropy, dtype, logits, labels, V, scratch=scratch)
    want_loss, want_dl = O.cross_entropy(logits.astype(np.float64), labels, n_valid)
    assert abs(loss - want_loss) / want_loss < 1e-5
    tol = 1e-5 if dtype == 0 else 6e-3
    assert np.abs(dl[:, :V] - want_dl).max() / np.abs(want_dl).max() < tol
    assert np.all(dl[:, V:] == 0)                  # padding columns are cleared
    assert np.all(dl[labels < 0] == 0)             # ignored rows carry no gradient
    # no valid row at all: loss 0, zero gradient
    loss, dl = run_cross_entropy(Bd.mslt_op_cross_entropy, dtype, logits, np.full(R, -1), V, scratch=scratch)
    assert loss == 0.0 and not dl.any()
    # loss only
    loss, _ = run_cross_entropy(Bd.mslt_op_cross_entropy, dtype, logits, labels, V, want_grad=False,
                                scratch=scratch)
    assert abs(loss - want_loss) / want_loss < 1e-5


def _t(x, dtype):
    import torch
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda().to(
        torch.bfloat16 if dtype == 1 else torch.float32)


def _stream():
    import torch
    return torch.cuda.current_stream().cuda_stream


@pytest.mark.parametrize("dtype", [0, 1], ids=["fp32", "bf16"])
@pytest.mark.parametrize("rows,H", [(5, 128), (37, 192), (130, 768), (64, 1024), (9, 320)])
def test_layernorm_forward_and_backward_match_oracle(dtype, rows, H):
    import torch
    from paper_2011_13635_b200 import binding as Bd
    rng = np.random.default_rng(rows * H)
    z = _t(rng.standard_normal((rows, H)) * 2 + 0.5, dtype)
    gamma = (1 + 0.1 * rng.standard_normal(H)).astype(np.float32)
    beta = (0.1 * rng.standard_normal(H)).astype(np.float32)
    dy = _t(rng.standard_normal((rows, H)), dtype)
    d_g, d_b = torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda()
    y = torch.empty_like(z)
    stats = torch.empty((rows, 2), device="cuda")
    Bd.mslt_op_layernorm(z, d_g, d_b, y, stats, 1e-12, _stream())
    z64, dy64 = z.double().cpu().numpy(), dy.double().cpu().numpy()
    y_ref, xhat, rstd = O.layer_norm(z64, gamma.astype(np.float64), beta.astype(np.float64), 1e-12)
    tol = 2e-5 if dtype == 0 else 6e-3
    assert np.abs(y.double().cpu().numpy() - y_ref).max() / np.abs(y_ref).max() < tol
    st = stats.cpu().numpy()
    np.testing.assert_allclose(st[:, 0], z64.mean(-1), atol=1e-5)
    np.testing.assert_allclose(st[:, 1], rstd[:, 0], rtol=1e-5)
    # without statistics (frozen layers)
    y2 = torch.empty_like(z)
    Bd.mslt_op_layernorm(z, d_g, d_b, y2, None, 1e-12, _stream())
    assert torch.equal(y, y2)
    # backward
    dz = torch.empty_like(z)
    dgam = torch.zeros(H, device="cuda"); dbet = torch.zeros(H, device="cuda")
    dbias = torch.zeros(H, device="cuda")
    Bd.mslt_op_layernorm_bwd(dy, z, stats, d_g, dz, dgam, dbet, _stream(), dbias=dbias)
    dz_ref, dg_ref, db_ref = O.layer_norm_backward(dy64, xhat, rstd, gamma.astype(np.float64))
    assert np.abs(dz.double().cpu().numpy() - dz_ref).max() / np.abs(dz_ref).max() < tol
    # the fused bias gradient: column sums of dz (they nearly cancel within a row, so compare
    # against the size of dz rather than of the sums)
    assert np.abs(dbias.cpu().numpy() - dz_ref.sum(axis=0)).max() < (1e-4 if dtype == 0 else 2e-2) * np.abs(dz_ref).max() * np.sqrt(dz_ref.shape[0])
    assert np.abs(dgam.cpu().numpy() - dg_ref).max() / np.abs(dg_ref).max() < 1e-4
    assert np.abs(dbet.cpu().numpy() - db_ref).max() / np.abs(db_ref).max() < 1e-4
    # the column sums are accumulated: a second call doubles them
    Bd.mslt_op_layernorm_bwd(dy, z, stats, d_g, dz, dgam, dbet, _stream())
    assert np.abs(dbet.cpu().numpy() - 2 * db_ref).max() / np.abs(db_ref).max() < 2e-4


@pytest.mark.parametrize("dtype", [0, 1], ids=["fp32", "bf16"])
@pytest.mark.parametrize("S", [8, 64, 72, 128, 512])
def test_softmax_forward_and_backward_match_oracle(dtype, S):
    import torch
    from paper_2011_13635_b200 import binding as Bd
    B, A = 3, 2
    rng = np.random.default_rng(S)
    sc = _t(rng.standard_normal((B * A * S, S)) * 3, dtype)
    lens = np.array([S, max(1, S // 3), 1], dtype=np.int32)
    d_lens = torch.from_numpy(lens).cuda()
    p = torch.empty_like(sc)
    Bd.mslt_op_softmax(sc, p, d_lens, A * S, 0.125, _stream())
    sc64 = sc.double().cpu().numpy().reshape(B, A, S, S)
    p_ref = O.masked_softmax(sc64 * 0.125, lens).reshape(B * A * S, S)
    got = p.double().cpu().numpy()
    tol = 2e-6 if dtype == 0 else 4e-3
    assert np.abs(got - p_ref).max() < tol
    assert np.all(got[p_ref == 0] == 0)
    # in place
    sc2 = sc.clone()
    Bd.mslt_op_softmax(sc2, sc2, d_lens, A * S, 0.125, _stream())
    assert torch.equal(sc2, p)
    # backward
    dp = _t(rng.standard_normal((B * A * S, S)), dtype)
    dp64 = dp.double().cpu().numpy()
    ref = O.softmax_backward(dp64, got) * 0.125
    Bd.mslt_op_softmax_bwd(dp, p, 0.125, _stream())
    assert np.abs(dp.double().cpu().numpy() - ref).max() / np.abs(ref).max() < (2e-5 if dtype == 0 else 6e-3)


@pytest.mark.parametrize("dtype", [0, 1], ids=["fp32", "bf16"])
@pytest.mark.parametrize("rows,N,ld", [(7, 8, 8), (300, 768, 768), (1000, 1040, 1048), (64, 30528, 30528)])
def test_colsum_matches_numpy(dtype, rows, N, ld):
    import torch
    from paper_2011_13635_b200 import binding as Bd
    rng = np.random.default_rng(rows + N)
    x = _t(rng.standard_normal((rows, ld)), dtype)
    out = torch.full((ld,), 0.5, device="cuda")
    Bd.mslt_op_colsum(x, N, out, _stream())
    ref = 0.5 + x.double().cpu().numpy()[:, :N].sum(0)
    got = out.cpu().numpy()
    assert np.abs(got[:N] - ref).max() < 1e-4 * max(1.0, np.abs(ref).max())
    assert np.all(got[N:] == 0.5)                   # nothing past N is touched


def test_op_argument_checks():
    import torch
    from paper_2011_13635_b200 import binding as Bd
    z = torch.zeros((4, 100), device="cuda")        # row length not a multiple of 8
    g = torch.zeros(100, device="cuda")
    with pytest.raises(Bd.MsltError) as ei:
        Bd.mslt_op_layernorm(z, g, g, z, None, 1e-12, _stream())
    assert ei.value.code == -1
    s = torch.zeros((4, 1024), device="cuda")       # row longer than the softmax kernels hold
    with pytest.raises(Bd.MsltError) as ei:
        Bd.mslt_op_softmax(s, s, None, 4, 1.0, _stream())
    assert ei.value.code == -1


@pytest.mark.parametrize("B,S,A,masked", [(2, 128, 2, False), (3, 128, 12, True), (2, 100, 3, True),
                                          (5, 64, 2, True), (1, 24, 1, False), (37, 128, 12, True),
                                          (2, 256, 2, False), (3, 512, 4, True), (2, 384, 3, True),
                                          (3, 200, 2, True), (40, 512, 16, True), (1, 136, 1, False)])
@pytest.mark.parametrize("want_probs", [True, False], ids=["probs", "noprobs"])
def test_fused_attention_matches_oracle(B, S, A, masked, want_probs):
    """Scores, masked softmax and context in one kernel against the oracle's definition
    (einsum, masked_softmax, einsum) on the same bf16-rounded inputs."""
    import math
    import torch
    from paper_2011_13635_b200 import binding as Bd
    d, H = 64, A * 64
    rng = np.random.default_rng(B * 1000 + S + A)
    qkv = torch.from_numpy((rng.standard_normal((B * S, 3 * H)) * 1.5).astype(np.float32)).cuda().bfloat16()
    lens = rng.integers(1, S + 1, size=B).astype(np.int32) if masked else np.full(B, S, np.int32)
    if masked:
        lens[0] = S
        lens[-1] = 1 if B > 1 else S
    d_lens = torch.from_numpy(lens).cuda() if masked else None
    probs = torch.full((B, A, S, S), 7.0, device="cuda", dtype=torch.bfloat16) if want_probs else None
    ctx = torch.full((B * S, H), 7.0, device="cuda", dtype=torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    scale = 1.0 / math.sqrt(d)
    for _ in range(2):   # twice: the second call must not depend on what the first left behind
        Bd.mslt_op_attention(qkv, probs, ctx, d_lens, B, S, A, scale, status, _stream())
    assert int(status.item()) == 0
    x = qkv.float().cpu().numpy().astype(np.float64).reshape(B, S, 3, A, d)
    q, k, v = (x[:, :, i].transpose(0, 2, 1, 3) for i in range(3))          # [B, A, S, d]
    p_ref = O.masked_softmax(np.einsum("bhid,bhjd->bhij", q, k) * scale, lens)
    c_ref = np.einsum("bhij,bhjd->bhid", p_ref, v).transpose(0, 2, 1, 3).reshape(B * S, H)
    if want_probs:
        got = probs.float().cpu().numpy()
        for b in range(B):
            # rows at padded query positions are unspecified (a long-row kernel skips tiles of them)
            assert np.abs(got[b, :, :lens[b]] - p_ref[b, :, :lens[b]]).max() < 6e-3   # bf16 resolution at p <= 1
            assert not got[b, :, :, lens[b]:].any()                          # masked keys exactly 0
            assert np.isfinite(got[b]).all()
    # rows at padded query positions are unspecified: compare valid rows only
    got = ctx.float().cpu().numpy().reshape(B, S, H)
    assert np.isfinite(got).all()                                            # padded rows too: later layers read them
    ref = c_ref.reshape(B, S, H)
    for b in range(B):
        err = np.abs(got[b, :lens[b]] - ref[b, :lens[b]]).max()
        assert err / np.abs(ref[b, :lens[b]]).max() < 1.5e-2, (b, err)


def test_fused_attention_rejects_other_shapes():
    import torch
    from paper_2011_13635_b200 import binding as Bd
    qkv = torch.zeros((256, 192), device="cuda", dtype=torch.bfloat16)
    ctx = torch.zeros((256, 64), device="cuda", dtype=torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(Bd.MsltError):
        Bd.mslt_op_attention(qkv, None, ctx, None, 1, 1024, 1, 0.125, status, _stream())
    with pytest.raises(Bd.MsltError):
        Bd.mslt_op_attention(qkv, None, ctx, None, 0, 128, 1, 0.125, status, _stream())


@pytest.mark.parametrize("B,S,A,masked", [(2, 128, 2, False), (3, 128, 12, True), (2, 104, 3, True),
                                          (5, 64, 2, True), (1, 24, 1, False), (37, 128, 12, True)])
def test_fused_attention_backward_matches_oracle(B, S, A, masked):
    """dQ, dK, dV of one kernel against the reverse-mode formulas written with the oracle's
    softmax_backward, on the same bf16-rounded inputs (probabilities from the oracle's softmax)."""
    import math
    import torch
    from paper_2011_13635_b200 import binding as Bd
    d, H = 64, A * 64
    rng = np.random.default_rng(B * 977 + S + A)
    bf = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda().bfloat16()
    qkv = bf(rng.standard_normal((B * S, 3 * H)) * 1.5)
    dctx = bf(rng.standard_normal((B * S, H)))
    lens = rng.integers(1, S + 1, size=B).astype(np.int32) if masked else np.full(B, S, np.int32)
    scale = 1.0 / math.sqrt(d)
    x = qkv.float().cpu().numpy().astype(np.float64).reshape(B, S, 3, A, d)
    q, k, v = (x[:, :, i].transpose(0, 2, 1, 3) for i in range(3))            # [B, A, S, d]
    probs = bf(O.masked_softmax(np.einsum("bhid,bhjd->bhij", q, k) * scale, lens))
    p = probs.float().cpu().numpy().astype(np.float64)
    dc = dctx.float().cpu().numpy().astype(np.float64).reshape(B, S, A, d).transpose(0, 2, 1, 3)
    dv = np.einsum("bhij,bhid->bhjd", p, dc)
    ds = O.softmax_backward(np.einsum("bhid,bhjd->bhij", dc, v), p) * scale
    dq = np.einsum("bhij,bhjd->bhid", ds, k)
    dk = np.einsum("bhij,bhid->bhjd", ds, q)
    want = np.stack([dq, dk, dv], axis=0).transpose(1, 3, 0, 2, 4).reshape(B * S, 3 * H)   # [B,S,3,A,d]
    dqkv = torch.full((B * S, 3 * H), 7.0, device="cuda", dtype=torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for _ in range(2):
        Bd.mslt_op_attention_bwd(qkv, probs, dctx, dqkv, B, S, A, scale, status, _stream())
    assert int(status.item()) == 0
    got = dqkv.float().cpu().numpy().reshape(B, S, 3, H)
    want = want.reshape(B, S, 3, H)
    for which, name in enumerate(("dq", "dk", "dv")):
        err = np.abs(got[:, :, which] - want[:, :, which]).max() / np.abs(want[:, :, which]).max()
        assert err < 1.5e-2, (name, err)


@pytest.mark.parametrize("which", ["forward", "forward_long_rows", "backward"])
def test_attention_wait_that_runs_out_is_reported_and_leaves_the_device_usable(which):
    """Every wait in the attention kernels is bounded.  With the test hook armed the next launch has
    an idle producer and a 20 ms limit: the kernel must come back with the status bit set (no
    fault, no hang), and the very next call must work and be correct again."""
    import math
    import torch
    from paper_2011_13635_b200 import binding as Bd
    B, A = 2, 2
    S = 256 if which == "forward_long_rows" else 128
    H = A * 64
    rng = np.random.default_rng(5)
    qkv = torch.from_numpy(rng.standard_normal((B * S, 3 * H)).astype(np.float32)).cuda().bfloat16()
    ctx = torch.zeros((B * S, H), device="cuda", dtype=torch.bfloat16)
    probs = torch.zeros((B, A, S, S), device="cuda", dtype=torch.bfloat16)
    dqkv = torch.zeros((B * S, 3 * H), device="cuda", dtype=torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    scale = 1.0 / math.sqrt(64)

    def call():
        if which == "backward":
            Bd.mslt_op_attention_bwd(qkv, probs, ctx, dqkv, B, S, A, scale, status, _stream())
        else:
            Bd.mslt_op_attention(qkv, probs, ctx, None, B, S, A, scale, status, _stream())

    Bd.lib.mslt_debug_starve_next_attention(1)
    with pytest.raises(Bd.MsltError) as ei:
        call()
    assert ei.value.code == -5
    assert int(status.item()) & 1
    status.zero_()
    Bd.mslt_op_attention(qkv, probs, ctx, None, B, S, A, scale, status, _stream())   # disarmed: works again
    assert int(status.item()) == 0
    x = qkv.float().cpu().numpy().astype(np.float64).reshape(B, S, 3, A, 64)
    q, k, v = (x[:, :, i].transpose(0, 2, 1, 3) for i in range(3))
    p_ref = O.masked_softmax(np.einsum("bhid,bhjd->bhij", q, k) * scale, np.full(B, S))
    c_ref = np.einsum("bhij,bhjd->bhid", p_ref, v).transpose(0, 2, 1, 3).reshape(B * S, H)
    assert np.abs(ctx.float().cpu().numpy() - c_ref).max() / np.abs(c_ref).max() < 1.5e-2
    if which == "backward":
        call()
        assert int(status.item()) == 0
