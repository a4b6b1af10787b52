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
