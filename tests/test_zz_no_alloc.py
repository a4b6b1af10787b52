"""The allocation-free loss entry point against the caller-scratch one.

Some users of this library run where device allocation is forbidden (a plugin with a fixed
memory budget, a real-time loop, code holding an allocator lock), so they cannot hand the loss
kernel a scratch buffer.  mslt_op_cross_entropy_noalloc serves them from an array built into the
library.  This file is collected last on purpose: a run that stops at the first failure has then
already exercised everything else.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _both(dtype, R, V, seed):
    import torch
    from paper_2011_13635_b200 import binding as Bd
    from tests.test_ops import run_cross_entropy
    rng = np.random.default_rng(seed)
    logits = (rng.standard_normal((R, V)) * 3).astype(np.float32)
    labels = rng.integers(0, V, size=R)
    labels[::7] = -1
    scratch = torch.empty(Bd.lib.mslt_op_cross_entropy_scratch_bytes(R), dtype=torch.uint8, device="cuda")
    ref = run_cross_entropy(Bd.mslt_op_cross_entropy, dtype, logits, labels, V, scratch=scratch)
    got = run_cross_entropy(Bd.mslt_op_cross_entropy_noalloc, dtype, logits, labels, V)
    from oracle import mslt_oracle as O
    want = O.cross_entropy(logits.astype(np.float64), labels, int((labels >= 0).sum()))
    return ref, got, want


@pytest.mark.parametrize("dtype", [0, 1], ids=["fp32", "bf16"])
def test_noalloc_matches_caller_scratch_on_two_calls_in_a_row(dtype):
    tol = 1e-5 if dtype == 0 else 6e-3           # the tolerances of tests/test_ops.py
    # the second call is smaller than the first: stale scratch from call one must not leak in
    for R, V, seed in ((300, 1037, 1), (64, 30522, 2)):
        (loss_ref, dl_ref), (loss, dl), (loss_o, dl_o) = _both(dtype, R, V, seed)
        assert abs(loss - loss_ref) <= 1e-5 * abs(loss_ref)
        assert np.abs(dl - dl_ref).max() <= tol * np.abs(dl_ref).max()
        # and against the CPU oracle itself
        assert abs(loss - loss_o) <= 1e-5 * abs(loss_o)
        assert np.abs(dl[:, :V] - dl_o).max() <= tol * np.abs(dl_o).max()


def test_noalloc_takes_no_device_memory_after_its_first_call():
    """What the call exists for: once the first call on a device has run (it may load the library
    image and look the built-in array up), later calls leave the free device memory and torch's
    allocator untouched."""
    import torch
    from paper_2011_13635_b200 import binding as Bd
    R, V = 512, 4096
    logits = torch.randn((R, V), device="cuda")
    labels = torch.randint(0, V, (R,), dtype=torch.int32, device="cuda")
    dl = torch.empty((R, V), device="cuda")
    loss = torch.zeros(1, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    Bd.mslt_op_cross_entropy_noalloc(0, logits, labels, V, dl, loss, stream)      # first call: set-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(3):
        Bd.mslt_op_cross_entropy_noalloc(0, logits, labels, V, dl, loss, stream)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, (free0, free1)
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (alloc0, reserved0)


def test_noalloc_rejects_sizes_beyond_its_scratch():
    import torch
    from paper_2011_13635_b200 import binding as Bd
    R, V = 16385, 8
    logits = torch.zeros((R, 8), device="cuda")
    labels = torch.zeros(R, dtype=torch.int32, device="cuda")
    loss = torch.zeros(1, device="cuda")
    with pytest.raises(Bd.MsltError) as ei:
        Bd.mslt_op_cross_entropy_noalloc(0, logits, labels, V, None, loss, torch.cuda.current_stream().cuda_stream)
    assert ei.value.code == -2 and "16384" in str(ei.value)
    # the largest supported size works
    Bd.mslt_op_cross_entropy_noalloc(0, logits[:16384], labels[:16384], V, None, loss,
                                     torch.cuda.current_stream().cuda_stream)
    assert abs(float(loss.item()) - np.log(8)) < 1e-5
