"""CPU-side checks of the boundary: the shared library loads, exports every symbol the header
declares, validates arguments on the host, and refuses to compute without a CUDA device."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2011_13635_b200 import build
    build.build()
    from paper_2011_13635_b200 import binding as Bd
    return Bd


def test_every_declared_symbol_is_exported(binding):
    header = open(os.path.join(ROOT, "include", "mslt.h")).read()
    declared = set(re.findall(r"\b(mslt_[a-z_0-9]+)\s*\(", header))
    assert {"mslt_create", "mslt_add_layers", "mslt_set_trainable", "mslt_step", "mslt_forward"} <= declared
    for name in declared:
        assert hasattr(binding.lib, name), name
    assert declared == set(binding.EXPORTS)


def test_host_side_validation(binding):
    a = binding.Arch(768, 12, 3072, 30522, 512, 3, 12, 128, 128, 20, 1, 1e-12)
    pb, wb = binding.mslt_query_bytes(a)
    n_params = (30522 * 768 + 512 * 768 + 2 * 768) + 12 * (12 * 768 * 768 + 13 * 768) + (768 * 768 + 3 * 768 + 30522)
    assert 18 * n_params <= pb <= 18 * n_params * 1.001
    assert wb > 12 * 16 * 128 * 128 * 768 * 2          # saved activations of 12 trainable layers
    for field, bad in [("hidden", 100), ("heads", 7), ("max_seq", 1000), ("dtype", 3), ("init_layers", 0),
                       ("max_layers", 2), ("max_pos", 64), ("ffn", 100)]:
        b = binding.Arch(768, 12, 3072, 30522, 512, 3, 12, 128, 128, 20, 1, 1e-12)
        setattr(b, field, bad)
        with pytest.raises(binding.MsltError) as ei:
            binding.mslt_query_bytes(b)
        assert ei.value.code == -1, field
    # saved activations are reserved for the layers that can be trainable at once: 9 + 3 needs 3 slots
    a3 = binding.Arch(768, 12, 3072, 30522, 512, 3, 12, 128, 128, 20, 1, 1e-12, 3)
    pb3, wb3 = binding.mslt_query_bytes(a3)
    T, H, F, A, S = 128 * 128, 768, 3072, 12, 128
    slot = 2 * (3 * T * H + 128 * A * S * S + 5 * T * H + 2 * T * F)      # bf16 bytes of one layer's slot
    assert pb3 == pb
    assert 9 * slot <= wb - wb3 <= 9 * slot * 1.01
    assert wb3 < 0.45 * wb
    a3.max_trainable = 13
    with pytest.raises(binding.MsltError) as ei:
        binding.mslt_query_bytes(a3)
    assert ei.value.code == -1
    # fp32 path has no bf16 copy
    a32 = binding.Arch(128, 2, 512, 1024, 64, 2, 2, 8, 64, 10, 0, 1e-12)
    pb32, _ = binding.mslt_query_bytes(a32)
    assert pb32 % 16 == 0


def test_no_cpu_path(binding):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    a = binding.Arch(128, 2, 512, 1024, 64, 2, 2, 8, 64, 10, 0, 1e-12)
    buf = (C.c_char * 4096)()
    addr = (C.addressof(buf) + 255) // 256 * 256
    h = C.c_void_p()
    rc = binding.lib.mslt_create(C.byref(a), addr, 1 << 40, addr, 1 << 40, None, C.byref(h))
    assert rc == -4 and b"no CUDA device" in binding.lib.mslt_last_error(None)
    d = binding.GemmDesc()
    d.dtype, d.M, d.N, d.K, d.batch, d.hdiv = 0, 8, 8, 8, 1, 1
    d.A = d.B = d.D = addr
    d.a_rs, d.a_ks, d.b_rs, d.b_ks, d.ldd = 8, 1, 8, 1, 8
    assert binding.lib.mslt_op_gemm(C.byref(d), None, None) == -4
    with pytest.raises(binding.MsltError):
        binding.Mslt(hidden=128, heads=2, ffn=512, vocab=1024, max_pos=64, init_layers=2, max_layers=2,
                     max_batch=8, max_seq=64, max_pred=10, dtype="fp32")
