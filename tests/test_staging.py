"""Stage hand-over, invariants and error paths of the C ABI on the GPU."""
import numpy as np
import pytest

from oracle import mslt_oracle as O
from paper_2011_13635_b200 import inputs as I
from tests import parity as PT

pytestmark = pytest.mark.gpu

CFG32 = I.StageConfig("stage32", hidden=128, heads=2, ffn=256, vocab=515, max_pos=64, layers=4,
                      trainable=2, batch=4, seq=32, pred=5, dtype="fp32", varlen=None, seed_index=21)
CFG16 = I.scaled(CFG32, name="stage16", hidden=128, heads=2, dtype="bf16", seed_index=22)


@pytest.mark.parametrize("cfg", [CFG32, CFG16], ids=["fp32", "bf16"])
def test_schedule_of_stages_matches_oracle(cfg):
    """Stage 1 trains 2 layers with everything trainable; 2 layers are stacked by copy; stage 2
    trains only the new layers and the output layer; joint retraining trains all again."""
    import torch
    lr = 1e-3 if cfg.dtype == "fp32" else 1e-4
    m, oracle = PT.build_pair(cfg, lr=lr, init_layers=2, max_layers=4)
    tol = PT.TOL[cfg.dtype]
    assert m.num_layers == 2 and m.num_trainable == 2
    seed = I.config_seed(cfg)
    for s in range(2):
        PT.compare_step(m, oracle, cfg, I.make_batch(cfg, seed=seed + s), tol)
    # stacking: new layers are byte copies of the previous top layers, in order
    m.mslt_add_layers(2)
    oracle.add_layers(2)
    assert m.num_layers == 4
    for t in O.LAYER_TENSORS:
        for i in (0, 1):
            assert np.array_equal(m.mslt_get_param(f"layer.{2 + i}.{t}"), m.mslt_get_param(f"layer.{i}.{t}"))
            assert np.array_equal(m.mslt_get_param_raw(f"layer.{2 + i}.{t}"),
                                  m.mslt_get_param_raw(f"layer.{i}.{t}"))
    m.mslt_set_trainable(2)
    oracle.set_trainable(2)
    info = m.tensors()
    assert not info["emb.word"]["trainable"] and not info["layer.1.qkv.weight"]["trainable"]
    assert info["layer.2.qkv.weight"]["trainable"] and info["head.decoder.bias"]["trainable"]
    # optimizer state starts again from zero
    assert not m.mslt_get_opt_state("layer.3.ffn1.weight", 0).any()
    for s in range(2, 4):
        PT.compare_step(m, oracle, cfg, I.make_batch(cfg, seed=seed + s), tol)
    # joint retraining
    m.mslt_set_trainable(4)
    oracle.set_trainable(4)
    PT.compare_step(m, oracle, cfg, I.make_batch(cfg, seed=seed + 9), tol)
    with pytest.raises(Exception) as ei:
        m.mslt_add_layers(1)                    # arena full
    assert ei.value.code == -3
    m.close()


@pytest.mark.parametrize("cfg", [CFG32, CFG16], ids=["fp32", "bf16"])
def test_grouped_parameter_sharing_schedule_matches_oracle(cfg):
    """Section 3.3: layers of a group share one parameter block; a stage adds a group and trains only
    that group and the output layer; the shared block's gradient is the sum over its layers."""
    from paper_2011_13635_b200 import binding as Bd
    cfg = I.scaled(cfg, share_group=2)
    lr = 1e-3 if cfg.dtype == "fp32" else 1e-4
    tol = PT.TOL[cfg.dtype]
    m, oracle = PT.build_pair(cfg, lr=lr, init_layers=2, max_layers=4)
    assert m.num_layers == 2 and len([n for n in m.tensors() if n.startswith("layer.")]) == 12   # one block
    seed = I.config_seed(cfg)
    PT.compare_step(m, oracle, cfg, I.make_batch(cfg, seed=seed), tol)            # both layers feed block 0
    with pytest.raises(Bd.MsltError) as ei:
        m.mslt_add_layers(1)
    assert ei.value.code == -3
    m.mslt_add_layers(2)
    oracle.add_layers(2)
    assert m.num_layers == 4
    assert np.array_equal(m.mslt_get_param("layer.1.ffn2.weight"), m.mslt_get_param("layer.0.ffn2.weight"))
    with pytest.raises(Bd.MsltError) as ei:
        m.mslt_set_trainable(1)
    assert ei.value.code == -3
    m.mslt_set_trainable(2)
    oracle.set_trainable(2)
    info = m.tensors()
    assert info["layer.1.qkv.weight"]["trainable"] and not info["layer.0.qkv.weight"]["trainable"]
    for s in (1, 2):
        PT.compare_step(m, oracle, cfg, I.make_batch(cfg, seed=seed + s), tol)
    assert len(m.grad_buckets()) == 2                                              # output layer + one group
    m.mslt_set_trainable(4)
    oracle.set_trainable(4)
    PT.compare_step(m, oracle, cfg, I.make_batch(cfg, seed=seed + 3), tol)
    m.close()


@pytest.mark.parametrize("cfg", [CFG32, CFG16], ids=["fp32", "bf16"])
def test_saved_activation_slots_only_for_the_trainable_layers(cfg):
    """A context sized for two trainable layers out of four: smaller workspace, same results, and a
    request for more trainable layers than it has slots for is refused."""
    from paper_2011_13635_b200 import binding as Bd
    lr = 1e-3 if cfg.dtype == "fp32" else 1e-4
    m, oracle = PT.build_pair(cfg, lr=lr, max_trainable=2)
    assert m.num_layers == 4 and m.num_trainable == 2
    full_ws = Bd.mslt_query_bytes(Bd.Arch(cfg.hidden, cfg.heads, cfg.ffn, cfg.vocab, cfg.max_pos, 4, 4, cfg.batch,
                                          cfg.seq, cfg.pred, 0 if cfg.dtype == "fp32" else 1, 1e-12, 0))[1]
    assert m.workspace_bytes < full_ws
    seed = I.config_seed(cfg)
    for s in range(2):
        PT.compare_step(m, oracle, cfg, I.make_batch(cfg, seed=seed + s), PT.TOL[cfg.dtype])
    m.mslt_set_trainable(1)
    oracle.set_trainable(1)
    PT.compare_step(m, oracle, cfg, I.make_batch(cfg, seed=seed + 2), PT.TOL[cfg.dtype])
    with pytest.raises(Bd.MsltError) as ei:
        m.mslt_set_trainable(3)
    assert ei.value.code == -2 and "max_trainable" in str(ei.value)
    assert m.num_trainable == 1
    m.close()


@pytest.mark.parametrize("cfg", [CFG32, CFG16], ids=["fp32", "bf16"])
def test_truncation_leaves_top_gradients_unchanged(cfg):
    """Gradients of the trainable slice from a staged step equal the same tensors' gradients
    from an all-trainable step at identical weights."""
    import torch
    batch = I.make_batch(cfg)
    grads = {}
    for k in (cfg.layers, 2, 0):
        m, _ = PT.build_pair(I.scaled(cfg, trainable=k), lr=0.0)
        d = PT.to_cuda(torch, batch[0], None, batch[2], batch[3])
        m.mslt_step(*d)
        grads[k] = {n: m.mslt_get_grad(n) for n, i in m.tensors().items() if i["trainable"]}
        m.close()
    tol = 1e-5 if cfg.dtype == "fp32" else 2e-2    # atomics reorder sums; bf16 rounds activations
    for k in (2, 0):
        assert "emb.word" not in grads[k] and "layer.1.qkv.weight" not in grads[k]
        for n, g in grads[k].items():
            assert PT.max_rel(g, grads[cfg.layers][n]) < tol, n


def test_frozen_parameters_stay_bit_identical_over_many_steps():
    import torch
    cfg = CFG16
    m, _ = PT.build_pair(cfg, lr=1e-2)
    before = {n: (m.mslt_get_param(n), m.mslt_get_param_raw(n)) for n in m.tensors()}
    for s in range(10):
        d = PT.to_cuda(torch, *I.make_batch(cfg, seed=100 + s))
        m.mslt_step(d[0], None, d[2], d[3])
    for n, info in m.tensors().items():
        same = np.array_equal(before[n][0], m.mslt_get_param(n))
        same_raw = np.array_equal(before[n][1], m.mslt_get_param_raw(n))
        assert same == (not info["trainable"]), n
        assert same_raw == (not info["trainable"]), n
    m.close()


def test_padding_content_does_not_matter():
    import torch
    cfg = I.scaled(CFG32, varlen=(9, 32), trainable=4)
    tok, lens, pos, lab = I.make_batch(cfg)
    tok2 = tok.copy()
    for b in range(cfg.batch):
        tok2[b, lens[b]:] = 7
    out = []
    for t in (tok, tok2):
        m, _ = PT.build_pair(cfg, lr=0.0)
        d = PT.to_cuda(torch, t, lens, pos, lab)
        loss = m.mslt_step(*d)
        out.append((loss, m.mslt_get_grad("layer.0.qkv.weight"), m.mslt_get_grad("emb.pos")))
        m.close()
    assert abs(out[0][0] - out[1][0]) < 1e-6
    assert PT.max_rel(out[0][1], out[1][1]) < 1e-5
    assert PT.max_rel(out[0][2], out[1][2]) < 1e-5


def test_error_paths_return_codes():
    import torch
    from paper_2011_13635_b200.binding import Mslt, MsltError
    cfg = CFG32
    with pytest.raises(MsltError) as ei:
        Mslt.from_config(I.scaled(cfg, hidden=100))
    assert ei.value.code == -1
    with pytest.raises(MsltError) as ei:
        Mslt.from_config(I.scaled(cfg, dtype="bf16", heads=4))       # head dim 32 on the bf16 path
    assert ei.value.code == -1
    m, _ = PT.build_pair(cfg, lr=1e-3, init_layers=2, max_layers=4)
    tok, lens, pos, lab = I.make_batch(cfg)
    d_tok, d_pos, d_lab = PT.to_cuda(torch, tok, pos, lab)
    with pytest.raises(MsltError) as ei:
        m.mslt_add_layers(3)                                          # k > L
    assert ei.value.code == -3
    with pytest.raises(MsltError) as ei:
        m.mslt_set_trainable(3)                                       # top_k > L
    assert ei.value.code == -3
    big = torch.zeros((cfg.batch + 1, cfg.seq), dtype=torch.int32, device="cuda")
    with pytest.raises(MsltError) as ei:
        m.mslt_step(big, None, d_pos, d_lab)                          # batch beyond capacity
    assert ei.value.code == -2
    with pytest.raises(MsltError) as ei:
        m.mslt_get_grad("layer.3.qkv.weight")                         # layer not present
    assert ei.value.code == -1
    bad = d_tok.clone()
    bad[0, 0] = cfg.vocab + 5
    with pytest.raises(MsltError) as ei:
        m.mslt_step(bad, None, d_pos, d_lab)                          # token id out of range
    assert ei.value.code == -5
    badp = d_pos.clone()
    badp[0, 0] = cfg.seq
    with pytest.raises(MsltError) as ei:
        m.mslt_step(d_tok, None, badp, d_lab)                         # MLM position out of range
    assert ei.value.code == -5
    # the context is still usable afterwards
    loss = m.mslt_step(d_tok, None, d_pos, d_lab)
    assert np.isfinite(loss)
    # no valid slot: loss 0, head gradients 0
    none = torch.full_like(d_lab, -1)
    assert m.mslt_step(d_tok, None, d_pos, none) == 0.0
    assert not m.mslt_get_grad("head.transform.weight").any()
    m.close()


def test_captured_step_replays_like_eager_steps():
    """mslt_step without loss read-back only enqueues work, so it can be captured in a CUDA graph:
    replays advance Adam's step count on the device and match eagerly launched steps."""
    import torch
    cfg = CFG16
    tok, lens, pos, lab = I.make_batch(cfg)
    res = []
    for use_graph in (False, True):
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            from paper_2011_13635_b200.binding import Mslt
            m = Mslt.from_config(cfg, stream=stream)
            m.set_params(I.make_weights(cfg, variant="parity"))
            m.mslt_set_trainable(cfg.trainable)
            m.mslt_set_optimizer(lr=1e-3)
            d = PT.to_cuda(torch, tok, pos, lab)
            m.mslt_step(d[0], None, d[1], d[2])                 # step 1, eager on both sides
            if use_graph:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    m.mslt_step(d[0], None, d[1], d[2], sync=False)
                g.replay(); g.replay()                          # steps 2 and 3 (capture runs nothing)
            else:
                for _ in range(2):
                    m.mslt_step(d[0], None, d[1], d[2], sync=False)
            loss = m.mslt_read_loss()
            res.append((loss, m.mslt_get_param("layer.3.ffn1.weight"), m.mslt_get_opt_state("head.ln.gamma", 1)))
            m.close()
    (l0, w0, v0), (l1, w1, v1) = res
    assert abs(l0 - l1) < 1e-3 * abs(l0)
    assert PT.max_rel(w1, w0) < 1e-3                            # atomics reorder sums, nothing more
    assert PT.max_rel(v1, v0) < 1e-2


def test_embedding_gradients_have_the_same_bits_on_every_run():
    """The embedding backward groups rows by token id in a fixed order and sums positions over the
    batch without atomics: two runs of the same all-trainable step give identical bits (fp32 path;
    on the bf16 path the tied decoder's split-k weight gradient, which lands in the same table, is
    summed with vector reductions, so only the position table is compared there)."""
    import torch
    for cfg in (I.scaled(CFG32, trainable=4), I.scaled(CFG16, trainable=4)):
        got = []
        for _ in range(2):
            m, _ = PT.build_pair(cfg, lr=1e-3)
            d = PT.to_cuda(torch, *I.make_batch(cfg))
            m.mslt_step(d[0], None, d[2], d[3])
            got.append((m.mslt_get_grad("emb.pos"), m.mslt_get_grad("emb.word")))
            m.close()
        assert np.array_equal(got[0][0], got[1][0])
        assert np.abs(got[0][0]).max() > 0
        if cfg.dtype == "fp32":
            assert np.array_equal(got[0][1], got[1][1])
