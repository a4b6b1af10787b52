"""GPU parity of the whole stage step against the CPU oracle, element by element, through the
C ABI.  Sizes are chosen so that the oracle finishes in seconds while the contractions still
span several tiles and ragged tails."""
import math

import numpy as np
import pytest

from paper_2011_13635_b200 import inputs as I
from tests import parity as PT

pytestmark = pytest.mark.gpu

TINY = I.CONFIGS["tiny"]


def _run(cfg, steps, lr, batch_seed=None, **opt):
    m, oracle = PT.build_pair(cfg, lr=lr, **opt)
    tol = PT.TOL[cfg.dtype]
    rep = []
    for s in range(steps):
        batch = I.make_batch(cfg, seed=(batch_seed or I.config_seed(cfg)) + s)
        PT.compare_step(m, oracle, cfg, batch, tol, rep)
    m.close()
    return rep


# -- fp32 path -------------------------------------------------------------------------------

def test_tiny_fp32_staged_step():
    """The small configuration as given: 1 frozen + 1 trainable layer, fp32."""
    rep = _run(TINY, steps=3, lr=1e-3)
    assert abs(rep[0]["loss_gpu"] - math.log(TINY.vocab)) < 0.2


@pytest.mark.parametrize("top_k", [0, 2])
def test_fp32_head_only_and_all_trainable(top_k):
    _run(I.scaled(TINY, trainable=top_k), steps=2, lr=1e-3)


def test_fp32_ragged_shapes_with_padding():
    cfg = I.StageConfig("ragged32", hidden=192, heads=3, ffn=320, vocab=1037, max_pos=80, layers=3,
                        trainable=2, batch=3, seq=72, pred=7, dtype="fp32", varlen=(20, 72),
                        seed_index=11)
    _run(cfg, steps=2, lr=1e-3)
    _run(I.scaled(cfg, trainable=3), steps=2, lr=1e-3)


def test_fp32_lamb_staged_and_all_trainable():
    """LAMB at the learning rate of the paper's experiments (Section 4.1): per-tensor trust ratios."""
    _run(TINY, steps=3, lr=0.00088, lamb=1)
    _run(I.scaled(TINY, trainable=2), steps=2, lr=0.00088, lamb=1, weight_decay=0.0)


def _run_nsp(cfg, steps, lr, drop_labels=False):
    """Both objectives (Section 4.1): segment embeddings, pooler and two-way classifier."""
    m, oracle = PT.build_pair(cfg, lr=lr)
    assert oracle.nsp and "emb.type" in m.tensors() and "head.nsp.weight" in m.tensors()
    rep = []
    for s in range(steps):
        seed = I.config_seed(cfg) + s
        tok, lens, pos, lab = I.make_batch(cfg, seed=seed)
        seg, nlab = I.make_nsp(cfg, lens, seed=seed)
        if s == 1:
            nlab[0] = -1                               # an ignored sequence
        PT.compare_step(m, oracle, cfg, (tok, lens, pos, lab, seg, None if drop_labels else nlab),
                        PT.TOL[cfg.dtype], rep)
    m.close()
    return rep


def test_fp32_nsp_objective_staged_and_all_trainable():
    cfg = I.scaled(TINY, nsp=True, varlen=(20, 64))
    rep = _run_nsp(cfg, steps=2, lr=1e-3)
    assert abs(rep[0]["loss_gpu"] - (math.log(cfg.vocab) + math.log(2))) < 0.3      # MLM + NSP at the start
    _run_nsp(I.scaled(cfg, trainable=2), steps=2, lr=1e-3)
    rep = _run_nsp(cfg, steps=1, lr=1e-3, drop_labels=True)                         # segments only
    assert abs(rep[0]["loss_gpu"] - math.log(cfg.vocab)) < 0.2


# -- bf16 path ---------------------------------------------------------------------------------

BASE_SMALL = I.scaled(I.CONFIGS["base_stage"], layers=3, trainable=2, batch=4)


def test_bf16_base_shapes_staged():
    """BERT-Base widths and vocabulary, 1 frozen + 2 trainable layers, 4 sequences of 128."""
    rep = _run(BASE_SMALL, steps=2, lr=1e-4)
    assert abs(rep[0]["loss_gpu"] - math.log(30522)) < 0.3


def test_bf16_base_shapes_all_trainable():
    _run(I.scaled(BASE_SMALL, layers=2, trainable=2, batch=3), steps=2, lr=1e-4)


def test_bf16_lamb_base_shapes():
    _run(BASE_SMALL, steps=2, lr=0.00088, lamb=1)
    _run(I.scaled(BASE_SMALL, layers=2, trainable=2, batch=2), steps=1, lr=0.00088, lamb=1)


def test_bf16_nsp_objective_base_shapes():
    cfg = I.scaled(BASE_SMALL, nsp=True)
    _run_nsp(cfg, steps=2, lr=1e-4)
    _run_nsp(I.scaled(cfg, layers=2, trainable=2, batch=3), steps=1, lr=1e-4)


def test_bf16_head_only():
    _run(I.scaled(BASE_SMALL, layers=1, trainable=0, batch=2), steps=1, lr=1e-4)


def test_bf16_ragged_shapes_with_padding():
    cfg = I.StageConfig("ragged16", hidden=192, heads=3, ffn=320, vocab=1037, max_pos=80, layers=2,
                        trainable=1, batch=3, seq=72, pred=7, dtype="bf16", varlen=(20, 72),
                        seed_index=12)
    _run(cfg, steps=2, lr=1e-4)
    _run(I.scaled(cfg, trainable=2), steps=1, lr=1e-4)


def test_bf16_large_long_shapes():
    """BERT-Large widths at sequence length 512 with per-sequence padding."""
    cfg = I.scaled(I.CONFIGS["large_long"], layers=2, trainable=1, batch=2)
    _run(cfg, steps=1, lr=1e-4)


# -- forward-only entry point ----------------------------------------------------------------------

@pytest.mark.parametrize("cfg", [TINY, I.scaled(BASE_SMALL, batch=2),
                                 I.scaled(I.CONFIGS["large_long"], layers=2, trainable=1, batch=2)],
                         ids=["tiny", "base", "large_long"])
def test_forward_matches_oracle(cfg):
    import torch
    m, oracle = PT.build_pair(cfg, lr=1e-3)
    tok, lens, pos, lab = I.make_batch(cfg)
    d_tok, d_lens, d_pos = PT.to_cuda(torch, tok, lens if cfg.varlen else None, pos)
    hidden, logits = m.mslt_forward(d_tok, d_lens, d_pos)
    h_ref, l_ref = oracle.forward(tok, lens, pos)
    hidden = hidden.float().cpu().numpy()
    tol = PT.TOL[cfg.dtype]["hidden"]
    for b in range(cfg.batch):       # rows at padded positions are unspecified
        n = int(lens[b])
        assert PT.max_rel(hidden[b, :n], h_ref[b, :n]) < tol
    ok = (pos >= 0).reshape(-1)
    lg = logits.cpu().numpy()
    assert PT.max_rel(lg[ok], l_ref[ok]) < tol
    # the loss recomputed from these logits equals the loss the training step reports
    labels = np.where(ok, lab.reshape(-1), -1)
    lg64 = lg.astype(np.float64)
    lse = np.log(np.exp(lg64 - lg64.max(1, keepdims=True)).sum(1)) + lg64.max(1)
    nll = (lse - lg64[np.arange(len(labels)), np.maximum(labels, 0)])[ok]
    d_lab = PT.to_cuda(torch, lab)[0]
    m.mslt_set_optimizer(lr=0.0)
    loss = m.mslt_step(d_tok, d_lens, d_pos, d_lab)
    assert abs(loss - nll.mean()) / nll.mean() < 1e-5
    assert m.mslt_debug_check_guards() == 0
    m.close()


def test_bf16_step_with_unfused_attention_in_a_child_process():
    """The batched-product attention path (what longer rows and odd lengths fall back to) is selected
    by an environment switch the library reads once, so it runs in a child process: same parity
    check as above on BERT-Base widths with a padding mask."""
    import os
    import subprocess
    import sys
    code = (
        "import math\n"
        "from paper_2011_13635_b200 import inputs as I\n"
        "from tests import parity as PT\n"
        "cfg = I.scaled(I.CONFIGS['base_stage'], layers=2, trainable=1, batch=3)\n"
        "cfg = I.StageConfig('unfused', hidden=cfg.hidden, heads=cfg.heads, ffn=cfg.ffn, vocab=cfg.vocab,\n"
        "                    max_pos=cfg.max_pos, layers=2, trainable=1, batch=3, seq=128, pred=cfg.pred,\n"
        "                    dtype='bf16', varlen=(40, 128), seed_index=23)\n"
        "m, oracle = PT.build_pair(cfg, lr=1e-4)\n"
        "before = m.launch_count\n"
        "PT.compare_step(m, oracle, cfg, I.make_batch(cfg), PT.TOL[cfg.dtype])\n"
        "print('launches', m.launch_count - before)\n"
        "m.close()\n")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    counts = {}
    for unfused in ("0", "1"):
        env = dict(os.environ, MSLT_UNFUSED_ATTENTION=unfused, PYTHONPATH=root)
        r = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True,
                           timeout=600)
        assert r.returncode == 0, r.stdout + r.stderr
        counts[unfused] = int(r.stdout.strip().split()[-1])
    # two launches per layer forward become three, one per trainable layer backward becomes five
    assert counts["1"] > counts["0"]
