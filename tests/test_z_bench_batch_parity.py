"""One whole training step at the launch configuration that bench.py times (BERT-Base stage,
9 frozen + 3 trainable layers, batch 128, sequence length 128), on both sides: loss, every
trainable gradient, the updated weights and the frozen slice against the CPU oracle.

This is the only comparison in which the oracle sees the weight-gradient contractions over all
16384 token rows (automatic split-k with vector reductions) and the 256 x 256 CTA-pair tiles at
128 row tiles.  The oracle needs a few minutes and a few GB for it, so the file is collected late.
"""
import math

import pytest

from paper_2011_13635_b200 import inputs as I
from tests import parity as PT

pytestmark = pytest.mark.gpu


def test_base_stage_batch_128_whole_step_against_the_oracle():
    cfg = I.CONFIGS["base_stage"]
    assert (cfg.batch, cfg.seq, cfg.layers, cfg.trainable) == (128, 128, 12, 3)
    m, oracle = PT.build_pair(cfg, lr=1e-4, max_trainable=cfg.trainable)     # as bench.py creates it
    rep = []
    PT.compare_step(m, oracle, cfg, I.make_batch(cfg), PT.TOL[cfg.dtype], rep)
    r = rep[0]
    print(f"\nbatch-128 step: loss gpu {r['loss_gpu']:.6f} oracle {r['loss_oracle']:.6f}; worst gradient "
          f"{r['grad']}; worst weight {r['weight']}; update mean-abs {r['update']}; update max-abs on clear "
          f"gradients {r['update_max_clear']}, over all elements {r['update_max_all']}")
    assert abs(r["loss_gpu"] - math.log(cfg.vocab)) < 0.5
    m.close()
