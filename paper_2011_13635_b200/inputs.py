"""Seeded synthetic inputs for the MSLT per-stage BERT training step.

This module only draws random numbers and names tensors; it holds none of the
method's arithmetic.  Both the CUDA library's tests/benchmarks and the CPU
oracle's tests are fed from here, so neither side needs the other's code.

The batches stand in for BERT pre-training batches (masked-language-model
objective, 15 % of the positions chosen as targets; Section 4.1 of the paper):
only the shapes, the masking rate, the 128/512 sequence lengths and a
Zipf-like token frequency are reproduced.

Generator: numpy's Philox counter-based bit generator, one stream per
(seed, purpose) pair, so that tokens, masks and weights do not shift when one
of them changes size.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, replace
from typing import Dict, Tuple

import numpy as np

BASE_SEED = 201113635


@dataclass(frozen=True)
class StageConfig:
    """One stage configuration: architecture, stack depth and batch shape."""
    name: str
    hidden: int
    heads: int
    ffn: int
    vocab: int
    max_pos: int
    layers: int          # L: encoder layers in the stack
    trainable: int       # k: top layers that take part in backward
    batch: int           # B
    seq: int             # S
    pred: int            # P: MLM slots per sequence
    dtype: str           # "fp32" or "bf16"
    varlen: Tuple[int, int] | None = None   # (lo, hi) inclusive, None = all S
    seed_index: int = 0
    share_group: int = 1  # layers per shared parameter block (Section 3.3); 1 = every layer its own
    nsp: bool = False     # next-sentence-prediction head and segment embeddings (Section 4.1)

    @property
    def frozen(self) -> int:
        return self.layers - self.trainable


CONFIGS: Dict[str, StageConfig] = {
    "tiny": StageConfig("tiny", 128, 2, 512, 1024, 64, 2, 1, 8, 64, 10, "fp32", None, 1),
    "base_stage": StageConfig("base_stage", 768, 12, 3072, 30522, 512, 12, 3, 128, 128, 20,
                              "bf16", None, 2),
    # same seed index as base_stage: identical data and weights, all layers trainable
    "base_full": StageConfig("base_full", 768, 12, 3072, 30522, 512, 12, 12, 128, 128, 20,
                             "bf16", None, 2),
    "large_stage": StageConfig("large_stage", 1024, 16, 4096, 30522, 512, 24, 3, 64, 128, 20,
                               "bf16", None, 4),
    "large_long": StageConfig("large_long", 1024, 16, 4096, 30522, 512, 24, 6, 16, 512, 80,
                              "bf16", (256, 512), 5),
}


def scaled(cfg: StageConfig, **kw) -> StageConfig:
    """A copy of a configuration with some fields replaced (smaller batch, ...)."""
    return replace(cfg, **kw)


def _rng(seed: int, purpose: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, purpose]))


def config_seed(cfg: StageConfig) -> int:
    return BASE_SEED + cfg.seed_index


def zipf_tokens(rng: np.random.Generator, vocab: int, shape, exponent: float = 1.1) -> np.ndarray:
    """i.i.d. ranks r in 1..V with p(r) ~ r^-exponent, by inverse CDF; id = r - 1."""
    w = np.arange(1, vocab + 1, dtype=np.float64) ** (-exponent)
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    u = rng.random(size=shape)
    ids = np.searchsorted(cdf, u, side="left")
    return np.minimum(ids, vocab - 1).astype(np.int32)


def make_batch(cfg: StageConfig, seed: int | None = None):
    """tokens [B,S], seq_lens [B], mlm_positions [B,P], mlm_labels [B,P]; all int32.

    Empty MLM slots hold -1 in both position and label.  Positions within one
    sequence are distinct, sorted and lie below that sequence's length; tokens
    past the length are id 0.
    """
    seed = config_seed(cfg) if seed is None else seed
    B, S, P, V = cfg.batch, cfg.seq, cfg.pred, cfg.vocab
    tokens = zipf_tokens(_rng(seed, 1), V, (B, S))
    r_len = _rng(seed, 2)
    if cfg.varlen is None:
        seq_lens = np.full((B,), S, dtype=np.int32)
    else:
        lo, hi = cfg.varlen
        seq_lens = r_len.integers(lo, hi + 1, size=(B,)).astype(np.int32)
        seq_lens = np.minimum(seq_lens, S)
    r_mlm = _rng(seed, 3)
    pos = np.full((B, P), -1, dtype=np.int32)
    lab = np.full((B, P), -1, dtype=np.int32)
    for b in range(B):
        n = int(seq_lens[b])
        tokens[b, n:] = 0
        nb = min(P, max(1, int(round(0.15 * n))))
        chosen = np.sort(r_mlm.choice(n, size=nb, replace=False)).astype(np.int32)
        pos[b, :nb] = chosen
        lab[b, :nb] = r_mlm.integers(0, V, size=nb).astype(np.int32)
    return tokens, seq_lens, pos, lab


def param_shapes(cfg: StageConfig, n_layers: int | None = None) -> Dict[str, Tuple[int, ...]]:
    """Ordered tensor names and shapes; weights are [out, in] row-major."""
    H, F, V = cfg.hidden, cfg.ffn, cfg.vocab
    L = cfg.layers if n_layers is None else n_layers
    d: Dict[str, Tuple[int, ...]] = {
        "emb.word": (V, H), "emb.pos": (cfg.max_pos, H),
        "emb.ln.gamma": (H,), "emb.ln.beta": (H,),
    }
    if cfg.nsp:
        d["emb.type"] = (2, H)
    for i in range(L // cfg.share_group):   # one parameter block per group of layers
        p = f"layer.{i}."
        d[p + "qkv.weight"] = (3 * H, H)
        d[p + "qkv.bias"] = (3 * H,)
        d[p + "out.weight"] = (H, H)
        d[p + "out.bias"] = (H,)
        d[p + "ln1.gamma"] = (H,)
        d[p + "ln1.beta"] = (H,)
        d[p + "ffn1.weight"] = (F, H)
        d[p + "ffn1.bias"] = (F,)
        d[p + "ffn2.weight"] = (H, F)
        d[p + "ffn2.bias"] = (H,)
        d[p + "ln2.gamma"] = (H,)
        d[p + "ln2.beta"] = (H,)
    d["head.transform.weight"] = (H, H)
    d["head.transform.bias"] = (H,)
    d["head.ln.gamma"] = (H,)
    d["head.ln.beta"] = (H,)
    d["head.decoder.bias"] = (V,)
    if cfg.nsp:
        d["head.pooler.weight"] = (H, H)
        d["head.pooler.bias"] = (H,)
        d["head.nsp.weight"] = (2, H)
        d["head.nsp.bias"] = (2,)
    return d


def make_nsp(cfg: StageConfig, seq_lens: np.ndarray, seed: int | None = None):
    """segment ids [B,S] (0 up to a random split point inside the sequence, 1 after it, 0 on the
    padding) and next-sentence labels [B] in {0, 1}; all int32."""
    seed = config_seed(cfg) if seed is None else seed
    r = _rng(seed, 4)
    seg = np.zeros((cfg.batch, cfg.seq), dtype=np.int32)
    for b in range(cfg.batch):
        n = int(seq_lens[b])
        cut = int(r.integers(1, max(2, n)))
        seg[b, cut:n] = 1
    lab = r.integers(0, 2, size=(cfg.batch,)).astype(np.int32)
    return seg, lab


def make_weights(cfg: StageConfig, seed: int | None = None, variant: str = "parity",
                 n_layers: int | None = None, std: float = 0.02) -> Dict[str, np.ndarray]:
    """fp32 weights: matrices and tables N(0, std).

    variant "parity": biases ~ N(0, std), LayerNorm gamma ~ 1 + N(0, std),
    beta ~ N(0, std), so that every path carries signal.
    variant "bench": biases 0, gamma 1, beta 0.
    Each tensor has its own stream keyed by a checksum of its name, so a deeper
    stack starts with the same values as a shallower one.
    """
    seed = config_seed(cfg) if seed is None else seed
    out: Dict[str, np.ndarray] = {}
    for name, shape in param_shapes(cfg, n_layers).items():
        rng = _rng(seed, 1000 + zlib.crc32(name.encode()))
        if len(shape) == 2:
            w = rng.standard_normal(size=shape) * std
        elif variant == "parity":
            w = rng.standard_normal(size=shape) * std
            if name.endswith("gamma"):
                w = 1.0 + w
        else:
            w = np.ones(shape) if name.endswith("gamma") else np.zeros(shape)
        out[name] = np.ascontiguousarray(w, dtype=np.float32)
    return out


ADAM_DEFAULTS = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-6, weight_decay=0.01,
                     bias_correction=1)
