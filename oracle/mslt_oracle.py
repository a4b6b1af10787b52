"""CPU fp64 oracle for the MSLT per-stage BERT training step.  TEST INFRASTRUCTURE.

This file is the slow, plain definition that the CUDA library is checked
against.  Only the tests, the smoke check and the benchmark's CPU-baseline leg
may use it; the product path never does.  It shares no code with the CUDA
path and imports nothing from it.

What it computes (paper, Section 3.1 last paragraph and Section 3.2):
  * the bottom layers, trained in earlier stages, take part in the forward
    pass only and supply the input of the top layers;
  * the newly added top layers and the output layer take part in forward and
    backward, and are the only parameters that are updated;
  * the word-embedding matrix is shared between the input and the output
    layer and is updated only when every layer is trainable (first stage,
    joint retraining);
  * new layers are initialised by copying the top layers of the previous
    stage's model.
The network itself is the BERT encoder the paper defers to (Section 4.1): a
post-LayerNorm Transformer encoder with exact (erf) GELU, a masked-language-
model head with a tied decoder, and mean cross-entropy over the valid slots.
The method is ordinary back-propagation truncated at a layer boundary, so the
oracle is that definition written out: full forward in float64, reverse-mode
gradients for the trainable tensors only, then Adam on those.

Everything is float64 numpy; matrix products use numpy's matmul/einsum as a
library step.  No blocking, fusion or reordering beyond the definition.

Pins (tests/test_oracle_pins.py): central finite differences on every
trainable tensor, softmax rows summing to one with exact zeros under the mask,
LayerNorm moments, loss = ln V for a zero decoder, hand-worked head-only
soft-max regression, Adam closed forms, padding invariance, batch additivity,
truncation invariance and bit-identical frozen tensors.
Parity unpinned by the paper (fixed only by this file and the CUDA path
following the same written rule): Adam hyper-parameter defaults, the reset of
the optimizer state when the trainable slice changes, loss normalisation by
the number of valid slots.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional

import numpy as np
from scipy.special import erf

F64 = np.float64


# ----------------------------------------------------------------------------
# element-wise and row-wise operations, forward and backward
# ----------------------------------------------------------------------------

def gelu(u: np.ndarray) -> np.ndarray:
    """gelu(u) = u * Phi(u), Phi the standard normal CDF (exact erf form)."""
    return 0.5 * u * (1.0 + erf(u / math.sqrt(2.0)))


def gelu_grad(u: np.ndarray) -> np.ndarray:
    """d gelu / du = Phi(u) + u * phi(u)."""
    cdf = 0.5 * (1.0 + erf(u / math.sqrt(2.0)))
    pdf = np.exp(-0.5 * u * u) / math.sqrt(2.0 * math.pi)
    return cdf + u * pdf


def layer_norm(z: np.ndarray, gamma: np.ndarray, beta: np.ndarray, eps: float):
    """Row-wise LayerNorm over the last axis with the biased (1/H) variance.

    Returns (y, xhat, rstd) with y = gamma * xhat + beta.
    """
    mean = z.mean(axis=-1, keepdims=True)
    var = ((z - mean) ** 2).mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + eps)
    xhat = (z - mean) * rstd
    return gamma * xhat + beta, xhat, rstd


def layer_norm_backward(dy: np.ndarray, xhat: np.ndarray, rstd: np.ndarray, gamma: np.ndarray):
    """Returns (dz, dgamma, dbeta) of y = gamma * xhat(z) + beta."""
    red = tuple(range(dy.ndim - 1))
    dgamma = (dy * xhat).sum(axis=red)
    dbeta = dy.sum(axis=red)
    dxhat = dy * gamma
    m1 = dxhat.mean(axis=-1, keepdims=True)
    m2 = (dxhat * xhat).mean(axis=-1, keepdims=True)
    dz = rstd * (dxhat - m1 - xhat * m2)
    return dz, dgamma, dbeta


def masked_softmax(scores: np.ndarray, seq_lens: np.ndarray) -> np.ndarray:
    """Softmax over the last axis of scores [B, A, S, S]; key j of sequence b
    is valid iff j < seq_lens[b]; masked keys get probability exactly 0."""
    B, _, _, S = scores.shape
    valid = np.arange(S)[None, :] < np.asarray(seq_lens)[:, None]          # [B, S]
    valid = valid[:, None, None, :]
    sc = np.where(valid, scores, -np.inf)
    mx = sc.max(axis=-1, keepdims=True)
    e = np.where(valid, np.exp(sc - mx), 0.0)
    return e / e.sum(axis=-1, keepdims=True)


def softmax_backward(dp: np.ndarray, p: np.ndarray) -> np.ndarray:
    """d scores of p = softmax(scores): p * (dp - sum_j dp*p)."""
    return p * (dp - (dp * p).sum(axis=-1, keepdims=True))


def cross_entropy(logits: np.ndarray, labels: np.ndarray, n_valid: int):
    """Per-row nll = logsumexp(logits) - logits[label]; rows with label < 0
    contribute nothing.  Returns (sum nll / n_valid, dlogits)."""
    R = logits.shape[0]
    ok = labels >= 0
    mx = logits.max(axis=-1, keepdims=True)
    lse = mx[:, 0] + np.log(np.exp(logits - mx).sum(axis=-1))
    safe = np.where(ok, labels, 0)
    nll = np.where(ok, lse - logits[np.arange(R), safe], 0.0)
    if n_valid == 0:
        return 0.0, np.zeros_like(logits)
    loss = nll.sum() / n_valid
    sm = np.exp(logits - lse[:, None])
    sm[np.arange(R), safe] -= 1.0
    dlogits = sm * (ok[:, None] / n_valid)
    return float(loss), dlogits


def adam_update(w, g, m, v, t: int, lr, beta1, beta2, eps, weight_decay, bias_correction: bool):
    """One Adam step with decoupled weight decay on one tensor; t is the step
    count after this update (1 for the first).  Returns (w, m, v)."""
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    if bias_correction:
        mh = m / (1.0 - beta1 ** t)
        vh = v / (1.0 - beta2 ** t)
    else:
        mh, vh = m, v
    w = w - lr * (mh / (np.sqrt(vh) + eps) + weight_decay * w)
    return w, m, v


def lamb_update(w, g, m, v, t: int, lr, beta1, beta2, eps, weight_decay, bias_correction: bool):
    """One LAMB step on one tensor (the optimizer of the paper's experiments, Section 4.1; You
    et al., "Large batch optimization for deep learning", Algorithm 2 with the identity as scaling
    function).  The Adam direction plus decoupled decay, r = m_hat / (sqrt(v_hat) + eps) + wd * w,
    is rescaled per tensor by the trust ratio ||w|| / ||r|| (Euclidean norms over the whole
    tensor; the ratio is 1 when either norm is 0):  w <- w - lr * (||w|| / ||r||) * r.
    t is the step count after this update.  Returns (w, m, v)."""
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    if bias_correction:
        mh = m / (1.0 - beta1 ** t)
        vh = v / (1.0 - beta2 ** t)
    else:
        mh, vh = m, v
    r = mh / (np.sqrt(vh) + eps) + weight_decay * w
    wn = math.sqrt(float(np.sum(w * w)))
    rn = math.sqrt(float(np.sum(r * r)))
    ratio = wn / rn if (wn > 0.0 and rn > 0.0) else 1.0
    w = w - lr * ratio * r
    return w, m, v


# ----------------------------------------------------------------------------
# the model
# ----------------------------------------------------------------------------

LAYER_TENSORS = ("qkv.weight", "qkv.bias", "out.weight", "out.bias", "ln1.gamma", "ln1.beta",
                 "ffn1.weight", "ffn1.bias", "ffn2.weight", "ffn2.bias", "ln2.gamma", "ln2.beta")
HEAD_TENSORS = ("head.transform.weight", "head.transform.bias", "head.ln.gamma", "head.ln.beta",
                "head.decoder.bias")
EMB_TENSORS = ("emb.word", "emb.pos", "emb.ln.gamma", "emb.ln.beta")
# next-sentence-prediction objective (Section 4.1: "the same MLM and NSP objectives" as BERT): a
# segment (token-type) table in the embeddings, a tanh pooler on the first token and a two-way
# classifier.  Present only when the parameter set holds them.
NSP_EMB_TENSORS = ("emb.type",)
NSP_HEAD_TENSORS = ("head.pooler.weight", "head.pooler.bias", "head.nsp.weight", "head.nsp.bias")


class MsltOracle:
    """BERT stack with a frozen/trainable boundary, in float64."""

    def __init__(self, params: Dict[str, np.ndarray], heads: int, ln_eps: float = 1e-12,
                 max_layers: Optional[int] = None, share_group: int = 1):
        """share_group = g > 1: the grouped parameter sharing of Section 3.3 (the paper's change to
        ALBERT): encoder layers l with the same l // g use one parameter block, named
        "layer.<l // g>."; a stage adds one or more whole groups and only those train."""
        self.p: Dict[str, np.ndarray] = {k: np.array(v, dtype=F64) for k, v in params.items()}
        self.heads = heads
        self.eps = ln_eps
        self.g = int(share_group)
        self.L = self.g * (1 + max(int(k.split(".")[1]) for k in self.p if k.startswith("layer.")))
        self.max_layers = self.L if max_layers is None else max_layers
        self.H = self.p["emb.word"].shape[1]
        self.V = self.p["emb.word"].shape[0]
        self.nsp = "head.nsp.weight" in self.p
        self.top_k = self.L
        self.opt = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-6, weight_decay=0.01,
                        bias_correction=1, lamb=0)
        self.grads: Dict[str, np.ndarray] = {}
        self._reset_optimizer()

    # -- staging (Section 3.2) -------------------------------------------------
    def trainable_names(self) -> List[str]:
        names: List[str] = []
        if self.top_k == self.L:
            names += list(EMB_TENSORS) + (list(NSP_EMB_TENSORS) if self.nsp else [])
        for b in range((self.L - self.top_k) // self.g, self.L // self.g):
            names += [f"layer.{b}.{t}" for t in LAYER_TENSORS]
        names += list(HEAD_TENSORS) + (list(NSP_HEAD_TENSORS) if self.nsp else [])
        return names

    def _reset_optimizer(self):
        self.t = 0
        self.m = {n: np.zeros_like(self.p[n]) for n in self.trainable_names()}
        self.v = {n: np.zeros_like(self.p[n]) for n in self.trainable_names()}

    def set_optimizer(self, **kw):
        self.opt.update(kw)

    def set_trainable(self, top_k: int):
        if not 0 <= top_k <= self.L or top_k % self.g:
            raise ValueError("top_k out of range, or not a whole number of groups")
        self.top_k = top_k
        self._reset_optimizer()

    def add_layers(self, k: int):
        """New layer L+i is a copy of layer L-k+i (order preserved)."""
        if not 1 <= k <= self.L or self.L + k > self.max_layers or k % self.g:
            raise ValueError("cannot add layers")
        for i in range(k // self.g):
            for t in LAYER_TENSORS:
                self.p[f"layer.{self.L // self.g + i}.{t}"] = self.p[f"layer.{(self.L - k) // self.g + i}.{t}"].copy()
        self.L += k
        self.top_k = min(self.top_k, self.L)
        self._reset_optimizer()

    # -- forward ------------------------------------------------------------------
    def _embed(self, tokens, segments=None):
        S = tokens.shape[1]
        z = self.p["emb.word"][tokens] + self.p["emb.pos"][:S][None, :, :]
        if self.nsp:
            seg = np.zeros_like(tokens) if segments is None else np.asarray(segments)
            z = z + self.p["emb.type"][seg]
        y, xhat, rstd = layer_norm(z, self.p["emb.ln.gamma"], self.p["emb.ln.beta"], self.eps)
        return y, (xhat, rstd)

    def _layer_forward(self, l: int, x, seq_lens):
        P = lambda t: self.p[f"layer.{l // self.g}.{t}"]
        B, S, H = x.shape
        A, d = self.heads, H // self.heads
        qkv = x @ P("qkv.weight").T + P("qkv.bias")                 # [B,S,3H]
        q, k, v = (qkv[..., i * H:(i + 1) * H].reshape(B, S, A, d).transpose(0, 2, 1, 3)
                   for i in range(3))                                # [B,A,S,d]
        sc = np.einsum("bhid,bhjd->bhij", q, k) / math.sqrt(d)
        p = masked_softmax(sc, seq_lens)
        c = np.einsum("bhij,bhjd->bhid", p, v).transpose(0, 2, 1, 3).reshape(B, S, H)
        o = c @ P("out.weight").T + P("out.bias")
        y, xh1, rs1 = layer_norm(x + o, P("ln1.gamma"), P("ln1.beta"), self.eps)
        u = y @ P("ffn1.weight").T + P("ffn1.bias")
        g = gelu(u)
        dn = g @ P("ffn2.weight").T + P("ffn2.bias")
        xo, xh2, rs2 = layer_norm(y + dn, P("ln2.gamma"), P("ln2.beta"), self.eps)
        stash = dict(x=x, q=q, k=k, v=v, p=p, c=c, xh1=xh1, rs1=rs1, y=y, u=u, g=g,
                     xh2=xh2, rs2=rs2)
        return xo, stash

    def encode(self, tokens, seq_lens=None, keep_from: Optional[int] = None, segments=None):
        """Hidden states after the last layer, [B,S,H].  Frozen and trainable
        layers run the same forward function; stashes are kept only for layers
        >= keep_from."""
        tokens = np.asarray(tokens)
        B, S = tokens.shape
        seq_lens = np.full((B,), S) if seq_lens is None else np.asarray(seq_lens)
        x, emb_stash = self._embed(tokens, segments)
        stashes = {}
        for l in range(self.L):
            x, st = self._layer_forward(l, x, seq_lens)
            if keep_from is not None and l >= keep_from:
                stashes[l] = st
        return x, emb_stash, stashes

    def _head_forward(self, x, positions, labels):
        B, P_ = positions.shape
        ok = (positions >= 0) & (labels >= 0)
        pos = np.where(ok, positions, 0)
        hm = x[np.arange(B)[:, None], pos]                           # [B,P,H]
        hm = hm.reshape(B * P_, -1)
        ut = hm @ self.p["head.transform.weight"].T + self.p["head.transform.bias"]
        gt = gelu(ut)
        tm, xh, rs = layer_norm(gt, self.p["head.ln.gamma"], self.p["head.ln.beta"], self.eps)
        logits = tm @ self.p["emb.word"].T + self.p["head.decoder.bias"]
        return logits, dict(hm=hm, ut=ut, xh=xh, rs=rs, tm=tm, ok=ok.reshape(-1), pos=pos)

    def _nsp_forward(self, x, nsp_labels):
        """Pooler and two-way classifier on the first token of every sequence; mean cross-entropy
        over the sequences whose label is >= 0."""
        cls = x[:, 0, :]
        up = cls @ self.p["head.pooler.weight"].T + self.p["head.pooler.bias"]
        pooled = np.tanh(up)
        logits = pooled @ self.p["head.nsp.weight"].T + self.p["head.nsp.bias"]      # [B,2]
        lab = np.asarray(nsp_labels)
        loss, dlogits = cross_entropy(logits, lab, int((lab >= 0).sum()))
        return loss, dlogits, dict(cls=cls, pooled=pooled, logits=logits)

    def forward(self, tokens, seq_lens=None, positions=None, segments=None):
        """(hidden [B,S,H], logits [B*P,V] or None): the inference-only path."""
        x, _, _ = self.encode(tokens, seq_lens, segments=segments)
        if positions is None:
            return x, None
        positions = np.asarray(positions)
        logits, _ = self._head_forward(x, positions, np.zeros_like(positions))
        return x, logits

    def loss(self, tokens, seq_lens, positions, labels, segments=None, nsp_labels=None) -> float:
        """MLM loss, plus the NSP loss when nsp_labels are given."""
        x, _, _ = self.encode(tokens, seq_lens, segments=segments)
        positions, labels = np.asarray(positions), np.asarray(labels)
        logits, hs = self._head_forward(x, positions, labels)
        lab = np.where(hs["ok"], labels.reshape(-1), -1)
        total = cross_entropy(logits, lab, int(hs["ok"].sum()))[0]
        if self.nsp and nsp_labels is not None:
            total += self._nsp_forward(x, nsp_labels)[0]
        return total

    # -- forward + backward, gradients for the trainable tensors only -------------------
    def loss_and_grads(self, tokens, seq_lens, positions, labels, segments=None, nsp_labels=None):
        tokens = np.asarray(tokens)
        positions, labels = np.asarray(positions), np.asarray(labels)
        B, S = tokens.shape
        H, A = self.H, self.heads
        d = H // A
        seq_lens = np.full((B,), S) if seq_lens is None else np.asarray(seq_lens)
        first = self.L - self.top_k                       # first trainable layer
        full = self.top_k == self.L
        x, emb_stash, st = self.encode(tokens, seq_lens, keep_from=first, segments=segments)
        logits, hs = self._head_forward(x, positions, labels)
        lab = np.where(hs["ok"], labels.reshape(-1), -1)
        n_valid = int(hs["ok"].sum())
        loss, dlogits = cross_entropy(logits, lab, n_valid)
        g: Dict[str, np.ndarray] = {}

        # MLM head: decoder (tied to the word embedding), LayerNorm, GELU, transform
        g["head.decoder.bias"] = dlogits.sum(axis=0)
        dtm = dlogits @ self.p["emb.word"]
        if full:
            g["emb.word"] = dlogits.T @ hs["tm"]
        dgt, g["head.ln.gamma"], g["head.ln.beta"] = layer_norm_backward(
            dtm, hs["xh"], hs["rs"], self.p["head.ln.gamma"])
        dut = dgt * gelu_grad(hs["ut"])
        g["head.transform.weight"] = dut.T @ hs["hm"]
        g["head.transform.bias"] = dut.sum(axis=0)
        dhm = (dut @ self.p["head.transform.weight"]).reshape(B, -1, H)
        dx = np.zeros((B, S, H), dtype=F64)
        okm = hs["ok"].reshape(B, -1)
        for b in range(B):
            for j in range(positions.shape[1]):
                if okm[b, j]:
                    dx[b, hs["pos"][b, j]] += dhm[b, j]

        self.losses = dict(mlm=loss, nsp=0.0)
        if self.nsp:
            for n in NSP_HEAD_TENSORS:
                g[n] = np.zeros_like(self.p[n])
            if nsp_labels is not None:
                # second objective: loss = MLM + NSP; its gradient enters the last hidden state at token 0
                nsp_loss, dl2, ns = self._nsp_forward(x, nsp_labels)
                loss = loss + nsp_loss
                self.losses["nsp"] = nsp_loss
                g["head.nsp.weight"] = dl2.T @ ns["pooled"]
                g["head.nsp.bias"] = dl2.sum(axis=0)
                dup = (dl2 @ self.p["head.nsp.weight"]) * (1.0 - ns["pooled"] ** 2)
                g["head.pooler.weight"] = dup.T @ ns["cls"]
                g["head.pooler.bias"] = dup.sum(axis=0)
                dx[:, 0, :] += dup @ self.p["head.pooler.weight"]

        # trainable encoder layers, top-down; stop at the frozen boundary
        def acc(name, value):          # layers of one group add their gradients into the shared block
            g[name] = g[name] + value if name in g else value

        for l in range(self.L - 1, first - 1, -1):
            P = lambda t: self.p[f"layer.{l // self.g}.{t}"]
            s = st[l]
            n = f"layer.{l // self.g}."
            dz2, dgam, dbet = layer_norm_backward(dx, s["xh2"], s["rs2"], P("ln2.gamma"))
            acc(n + "ln2.gamma", dgam); acc(n + "ln2.beta", dbet)
            acc(n + "ffn2.weight", np.einsum("bso,bsi->oi", dz2, s["g"]))
            acc(n + "ffn2.bias", dz2.sum(axis=(0, 1)))
            du = (dz2 @ P("ffn2.weight")) * gelu_grad(s["u"])
            acc(n + "ffn1.weight", np.einsum("bso,bsi->oi", du, s["y"]))
            acc(n + "ffn1.bias", du.sum(axis=(0, 1)))
            dy = du @ P("ffn1.weight") + dz2
            dz1, dgam, dbet = layer_norm_backward(dy, s["xh1"], s["rs1"], P("ln1.gamma"))
            acc(n + "ln1.gamma", dgam); acc(n + "ln1.beta", dbet)
            acc(n + "out.weight", np.einsum("bso,bsi->oi", dz1, s["c"]))
            acc(n + "out.bias", dz1.sum(axis=(0, 1)))
            dc = (dz1 @ P("out.weight")).reshape(B, S, A, d).transpose(0, 2, 1, 3)   # [B,A,S,d]
            dv = np.einsum("bhij,bhid->bhjd", s["p"], dc)
            dp = np.einsum("bhid,bhjd->bhij", dc, s["v"])
            dsc = softmax_backward(dp, s["p"]) / math.sqrt(d)
            dq = np.einsum("bhij,bhjd->bhid", dsc, s["k"])
            dk = np.einsum("bhij,bhid->bhjd", dsc, s["q"])
            dqkv = np.concatenate([t.transpose(0, 2, 1, 3).reshape(B, S, H) for t in (dq, dk, dv)],
                                  axis=-1)
            acc(n + "qkv.weight", np.einsum("bso,bsi->oi", dqkv, s["x"]))
            acc(n + "qkv.bias", dqkv.sum(axis=(0, 1)))
            if l > first or full:
                dx = dqkv @ P("qkv.weight") + dz1

        if full:
            dz0, g["emb.ln.gamma"], g["emb.ln.beta"] = layer_norm_backward(
                dx, emb_stash[0], emb_stash[1], self.p["emb.ln.gamma"])
            g["emb.pos"] = np.zeros_like(self.p["emb.pos"])
            g["emb.pos"][:S] = dz0.sum(axis=0)
            np.add.at(g["emb.word"], tokens.reshape(-1), dz0.reshape(B * S, H))
            if self.nsp:
                seg = np.zeros_like(tokens) if segments is None else np.asarray(segments)
                g["emb.type"] = np.zeros_like(self.p["emb.type"])
                np.add.at(g["emb.type"], seg.reshape(-1), dz0.reshape(B * S, H))
        self.grads = g
        return loss, g

    # -- one training step ------------------------------------------------------------
    def step(self, tokens, seq_lens, positions, labels, segments=None, nsp_labels=None) -> float:
        """Forward, truncated backward, Adam (or LAMB, opt["lamb"] = 1) on the trainable tensors only."""
        loss, g = self.loss_and_grads(tokens, seq_lens, positions, labels, segments, nsp_labels)
        self.t += 1
        o = self.opt
        update = lamb_update if o.get("lamb") else adam_update
        for n in self.trainable_names():
            wd = o["weight_decay"] if self.p[n].ndim == 2 else 0.0
            self.p[n], self.m[n], self.v[n] = update(
                self.p[n], g[n], self.m[n], self.v[n], self.t, o["lr"], o["beta1"], o["beta2"],
                o["eps"], wd, bool(o["bias_correction"]))
        return loss
