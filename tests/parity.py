"""Shared helpers of the GPU parity tests: drive the CUDA library and the CPU oracle on the
same seeded inputs and compare them element by element."""
from __future__ import annotations

import numpy as np

from oracle import mslt_oracle as O
from paper_2011_13635_b200 import inputs as I

# Tolerances (loss: relative; tensors: max-abs error over max-abs reference value).
#   fp32 path: every contraction accumulates in fp32 in k order, statistics in fp32.
#   bf16 path: activations, saved activations and activation gradients are rounded to bf16
#   (relative 2^-9 per rounding); weight gradients accumulate in fp32.
#   update: the change dw = w_after - w_before of one step, in two forms.  update_l1 is
#   mean|dw - dw_ref| / mean|dw_ref| over the whole tensor.  update_max is the max-abs form
#   max|dw - dw_ref| / max|dw_ref|; Adam's first step is -lr * g / (|g| + eps), i.e. sign-like, so
#   an element whose gradient lies within the gradient tolerance of zero may legitimately take the
#   opposite sign (an error of 2 in that form).  The max-abs form is therefore asserted on the
#   elements whose reference gradient is clear of zero by twice the gradient tolerance
#   (|g_ref| > 2 * tol_grad * G with G = max|g_ref|, where both sides must agree on the sign) and
#   reported (not asserted) over all elements.  Its tolerance follows from the gradient tolerance:
#   h(g) = g / (|g| + eps) has slope eps / (|g| + eps)^2, a gradient error of at most tol_grad * G
#   is at most half of such an element, so its first-step update is off by at most
#   lr * eps * tol_grad * G / (|g_ref| / 2 + eps)^2 (never more than lr / 4), plus update_max for
#   the rounding of the arithmetic itself.
#   (fp32 update_l1: gradients as small as eps = 1e-6, e.g. those of the pooler under the second
#   objective, make g / (|g| + eps) amplify a 1e-4 gradient error to a few 1e-3 in the mean.)
TOL = {"fp32": dict(loss=2e-3, grad=1e-4, weight=1e-4, hidden=1e-4, update_l1=5e-3, update_max=1e-4),
       "bf16": dict(loss=2e-3, grad=3e-2, weight=3e-2, hidden=3e-2, update_l1=0.15, update_max=1e-3)}


def max_rel(a: np.ndarray, r: np.ndarray) -> float:
    """max_i |a_i - r_i| / max_i |r_i|."""
    a = np.asarray(a, dtype=np.float64)
    r = np.asarray(r, dtype=np.float64)
    den = np.abs(r).max()
    num = np.abs(a - r).max()
    if den == 0.0:
        return 0.0 if num == 0.0 else float("inf")
    return float(num / den)


def to_cuda(torch, *arrays):
    return [None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda() for a in arrays]


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16 bit patterns (uint16), by integer arithmetic."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    bias = ((u >> 16) & 1) + 0x7FFF
    return ((u + bias) >> 16).astype(np.uint16)


def build_pair(cfg: I.StageConfig, lr: float, max_layers=None, init_layers=None, seed=None,
               max_trainable: int = 0, **opt):
    """(library context, oracle) with identical weights, boundary and hyper-parameters."""
    from paper_2011_13635_b200.binding import Mslt
    L0 = cfg.layers if init_layers is None else init_layers
    w = I.make_weights(cfg, seed=seed, variant="parity", n_layers=L0)
    oracle = O.MsltOracle(w, cfg.heads, ln_eps=1e-12, max_layers=max_layers or cfg.layers,
                          share_group=cfg.share_group)
    hyper = dict(I.ADAM_DEFAULTS)
    hyper.update(opt)
    hyper["lr"] = lr
    # both sides get the same numbers: the C ABI carries hyper-parameters as float32
    hyper = {k: (float(np.float32(v)) if k not in ("bias_correction", "lamb") else v) for k, v in hyper.items()}
    oracle.set_optimizer(**hyper)
    m = Mslt.from_config(cfg, init_layers=L0, max_layers=max_layers or cfg.layers, max_trainable=max_trainable)
    m.set_params(w)
    m.mslt_set_optimizer(**hyper)
    if init_layers is None:
        oracle.set_trainable(cfg.trainable)
        m.mslt_set_trainable(cfg.trainable)
    return m, oracle


def compare_step(m, oracle, cfg, batch, tol, report=None):
    """One step on both sides; asserts loss, gradients, weights and the frozen slice."""
    import torch
    tok, lens, pos, lab = batch[:4]
    seg, nlab = (batch[4], batch[5]) if len(batch) == 6 else (None, None)   # both objectives
    names = oracle.trainable_names()
    all_names = list(oracle.p.keys())
    frozen = [n for n in all_names if n not in names]
    w_before = {n: m.mslt_get_param(n) for n in names}
    m_before = {n: m.mslt_get_opt_state(n, 0) for n in names}
    v_before = {n: m.mslt_get_opt_state(n, 1) for n in names}
    raw_frozen = {n: (m.mslt_get_param(n), m.mslt_get_param_raw(n)) for n in frozen}
    ow_before = {n: oracle.p[n].copy() for n in names}

    d_tok, d_lens, d_pos, d_lab = to_cuda(torch, tok, lens if cfg.varlen else None, pos, lab)
    if len(batch) == 6:
        d_seg, d_nlab = to_cuda(torch, seg, nlab)
        loss_g = m.mslt_step_nsp(d_tok, d_lens, d_seg, d_pos, d_lab, d_nlab)
        loss_o = oracle.step(tok, lens, pos, lab, seg, nlab)
    else:
        loss_g = m.mslt_step(d_tok, d_lens, d_pos, d_lab)
        loss_o = oracle.step(tok, lens, pos, lab)
    rel_loss = abs(loss_g - loss_o) / abs(loss_o)
    assert rel_loss < tol["loss"], (loss_g, loss_o)

    worst = dict(grad=("", 0.0), weight=("", 0.0), update=("", 0.0), update_max_clear=("", 0.0),
                 update_max_all=("", 0.0))
    o = oracle.opt
    t = oracle.t
    for n in names:
        g = m.mslt_get_grad(n)
        e = max_rel(g, oracle.grads[n])
        if e > worst["grad"][1]:
            worst["grad"] = (n, e)
        assert e < tol["grad"], ("grad", n, e)
        w_after = m.mslt_get_param(n)
        e = max_rel(w_after, oracle.p[n])
        if e > worst["weight"][1]:
            worst["weight"] = (n, e)
        assert e < tol["weight"], ("weight", n, e)
        # the update itself: mean |dw - dw_ref| / mean |dw_ref| (Adam's first steps are
        # sign-like, so single elements with a near-zero gradient may flip under rounding)
        dw, dwo = w_after - w_before[n], oracle.p[n] - ow_before[n]
        e = float(np.abs(dw - dwo).mean() / max(np.abs(dwo).mean(), 1e-30))
        if e > worst["update"][1]:
            worst["update"] = (n, e)
        assert e < tol["update_l1"], ("update", n, e)
        # max-abs form of the update: over all elements (a number for the report) and, asserted,
        # over the elements whose reference gradient is clear of zero
        den = max(np.abs(dwo).max(), 1e-30)
        e_all = float(np.abs(dw - dwo).max() / den)
        if e_all > worst["update_max_all"][1]:
            worst["update_max_all"] = (n, e_all)
        g_ref = oracle.grads[n]
        clear = np.abs(g_ref) > 2.0 * tol["grad"] * np.abs(g_ref).max()
        if t == 1 and clear.any() and o["bias_correction"] and not o.get("lamb"):
            e = float(np.abs(dw - dwo)[clear].max() / den)
            if e > worst["update_max_clear"][1]:
                worst["update_max_clear"] = (n, e)
            gc = np.abs(g_ref[clear])
            allow = o["lr"] * (o["eps"] * tol["grad"] * np.abs(g_ref).max() / (gc / 2 + o["eps"]) ** 2).max() / den
            assert e < allow + tol["update_max"], ("update, max-abs form on clear gradients", n, e, allow)
            assert np.abs(dw[clear]).min() > 0.0, ("an element with a clear gradient did not move", n)
        # the Adam kernel alone: the oracle's update formula applied to the library's own inputs
        wd = o["weight_decay"] if w_before[n].ndim == 2 else 0.0
        rule = O.lamb_update if o.get("lamb") else O.adam_update
        w_ref, m_ref, v_ref = rule(w_before[n].astype(np.float64), g.astype(np.float64),
                                m_before[n].astype(np.float64), v_before[n].astype(np.float64),
                                t, o["lr"], o["beta1"], o["beta2"], o["eps"], wd, bool(o["bias_correction"]))
        assert max_rel(w_after, w_ref) < 2e-6, ("adam w", n)
        assert max_rel(m.mslt_get_opt_state(n, 0), m_ref) < 2e-6, ("adam m", n)
        assert max_rel(m.mslt_get_opt_state(n, 1), v_ref) < 2e-6, ("adam v", n)
        if cfg.dtype == "bf16" and w_after.ndim == 2:
            assert np.array_equal(m.mslt_get_param_raw(n), bf16_round(w_after)), ("bf16 copy", n)
    for n in frozen:
        assert np.array_equal(m.mslt_get_param(n), raw_frozen[n][0]), ("frozen master moved", n)
        assert np.array_equal(m.mslt_get_param_raw(n), raw_frozen[n][1]), ("frozen copy moved", n)
    assert m.mslt_debug_check_guards() == 0, "a kernel wrote outside its workspace buffer"
    if report is not None:
        report.append(dict(loss_gpu=loss_g, loss_oracle=loss_o, rel_loss=rel_loss, **worst))
    return loss_g, loss_o, worst
