"""Pins for the CPU oracle: each test checks it against something other than itself
(finite differences, closed forms, library routines, brute force, invariants)."""
import math

import numpy as np
import pytest
import torch

from oracle import mslt_oracle as O
from paper_2011_13635_b200 import inputs as I

TINY = I.StageConfig("pin", hidden=8, heads=2, ffn=16, vocab=11, max_pos=6, layers=2, trainable=1,
                     batch=2, seq=5, pred=3, dtype="fp32", varlen=(3, 5), seed_index=77)


def tiny_model(cfg=TINY, std=0.3, top_k=None, seed=5):
    w = I.make_weights(cfg, seed=seed, variant="parity", std=std)
    m = O.MsltOracle(w, cfg.heads, ln_eps=1e-12)
    m.set_trainable(cfg.trainable if top_k is None else top_k)
    return m


def tiny_batch(cfg=TINY, seed=9):
    return I.make_batch(cfg, seed=seed)


# -- backward formulas: central finite differences on every trainable element ---------------

@pytest.mark.parametrize("top_k", [0, 1, 2])
def test_gradients_match_finite_differences(top_k):
    m = tiny_model(top_k=top_k)
    tok, lens, pos, lab = tiny_batch()
    assert lens.min() < TINY.seq, "the case must contain padding"
    loss, g = m.loss_and_grads(tok, lens, pos, lab)
    assert set(g.keys()) == set(m.trainable_names())
    h = 1e-5
    for name in m.trainable_names():
        w = m.p[name]
        fd = np.zeros_like(w)
        it = np.nditer(w, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = w[idx]
            w[idx] = keep + h
            lp = m.loss(tok, lens, pos, lab)
            w[idx] = keep - h
            lm = m.loss(tok, lens, pos, lab)
            w[idx] = keep
            fd[idx] = (lp - lm) / (2 * h)
        scale = max(np.abs(fd).max(), 1e-8)
        err = np.abs(fd - g[name]).max() / scale
        assert err < 1e-6, (name, err)
        if name != "emb.pos":      # rows past S are legitimately zero
            assert np.abs(g[name]).max() > 0, name


def test_frozen_tensor_has_gradient_but_is_not_updated():
    m = tiny_model(top_k=1)
    tok, lens, pos, lab = tiny_batch()
    name = "layer.0.ffn1.weight"
    w = m.p[name]
    keep = w[0, 0]
    w[0, 0] = keep + 1e-5
    lp = m.loss(tok, lens, pos, lab)
    w[0, 0] = keep - 1e-5
    lm = m.loss(tok, lens, pos, lab)
    w[0, 0] = keep
    assert abs(lp - lm) > 1e-12          # the loss does depend on it
    before = {k: v.copy() for k, v in m.p.items()}
    for _ in range(3):
        m.step(tok, lens, pos, lab)
    for k in before:
        frozen = k.startswith("emb.") or k.startswith("layer.0.")
        same = np.array_equal(before[k], m.p[k])
        assert same == frozen, k


# -- forward conventions against library routines ----------------------------------------------

def test_encoder_layer_matches_torch_transformer_encoder_layer():
    cfg = TINY
    m = tiny_model()
    rng = np.random.default_rng(0)
    x = rng.standard_normal((cfg.batch, cfg.seq, cfg.hidden))
    lens = np.array([3, 5])
    ref = torch.nn.TransformerEncoderLayer(cfg.hidden, cfg.heads, cfg.ffn, dropout=0.0,
                                           activation="gelu", layer_norm_eps=1e-12,
                                           batch_first=True, norm_first=False).double()
    P = lambda t: torch.from_numpy(m.p["layer.1." + t])
    with torch.no_grad():
        ref.self_attn.in_proj_weight.copy_(P("qkv.weight"))
        ref.self_attn.in_proj_bias.copy_(P("qkv.bias"))
        ref.self_attn.out_proj.weight.copy_(P("out.weight"))
        ref.self_attn.out_proj.bias.copy_(P("out.bias"))
        ref.norm1.weight.copy_(P("ln1.gamma")); ref.norm1.bias.copy_(P("ln1.beta"))
        ref.linear1.weight.copy_(P("ffn1.weight")); ref.linear1.bias.copy_(P("ffn1.bias"))
        ref.linear2.weight.copy_(P("ffn2.weight")); ref.linear2.bias.copy_(P("ffn2.bias"))
        ref.norm2.weight.copy_(P("ln2.gamma")); ref.norm2.bias.copy_(P("ln2.beta"))
    ref.train()   # keeps torch on its plain (non-fused, non-nested) path; dropout is 0
    pad = torch.from_numpy(np.arange(cfg.seq)[None, :] >= lens[:, None])
    want = ref(torch.from_numpy(x), src_key_padding_mask=pad).detach().numpy()
    got, _ = m._layer_forward(1, x, lens)
    for b in range(cfg.batch):           # rows at padded positions are unspecified
        np.testing.assert_allclose(got[b, :lens[b]], want[b, :lens[b]], rtol=0, atol=1e-12)


def test_head_and_loss_match_torch_functional():
    m = tiny_model()
    tok, lens, pos, lab = tiny_batch()
    x, _, _ = m.encode(tok, lens)
    F = torch.nn.functional
    xt = torch.from_numpy(x)
    rows, labels = [], []
    for b in range(tok.shape[0]):
        for j in range(pos.shape[1]):
            if pos[b, j] >= 0:
                rows.append(xt[b, pos[b, j]]); labels.append(int(lab[b, j]))
    hm = torch.stack(rows)
    T = lambda n: torch.from_numpy(m.p[n])
    t = F.gelu(F.linear(hm, T("head.transform.weight"), T("head.transform.bias")))
    t = F.layer_norm(t, (TINY.hidden,), T("head.ln.gamma"), T("head.ln.beta"), eps=1e-12)
    logits = F.linear(t, T("emb.word"), T("head.decoder.bias"))
    want = F.cross_entropy(logits, torch.tensor(labels)).item()
    assert abs(m.loss(tok, lens, pos, lab) - want) < 1e-12


def test_embedding_matches_torch():
    m = tiny_model()
    tok, _, _, _ = tiny_batch()
    F = torch.nn.functional
    e = F.embedding(torch.from_numpy(tok.astype(np.int64)), torch.from_numpy(m.p["emb.word"]))
    e = e + torch.from_numpy(m.p["emb.pos"][: tok.shape[1]])
    want = F.layer_norm(e, (TINY.hidden,), torch.from_numpy(m.p["emb.ln.gamma"]),
                        torch.from_numpy(m.p["emb.ln.beta"]), eps=1e-12).numpy()
    got, _ = m._embed(tok)
    np.testing.assert_allclose(got, want, atol=1e-12, rtol=0)


def test_gelu_values_and_derivative():
    # Phi(1) = 0.841344746068543 (standard normal table), so gelu(1) = Phi(1)
    assert abs(O.gelu(np.array([1.0]))[0] - 0.841344746068543) < 1e-14
    assert O.gelu(np.array([0.0]))[0] == 0.0
    u = np.linspace(-4, 4, 41)
    fd = (O.gelu(u + 1e-6) - O.gelu(u - 1e-6)) / 2e-6
    np.testing.assert_allclose(O.gelu_grad(u), fd, atol=1e-9)
    # the tanh approximation is visibly different: the exact form is what is used
    tanh_form = 0.5 * u * (1 + np.tanh(math.sqrt(2 / math.pi) * (u + 0.044715 * u ** 3)))
    assert np.abs(tanh_form - O.gelu(u)).max() > 1e-4


# -- softmax and LayerNorm invariants -------------------------------------------------------------

def test_softmax_rows_sum_to_one_and_mask_is_exact_zero():
    rng = np.random.default_rng(1)
    sc = rng.standard_normal((3, 2, 7, 7)) * 5
    lens = np.array([7, 4, 1])
    p = O.masked_softmax(sc, lens)
    np.testing.assert_allclose(p.sum(-1), 1.0, atol=1e-14)
    for b, n in enumerate(lens):
        assert np.all(p[b, :, :, n:] == 0.0)
        assert np.all(p[b, :, :, :n] > 0.0)
    assert np.all(p[2, :, :, 0] == 1.0)        # a single valid key takes all the mass


def test_single_token_sequence_context_equals_value():
    cfg = I.scaled(TINY, seq=1, batch=1, varlen=None, pred=1)
    m = tiny_model(cfg)
    x = np.random.default_rng(2).standard_normal((1, 1, cfg.hidden))
    _, st = m._layer_forward(0, x, np.array([1]))
    v = st["v"].transpose(0, 2, 1, 3).reshape(1, 1, cfg.hidden)
    np.testing.assert_allclose(st["c"], v, atol=1e-15)


def test_layer_norm_moments():
    rng = np.random.default_rng(3)
    z = rng.standard_normal((5, 64)) * 3 + 2
    y, xhat, _ = O.layer_norm(z, np.ones(64), np.zeros(64), 1e-12)
    np.testing.assert_allclose(xhat.mean(-1), 0, atol=1e-13)
    np.testing.assert_allclose((xhat ** 2).mean(-1), 1, atol=1e-10)
    assert np.array_equal(y, xhat)
    g = rng.standard_normal(64); b = rng.standard_normal(64)
    y2, _, _ = O.layer_norm(z, g, b, 1e-12)
    np.testing.assert_allclose(y2, xhat * g + b, atol=1e-15)


# -- loss closed forms ----------------------------------------------------------------------------

def test_zero_decoder_gives_log_vocab():
    for V in (11, 1024, 30522):
        cfg = I.scaled(TINY, vocab=V)
        w = I.make_weights(cfg, seed=4, std=0.3)
        w["emb.word"][:] = 0
        w["head.decoder.bias"][:] = 0
        m = O.MsltOracle(w, cfg.heads)
        tok, lens, pos, lab = I.make_batch(cfg, seed=4)
        assert abs(m.loss(tok, lens, pos, lab) - math.log(V)) < 1e-12
    assert abs(math.log(30522) - 10.326203) < 1e-6 and abs(math.log(1024) - 6.931472) < 1e-6


def test_initial_loss_is_close_to_log_vocab():
    cfg = I.scaled(I.CONFIGS["tiny"], batch=2)
    m = O.MsltOracle(I.make_weights(cfg), cfg.heads)
    tok, lens, pos, lab = I.make_batch(cfg)
    assert abs(m.loss(tok, lens, pos, lab) - math.log(cfg.vocab)) < 0.15


def test_cross_entropy_gradient_properties():
    rng = np.random.default_rng(5)
    logits = rng.standard_normal((6, 9)) * 3
    labels = np.array([1, -1, 8, 0, -1, 3])
    loss, dl = O.cross_entropy(logits, labels, 4)
    np.testing.assert_allclose(dl.sum(-1), 0, atol=1e-15)      # each row sums to zero
    assert np.all(dl[1] == 0) and np.all(dl[4] == 0)
    # brute force, one slot at a time
    want = 0.0
    for r, y in enumerate(labels):
        if y >= 0:
            want += math.log(sum(math.exp(v) for v in logits[r])) - logits[r, y]
    assert abs(loss - want / 4) < 1e-13
    assert O.cross_entropy(logits, np.full(6, -1), 0)[0] == 0.0


def test_head_only_training_is_softmax_regression_by_hand():
    """top_k = 0: features are fixed, so d loss / d decoder-bias = mean(softmax - onehot)
    and d loss / d transform-weight follows by the chain rule, written out per slot."""
    m = tiny_model(top_k=0)
    tok, lens, pos, lab = tiny_batch()
    _, g = m.loss_and_grads(tok, lens, pos, lab)
    assert set(g) == set(O.HEAD_TENSORS)
    x, _, _ = m.encode(tok, lens)
    E, bv = m.p["emb.word"], m.p["head.decoder.bias"]
    slots = [(b, j) for b in range(tok.shape[0]) for j in range(pos.shape[1]) if pos[b, j] >= 0]
    dbv = np.zeros_like(bv)
    for b, j in slots:
        h = x[b, pos[b, j]]
        u = m.p["head.transform.weight"] @ h + m.p["head.transform.bias"]
        a = np.array([0.5 * t * (1 + math.erf(t / math.sqrt(2))) for t in u])
        mu = a.mean(); var = ((a - mu) ** 2).mean()
        t = m.p["head.ln.gamma"] * (a - mu) / math.sqrt(var + 1e-12) + m.p["head.ln.beta"]
        z = E @ t + bv
        s = np.exp(z - z.max()); s /= s.sum()
        s[lab[b, j]] -= 1
        dbv += s / len(slots)
    np.testing.assert_allclose(g["head.decoder.bias"], dbv, atol=1e-14)


# -- Adam closed forms ---------------------------------------------------------------------------------

def test_adam_closed_forms():
    rng = np.random.default_rng(6)
    w = rng.standard_normal(50); g = rng.standard_normal(50)
    z = np.zeros(50)
    lr, eps = 1e-2, 1e-6
    # step 1 with bias correction and no decay: dw = -lr * g / (|g| + eps)
    w1, m1, v1 = O.adam_update(w, g, z, z, 1, lr, 0.9, 0.999, eps, 0.0, True)
    np.testing.assert_allclose(w1 - w, -lr * g / (np.abs(g) + eps), atol=1e-15)
    np.testing.assert_allclose(m1, 0.1 * g); np.testing.assert_allclose(v1, 0.001 * g * g)
    # zero gradient: only the decay term moves the weight
    w2, _, _ = O.adam_update(w, z, z, z, 1, lr, 0.9, 0.999, eps, 0.1, True)
    np.testing.assert_allclose(w2, w * (1 - lr * 0.1), atol=1e-15)
    # beta1 = beta2 = 0 without bias correction: sign-like step at any t
    w3, _, _ = O.adam_update(w, g, rng.standard_normal(50), np.abs(rng.standard_normal(50)), 7,
                             lr, 0.0, 0.0, eps, 0.0, False)
    np.testing.assert_allclose(w3 - w, -lr * g / (np.abs(g) + eps), atol=1e-15)
    # two steps with a constant gradient: m_hat = g, v_hat = g^2 again
    wa, ma, va = O.adam_update(w, g, z, z, 1, lr, 0.9, 0.999, eps, 0.0, True)
    wb, _, _ = O.adam_update(wa, g, ma, va, 2, lr, 0.9, 0.999, eps, 0.0, True)
    np.testing.assert_allclose(wb - wa, -lr * g / (np.abs(g) + eps), atol=1e-14)


def test_step_applies_decay_to_matrices_only():
    m = tiny_model(top_k=0)
    m.set_optimizer(lr=0.0)
    tok, lens, pos, lab = tiny_batch()
    before = {k: v.copy() for k, v in m.p.items()}
    m.step(tok, lens, pos, lab)
    for k in before:
        assert np.array_equal(before[k], m.p[k])       # lr = 0 moves nothing
    m2 = tiny_model(top_k=0)
    m2.set_optimizer(lr=1e-3, weight_decay=0.5, beta1=0.0, beta2=0.0, bias_correction=0, eps=1e-6)
    _, g = m2.loss_and_grads(tok, lens, pos, lab)
    w0 = {k: v.copy() for k, v in m2.p.items()}
    m2.step(tok, lens, pos, lab)
    for n in O.HEAD_TENSORS:
        wd = 0.5 if w0[n].ndim == 2 else 0.0
        want = w0[n] - 1e-3 * (g[n] / (np.abs(g[n]) + 1e-6) + wd * w0[n])
        np.testing.assert_allclose(m2.p[n], want, atol=1e-14)


def _first_step_form(m, g, w0, lr, eps):
    """With bias correction and no decay the first Adam step moves every weight by
    -lr * g / (|g| + eps): m_hat = g and v_hat = g^2 whatever the betas are.  It holds only while
    the counter that enters the bias correction reads 1, so it pins the counter itself."""
    for n in m.trainable_names():
        np.testing.assert_allclose(m.p[n] - w0[n], -lr * g[n] / (np.abs(g[n]) + eps), atol=1e-13, err_msg=n)


def test_step_counter_starts_at_one_and_restarts_with_every_stage_change():
    lr, eps = 1e-2, 1e-6
    cfg = I.scaled(TINY, layers=2)
    w = I.make_weights(cfg, seed=5, variant="parity", std=0.3)
    m = O.MsltOracle(w, cfg.heads, max_layers=4)
    m.set_optimizer(lr=lr, eps=eps, weight_decay=0.0, beta1=0.9, beta2=0.999, bias_correction=1)
    tok, lens, pos, lab = tiny_batch()

    def one_step():
        w0 = {k: v.copy() for k, v in m.p.items()}
        _, g = m.loss_and_grads(tok, lens, pos, lab)
        g = {k: v.copy() for k, v in g.items()}
        m.step(tok, lens, pos, lab)
        return w0, g

    m.set_trainable(1)
    w0, g = one_step()
    _first_step_form(m, g, w0, lr, eps)             # a counter that started at 0 or 2 fails here
    # the second step is not of that form (m and v now carry history) ...
    w0, g = one_step()
    moved = np.concatenate([(m.p[n] - w0[n]).ravel() for n in m.trainable_names()])
    first = np.concatenate([(-lr * g[n] / (np.abs(g[n]) + eps)).ravel() for n in m.trainable_names()])
    assert np.abs(moved - first).max() > 1e-4
    assert m.t == 2
    # changing the trainable slice clears the moments and the counter: first-step form again,
    # also for tensors that were trainable (and had history) before
    m.set_trainable(2)
    assert m.t == 0
    w0, g = one_step()
    _first_step_form(m, g, w0, lr, eps)
    # so does stacking (the new layers and the head both restart)
    one_step()
    m.add_layers(2)
    assert m.t == 0 and m.top_k == 2
    w0, g = one_step()
    _first_step_form(m, g, w0, lr, eps)
    # without the restart the same call would not have the first-step form: plant the mistake
    m.t = 3
    w0, g = one_step()
    with pytest.raises(AssertionError):
        _first_step_form(m, g, w0, lr, eps)


def test_second_step_bias_correction_closed_form():
    # constant gradient through step(): with g fixed, m_hat = g and v_hat = g^2 at every t, so each of
    # the first steps moves head.decoder.bias by the same -lr * g / (|g| + eps) only if t counts 1, 2, ...
    lr, eps = 1e-3, 1e-6
    m = tiny_model(top_k=0)
    m.set_optimizer(lr=lr, eps=eps, weight_decay=0.0, bias_correction=1)
    g = np.linspace(-1.0, 1.0, m.p["head.decoder.bias"].size)
    g[np.abs(g) < 1e-3] = 0.5
    m.loss_and_grads = lambda *a: (0.0, {n: (g.copy() if n == "head.decoder.bias" else np.zeros_like(m.p[n]))
                                         for n in m.trainable_names()})
    tok, lens, pos, lab = tiny_batch()
    for t in (1, 2, 3):
        w0 = m.p["head.decoder.bias"].copy()
        m.step(tok, lens, pos, lab)
        assert m.t == t
        np.testing.assert_allclose(m.p["head.decoder.bias"] - w0, -lr * g / (np.abs(g) + eps), atol=1e-15)


# -- staging ------------------------------------------------------------------------------------------------

def test_truncated_gradients_equal_full_gradients_on_the_trainable_slice():
    tok, lens, pos, lab = tiny_batch()
    full = tiny_model(top_k=2)
    _, gf = full.loss_and_grads(tok, lens, pos, lab)
    for k in (0, 1):
        part = tiny_model(top_k=k)
        _, gp = part.loss_and_grads(tok, lens, pos, lab)
        for n in gp:
            np.testing.assert_allclose(gp[n], gf[n], atol=1e-15, rtol=0)
        assert "emb.word" not in gp and "layer.0.qkv.weight" not in gp


def test_add_layers_copies_top_layers_in_order():
    cfg = I.scaled(TINY, layers=2)
    w = I.make_weights(cfg, seed=5, std=0.3)
    m = O.MsltOracle(w, cfg.heads, max_layers=4)
    tok, lens, pos, lab = tiny_batch()
    h_before, _ = m.forward(tok, lens)
    m.add_layers(2)
    assert m.L == 4
    for t in O.LAYER_TENSORS:
        assert np.array_equal(m.p[f"layer.2.{t}"], m.p[f"layer.0.{t}"])
        assert np.array_equal(m.p[f"layer.3.{t}"], m.p[f"layer.1.{t}"])
    assert not np.array_equal(m.p["layer.2.qkv.weight"], m.p["layer.3.qkv.weight"])
    # the old prefix still computes the same thing
    m2 = O.MsltOracle(w, cfg.heads)
    h2, _ = m2.forward(tok, lens)
    assert np.array_equal(h_before, h2)
    with pytest.raises(ValueError):
        m.add_layers(1)                      # arena full
    m3 = O.MsltOracle(w, cfg.heads, max_layers=8)
    with pytest.raises(ValueError):
        m3.add_layers(3)                     # k > L
    # staged training after stacking: new layers move, old ones do not
    m.set_trainable(2)
    before = {k: v.copy() for k, v in m.p.items()}
    m.step(tok, lens, pos, lab)
    for k in before:
        frozen = k.startswith("emb.") or k.startswith("layer.0.") or k.startswith("layer.1.")
        assert np.array_equal(before[k], m.p[k]) == frozen, k


def test_forward_equals_forward_inside_step():
    m = tiny_model(top_k=1)
    tok, lens, pos, lab = tiny_batch()
    h, logits = m.forward(tok, lens, pos)
    x, _, _ = m.encode(tok, lens, keep_from=1)
    assert np.array_equal(h, x)
    l2, _ = m._head_forward(x, pos, lab)
    ok = (pos >= 0).reshape(-1)
    assert np.array_equal(logits[ok], l2[ok])


# -- masking and batch structure ---------------------------------------------------------------------------------

def test_padding_content_does_not_matter():
    m = tiny_model(top_k=2)
    tok, lens, pos, lab = tiny_batch()
    l1, g1 = m.loss_and_grads(tok, lens, pos, lab)
    tok2 = tok.copy()
    for b in range(tok.shape[0]):
        tok2[b, lens[b]:] = (tok2[b, lens[b]:] + 3) % TINY.vocab
    assert not np.array_equal(tok, tok2)
    l2, g2 = m.loss_and_grads(tok2, lens, pos, lab)
    assert abs(l1 - l2) < 1e-15
    for n in g1:
        if n == "emb.word":
            continue       # rows of the padded token ids receive (zero) scatter entries
        np.testing.assert_allclose(g1[n], g2[n], atol=1e-15, rtol=0)
    np.testing.assert_allclose(g1["emb.word"], g2["emb.word"], atol=1e-15, rtol=0)


def test_batch_loss_and_gradients_are_slot_weighted_sums():
    m = tiny_model(top_k=2)
    tok, lens, pos, lab = tiny_batch()
    L, G = m.loss_and_grads(tok, lens, pos, lab)
    n_all = int((pos >= 0).sum())
    acc_l, acc_g = 0.0, None
    for b in range(tok.shape[0]):
        sl = slice(b, b + 1)
        nb = int((pos[sl] >= 0).sum())
        lb, gb = m.loss_and_grads(tok[sl], lens[sl], pos[sl], lab[sl])
        acc_l += lb * nb / n_all
        gb = {k: v * nb / n_all for k, v in gb.items()}
        acc_g = gb if acc_g is None else {k: acc_g[k] + gb[k] for k in gb}
    assert abs(L - acc_l) < 1e-14
    for n in G:
        np.testing.assert_allclose(G[n], acc_g[n], atol=1e-14, rtol=0)


def test_training_reduces_the_loss():
    m = tiny_model(top_k=1)
    m.set_optimizer(lr=1e-2)
    tok, lens, pos, lab = tiny_batch()
    losses = [m.step(tok, lens, pos, lab) for _ in range(20)]
    assert losses[-1] < losses[0] - 0.1


# -- the input generators ------------------------------------------------------------------------------------------

def test_batches_follow_the_recipe():
    cfg = I.scaled(I.CONFIGS["large_long"], batch=8)
    tok, lens, pos, lab = I.make_batch(cfg)
    assert tok.dtype == np.int32 and tok.shape == (8, 512)
    assert lens.min() >= 256 and lens.max() <= 512
    for b in range(8):
        n = int((pos[b] >= 0).sum())
        assert n == min(cfg.pred, max(1, round(0.15 * lens[b])))
        assert np.all(pos[b, :n] < lens[b]) and len(set(pos[b, :n])) == n
        assert np.all((lab[b, :n] >= 0) & (lab[b, :n] < cfg.vocab))
        assert np.all(pos[b, n:] == -1) and np.all(lab[b, n:] == -1)
        assert np.all(tok[b, lens[b]:] == 0)
    t2, _, _, _ = I.make_batch(cfg)
    assert np.array_equal(tok, t2)
    big = I.zipf_tokens(I._rng(1, 1), 30522, (200000,))
    assert 0.05 < (big == 0).mean() < 0.2 and big.max() > 10000   # Zipf head and tail
    a = I.make_batch(I.scaled(I.CONFIGS["base_stage"], batch=2))
    b = I.make_batch(I.scaled(I.CONFIGS["base_full"], batch=2))
    assert all(np.array_equal(x, y) for x, y in zip(a, b))         # same seed, same data


# -- LAMB (the optimizer of the paper's experiments, Section 4.1) -----------------------------------

def _lamb_by_hand(w, g, m, v, t, lr, b1, b2, eps, wd, bc):
    """The same rule element by element with plain Python floats."""
    n = len(w)
    m2 = [b1 * m[i] + (1 - b1) * g[i] for i in range(n)]
    v2 = [b2 * v[i] + (1 - b2) * g[i] * g[i] for i in range(n)]
    c1 = 1 - b1 ** t if bc else 1.0
    c2 = 1 - b2 ** t if bc else 1.0
    r = [(m2[i] / c1) / (math.sqrt(v2[i] / c2) + eps) + wd * w[i] for i in range(n)]
    wn = math.sqrt(sum(x * x for x in w)); rn = math.sqrt(sum(x * x for x in r))
    ratio = wn / rn if wn > 0 and rn > 0 else 1.0
    return [w[i] - lr * ratio * r[i] for i in range(n)], m2, v2


def test_lamb_closed_forms():
    rng = np.random.default_rng(16)
    n = 40
    w = rng.standard_normal(n); g = rng.standard_normal(n) * 3
    z = np.zeros(n)
    lr, eps = 0.00088, 1e-6
    # brute force, with history and decay
    m0 = rng.standard_normal(n) * 0.1; v0 = np.abs(rng.standard_normal(n)) * 0.1
    got = O.lamb_update(w, g, m0, v0, 5, lr, 0.9, 0.999, eps, 0.01, True)
    want = _lamb_by_hand(list(w), list(g), list(m0), list(v0), 5, lr, 0.9, 0.999, eps, 0.01, True)
    for a, b in zip(got, want):
        np.testing.assert_allclose(a, np.array(b), rtol=1e-12, atol=1e-15)
    # first step, no decay: the direction is g / (|g| + eps), one unit per element, so the step of every
    # element has size lr * ||w|| / sqrt(n) (up to eps / |g|) whatever the size of the gradient
    w1, _, _ = O.lamb_update(w, g, z, z, 1, lr, 0.9, 0.999, eps, 0.0, True)
    r = g / (np.abs(g) + eps)
    np.testing.assert_allclose(w1 - w, -lr * np.linalg.norm(w) / np.linalg.norm(r) * r, atol=1e-15)
    big = np.abs(g) > 1e-2
    np.testing.assert_allclose(np.abs(w1 - w)[big], lr * np.linalg.norm(w) / math.sqrt(n), rtol=2e-4)
    # the update does not change when the gradient is rescaled (eps aside) ...
    w1b, _, _ = O.lamb_update(w, 100.0 * g, z, z, 1, lr, 0.9, 0.999, 0.0 + 1e-30, 0.0, True)
    w1c, _, _ = O.lamb_update(w, g, z, z, 1, lr, 0.9, 0.999, 0.0 + 1e-30, 0.0, True)
    np.testing.assert_allclose(w1b, w1c, atol=1e-14)
    # ... and scales with the weights: the step is relative to ||w||
    w3, _, _ = O.lamb_update(3.0 * w, g, z, z, 1, lr, 0.9, 0.999, eps, 0.0, True)
    np.testing.assert_allclose(w3 - 3.0 * w, 3.0 * (w1 - w), atol=1e-14)
    # the norm of the whole step is lr * ||w|| exactly (that is what the trust ratio does)
    assert abs(np.linalg.norm(w1 - w) - lr * np.linalg.norm(w)) < 1e-14
    wd_step, _, _ = O.lamb_update(w, g, m0, v0, 7, lr, 0.9, 0.999, eps, 0.05, True)
    assert abs(np.linalg.norm(wd_step - w) - lr * np.linalg.norm(w)) < 1e-14
    # zero gradient and no decay: nothing moves; zero gradient with decay: pure shrink by lr (ratio = 1 / wd)
    w4, _, _ = O.lamb_update(w, z, z, z, 1, lr, 0.9, 0.999, eps, 0.0, True)
    assert np.array_equal(w4, w)
    w5, _, _ = O.lamb_update(w, z, z, z, 1, lr, 0.9, 0.999, eps, 0.1, True)
    np.testing.assert_allclose(w5, w * (1 - lr), atol=1e-15)
    # a tensor of zeros has no norm to be relative to: trust ratio 1, i.e. a plain Adam step
    w6, _, _ = O.lamb_update(z, g, z, z, 1, lr, 0.9, 0.999, eps, 0.0, True)
    w6a, _, _ = O.adam_update(z, g, z, z, 1, lr, 0.9, 0.999, eps, 0.0, True)
    np.testing.assert_allclose(w6, w6a, atol=1e-18)
    # moments are Adam's
    _, mm, vv = O.lamb_update(w, g, m0, v0, 5, lr, 0.9, 0.999, eps, 0.01, True)
    _, ma, va = O.adam_update(w, g, m0, v0, 5, lr, 0.9, 0.999, eps, 0.01, True)
    assert np.array_equal(mm, ma) and np.array_equal(vv, va)


def test_step_with_lamb_updates_every_trainable_tensor_by_its_own_norm():
    m = tiny_model(top_k=1)
    lr = 0.00088
    m.set_optimizer(lr=lr, weight_decay=0.0, lamb=1)
    tok, lens, pos, lab = tiny_batch()
    before = {k: v.copy() for k, v in m.p.items()}
    m.step(tok, lens, pos, lab)
    names = set(m.trainable_names())
    for k in before:
        if k in names:
            # the trust ratio is per tensor: each tensor's step has norm lr * its own norm
            assert abs(np.linalg.norm(m.p[k] - before[k]) - lr * np.linalg.norm(before[k])) < 1e-12, k
        else:
            assert np.array_equal(m.p[k], before[k]), k


# -- grouped parameter sharing (Section 3.3: the paper's change to ALBERT) ------------------------------

SHARED = I.scaled(TINY, layers=4, trainable=2, share_group=2, seed_index=78)


def _unshared_twin(m):
    """The same network with every layer given its own copy of its group's block."""
    w = {k: v.copy() for k, v in m.p.items() if not k.startswith("layer.")}
    for l in range(m.L):
        for t in O.LAYER_TENSORS:
            w[f"layer.{l}.{t}"] = m.p[f"layer.{l // m.g}.{t}"].copy()
    return O.MsltOracle(w, m.heads, ln_eps=m.eps)


@pytest.mark.parametrize("top_k", [2, 4])
def test_shared_group_gradient_is_the_sum_over_its_layers(top_k):
    w = I.make_weights(SHARED, seed=5, variant="parity", std=0.3)
    assert "layer.1.qkv.weight" in w and "layer.2.qkv.weight" not in w      # two blocks for four layers
    m = O.MsltOracle(w, SHARED.heads, share_group=2)
    assert m.L == 4
    m.set_trainable(top_k)
    tok, lens, pos, lab = tiny_batch(SHARED)
    twin = _unshared_twin(m)
    twin.set_trainable(top_k)
    # same function of the same numbers ...
    h, _ = m.forward(tok, lens)
    h2, _ = twin.forward(tok, lens)
    assert np.array_equal(h, h2)
    loss, g = m.loss_and_grads(tok, lens, pos, lab)
    loss2, g2 = twin.loss_and_grads(tok, lens, pos, lab)
    assert loss == loss2
    # ... and the gradient of a shared block is the sum of the gradients its layers would get alone
    assert set(g) == set(m.trainable_names())
    for b in range((4 - top_k) // 2, 2):
        for t in O.LAYER_TENSORS:
            np.testing.assert_allclose(g[f"layer.{b}.{t}"], g2[f"layer.{2 * b}.{t}"] + g2[f"layer.{2 * b + 1}.{t}"],
                                       rtol=0, atol=1e-13)
    for n in O.HEAD_TENSORS:
        np.testing.assert_allclose(g[n], g2[n], rtol=0, atol=1e-14)


def test_shared_group_gradients_match_finite_differences():
    w = I.make_weights(SHARED, seed=5, variant="parity", std=0.3)
    m = O.MsltOracle(w, SHARED.heads, share_group=2)
    m.set_trainable(2)
    tok, lens, pos, lab = tiny_batch(SHARED)
    _, g = m.loss_and_grads(tok, lens, pos, lab)
    h = 1e-5
    for name in ("layer.1.qkv.weight", "layer.1.ln1.gamma", "layer.1.ffn2.bias", "layer.1.out.weight"):
        wt = m.p[name]
        fd = np.zeros_like(wt)
        it = np.nditer(wt, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = wt[idx]
            wt[idx] = keep + h; lp = m.loss(tok, lens, pos, lab)
            wt[idx] = keep - h; lm = m.loss(tok, lens, pos, lab)
            wt[idx] = keep
            fd[idx] = (lp - lm) / (2 * h)
        assert np.abs(fd - g[name]).max() / max(np.abs(fd).max(), 1e-8) < 1e-6, name


def test_shared_groups_stack_and_train_by_whole_groups():
    cfg = I.scaled(SHARED, layers=2)
    w = I.make_weights(cfg, seed=5, variant="parity", std=0.3)
    m = O.MsltOracle(w, cfg.heads, max_layers=4, share_group=2)
    assert m.L == 2 and m.trainable_names().count("layer.0.qkv.weight") == 1
    with pytest.raises(ValueError):
        m.add_layers(1)                       # half a group
    with pytest.raises(ValueError):
        m.set_trainable(1)
    m.add_layers(2)                           # the new group starts as a copy of the top group
    assert m.L == 4 and np.array_equal(m.p["layer.1.ffn1.weight"], m.p["layer.0.ffn1.weight"])
    m.set_trainable(2)
    assert "layer.1.ffn1.weight" in m.trainable_names() and "layer.0.ffn1.weight" not in m.trainable_names()
    before = {k: v.copy() for k, v in m.p.items()}
    m.step(*tiny_batch(SHARED))
    for k in before:                          # only the new group and the output layer move
        moved = not np.array_equal(before[k], m.p[k])
        assert moved == (k.startswith("layer.1.") or k.startswith("head.")), k


# -- next-sentence prediction and segment embeddings (Section 4.1: "the same MLM and NSP objectives") ----

NSP = I.scaled(TINY, nsp=True, seed_index=79)


def _nsp_case(top_k):
    w = I.make_weights(NSP, seed=5, variant="parity", std=0.3)
    m = O.MsltOracle(w, NSP.heads)
    m.set_trainable(top_k)
    tok, lens, pos, lab = tiny_batch(NSP)
    seg, nlab = I.make_nsp(NSP, lens, seed=9)
    assert seg.max() == 1 and seg.min() == 0
    return m, (tok, lens, pos, lab, seg, nlab)


@pytest.mark.parametrize("top_k", [0, 1, 2])
def test_nsp_gradients_match_finite_differences(top_k):
    m, batch = _nsp_case(top_k)
    assert m.nsp
    loss, g = m.loss_and_grads(*batch)
    names = m.trainable_names()
    assert set(g) == set(names) and "head.nsp.weight" in names
    assert ("emb.type" in names) == (top_k == 2)
    assert abs(loss - (m.losses["mlm"] + m.losses["nsp"])) < 1e-14 and m.losses["nsp"] > 0
    h = 1e-5
    for name in names:
        wt = m.p[name]
        fd = np.zeros_like(wt)
        it = np.nditer(wt, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = wt[idx]
            wt[idx] = keep + h; lp = m.loss(*batch)
            wt[idx] = keep - h; lm = m.loss(*batch)
            wt[idx] = keep
            fd[idx] = (lp - lm) / (2 * h)
        assert np.abs(fd - g[name]).max() / max(np.abs(fd).max(), 1e-8) < 1e-6, name
        if name != "emb.pos":
            assert np.abs(g[name]).max() > 0, name


def test_nsp_head_matches_torch_functional_and_zero_classifier_gives_log_two():
    m, (tok, lens, pos, lab, seg, nlab) = _nsp_case(1)
    x, _, _ = m.encode(tok, lens, segments=seg)
    F = torch.nn.functional
    T = lambda n: torch.from_numpy(m.p[n])
    pooled = torch.tanh(F.linear(torch.from_numpy(x[:, 0, :]), T("head.pooler.weight"), T("head.pooler.bias")))
    want = F.cross_entropy(F.linear(pooled, T("head.nsp.weight"), T("head.nsp.bias")),
                           torch.from_numpy(nlab.astype(np.int64))).item()
    assert abs(m._nsp_forward(x, nlab)[0] - want) < 1e-12
    # embeddings with segments against torch
    e = F.embedding(torch.from_numpy(tok.astype(np.int64)), T("emb.word")) + T("emb.pos")[: tok.shape[1]]
    e = e + F.embedding(torch.from_numpy(seg.astype(np.int64)), T("emb.type"))
    want_e = F.layer_norm(e, (NSP.hidden,), T("emb.ln.gamma"), T("emb.ln.beta"), eps=1e-12).numpy()
    np.testing.assert_allclose(m._embed(tok, seg)[0], want_e, atol=1e-12, rtol=0)
    # a zero classifier cannot tell the two classes apart: loss ln 2 exactly
    m.p["head.nsp.weight"][:] = 0.0; m.p["head.nsp.bias"][:] = 0.0
    assert abs(m._nsp_forward(x, nlab)[0] - math.log(2.0)) < 1e-15
    # ignored labels drop out of the mean
    nl2 = nlab.copy(); nl2[0] = -1
    m2, _ = _nsp_case(1)
    full = m2._nsp_forward(x, nlab)[0]
    part = m2._nsp_forward(x, nl2)[0]
    one = m2._nsp_forward(x[1:], nlab[1:])[0]
    assert abs(part - one) < 1e-14 and abs(full - part) > 1e-6


def test_without_nsp_labels_the_nsp_parameters_get_zero_gradient_and_mlm_is_unchanged():
    m, (tok, lens, pos, lab, seg, nlab) = _nsp_case(1)
    loss, g = m.loss_and_grads(tok, lens, pos, lab, seg, None)
    assert loss == m.losses["mlm"] and m.losses["nsp"] == 0.0
    for n in O.NSP_HEAD_TENSORS:
        assert not g[n].any()
