"""Pins for the whole-step oracle: finite differences, an independent library route
(the same model in torch float64 autograd + torch.optim.AdamW), and invariants of the
GPT-2 training step.  No CUDA involved.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import seeded_inputs as si

TINY = si.make_config(n_layers=2, d_model=16, n_heads=2, seq_len=6, vocab_size=11, padded_vocab_size=12)


def _model(cfg, seed=0, jitter=0.05):
    m = oracle.Model(cfg)
    params = si.init_params(cfg, seed, jitter=jitter)
    m.set_params(params)
    return m, params


# ------------------------------------------------------------------ torch float64 route

def torch_gpt2_loss(cfg, params, tok, tgt):
    """The same network written with torch library ops in float64 (independent of oracle.c)."""
    F = torch.nn.functional
    L, C, H, T = cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["seq_len"]
    B = tok.shape[0]
    d = C // H
    tok_t = torch.tensor(tok, dtype=torch.long)
    x = params["wte"][tok_t] + params["wpe"][None, :T]
    for l in range(L):
        p = lambda s: params[f"h{l}.{s}"]
        a = F.layer_norm(x, (C,), p("ln1.g"), p("ln1.b"), 1e-5)
        qkv = F.linear(a, p("attn.qkv.w"), p("attn.qkv.b"))
        q, k, v = qkv.view(B, T, 3, H, d).permute(2, 0, 3, 1, 4)
        o = F.scaled_dot_product_attention(q, k, v, is_causal=True)
        o = o.permute(0, 2, 1, 3).reshape(B, T, C)
        x = x + F.linear(o, p("attn.proj.w"), p("attn.proj.b"))
        mm = F.layer_norm(x, (C,), p("ln2.g"), p("ln2.b"), 1e-5)
        h = F.linear(mm, p("mlp.fc.w"), p("mlp.fc.b"))
        x = x + F.linear(F.gelu(h), p("mlp.proj.w"), p("mlp.proj.b"))
    xf = F.layer_norm(x, (C,), params["lnf.g"], params["lnf.b"], 1e-5)
    logits = F.linear(xf, params["wte"])
    loss = F.cross_entropy(logits.view(B * T, -1), torch.tensor(tgt, dtype=torch.long).view(-1))
    return loss, logits


def _torch_params(params):
    return {k: torch.tensor(np.asarray(v, dtype=np.float64), requires_grad=True) for k, v in params.items()}


@pytest.mark.parametrize("cfg", [TINY, si.make_config(1, 16, 4, 5, 9, 9)])
def test_loss_and_gradients_match_torch_autograd(cfg):
    m, params = _model(cfg, seed=3)
    tok, tgt = si.uniform_tokens(5, 3, cfg["seq_len"], cfg["vocab_size"])
    loss = m.loss_and_grad(tok, tgt)
    tp = _torch_params(params)
    tl, tlogits = torch_gpt2_loss(cfg, tp, tok, tgt)
    tl.backward()
    assert abs(loss - float(tl.detach())) < 1e-12
    np.testing.assert_allclose(m.activation("logits"), tlogits.detach().numpy().reshape(-1, cfg["padded_vocab_size"]),
                               rtol=1e-11, atol=1e-13)
    for name, g in m.grads().items():
        ref = tp[name].grad.numpy().ravel()
        assert np.abs(g - ref).max() <= 1e-11 * max(1.0, np.abs(ref).max()), name


def test_three_training_steps_match_torch_adamw():
    cfg = TINY
    m, params = _model(cfg, seed=7)
    tp = _torch_params(params)
    decay = [tp[n] for n in tp if m.decay(n)]
    nodecay = [tp[n] for n in tp if not m.decay(n)]
    hp = si.ADAMW
    opt = torch.optim.AdamW([{"params": decay, "weight_decay": hp["weight_decay"]},
                             {"params": nodecay, "weight_decay": 0.0}],
                            lr=hp["lr"], betas=(hp["beta1"], hp["beta2"]), eps=hp["eps"])
    for step in range(3):
        tok, tgt = si.uniform_tokens(100 + step, 2, cfg["seq_len"], cfg["vocab_size"])
        loss = m.loss_and_grad(tok, tgt)
        # scale the gradients up so that the clip is active on some steps
        if step == 1:
            for n in m.names():
                m.set_tensor(n, m.get(n, 1) * 50.0, kind=1)
        gn = m.adamw_step(hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"], hp["grad_clip"])
        opt.zero_grad()
        tl, _ = torch_gpt2_loss(cfg, tp, tok, tgt)
        tl.backward()
        if step == 1:
            for q in tp.values():
                q.grad *= 50.0
        tgn = torch.nn.utils.clip_grad_norm_(list(tp.values()), hp["grad_clip"])
        opt.step()
        assert abs(loss - float(tl.detach())) < 1e-11
        assert abs(gn - float(tgn)) < 1e-10 * max(1.0, gn)
        if step == 1:
            assert gn > 1.0 and m.last_scale() < 1.0
        for n in m.names():
            np.testing.assert_allclose(m.get(n), tp[n].detach().numpy().ravel(), rtol=1e-10, atol=1e-12, err_msg=n)


# ------------------------------------------------------------------ finite differences

@pytest.mark.parametrize("cfg,seed", [(TINY, 11), (si.make_config(1, 16, 2, 4, 7, 8), 12)])
def test_gradients_match_finite_differences(cfg, seed):
    m, params = _model(cfg, seed=seed)
    tok, tgt = si.uniform_tokens(seed, 2, cfg["seq_len"], cfg["vocab_size"])
    m.loss_and_grad(tok, tgt)
    grads = m.grads()
    rng = np.random.default_rng(seed)
    for name in m.names():
        p = m.get(name)
        k = min(p.size, 6)
        for i in rng.choice(p.size, k, replace=False):
            h = 1e-5 * max(1.0, abs(p[i]))
            q = p.copy()
            q[i] = p[i] + h
            m.set_tensor(name, q)
            lp = m.loss(tok, tgt)
            q[i] = p[i] - h
            m.set_tensor(name, q)
            lm = m.loss(tok, tgt)
            fd = (lp - lm) / (2 * h)
            assert abs(fd - grads[name][i]) <= 1e-6 * max(abs(fd), 1e-3), (name, i, fd, grads[name][i])
        m.set_tensor(name, p)


def test_tied_embedding_gradient_is_sum_of_both_uses():
    """A token row of wte is used by the gather and by the LM head; FD sees the sum."""
    cfg = TINY
    m, _ = _model(cfg, seed=21)
    tok, tgt = si.uniform_tokens(21, 2, cfg["seq_len"], cfg["vocab_size"])
    m.loss_and_grad(tok, tgt)
    g = m.get("wte", 1).reshape(cfg["padded_vocab_size"], -1)
    used = int(tok[0, 0])
    unused = cfg["padded_vocab_size"] - 1           # padding row: never an input token
    assert used != unused
    p = m.get("wte")
    C = cfg["d_model"]
    for row in (used, unused):
        i = row * C + 3
        h = 1e-5
        q = p.copy(); q[i] += h; m.set_tensor("wte", q); lp = m.loss(tok, tgt)
        q[i] -= 2 * h; m.set_tensor("wte", q); lm = m.loss(tok, tgt)
        m.set_tensor("wte", p)
        assert abs((lp - lm) / (2 * h) - g[row, 3]) < 1e-7
    # the padding row still gets an LM-head gradient (softmax runs over the padded vocabulary)
    assert np.abs(g[unused]).max() > 0.0


# ------------------------------------------------------------------ invariants of the step

def test_initial_loss_is_log_vocab_plus_half_logit_variance():
    cfg = si.config(0)
    m = oracle.Model(cfg)
    m.set_params(si.init_params(cfg, 0))
    tok, tgt = si.tokens_for(cfg, 0)
    loss = m.loss(tok, tgt)
    C, Vp = cfg["d_model"], cfg["padded_vocab_size"]
    # logits of a unit-variance LayerNorm output against N(0, 0.02^2) rows have variance C * 0.02^2
    expect = math.log(Vp) + 0.5 * C * 0.02 ** 2
    assert abs(loss - expect) < 0.05, (loss, expect)
    assert abs(loss - math.log(cfg["vocab_size"])) < 0.1


def test_model_is_causal():
    cfg = TINY
    m, _ = _model(cfg, seed=5)
    tok, tgt = si.uniform_tokens(5, 2, cfg["seq_len"], cfg["vocab_size"])
    m.loss(tok, tgt)
    l1 = m.activation("logits")
    tok2 = tok.copy()
    t0 = 3
    tok2[0, t0] = (tok2[0, t0] + 1) % cfg["vocab_size"]
    m.loss(tok2, tgt)
    l2 = m.activation("logits")
    T = cfg["seq_len"]
    assert np.array_equal(l1[:t0], l2[:t0])
    assert np.array_equal(l1[T:], l2[T:])
    assert not np.array_equal(l1[t0], l2[t0])


def test_key_bias_gradient_vanishes():
    """Softmax is invariant to a per-row shift of the scores, so d loss / d (key bias) = 0."""
    cfg = TINY
    m, _ = _model(cfg, seed=9)
    tok, tgt = si.uniform_tokens(9, 3, cfg["seq_len"], cfg["vocab_size"])
    m.loss_and_grad(tok, tgt)
    C = cfg["d_model"]
    gb = m.get("h0.attn.qkv.b", 1)
    assert np.abs(gb[C:2 * C]).max() < 1e-16 * 1e3
    assert np.abs(gb[:C]).max() > 1e-6 and np.abs(gb[2 * C:]).max() > 1e-6


def test_chunked_batch_equals_whole_batch():
    cfg = TINY
    m, _ = _model(cfg, seed=13)
    tok, tgt = si.uniform_tokens(13, 4, cfg["seq_len"], cfg["vocab_size"])
    l_all = m.loss_and_grad(tok, tgt)
    g_all = m.grads()
    l_chunk = m.loss_and_grad(tok, tgt, chunk=1)
    assert abs(l_all - l_chunk) < 1e-13
    for n, g in m.grads().items():
        np.testing.assert_allclose(g, g_all[n], rtol=1e-10, atol=1e-15, err_msg=n)


def test_zipf_generator_statistics():
    tok, tgt = si.zipf_tokens(2, 8, 1024, 50257)
    assert tok.shape == (8, 1024) and np.array_equal(tok[:, 1:], tgt[:, :-1])
    assert tok.min() >= 0 and tok.max() < 50257
    w = np.arange(1, 50258, dtype=np.float64) ** -1.1
    p0 = w[0] / w.sum()
    frac0 = float((tok == 0).mean())
    assert abs(frac0 - p0) < 0.02                    # rank-1 token carries about 14% of positions
    assert 1500 < np.unique(tok).size < 3500
