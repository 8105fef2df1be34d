"""Pins for the per-op functions of the CPU oracle.

Each check ties the oracle to something other than its own code: a library routine
(numpy matmul, scipy erf / logsumexp, torch float64 autograd and optimizers), a closed
form, an invariant the mathematics forces, central finite differences, or a brute-force
loop on a tiny input.  None of them uses the CUDA path.
"""
import json
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

import oracle
import seeded_inputs as si

rng = np.random.default_rng(1234)


def fd_grad(f, x, idx, h=1e-6):
    """Central difference of scalar f at flat positions idx of array x (modified in place, restored)."""
    out = []
    flat = x.reshape(-1)
    for i in idx:
        old = flat[i]
        step = h * max(1.0, abs(old))
        flat[i] = old + step
        fp = f()
        flat[i] = old - step
        fm = f()
        flat[i] = old
        out.append((fp - fm) / (2 * step))
    return np.array(out)


# ------------------------------------------------------------------ golden: the paper's table

def test_hyperparameters_match_paper_table():
    with open(os.path.join(os.path.dirname(__file__), "golden", "hyperparameters.json")) as f:
        gold = json.load(f)
    cfg = si.config(2)
    m = gold["model"]
    assert cfg["d_model"] == m["d_model"] and cfg["n_layers"] == m["n_layers"]
    assert cfg["n_heads"] == m["n_heads"] and cfg["d_model"] // cfg["n_heads"] == m["head_dim"]
    assert 4 * cfg["d_model"] == m["ffn_hidden"] and cfg["seq_len"] == m["seq_len"]
    assert cfg["vocab_size"] == m["vocab_size"] and cfg["padded_vocab_size"] == m["padded_vocab_size"]
    o = gold["optim"]
    for k in ("lr", "beta1", "beta2", "eps", "weight_decay", "grad_clip"):
        assert si.ADAMW[k] == o[k]
    # "124M": tied embeddings, logical vocabulary
    n = si.num_params(cfg) - (cfg["padded_vocab_size"] - cfg["vocab_size"]) * cfg["d_model"]
    assert round(n / 1e6) == m["size_millions"]
    # init distribution of the registry
    reg = {name: init for name, _, _, init in si.tensor_registry(cfg)}
    assert reg["wte"] == ("normal", 0.02) and reg["wpe"] == ("normal", 0.02)
    assert reg["h3.attn.proj.w"][1] == pytest.approx(0.02 / math.sqrt(24))
    assert reg["h3.mlp.proj.w"][1] == pytest.approx(0.02 / math.sqrt(24))
    assert reg["h3.mlp.fc.w"] == ("normal", 0.02) and reg["h3.attn.qkv.b"] == ("const", 0.0)
    assert reg["h0.ln1.g"] == ("const", 1.0)


# ------------------------------------------------------------------ linear

def test_linear_matches_numpy_matmul():
    x, w, b = rng.standard_normal((37, 29)), rng.standard_normal((23, 29)), rng.standard_normal(23)
    y = oracle.linear_fwd(x, w, b)
    np.testing.assert_allclose(y, x @ w.T + b, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(oracle.linear_fwd(x, w), x @ w.T, rtol=1e-13, atol=1e-13)
    dy = rng.standard_normal((37, 23))
    dx, dw, db = oracle.linear_bwd(dy, x, w)
    np.testing.assert_allclose(dx, dy @ w, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(dw, dy.T @ x, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(db, dy.sum(0), rtol=1e-13, atol=1e-13)


def test_linear_is_not_transposed():
    # a one-hot weight picks a single input feature: catches a swapped [out,in] convention
    x = rng.standard_normal((5, 4))
    w = np.zeros((3, 4))
    w[2, 1] = 1.0
    y = oracle.linear_fwd(x, w)
    assert np.array_equal(y[:, 2], x[:, 1]) and not y[:, :2].any()


# ------------------------------------------------------------------ GELU

def test_gelu_closed_form_and_special_values():
    x = np.concatenate([np.linspace(-8, 8, 2001), rng.standard_normal(1000) * 3])
    ref = 0.5 * x * (1.0 + scipy.special.erf(x / np.sqrt(2.0)))
    np.testing.assert_allclose(oracle.gelu_fwd(x), ref, rtol=1e-14, atol=1e-15)
    np.testing.assert_allclose(oracle.gelu_fwd(x), x * scipy.special.ndtr(x), rtol=1e-12, atol=1e-15)
    assert oracle.gelu_fwd(np.zeros(1))[0] == 0.0
    assert oracle.gelu_bwd(np.zeros(1), np.ones(1))[0] == 0.5
    big = np.array([12.0, 30.0])
    np.testing.assert_allclose(oracle.gelu_fwd(big), big, rtol=1e-15)
    np.testing.assert_allclose(oracle.gelu_fwd(-big), 0.0, atol=1e-30)
    # GELU(-x) = GELU(x) - x
    np.testing.assert_allclose(oracle.gelu_fwd(-x), oracle.gelu_fwd(x) - x, atol=1e-14)


@pytest.mark.parametrize("tanh_form", [False, True])
def test_gelu_backward_matches_torch_and_fd(tanh_form):
    x = rng.standard_normal(500) * 2.5
    dy = rng.standard_normal(500)
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    yt = torch.nn.functional.gelu(xt, approximate="tanh" if tanh_form else "none")
    np.testing.assert_allclose(oracle.gelu_fwd(x, tanh_form), yt.detach().numpy(), rtol=1e-13, atol=1e-15)
    yt.backward(torch.tensor(dy))
    np.testing.assert_allclose(oracle.gelu_bwd(x, dy, tanh_form), xt.grad.numpy(), rtol=1e-12, atol=1e-14)
    h = 1e-6
    fd = (oracle.gelu_fwd(x + h, tanh_form) - oracle.gelu_fwd(x - h, tanh_form)) / (2 * h)
    np.testing.assert_allclose(oracle.gelu_bwd(x, np.ones_like(x), tanh_form), fd, rtol=1e-7, atol=1e-9)


# ------------------------------------------------------------------ LayerNorm

def test_layernorm_forward_invariants_and_library():
    N, C = 19, 48
    x = rng.standard_normal((N, C)) * 3 + 1.5
    y, mean, rstd = oracle.layernorm_fwd(x, np.ones(C), np.zeros(C))
    assert np.abs(y.mean(1)).max() < 1e-14
    var = x.var(1)                                  # biased variance
    np.testing.assert_allclose(y.var(1), var / (var + 1e-5), rtol=1e-12)
    np.testing.assert_allclose(mean, x.mean(1), rtol=1e-14)
    np.testing.assert_allclose(rstd, 1 / np.sqrt(var + 1e-5), rtol=1e-13)
    g, b = rng.standard_normal(C), rng.standard_normal(C)
    y2, _, _ = oracle.layernorm_fwd(x, g, b)
    ref = torch.nn.functional.layer_norm(torch.tensor(x), (C,), torch.tensor(g), torch.tensor(b), 1e-5)
    np.testing.assert_allclose(y2, ref.numpy(), rtol=1e-12, atol=1e-13)


def test_layernorm_backward_library_fd_and_invariants():
    N, C = 11, 40
    x = rng.standard_normal((N, C)) * 2 - 0.7
    g, b = rng.standard_normal(C) + 1.0, rng.standard_normal(C)
    dy = rng.standard_normal((N, C))
    _, mean, rstd = oracle.layernorm_fwd(x, g, b)
    dx, dg, db = oracle.layernorm_bwd(dy, x, g, mean, rstd)
    xt = torch.tensor(x, requires_grad=True)
    gt, bt = torch.tensor(g, requires_grad=True), torch.tensor(b, requires_grad=True)
    torch.nn.functional.layer_norm(xt, (C,), gt, bt, 1e-5).backward(torch.tensor(dy))
    np.testing.assert_allclose(dx, xt.grad.numpy(), rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(dg, gt.grad.numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(db, bt.grad.numpy(), rtol=1e-12, atol=1e-13)
    # the normalisation removes the mean and the xhat component of every row gradient
    xhat = (x - mean[:, None]) * rstd[:, None]
    assert np.abs(dx.sum(1)).max() < 1e-13
    # ... the latter up to the eps in the variance: sum_c dx*xhat = eps * rstd^3 * sum_c dxhat*xhat
    np.testing.assert_allclose((dx * xhat).sum(1), 1e-5 * rstd ** 3 * (dy * g * xhat).sum(1), rtol=1e-7, atol=1e-13)
    f = lambda: float((oracle.layernorm_fwd(x, g, b)[0] * dy).sum())
    idx = rng.choice(N * C, 12, replace=False)
    np.testing.assert_allclose(dx.reshape(-1)[idx], fd_grad(f, x, idx), rtol=1e-6, atol=1e-8)


# ------------------------------------------------------------------ attention

def _torch_attention(qkv, B, T, H):
    C = qkv.shape[-1] // 3
    d = C // H
    q, k, v = qkv.view(B, T, 3, H, d).permute(2, 0, 3, 1, 4)
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)
    return o.permute(0, 2, 1, 3).reshape(B * T, C)


def test_attention_matches_library_forward_and_backward():
    B, T, H, d = 2, 13, 3, 8
    C = H * d
    qkv = rng.standard_normal((B * T, 3 * C))
    d_o = rng.standard_normal((B * T, C))
    o, lse, P = oracle.attention_fwd(qkv, B, T, H, want_probs=True)
    qt = torch.tensor(qkv, requires_grad=True)
    ot = _torch_attention(qt, B, T, H)
    np.testing.assert_allclose(o, ot.detach().numpy(), rtol=1e-12, atol=1e-13)
    ot.backward(torch.tensor(d_o))
    np.testing.assert_allclose(oracle.attention_bwd(qkv, d_o, B, T, H), qt.grad.numpy(), rtol=1e-11, atol=1e-13)
    # softmax rows: probabilities, exact zeros above the diagonal, unit sums
    assert P.min() >= 0.0 and P.max() <= 1.0
    assert np.abs(P.sum(-1) - 1.0).max() < 1e-14
    iu = np.triu_indices(T, 1)
    assert not P[:, :, iu[0], iu[1]].any()
    # lse is the log of the row normaliser of the scaled scores
    q = qkv[:, :C].reshape(B, T, H, d).transpose(0, 2, 1, 3)
    k = qkv[:, C:2 * C].reshape(B, T, H, d).transpose(0, 2, 1, 3)
    S = q @ k.transpose(0, 1, 3, 2) / math.sqrt(d)
    S[:, :, iu[0], iu[1]] = -np.inf
    np.testing.assert_allclose(lse, scipy.special.logsumexp(S, axis=-1), rtol=1e-13)


def test_attention_special_cases():
    H, d = 2, 4
    C = H * d
    # T = 1: the only key is the query's own position, so o = v
    qkv = rng.standard_normal((3, 3 * C))
    o, _ = oracle.attention_fwd(qkv, 3, 1, H)
    np.testing.assert_allclose(o, qkv[:, 2 * C:], rtol=1e-15)
    # q = 0: uniform weights over the prefix, o_i = mean_{j<=i} v_j
    T = 9
    qkv = rng.standard_normal((T, 3 * C))
    qkv[:, :C] = 0.0
    o, _ = oracle.attention_fwd(qkv, 1, T, H)
    ref = np.cumsum(qkv[:, 2 * C:], 0) / np.arange(1, T + 1)[:, None]
    np.testing.assert_allclose(o, ref, rtol=1e-13, atol=1e-14)


def test_attention_is_causal_and_per_sequence():
    B, T, H, d = 2, 10, 2, 4
    C = H * d
    qkv = rng.standard_normal((B * T, 3 * C))
    o1, _ = oracle.attention_fwd(qkv, B, T, H)
    q2 = qkv.copy()
    q2[6] += 1.0                       # position 6 of sequence 0
    o2, _ = oracle.attention_fwd(q2, B, T, H)
    assert np.array_equal(o1[:6], o2[:6])          # earlier positions untouched, bit for bit
    assert np.array_equal(o1[T:], o2[T:])          # other sequence untouched
    assert not np.array_equal(o1[6:T], o2[6:T])


def test_attention_backward_fd():
    B, T, H, d = 1, 7, 2, 4
    C = H * d
    qkv = rng.standard_normal((B * T, 3 * C))
    d_o = rng.standard_normal((B * T, C))
    dqkv = oracle.attention_bwd(qkv, d_o, B, T, H)
    f = lambda: float((oracle.attention_fwd(qkv, B, T, H)[0] * d_o).sum())
    idx = rng.choice(qkv.size, 24, replace=False)
    np.testing.assert_allclose(dqkv.reshape(-1)[idx], fd_grad(f, qkv, idx), rtol=1e-6, atol=1e-9)


# ------------------------------------------------------------------ cross-entropy

def test_softmax_xent_library_and_invariants():
    N, V = 17, 53
    z = rng.standard_normal((N, V)) * 4
    y = rng.integers(0, V, N)
    losses, dz = oracle.softmax_xent(z, y)
    ref = scipy.special.logsumexp(z, axis=1) - z[np.arange(N), y]
    np.testing.assert_allclose(losses, ref, rtol=1e-13)
    zt = torch.tensor(z, requires_grad=True)
    torch.nn.functional.cross_entropy(zt, torch.tensor(y), reduction="mean").backward()
    np.testing.assert_allclose(dz, zt.grad.numpy(), rtol=1e-11, atol=1e-15)
    assert np.abs(dz.sum(1)).max() < 1e-15           # each row sums to zero
    assert np.abs(dz).sum() <= 2.0 + 1e-12
    sm = dz * N
    sm[np.arange(N), y] += 1.0
    assert np.abs(sm.sum(1) - 1.0).max() < 1e-13 and sm.min() >= 0.0
    # shift invariance and a huge-logit row (stability)
    l2, _ = oracle.softmax_xent(z + 1000.0, y)
    np.testing.assert_allclose(l2, losses, rtol=1e-9)
    # uniform logits: loss = ln V exactly
    l3, _ = oracle.softmax_xent(np.zeros((2, V)), np.array([0, 5]))
    np.testing.assert_allclose(l3, math.log(V), rtol=1e-15)


# ------------------------------------------------------------------ embedding

def test_embedding_brute_force_and_fp32_rounding():
    T, C, V, B = 5, 6, 11, 3
    wte = si.normal_f32(1, (V, C))
    wpe = si.normal_f32(2, (T, C))
    tok = rng.integers(0, V, (B, T)).astype(np.int32)
    x = oracle.embedding_fwd(tok, wte, wpe, T)
    xr = oracle.embedding_fwd(tok, wte, wpe, T, round_fp32=True)
    for b in range(B):
        for t in range(T):
            for c in range(C):
                assert x[b * T + t, c] == float(wte[tok[b, t], c]) + float(wpe[t, c])
                assert xr[b * T + t, c] == float(np.float32(wte[tok[b, t], c]) + np.float32(wpe[t, c]))
    dx = rng.standard_normal((B * T, C))
    dwte, dwpe = oracle.embedding_bwd(tok, dx, T, V)
    ref = np.zeros((V, C))
    np.add.at(ref, tok.ravel(), dx)
    np.testing.assert_allclose(dwte, ref, rtol=1e-14, atol=1e-15)
    np.testing.assert_allclose(dwpe, dx.reshape(B, T, C).sum(0), rtol=1e-14, atol=1e-15)


# ------------------------------------------------------------------ clip and AdamW

def test_adamw_first_step_closed_form():
    n = 200
    p, g = rng.standard_normal(n), rng.standard_normal(n) * 1e-3
    g[:5] = 0.0
    lr, b1, b2, eps, wd = 6e-4, 0.9, 0.95, 1e-8, 0.1
    p1, m1, v1 = oracle.adamw(p, g, np.zeros(n), np.zeros(n), lr, b1, b2, eps, wd, 1, 1)
    # at t = 1 with zero moments: mhat = g, vhat = g^2
    np.testing.assert_allclose(p1, p * (1 - lr * wd) - lr * g / (np.abs(g) + eps), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(m1, (1 - b1) * g, rtol=1e-14)
    np.testing.assert_allclose(v1, (1 - b2) * g * g, rtol=1e-12)
    # no decay flag and zero gradient: the parameter does not move
    p2, _, _ = oracle.adamw(p, np.zeros(n), np.zeros(n), np.zeros(n), lr, b1, b2, eps, wd, 0, 1)
    assert np.array_equal(p2, p)
    # the clip scale multiplies the gradient before the moments
    p3, m3, _ = oracle.adamw(p, g, np.zeros(n), np.zeros(n), lr, b1, b2, eps, wd, 1, 1, scale=0.25)
    np.testing.assert_allclose(m3, (1 - b1) * 0.25 * g, rtol=1e-14)


@pytest.mark.parametrize("decay", [0, 1])
def test_adamw_matches_torch_optimizer_over_steps(decay):
    n = 64
    lr, b1, b2, eps, wd = 6e-4, 0.9, 0.95, 1e-8, 0.1
    p = rng.standard_normal(n)
    pt = torch.tensor(p.copy(), requires_grad=True)
    opt = torch.optim.AdamW([pt], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd if decay else 0.0)
    m, v = np.zeros(n), np.zeros(n)
    for t in range(1, 8):
        g = rng.standard_normal(n) * 10.0 ** rng.integers(-6, 1)
        pt.grad = torch.tensor(g.copy())
        opt.step()
        p, m, v = oracle.adamw(p, g, m, v, lr, b1, b2, eps, wd, decay, t)
        np.testing.assert_allclose(p, pt.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_clip_matches_torch_clip_grad_norm():
    shapes = [(7, 3), (11,), (2, 5)]
    for mag in (1e-3, 5.0):
        grads = [rng.standard_normal(s) * mag for s in shapes]
        gn = oracle.grad_norm(grads)
        np.testing.assert_allclose(gn, np.linalg.norm(np.concatenate([g.ravel() for g in grads])), rtol=1e-14)
        ps = [torch.zeros(s, dtype=torch.float64, requires_grad=True) for s in shapes]
        for q, g in zip(ps, grads):
            q.grad = torch.tensor(g.copy())
        total = torch.nn.utils.clip_grad_norm_(ps, 1.0)
        s = oracle.clip_scale(gn, 1.0)
        np.testing.assert_allclose(float(total), gn, rtol=1e-13)
        for q, g in zip(ps, grads):
            np.testing.assert_allclose(q.grad.numpy(), s * g, rtol=1e-12)
        if gn <= 1.0:
            assert s == 1.0
        else:
            np.testing.assert_allclose(s * gn, gn / (gn + 1e-6), rtol=1e-13)


def test_lr_schedule_pins():
    """Learning-rate schedule against what the hyper-parameter table fixes (Table of GPT-2 124M
    hyper-parameters: max 6e-4, min 6e-5, 715 warmup steps, 19,073 training steps) and the shape
    of the reading: end points, the linear ramp, the cosine's midpoint and symmetry, monotonicity."""
    mx, mn, wu, ms = 6e-4, 6e-5, 715, 19073
    f = lambda t: oracle.lr_schedule(t, mx, mn, wu, ms)
    assert f(0) == 0.0
    assert f(wu) == mx and f(ms) == mn and f(ms + 1000) == mn
    assert abs(f(1) - mx / wu) < 1e-18 and abs(f(wu // 5) - mx * (wu // 5) / wu) < 1e-18
    mid = (wu + ms) // 2          # (715 + 19073) / 2 = 9894 exactly: cos(pi/2) = 0
    assert (wu + ms) % 2 == 0 and abs(f(mid) - 0.5 * (mx + mn)) < 1e-15
    for k in (1, 100, 5000):       # cos(pi - x) = -cos(x): the curve is point-symmetric about the midpoint
        assert abs((f(mid - k) - 0.5 * (mx + mn)) + (f(mid + k) - 0.5 * (mx + mn))) < 1e-15
    ramp = [f(t) for t in range(1, wu + 1)]
    decay = [f(t) for t in range(wu, ms + 1)]
    assert all(a < b for a, b in zip(ramp, ramp[1:]))
    assert all(a > b for a, b in zip(decay, decay[1:]))
    # a quarter of the way down the cosine: (1 + cos(pi/4)) / 2 of the range above min
    q = wu + (ms - wu) // 4
    assert (ms - wu) % 4 != 0 or abs(f(q) - (mn + 0.5 * (1 + 2 ** -0.5) * (mx - mn))) < 1e-15
    # no warmup, no decay
    assert oracle.lr_schedule(1, 1e-3, 1e-3, 0, 10) == 1e-3


def test_dense_attention_route_equals_row_by_row_routine():
    """The matrix-form attention (library matmuls, used for long contexts) against the row-by-row C
    routine, which the tests above pin to the library, to finite differences and to special cases."""
    B, T, H, d = 2, 150, 3, 16
    qkv = si.normal_f32(901, (B * T, 3 * H * d)).astype(np.float64)
    d_o = si.normal_f32(902, (B * T, H * d), 1e-2).astype(np.float64)
    o, lse, dqkv = oracle.attention_dense(qkv, d_o, B, T, H)
    ro, rlse = oracle.attention_fwd(qkv, B, T, H)
    rd = oracle.attention_bwd(qkv, d_o, B, T, H)
    assert np.abs(o - ro).max() < 1e-13 and np.abs(lse - rlse).max() < 1e-12
    assert np.abs(dqkv - rd).max() < 1e-13 * max(1.0, np.abs(rd).max() / 1e-2)


def test_loader_windows_pins():
    """Batch cursor of Algorithm 2 against what the algorithm fixes: rank r starts at B*T*r, windows of
    one rank are B*T*world apart, the ranks' windows tile a shard without gaps or overlap, a window
    (plus its one-token-later target window) never crosses a shard's end, and shards are visited
    cyclically."""
    B, T = 2, 8
    bt = B * T
    world = 3
    lens = [bt * world * 4 + 1, bt * world * 2 + 5, bt * world + 1]
    per_rank = [oracle.loader_windows(lens, B, T, r, world, 40) for r in range(world)]
    for r, wins in enumerate(per_rank):
        assert wins[0] == (0, bt * r)
        for (s0, p0), (s1, p1) in zip(wins, wins[1:]):
            assert p0 + bt + 1 <= lens[s0]                       # tokens and targets fit
            if s1 == s0 and p1 > p0:
                assert p1 - p0 == bt * world                     # the global rank stride
            else:
                assert s1 == (s0 + 1) % len(lens) and p1 == bt * r
    # inside one pass over shard 0 the ranks interleave into a gap-free tiling
    first = sorted(p for wins in per_rank for (s, p) in wins[:4] if s == 0)
    assert first == [bt * k for k in range(len(first))]
    # shard 0 holds exactly 4 global batches + 1 token: every rank takes 4 windows there, then moves on
    assert [s for s, _ in per_rank[0][:8]] == [0, 0, 0, 0, 1, 1, 2, 0]
    # one rank, one shard of exactly one batch + 1: the same window for ever
    assert oracle.loader_windows([bt + 1], B, T, 0, 1, 3) == [(0, 0)] * 3
