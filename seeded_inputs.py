"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle harness.

This module holds no arithmetic of the training step.  It only names the model
configurations, lists the parameter tensors in registry order, and draws
parameters, tokens and activations from seeded generators so that the CUDA path
and the oracle are always fed the same arrays.

Recipes
-------
* Parameters: weight matrices and both embeddings ~ N(0, 0.02^2); the two residual
  projections per block (attention output, MLP down-projection) ~ N(0, (0.02 /
  sqrt(2 * n_layers))^2); biases 0; LayerNorm gain 1, shift 0 (the paper's
  hyper-parameter table, "Optimization & Initialization" column and its caption).
  Drawn with numpy's PCG64 as float64, scaled, cast to float32, in registry order.
* Tokens, tiny configuration: independent uniform integers in [0, vocab).
* Tokens, GPT-2 sized configurations: Zipf(s=1.1) over the logical vocabulary by
  inverse-CDF sampling; targets are the tokens shifted by one position (the data
  loader of the paper's Algorithm 2 hands out `t` and `t+1` windows).  These
  stand in for the tokenised web-text corpus the paper trains on, which is not
  available offline: what the path is sensitive to is the vocabulary size, the
  sequence shape and the heavy-tailed token frequencies.
"""
from __future__ import annotations

import math
from collections import OrderedDict

import numpy as np

# BASELINE configurations, by index.
CONFIGS = {
    0: dict(name="tiny", n_layers=2, d_model=64, n_heads=4, seq_len=64, vocab_size=512,
            padded_vocab_size=512, batch=4, tokens="uniform"),
    1: dict(name="gpt2-small-block", n_layers=1, d_model=768, n_heads=12, seq_len=1024,
            vocab_size=0, padded_vocab_size=0, batch=8, tokens="none", init_layers=12),
    2: dict(name="gpt2-124M-b8", n_layers=12, d_model=768, n_heads=12, seq_len=1024,
            vocab_size=50257, padded_vocab_size=50304, batch=8, tokens="zipf"),
    3: dict(name="gpt2-124M-b32", n_layers=12, d_model=768, n_heads=12, seq_len=1024,
            vocab_size=50257, padded_vocab_size=50304, batch=32, tokens="zipf"),
    4: dict(name="gpt2-350M-b8", n_layers=24, d_model=1024, n_heads=16, seq_len=1024,
            vocab_size=50257, padded_vocab_size=50304, batch=8, tokens="zipf"),
    5: dict(name="gpt2-124M-t16k-b2", n_layers=12, d_model=768, n_heads=12, seq_len=16384,
            vocab_size=50257, padded_vocab_size=50304, batch=2, tokens="zipf"),   # the long-context shape
    6: dict(name="gpt2-2.42B-b2", n_layers=20, d_model=3072, n_heads=24, seq_len=1024,
            vocab_size=50257, padded_vocab_size=50304, batch=2, tokens="zipf"),   # the paper's largest model
}

ADAMW = dict(lr=6e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1, grad_clip=1.0)


def config(i: int) -> dict:
    return dict(CONFIGS[i])


def make_config(n_layers, d_model, n_heads, seq_len, vocab_size, padded_vocab_size=None, batch=1,
                tokens="uniform", name="custom") -> dict:
    return dict(name=name, n_layers=n_layers, d_model=d_model, n_heads=n_heads, seq_len=seq_len,
                vocab_size=vocab_size, padded_vocab_size=padded_vocab_size or vocab_size,
                batch=batch, tokens=tokens)


def tensor_registry(cfg: dict):
    """[(name, shape, decay_flag, init)] in registry order; init is ("normal", std) | ("const", v)."""
    L, C, T, Vp = cfg["n_layers"], cfg["d_model"], cfg["seq_len"], cfg["padded_vocab_size"]
    F = 4 * C
    std = 0.02
    rstd = 0.02 / math.sqrt(2.0 * cfg.get("init_layers", L))
    reg = []
    if Vp > 0:
        reg.append(("wte", (Vp, C), 1, ("normal", std)))
        reg.append(("wpe", (T, C), 1, ("normal", std)))
    for l in range(L):
        p = f"h{l}."
        reg += [
            (p + "ln1.g", (C,), 0, ("const", 1.0)),
            (p + "ln1.b", (C,), 0, ("const", 0.0)),
            (p + "attn.qkv.w", (3 * C, C), 1, ("normal", std)),
            (p + "attn.qkv.b", (3 * C,), 0, ("const", 0.0)),
            (p + "attn.proj.w", (C, C), 1, ("normal", rstd)),
            (p + "attn.proj.b", (C,), 0, ("const", 0.0)),
            (p + "ln2.g", (C,), 0, ("const", 1.0)),
            (p + "ln2.b", (C,), 0, ("const", 0.0)),
            (p + "mlp.fc.w", (F, C), 1, ("normal", std)),
            (p + "mlp.fc.b", (F,), 0, ("const", 0.0)),
            (p + "mlp.proj.w", (C, F), 1, ("normal", rstd)),
            (p + "mlp.proj.b", (C,), 0, ("const", 0.0)),
        ]
    if Vp > 0:
        reg.append(("lnf.g", (C,), 0, ("const", 1.0)))
        reg.append(("lnf.b", (C,), 0, ("const", 0.0)))
    return reg


def num_params(cfg: dict) -> int:
    return sum(int(np.prod(s)) for _, s, _, _ in tensor_registry(cfg))


def init_params(cfg: dict, seed: int, jitter: float = 0.0) -> "OrderedDict[str, np.ndarray]":
    """Float32 parameter arrays in registry order.

    `jitter` > 0 perturbs the constant tensors (biases, LayerNorm gain/shift) with
    N(0, jitter^2) noise: tests use it so that those tensors are not at the special
    values 0 and 1, where a wrong index or a dropped term can hide.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    out = OrderedDict()
    for name, shape, _decay, (kind, val) in tensor_registry(cfg):
        if kind == "normal":
            a = rng.standard_normal(shape) * val
        else:
            a = np.full(shape, val, dtype=np.float64)
            if jitter > 0.0:
                a = a + rng.standard_normal(shape) * jitter
        out[name] = a.astype(np.float32)
    return out


def uniform_tokens(seed: int, batch: int, seq_len: int, vocab: int):
    """Tokens and targets as independent uniform draws (tiny configuration)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    tok = rng.integers(0, vocab, size=(batch, seq_len), dtype=np.int64).astype(np.int32)
    tgt = rng.integers(0, vocab, size=(batch, seq_len), dtype=np.int64).astype(np.int32)
    return tok, tgt


def zipf_tokens(seed: int, batch: int, seq_len: int, vocab: int, s: float = 1.1):
    """Zipf(s) token ids over [0, vocab): rank k (1-based) has probability ~ k^-s, id = k - 1.

    Draws batch x (seq_len + 1) ids; tokens are columns [0, T), targets columns [1, T].
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    w = np.arange(1, vocab + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    u = rng.random(size=(batch, seq_len + 1))
    ids = np.minimum(np.searchsorted(cdf, u, side="right"), vocab - 1).astype(np.int32)
    return np.ascontiguousarray(ids[:, :-1]), np.ascontiguousarray(ids[:, 1:])


def tokens_for(cfg: dict, seed: int, batch: int | None = None):
    B = batch if batch is not None else cfg["batch"]
    if cfg["tokens"] == "zipf":
        return zipf_tokens(seed, B, cfg["seq_len"], cfg["vocab_size"])
    return uniform_tokens(seed, B, cfg["seq_len"], cfg["vocab_size"])


def normal_f32(seed: int, shape, std: float = 1.0) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64(seed))
    return (rng.standard_normal(shape) * std).astype(np.float32)


def block_inputs(cfg: dict, seed: int, batch: int | None = None):
    """Single-block workload: input activations ~ N(0,1), upstream gradient ~ N(0, 1e-2^2)."""
    B = batch if batch is not None else cfg["batch"]
    shape = (B * cfg["seq_len"], cfg["d_model"])
    rng = np.random.Generator(np.random.PCG64(seed))
    x = rng.standard_normal(shape).astype(np.float32)
    dy = (rng.standard_normal(shape) * 1e-2).astype(np.float32)
    return x, dy
