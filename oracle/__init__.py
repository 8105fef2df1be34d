"""CPU oracle (float64) for the GPT-2 training step.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline legs may import
this package; the CUDA library and its Python binding never do.  The arithmetic
lives in `oracle.c` (plain C, double precision, OpenMP for the outer loops); this
module compiles it with gcc on first use and wraps it with ctypes + numpy.

Every function is pinned by `tests/test_oracle_*.py` against finite differences,
closed forms, invariants and library routines -- none is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import math
import hashlib
import os
import subprocess
from collections import OrderedDict

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_SIG = os.path.join(_HERE, "liboracle.sig")
_lib = None

_D = ctypes.POINTER(ctypes.c_double)
_I = ctypes.POINTER(ctypes.c_int32)
_i64 = ctypes.c_int64


def _signature() -> str:
    """Source hash plus the host's CPU feature flags (the library is built -march=native,
    so a copy built on another machine must be rebuilt)."""
    h = hashlib.sha256()
    with open(_SRC, "rb") as f:
        h.update(f.read())
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    h.update(line.encode())
                    break
    except OSError:
        pass
    return h.hexdigest()


def build(force: bool = False) -> str:
    """Compile oracle.c into liboracle.so (idempotent)."""
    sig = _signature()
    if not force and os.path.exists(_LIB) and os.path.exists(_SIG):
        with open(_SIG) as f:
            if f.read().strip() == sig:
                return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-fvisibility=hidden",
           "-std=gnu11", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    with open(_SIG, "w") as f:
        f.write(sig)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        L.orc_num_threads.restype = ctypes.c_int
        L.orc_embedding_fwd.argtypes = [_I, _D, _D, _i64, _i64, _i64, ctypes.c_int, _D]
        L.orc_embedding_bwd.argtypes = [_I, _D, _i64, _i64, _i64, _D, _D]
        L.orc_layernorm_fwd.argtypes = [_D, _D, _D, _i64, _i64, ctypes.c_double, _D, _D, _D]
        L.orc_layernorm_bwd.argtypes = [_D, _D, _D, _D, _D, _i64, _i64, _D, _D, _D]
        L.orc_linear_fwd.argtypes = [_D, _D, _D, _i64, _i64, _i64, _D]
        L.orc_linear_bwd.argtypes = [_D, _D, _D, _i64, _i64, _i64, _D, _D, _D]
        L.orc_attention_fwd.argtypes = [_D, _i64, _i64, _i64, _i64, _D, _D, _D]
        L.orc_attention_bwd.argtypes = [_D, _D, _i64, _i64, _i64, _i64, _D]
        L.orc_gelu_fwd.argtypes = [_D, _i64, ctypes.c_int, _D]
        L.orc_gelu_bwd.argtypes = [_D, _D, _i64, ctypes.c_int, _D]
        L.orc_softmax_xent.argtypes = [_D, _I, _i64, _i64, ctypes.c_double, _D, _D]
        L.orc_sum_squares.argtypes = [_D, _i64]
        L.orc_sum_squares.restype = ctypes.c_double
        L.orc_clip_scale.argtypes = [ctypes.c_double, ctypes.c_double]
        L.orc_clip_scale.restype = ctypes.c_double
        L.orc_adamw.argtypes = [_D, _D, _D, _D, _i64] + [ctypes.c_double] * 5 + [ctypes.c_int, _i64,
                                                                               ctypes.c_double]
        L.orc_model_create.argtypes = [_i64] * 6 + [ctypes.c_int]
        L.orc_model_create.restype = ctypes.c_void_p
        L.orc_model_destroy.argtypes = [ctypes.c_void_p]
        L.orc_model_num_tensors.argtypes = [ctypes.c_void_p]
        L.orc_model_tensor_info.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_char_p),
                                            ctypes.POINTER(_i64), ctypes.POINTER(ctypes.c_int)]
        L.orc_model_tensor_ptr.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int]
        L.orc_model_tensor_ptr.restype = _D
        L.orc_model_zero_grad.argtypes = [ctypes.c_void_p]
        L.orc_model_set_step.argtypes = [ctypes.c_void_p, _i64]
        L.orc_model_forward_backward.argtypes = [ctypes.c_void_p, _I, _I, _i64, _i64, ctypes.c_int]
        L.orc_model_forward_backward.restype = ctypes.c_double
        L.orc_model_grad_norm.argtypes = [ctypes.c_void_p]
        L.orc_model_grad_norm.restype = ctypes.c_double
        L.orc_model_adamw_step.argtypes = [ctypes.c_void_p] + [ctypes.c_double] * 6
        L.orc_model_adamw_step.restype = ctypes.c_double
        L.orc_model_last_scale.argtypes = [ctypes.c_void_p]
        L.orc_model_last_scale.restype = ctypes.c_double
        L.orc_model_activation.argtypes = [ctypes.c_void_p, ctypes.c_char_p, _i64]
        L.orc_model_activation.restype = _D
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _d(a):
    """float64 C-contiguous copy/view (float32 inputs widen exactly)."""
    return np.ascontiguousarray(a, dtype=np.float64)


def _i(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a):
    return a.ctypes.data_as(_D) if a is not None else None


def _pi(a):
    return a.ctypes.data_as(_I)


# ------------------------------------------------------------------ per-op wrappers

def embedding_fwd(tok, wte, wpe, T, round_fp32=False):
    tok, wte, wpe = _i(tok).ravel(), _d(wte), _d(wpe)
    N, C = tok.size, wte.shape[1]
    x = np.empty((N, C))
    lib().orc_embedding_fwd(_pi(tok), _p(wte), _p(wpe), N, T, C, int(round_fp32), _p(x))
    return x


def embedding_bwd(tok, dx, T, Vp):
    tok, dx = _i(tok).ravel(), _d(dx)
    N, C = dx.shape
    dwte, dwpe = np.zeros((Vp, C)), np.zeros((T, C))
    lib().orc_embedding_bwd(_pi(tok), _p(dx), N, T, C, _p(dwte), _p(dwpe))
    return dwte, dwpe


def layernorm_fwd(x, g, b, eps=1e-5):
    x, g, b = _d(x), _d(g), _d(b)
    N, C = x.shape
    y, mean, rstd = np.empty((N, C)), np.empty(N), np.empty(N)
    lib().orc_layernorm_fwd(_p(x), _p(g), _p(b), N, C, eps, _p(y), _p(mean), _p(rstd))
    return y, mean, rstd


def layernorm_bwd(dy, x, g, mean, rstd):
    dy, x, g, mean, rstd = _d(dy), _d(x), _d(g), _d(mean), _d(rstd)
    N, C = x.shape
    dx, dg, db = np.empty((N, C)), np.zeros(C), np.zeros(C)
    lib().orc_layernorm_bwd(_p(dy), _p(x), _p(g), _p(mean), _p(rstd), N, C, _p(dx), _p(dg), _p(db))
    return dx, dg, db


def linear_fwd(x, w, b=None):
    x, w = _d(x), _d(w)
    b = _d(b) if b is not None else None
    N, cin = x.shape
    out = w.shape[0]
    y = np.empty((N, out))
    lib().orc_linear_fwd(_p(x), _p(w), _p(b), N, cin, out, _p(y))
    return y


def linear_bwd(dy, x, w, want_db=True):
    dy, x, w = _d(dy), _d(x), _d(w)
    N, cin = x.shape
    out = w.shape[0]
    dx, dw = np.empty((N, cin)), np.zeros((out, cin))
    db = np.zeros(out) if want_db else None
    lib().orc_linear_bwd(_p(dy), _p(x), _p(w), N, cin, out, _p(dx), _p(dw), _p(db))
    return dx, dw, db


def attention_fwd(qkv, B, T, H, want_probs=False):
    qkv = _d(qkv)
    C = qkv.shape[-1] // 3
    o, lse = np.empty((B * T, C)), np.empty((B, H, T))
    probs = np.empty((B, H, T, T)) if want_probs else None
    lib().orc_attention_fwd(_p(qkv), B, T, C, H, _p(o), _p(lse), _p(probs))
    return (o, lse, probs) if want_probs else (o, lse)


def attention_bwd(qkv, d_o, B, T, H):
    qkv, d_o = _d(qkv), _d(d_o)
    C = qkv.shape[-1] // 3
    dqkv = np.empty((B * T, 3 * C))
    lib().orc_attention_bwd(_p(qkv), _p(d_o), B, T, C, H, _p(dqkv))
    return dqkv


def attention_dense(qkv, d_o, B, T, H):
    """Causal attention forward and backward by its matrix definition, one (sequence, head) at a
    time with float64 library matmuls: S = Q K^T / sqrt(d) with the strict upper triangle at -inf,
    P = row softmax(S), O = P V; then dV = P^T dO, dP = dO V^T, dS = P o (dP - rowsum(dO o O)),
    dQ = dS K / sqrt(d), dK = dS^T Q / sqrt(d).  It holds whole T x T matrices, so it serves where
    the row-by-row C routine is too slow (long contexts); a test pins it to that routine.
    Returns (o [B*T, C], lse [B, H, T], dqkv [B*T, 3C])."""
    qkv, d_o = _d(qkv), _d(d_o)
    C = qkv.shape[-1] // 3
    d = C // H
    o, lse, dqkv = np.empty((B * T, C)), np.empty((B, H, T)), np.empty((B * T, 3 * C))
    upper = np.triu(np.ones((T, T), dtype=bool), k=1)
    for b in range(B):
        rows = slice(b * T, (b + 1) * T)
        for h in range(H):
            cq, ck, cv = (slice(p * C + h * d, p * C + (h + 1) * d) for p in range(3))
            q, k, v, do = qkv[rows, cq], qkv[rows, ck], qkv[rows, cv], d_o[rows, h * d:(h + 1) * d]
            s = (q @ k.T) / math.sqrt(d)
            s[upper] = -np.inf
            mx = s.max(axis=1, keepdims=True)
            p = np.exp(s - mx)
            den = p.sum(axis=1, keepdims=True)
            p /= den
            lse[b, h] = (mx + np.log(den)).ravel()
            oh = p @ v
            o[rows, h * d:(h + 1) * d] = oh
            dp = do @ v.T
            ds = p * (dp - (do * oh).sum(axis=1, keepdims=True))
            dqkv[rows, cq] = (ds @ k) / math.sqrt(d)
            dqkv[rows, ck] = (ds.T @ q) / math.sqrt(d)
            dqkv[rows, cv] = p.T @ do
    return o, lse, dqkv


def gelu_fwd(x, tanh_form=False):
    x = _d(x)
    y = np.empty_like(x)
    lib().orc_gelu_fwd(_p(x), x.size, int(tanh_form), _p(y))
    return y


def gelu_bwd(x, dy, tanh_form=False):
    x, dy = _d(x), _d(dy)
    dx = np.empty_like(x)
    lib().orc_gelu_bwd(_p(x), _p(dy), x.size, int(tanh_form), _p(dx))
    return dx


def softmax_xent(logits, targets, inv_count=None, want_grad=True):
    logits, targets = _d(logits), _i(targets).ravel()
    N, Vp = logits.shape
    if inv_count is None:
        inv_count = 1.0 / N
    losses = np.empty(N)
    dl = np.empty((N, Vp)) if want_grad else None
    lib().orc_softmax_xent(_p(logits), _pi(targets), N, Vp, inv_count, _p(losses), _p(dl))
    return losses, dl


def grad_norm(grads) -> float:
    s = 0.0
    for g in grads:
        g = _d(g).ravel()
        s += lib().orc_sum_squares(_p(g), g.size)
    return float(np.sqrt(s))


def clip_scale(norm: float, clip: float) -> float:
    return float(lib().orc_clip_scale(norm, clip))


def adamw(p, g, m, v, lr, beta1, beta2, eps, weight_decay, decay, t, scale=1.0):
    """Returns updated (p, m, v) as new float64 arrays."""
    p, m, v = _d(p).copy(), _d(m).copy(), _d(v).copy()
    g = _d(g)
    lib().orc_adamw(_p(p), _p(g), _p(m), _p(v), p.size, lr, beta1, beta2, eps, weight_decay, int(decay),
                    int(t), scale)
    return p, m, v


# ------------------------------------------------------------------------- model

def loader_windows(shard_lens, B, T, rank, world, n_batches):
    """The batch cursor of Algorithm 2 (double-buffered batch production), without any copying:
    the (shard, position) of each of the first n_batches windows a rank reads.  A window is B*T
    tokens at `position` (the targets are the same window one token later); the rank starts at
    B*T*rank, moves on by B*T*world after each window, and opens the next shard (positions start
    again at B*T*rank) when the current one has fewer than B*T + 1 tokens left at the position --
    tested before a window is taken -- or fewer than B*T*world + 1 left after moving on."""
    bt = B * T
    cur, pos = 0, bt * rank
    out = []
    for _ in range(n_batches):
        if pos + bt + 1 > shard_lens[cur]:
            cur, pos = (cur + 1) % len(shard_lens), bt * rank
        out.append((cur, pos))
        pos += bt * world
        if pos + bt * world + 1 > shard_lens[cur]:
            cur, pos = (cur + 1) % len(shard_lens), bt * rank
    return out


def lr_schedule(step: int, max_lr: float, min_lr: float, warmup_steps: int, max_steps: int) -> float:
    """Learning rate of optimizer step `step` (first step = 1), from the four numbers of the
    hyper-parameter table (max / min learning rate, warmup steps, training steps).  The paper gives
    no curve; the reading taken: a straight line from 0 to max_lr over the warmup steps, then half
    a cosine period from max_lr (at step = warmup_steps) down to min_lr (at step = max_steps),
    min_lr from there on."""
    if step < 1:
        return 0.0
    if warmup_steps > 0 and step <= warmup_steps:
        return max_lr * step / warmup_steps
    if step >= max_steps or max_steps <= warmup_steps:
        return min_lr
    progress = (step - warmup_steps) / (max_steps - warmup_steps)
    return min_lr + 0.5 * (1.0 + math.cos(math.pi * progress)) * (max_lr - min_lr)


class Model:
    """The whole training step in float64."""

    def __init__(self, cfg: dict, gelu_tanh: bool = False):
        self.cfg = dict(cfg)
        self.h = lib().orc_model_create(cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["seq_len"],
                                        cfg["vocab_size"], cfg["padded_vocab_size"], int(gelu_tanh))
        if not self.h:
            raise ValueError("invalid model configuration")
        self._index = OrderedDict()
        name, numel, decay = ctypes.c_char_p(), _i64(), ctypes.c_int()
        for i in range(lib().orc_model_num_tensors(self.h)):
            lib().orc_model_tensor_info(self.h, i, ctypes.byref(name), ctypes.byref(numel), ctypes.byref(decay))
            self._index[name.value.decode()] = (i, int(numel.value), int(decay.value))
        self._rows = 0

    def __del__(self):
        if getattr(self, "h", None):
            lib().orc_model_destroy(self.h)
            self.h = None

    def names(self):
        return list(self._index)

    def decay(self, name):
        return self._index[name][2]

    def _view(self, name, kind):
        i, numel, _ = self._index[name]
        ptr = lib().orc_model_tensor_ptr(self.h, i, kind)
        return np.ctypeslib.as_array(ptr, shape=(numel,))

    def set_params(self, params):
        for name, a in params.items():
            self._view(name, 0)[:] = np.asarray(a, dtype=np.float64).ravel()

    def set_tensor(self, name, a, kind=0):
        self._view(name, kind)[:] = np.asarray(a, dtype=np.float64).ravel()

    def get(self, name, kind=0):
        return self._view(name, kind).copy()

    def params(self):
        return OrderedDict((n, self.get(n, 0)) for n in self._index)

    def grads(self):
        return OrderedDict((n, self.get(n, 1)) for n in self._index)

    def zero_grad(self):
        lib().orc_model_zero_grad(self.h)

    def loss(self, tok, tgt, chunk=0):
        tok, tgt = _i(tok), _i(tgt)
        B = tok.shape[0]
        self._rows = (chunk if 0 < chunk <= B else B) * self.cfg["seq_len"]
        return float(lib().orc_model_forward_backward(self.h, _pi(tok), _pi(tgt), B, chunk, 0))

    def loss_and_grad(self, tok, tgt, chunk=0):
        tok, tgt = _i(tok), _i(tgt)
        B = tok.shape[0]
        self._rows = (chunk if 0 < chunk <= B else B) * self.cfg["seq_len"]
        self.zero_grad()
        return float(lib().orc_model_forward_backward(self.h, _pi(tok), _pi(tgt), B, chunk, 1))

    def grad_norm(self):
        return float(lib().orc_model_grad_norm(self.h))

    def adamw_step(self, lr, beta1, beta2, eps, weight_decay, grad_clip):
        return float(lib().orc_model_adamw_step(self.h, lr, beta1, beta2, eps, weight_decay, grad_clip))

    def last_scale(self):
        return float(lib().orc_model_last_scale(self.h))

    def activation(self, name, layer=0):
        ptr = lib().orc_model_activation(self.h, name.encode(), layer)
        if not ptr:
            raise KeyError(name)
        C, Vp = self.cfg["d_model"], self.cfg["padded_vocab_size"]
        width = {"x": C, "a": C, "o": C, "x1": C, "m": C, "xL": C, "xf": C, "qkv": 3 * C, "h": 4 * C,
                 "g": 4 * C, "logits": Vp, "dlogits": Vp}.get(name, 1)
        return np.ctypeslib.as_array(ptr, shape=(self._rows, width)).copy()
