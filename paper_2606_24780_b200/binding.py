"""ctypes binding of libbt.so: the same names as include/bt.h, argument marshalling only.

Device arrays are passed as torch CUDA tensors (or raw integer addresses); torch is used only
for device memory and streams.  Every call raises BtError on a non-zero status.  There is no
fallback: if libbt.so is missing the import of the library fails with instructions.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbt.so")

BT_FLAG_GELU_TANH, BT_FLAG_GEMM_SIMT, BT_FLAG_ATTN_SIMT, BT_FLAG_GEMM_PAIR, BT_FLAG_GEMM_SINGLE = 1, 2, 4, 8, 16
BT_FLAG_DEBUG = 32
BT_FLAG_RECOMPUTE_LN = 64
BT_FLAG_LOGITS_IN_PLACE = 128
BT_FLAG_RECOMPUTE_GELU = 256
BT_GEMM_NT, BT_GEMM_NN, BT_GEMM_TN = 0, 1, 2
STATUS = {0: "BT_OK", 1: "BT_ERR_INVALID_ARG", 2: "BT_ERR_UNSUPPORTED", 3: "BT_ERR_OOM", 4: "BT_ERR_CUDA",
          5: "BT_ERR_DEVICE_TIMEOUT", 6: "BT_ERR_NOT_FOUND"}


class BtError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS.get(status, status)}: {message}")
        self.status = status


class bt_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("n_layers", "d_model", "n_heads", "seq_len", "vocab_size",
                                              "padded_vocab_size", "max_batch")] + [("flags", ctypes.c_uint32)]


class bt_adamw_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_float) for n in ("lr", "beta1", "beta2", "eps", "weight_decay", "grad_clip")]


class bt_lr_schedule(ctypes.Structure):
    _fields_ = [("max_lr", ctypes.c_float), ("min_lr", ctypes.c_float), ("warmup_steps", ctypes.c_int32),
                ("max_steps", ctypes.c_int32)]


_vp, _i32, _i64, _u32, _sz, _f = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32, ctypes.c_size_t,
                                  ctypes.c_float)
_SIGNATURES = {
    "bt_workspace_bytes": (_sz, [ctypes.POINTER(bt_config)]),
    "bt_workspace_part_bytes": (_sz, [ctypes.POINTER(bt_config), _i32]),
    "bt_model_create": (_i32, [ctypes.POINTER(bt_config), _vp, _sz, _vp, ctypes.POINTER(_vp)]),
    "bt_model_destroy": (None, [_vp]),
    "bt_model_init": (_i32, [_vp, ctypes.c_uint64]),
    "bt_num_tensors": (_i32, [_vp]),
    "bt_tensor_info": (_i32, [_vp, _i32, ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(_i64), ctypes.POINTER(_i32)]),
    "bt_tensor_ptr": (_i32, [_vp, ctypes.c_char_p, _i32, ctypes.POINTER(_vp)]),
    "bt_activation_ptr": (_i32, [_vp, ctypes.c_char_p, _i32, ctypes.POINTER(_vp), ctypes.POINTER(_i64)]),
    "bt_get_step": (_i64, [_vp]),
    "bt_set_step": (_i32, [_vp, _i64]),
    "bt_forward": (_i32, [_vp, _vp, _vp, _i32, ctypes.POINTER(_f)]),
    "bt_backward": (_i32, [_vp]),
    "bt_adamw_step": (_i32, [_vp, ctypes.POINTER(bt_adamw_config), ctypes.POINTER(_f)]),
    "bt_train_step": (_i32, [_vp, _vp, _vp, _i32, ctypes.POINTER(bt_adamw_config), ctypes.POINTER(_f)]),
    "bt_train_step_host": (_i32, [_vp, _vp, _vp, _i32, ctypes.POINTER(bt_adamw_config), ctypes.POINTER(_f)]),
    "bt_micro_step": (_i32, [_vp, _vp, _vp, _i32, _i32, _i32, ctypes.POINTER(_f)]),
    "bt_train_step_accum": (_i32, [_vp, _vp, _vp, _i32, _i32, ctypes.POINTER(bt_adamw_config), ctypes.POINTER(_f)]),
    "bt_lr_at": (_f, [ctypes.POINTER(bt_lr_schedule), _i64]),
    "bt_ddp_plan_create": (_i32, [ctypes.POINTER(bt_config), _i64, ctypes.POINTER(_vp)]),
    "bt_ddp_plan_destroy": (None, [_vp]),
    "bt_ddp_plan_num_buckets": (_i32, [_vp]),
    "bt_ddp_plan_bucket": (_i32, [_vp, _i32, ctypes.POINTER(_i64), ctypes.POINTER(_i64), ctypes.POINTER(_i32)]),
    "bt_ddp_plan_tensor": (_i32, [_vp, _i32, ctypes.POINTER(_i64), ctypes.POINTER(_i64)]),
    "bt_ddp_plan_reset": (None, [_vp]),
    "bt_ddp_plan_mark_ready": (_i32, [_vp, _i32, ctypes.POINTER(_i32)]),
    "bt_ddp_attach": (_i32, [_vp, _i64, _vp, _vp, _vp]),
    "bt_ddp_detach": (_i32, [_vp]),
    "bt_arena_ptr": (_i32, [_vp, _i32, ctypes.POINTER(_vp), ctypes.POINTER(_i64)]),
    "bt_loader_plan": (_i32, [ctypes.POINTER(_i64), _i32, _i32, _i32, _i32, _i32, _i32, ctypes.POINTER(_i32),
                              ctypes.POINTER(_i64)]),
    "bt_loader_create": (_i32, [ctypes.POINTER(_vp), ctypes.POINTER(_i64), _i32, _i32, _i32, _i32, _i32, _i32, _i32,
                                _vp, _vp, _vp, ctypes.POINTER(_vp)]),
    "bt_loader_next": (_i32, [_vp, ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_i32)]),
    "bt_loader_release": (_i32, [_vp, _i32]),
    "bt_loader_destroy": (None, [_vp]),
    "bt_get_loss": (_i32, [_vp, ctypes.POINTER(_f)]),
    "bt_launch_count": (_i64, [_vp]),
    "bt_last_error": (ctypes.c_char_p, []),
    "bt_profile_enable": (_i32, [_vp, _i32]),
    "bt_profile_num_categories": (_i32, []),
    "bt_profile_category_name": (ctypes.c_char_p, [_i32]),
    "bt_profile_read": (_i32, [_vp, _i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(_i64),
                               ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]),
    "bt_op_embedding_fwd": (_i32, [_vp, _vp, _vp, _i64, _i32, _i32, _i32, _vp, _vp, _vp]),
    "bt_op_embedding_bwd_scratch_bytes": (_sz, [_i64, _i32, _i32]),
    "bt_op_embedding_bwd": (_i32, [_vp, _vp, _i64, _i32, _i32, _i32, _vp, _vp, _vp, _sz, _vp]),
    "bt_first_invalid_id": (_i64, [_vp, _i64, _i32]),
    "bt_selftest_bounded_wait": (_i32, [_vp, _f]),
    "bt_probe_tf32_mma_rate": (_i32, [_i32, _i32, _vp, _vp, _vp]),
    "bt_probe_mma_issue_rate": (_i32, [_i32, _i32, _i32, _i32, _i32, _vp, _vp, _vp]),
    "bt_op_layernorm_fwd": (_i32, [_vp, _vp, _vp, _i64, _i32, _vp, _vp, _vp, _vp, _vp]),
    "bt_op_layernorm_bwd_scratch_bytes": (_sz, [_i64, _i32]),
    "bt_op_layernorm_bwd": (_i32, [_vp] * 6 + [_i64, _i32] + [_vp] * 5 + [_sz, _vp]),
    "bt_op_layernorm_bwd_colsum": (_i32, [_vp] * 6 + [_i64, _i32] + [_vp] * 6 + [_sz, _vp]),
    "bt_op_gemm_scratch_bytes": (_sz, [_i32, _i64, _i64, _i64]),
    "bt_op_split": (_i32, [_vp, _i64, _vp, _vp]),
    "bt_op_gemm_split_scratch_bytes": (_sz, []),
    "bt_op_gemm_split": (_i32, [_i32, _i64, _i64, _i64] + [_vp] * 6 + [_sz, _u32, _vp]),
    "bt_op_gemm_split_act": (_i32, [_i32, _i64, _i64, _i64] + [_vp] * 4 + [_i32] + [_vp] * 3 + [_sz, _u32, _vp]),
    "bt_op_gemm_gelu_bwd_scratch_bytes": (_sz, [_i64, _i64]),
    "bt_op_gemm_gelu_bwd": (_i32, [_i64, _i64, _i64] + [_vp] * 3 + [_i32] + [_vp] * 3 + [_sz, _u32, _vp]),
    "bt_op_gemm_check": (_i32, [_vp, _vp]),
    "bt_op_gemm_plan": (_i32, [_i64, _i64, _i64, _i32, _u32, _vp]),
    "bt_op_gemm": (_i32, [_i32, _i64, _i64, _i64] + [_vp] * 6 + [_sz, _u32, _vp]),
    "bt_op_attention_fwd": (_i32, [_vp, _vp, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _u32, _vp]),
    "bt_op_attention_bwd": (_i32, [_vp] * 6 + [_i32] * 4 + [_vp] * 3 + [_sz, _u32, _vp]),
    "bt_op_gelu_fwd": (_i32, [_vp, _i64, _i32, _vp, _vp, _vp]),
    "bt_op_gelu_bwd": (_i32, [_vp, _vp, _i64, _i32, _vp, _vp, _vp]),
    "bt_op_gelu_bwd_colsum": (_i32, [_vp, _vp, _i64, _i32, _i32, _vp, _vp, _vp, _vp, _sz, _vp]),
    "bt_op_softmax_xent": (_i32, [_vp, _vp, _i64, _i32, _f, _vp, _vp, _vp, _vp, _vp, _vp]),
    "bt_op_colsum_scratch_bytes": (_sz, [_i64, _i32]),
    "bt_op_colsum": (_i32, [_vp, _i64, _i32, _vp, _vp, _sz, _vp]),
    "bt_op_colsum_static_max_floats": (_sz, []),
    "bt_op_colsum_static": (_i32, [_vp, _i64, _i32, _vp, _vp]),
    "bt_op_grad_norm_scratch_bytes": (_sz, [_i64]),
    "bt_op_grad_norm": (_i32, [_vp, _i64, _f, _vp, _vp, _sz, _vp]),
    "bt_op_adamw_multi": (_i32, [_i32] + [ctypes.POINTER(_vp)] * 4 + [ctypes.POINTER(_i64), ctypes.POINTER(_i32),
                                 ctypes.POINTER(bt_adamw_config), _i64, _vp, _vp]),
}

_lib = None


def exported_symbols():
    """Names include/bt.h declares (used by the CPU test that checks the library exports them)."""
    return sorted(_SIGNATURES)


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2606_24780_b200.build` "
                              "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, torch.Tensor):
        if not t.is_contiguous():
            raise ValueError("tensor arguments must be contiguous")
        return t.data_ptr()
    raise TypeError(type(t))


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else None
    return stream


def _check(st):
    if st != 0:
        raise BtError(st, (lib().bt_last_error() or b"").decode())


def make_config(n_layers, d_model, n_heads, seq_len, vocab_size, padded_vocab_size, max_batch, flags=0):
    return bt_config(n_layers, d_model, n_heads, seq_len, vocab_size, padded_vocab_size, max_batch, flags)


def make_adamw(lr=6e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1, grad_clip=1.0):
    return bt_adamw_config(lr, beta1, beta2, eps, weight_decay, grad_clip)


# ------------------------------------------------------------------ model calls

def bt_workspace_bytes(cfg):
    return int(lib().bt_workspace_bytes(ctypes.byref(cfg)))


def bt_model_create(cfg, workspace, workspace_bytes=None, stream=None):
    out = _vp()
    nbytes = workspace_bytes if workspace_bytes is not None else (workspace.numel() * workspace.element_size()
                                                                  if isinstance(workspace, torch.Tensor) else 0)
    _check(lib().bt_model_create(ctypes.byref(cfg), _ptr(workspace), nbytes, _stream(stream), ctypes.byref(out)))
    return out.value


def bt_model_destroy(model):
    lib().bt_model_destroy(model)


def bt_model_init(model, seed):
    _check(lib().bt_model_init(model, seed))


def bt_num_tensors(model):
    return int(lib().bt_num_tensors(model))


def bt_tensor_info(model, index):
    name, numel, decay = ctypes.c_char_p(), _i64(), _i32()
    _check(lib().bt_tensor_info(model, index, ctypes.byref(name), ctypes.byref(numel), ctypes.byref(decay)))
    return name.value.decode(), int(numel.value), int(decay.value)


def bt_tensor_ptr(model, name, kind=0):
    p = _vp()
    _check(lib().bt_tensor_ptr(model, name.encode(), kind, ctypes.byref(p)))
    return p.value


def bt_activation_ptr(model, name, layer=0):
    p, n = _vp(), _i64()
    _check(lib().bt_activation_ptr(model, name.encode(), layer, ctypes.byref(p), ctypes.byref(n)))
    return p.value, int(n.value)


def bt_get_step(model):
    return int(lib().bt_get_step(model))


def bt_set_step(model, t):
    _check(lib().bt_set_step(model, t))


def bt_forward(model, tokens, targets, B, want_loss=True):
    loss = _f()
    _check(lib().bt_forward(model, _ptr(tokens), _ptr(targets), B, ctypes.byref(loss) if want_loss else None))
    return float(loss.value) if want_loss else None


def bt_backward(model):
    _check(lib().bt_backward(model))


def bt_adamw_step(model, opt, want_norm=True):
    gn = _f()
    _check(lib().bt_adamw_step(model, ctypes.byref(opt), ctypes.byref(gn) if want_norm else None))
    return float(gn.value) if want_norm else None


def bt_train_step(model, tokens, targets, B, opt, want_loss=True):
    loss = _f()
    _check(lib().bt_train_step(model, _ptr(tokens), _ptr(targets), B, ctypes.byref(opt),
                               ctypes.byref(loss) if want_loss else None))
    return float(loss.value) if want_loss else None


def bt_train_step_host(model, h_tokens, h_targets, B, opt, want_loss=True):
    """h_tokens / h_targets: CPU int32 torch tensors (pinned for an asynchronous copy)."""
    loss = _f()
    _check(lib().bt_train_step_host(model, _ptr(h_tokens), _ptr(h_targets), B, ctypes.byref(opt),
                                    ctypes.byref(loss) if want_loss else None))
    return float(loss.value) if want_loss else None


def bt_micro_step(model, tokens, targets, B, micro_index, n_micro, want_loss=True):
    loss = _f()
    _check(lib().bt_micro_step(model, _ptr(tokens), _ptr(targets), B, micro_index, n_micro,
                               ctypes.byref(loss) if want_loss else None))
    return float(loss.value) if want_loss else None


def bt_train_step_accum(model, tokens, targets, B, n_micro, opt, want_loss=True):
    """tokens / targets: device int32 [n_micro * B, seq_len]."""
    loss = _f()
    _check(lib().bt_train_step_accum(model, _ptr(tokens), _ptr(targets), B, n_micro, ctypes.byref(opt),
                                     ctypes.byref(loss) if want_loss else None))
    return float(loss.value) if want_loss else None


def bt_lr_at(schedule, step):
    return float(lib().bt_lr_at(ctypes.byref(schedule), step))


def bt_loader_plan(shard_lens, B, T, rank, world, n_batches):
    """Host only: [(shard, position)] of the first n_batches windows of this rank."""
    n = len(shard_lens)
    lens = (_i64 * n)(*shard_lens)
    out_s, out_p = (_i32 * n_batches)(), (_i64 * n_batches)()
    _check(lib().bt_loader_plan(lens, n, B, T, rank, world, n_batches, out_s, out_p))
    return [(int(out_s[i]), int(out_p[i])) for i in range(n_batches)]


ALLREDUCE_FN = ctypes.CFUNCTYPE(ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32,
                                ctypes.c_void_p)


WORKSPACE_PARTS = ("params_grads_moments", "weight_planes", "grad_accumulator", "activations", "logits",
                   "backward_temporaries", "scratch")


def bt_workspace_parts(cfg):
    """{section: bytes} of the workspace of a configuration; the values add up to bt_workspace_bytes."""
    return {name: int(lib().bt_workspace_part_bytes(ctypes.byref(cfg), i)) for i, name in enumerate(WORKSPACE_PARTS)}


class DdpPlan:
    """Host-only view of the gradient buckets of a configuration (no GPU needed): ranges of the flat
    gradient arena in gradient-ready order, the arena offsets of the registry tensors, and the
    in-order launch gate."""

    def __init__(self, cfg, bucket_cap_bytes=25 * 1000 * 1000):
        self.h = _vp()
        _check(lib().bt_ddp_plan_create(ctypes.byref(cfg), bucket_cap_bytes, ctypes.byref(self.h)))
        self.n_buckets = int(lib().bt_ddp_plan_num_buckets(self.h))

    def bucket(self, b):
        """(offset, count, n_tensors) of bucket b, offsets and counts in floats."""
        off, cnt, nt = _i64(), _i64(), _i32()
        _check(lib().bt_ddp_plan_bucket(self.h, b, ctypes.byref(off), ctypes.byref(cnt), ctypes.byref(nt)))
        return int(off.value), int(cnt.value), int(nt.value)

    def tensor(self, i):
        """(offset, padded length) of registry tensor i inside the arena, in floats."""
        off, ln = _i64(), _i64()
        _check(lib().bt_ddp_plan_tensor(self.h, i, ctypes.byref(off), ctypes.byref(ln)))
        return int(off.value), int(ln.value)

    def reset(self):
        lib().bt_ddp_plan_reset(self.h)

    def mark_ready(self, tensor):
        """Buckets the gate releases now that `tensor`'s gradient is final (in launch order)."""
        out = (_i32 * max(1, self.n_buckets))()
        n = int(lib().bt_ddp_plan_mark_ready(self.h, tensor, out))
        if n < 0:
            raise BtError(1, f"tensor {tensor} out of range or marked ready twice")
        return [int(out[i]) for i in range(n)]

    def close(self):
        if self.h and _lib is not None:
            _lib.bt_ddp_plan_destroy(self.h)
        self.h = None

    __del__ = close


def bt_arena_ptr(model, kind):
    p, n = _vp(), _i64()
    _check(lib().bt_arena_ptr(model, kind, ctypes.byref(p), ctypes.byref(n)))
    return p.value, int(n.value)


class Loader:
    """Prefetching batch production over host int32 token shards (CPU torch tensors, kept alive
    here).  `next()` returns (tokens, targets, slot): device int32 tensors of shape [B, T] and the
    ring slot they live in; call `release(slot)` after enqueuing the last kernel that reads them."""

    def __init__(self, shards, B, T, rank=0, world=1, pinned=True, vocab_size=0, n_slots=2, device="cuda",
                 stream=None):
        self.shards = [s.contiguous() for s in shards]
        self.B, self.T = B, T
        n = len(self.shards)
        ptrs = (_vp * n)(*[s.data_ptr() for s in self.shards])
        lens = (_i64 * n)(*[s.numel() for s in self.shards])
        self.d_buffers = torch.empty(2 * n_slots * B * T, dtype=torch.int32, device=device)
        self.h_pinned = torch.empty(2 * n_slots * B * T, dtype=torch.int32).pin_memory() if pinned else None
        self.h = _vp()
        _check(lib().bt_loader_create(ptrs, lens, n, B, T, rank, world, vocab_size, n_slots, _ptr(self.d_buffers),
                                      _ptr(self.h_pinned), _stream(stream), ctypes.byref(self.h)))

    def next(self):
        x, y, slot = _vp(), _vp(), _i32()
        _check(lib().bt_loader_next(self.h, ctypes.byref(x), ctypes.byref(y), ctypes.byref(slot)))
        base, n = self.d_buffers.data_ptr(), self.B * self.T
        ox, oy = (x.value - base) // 4, (y.value - base) // 4
        return (self.d_buffers[ox:ox + n].view(self.B, self.T), self.d_buffers[oy:oy + n].view(self.B, self.T),
                int(slot.value))

    def release(self, slot):
        _check(lib().bt_loader_release(self.h, slot))

    def close(self):
        if self.h:
            lib().bt_loader_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()


def bt_get_loss(model):
    loss = _f()
    _check(lib().bt_get_loss(model, ctypes.byref(loss)))
    return float(loss.value)


def bt_launch_count(model):
    return int(lib().bt_launch_count(model))


def bt_profile_enable(model, on):
    _check(lib().bt_profile_enable(model, int(on)))


def bt_profile_num_categories():
    return int(lib().bt_profile_num_categories())


def bt_profile_category_name(cat):
    return lib().bt_profile_category_name(cat).decode()


def bt_profile_read(model, cat):
    """(ms_total, launches, flops, bytes) of one category since bt_profile_enable."""
    ms, fl, by, n = ctypes.c_double(), ctypes.c_double(), ctypes.c_double(), _i64()
    _check(lib().bt_profile_read(model, cat, ctypes.byref(ms), ctypes.byref(n), ctypes.byref(fl), ctypes.byref(by)))
    return float(ms.value), int(n.value), float(fl.value), float(by.value)


# ------------------------------------------------------------------ per-op calls

def bt_op_embedding_fwd(tok, wte, wpe, N, T, C, V, x, d_bad=None, stream=None):
    _check(lib().bt_op_embedding_fwd(_ptr(tok), _ptr(wte), _ptr(wpe), N, T, C, V, _ptr(x), _ptr(d_bad), _stream(stream)))


def bt_op_embedding_bwd_scratch_bytes(N, C, V):
    return int(lib().bt_op_embedding_bwd_scratch_bytes(N, C, V))


def bt_op_embedding_bwd(tok, dx, N, T, C, V, dwte, dwpe, scratch, scratch_bytes, stream=None):
    _check(lib().bt_op_embedding_bwd(_ptr(tok), _ptr(dx), N, T, C, V, _ptr(dwte), _ptr(dwpe), _ptr(scratch),
                                     scratch_bytes, _stream(stream)))


def bt_first_invalid_id(h_ids, vocab_size):
    """Position of the first id outside [0, vocab_size) in a host int32 tensor, or -1 (host only)."""
    if not isinstance(h_ids, torch.Tensor) or h_ids.is_cuda or h_ids.dtype != torch.int32 or not h_ids.is_contiguous():
        raise TypeError("h_ids must be a contiguous int32 host tensor")
    return int(lib().bt_first_invalid_id(h_ids.data_ptr(), h_ids.numel(), vocab_size))


def bt_probe_tf32_mma_rate(n_ctas=148, iters=4000, stream=None):
    """Clocks per tcgen05.mma.kind::tf32 (128 x 256 x 8) on every CTA's SM: (min, median, max) over
    the CTAs.  262144 / clocks = dense TF32 MAC per clock per SM."""
    clocks = torch.zeros(n_ctas, dtype=torch.int64, device="cuda")
    err = torch.zeros(4, dtype=torch.int32, device="cuda")
    for _ in range(2):                       # the first launch also loads the kernel
        _check(lib().bt_probe_tf32_mma_rate(n_ctas, iters, _ptr(clocks), _ptr(err), _stream(stream)))
    torch.cuda.synchronize()
    if int(err[0]) != 0 or int(clocks.min()) < 0:
        raise BtError(5, f"rate probe: a bounded wait ran out (code {int(err[0])})")
    c = clocks.double() / iters
    return float(c.min()), float(c.median()), float(c.max())


def bt_probe_mma_issue_rate(n, a_in_tmem, issuers, n_ctas=148, iters=4096, stream=None):
    """Clocks per tcgen05.mma (128 x n x 8) with `issuers` issuing threads per CTA: median over the CTAs of
    (slowest thread's clocks) / (iters x issuers)."""
    clocks = torch.zeros(4 * n_ctas, dtype=torch.int64, device="cuda")
    err = torch.zeros(4, dtype=torch.int32, device="cuda")
    for _ in range(2):                       # the first launch also loads the kernel
        _check(lib().bt_probe_mma_issue_rate(n, int(a_in_tmem), issuers, n_ctas, iters, _ptr(clocks), _ptr(err),
                                             _stream(stream)))
    torch.cuda.synchronize()
    c = clocks.view(n_ctas, 4)[:, :issuers]
    if int(err[0]) != 0 or int(c.min()) < 0:
        raise BtError(5, f"issue-rate probe: a bounded wait ran out (code {int(err[0])})")
    return float((c.max(dim=1).values.double() / (iters * issuers)).median())


def bt_selftest_bounded_wait(model, limit_ms):
    """Runs the library's bounded barrier wait on a barrier nobody arrives at; raises BtError with
    status BT_ERR_DEVICE_TIMEOUT once the limit has passed (the expected outcome)."""
    _check(lib().bt_selftest_bounded_wait(model, limit_ms))


def bt_op_layernorm_fwd(x, gamma, beta, N, C, y, y_split, mean, rstd, stream=None):
    _check(lib().bt_op_layernorm_fwd(_ptr(x), _ptr(gamma), _ptr(beta), N, C, _ptr(y), _ptr(y_split), _ptr(mean),
                                     _ptr(rstd), _stream(stream)))


def bt_op_layernorm_bwd_scratch_bytes(N, C):
    return int(lib().bt_op_layernorm_bwd_scratch_bytes(N, C))


def bt_op_layernorm_bwd(dy, x, gamma, mean, rstd, dres, N, C, dx, dx_split, dgamma, dbeta, scratch, scratch_bytes,
                        stream=None):
    _check(lib().bt_op_layernorm_bwd(_ptr(dy), _ptr(x), _ptr(gamma), _ptr(mean), _ptr(rstd), _ptr(dres), N, C,
                                     _ptr(dx), _ptr(dx_split), _ptr(dgamma), _ptr(dbeta), _ptr(scratch),
                                     scratch_bytes, _stream(stream)))


def bt_op_layernorm_bwd_colsum(dy, x, gamma, mean, rstd, dres, N, C, dx, dx_split, dgamma, dbeta, dx_colsum, scratch,
                               scratch_bytes, stream=None):
    _check(lib().bt_op_layernorm_bwd_colsum(_ptr(dy), _ptr(x), _ptr(gamma), _ptr(mean), _ptr(rstd), _ptr(dres), N, C,
                                            _ptr(dx), _ptr(dx_split), _ptr(dgamma), _ptr(dbeta), _ptr(dx_colsum),
                                            _ptr(scratch), scratch_bytes, _stream(stream)))


def bt_op_gemm_scratch_bytes(layout, M, N, K):
    return int(lib().bt_op_gemm_scratch_bytes(layout, M, N, K))


def bt_op_gemm(layout, M, N, K, A, B, D, bias, residual, scratch, scratch_bytes, flags=0, stream=None):
    _check(lib().bt_op_gemm(layout, M, N, K, _ptr(A), _ptr(B), _ptr(D), _ptr(bias), _ptr(residual), _ptr(scratch),
                            scratch_bytes, flags, _stream(stream)))


def bt_op_split(x, n, x_split, stream=None):
    _check(lib().bt_op_split(_ptr(x), n, _ptr(x_split), _stream(stream)))


def bt_op_gemm_split_scratch_bytes():
    return int(lib().bt_op_gemm_split_scratch_bytes())


def bt_op_gemm_split_act(layout, M, N, K, A_split, B_split, D, D_act_split, act, bias, residual, scratch,
                         scratch_bytes, flags=0, stream=None):
    _check(lib().bt_op_gemm_split_act(layout, M, N, K, _ptr(A_split), _ptr(B_split), _ptr(D), _ptr(D_act_split), act,
                                      _ptr(bias), _ptr(residual), _ptr(scratch), scratch_bytes, flags, _stream(stream)))


def bt_op_gemm_split(layout, M, N, K, A_split, B_split, D, bias, residual, scratch, scratch_bytes, flags=0,
                     stream=None):
    _check(lib().bt_op_gemm_split(layout, M, N, K, _ptr(A_split), _ptr(B_split), _ptr(D), _ptr(bias), _ptr(residual),
                                  _ptr(scratch), scratch_bytes, flags, _stream(stream)))


def bt_op_gemm_gelu_bwd_scratch_bytes(M, N):
    return lib().bt_op_gemm_gelu_bwd_scratch_bytes(M, N)


def bt_op_gemm_gelu_bwd(M, N, K, dy_split, w_split, h, form, dh_split, colsum, scratch, scratch_bytes, flags=0,
                        stream=None):
    _check(lib().bt_op_gemm_gelu_bwd(M, N, K, _ptr(dy_split), _ptr(w_split), _ptr(h), int(form), _ptr(dh_split),
                                     _ptr(colsum), _ptr(scratch), scratch_bytes, flags, _stream(stream)))


def bt_op_gemm_plan(M, N, K, epilogue=False, flags=0):
    """The planner's choice for a product: dict with tile width, pair tiles, K splits, the tail split and the
    group height of the tile raster."""
    out = (ctypes.c_int32 * 7)()
    _check(lib().bt_op_gemm_plan(M, N, K, int(bool(epilogue)), flags, ctypes.cast(out, ctypes.c_void_p)))
    return dict(zip(("bn", "pair", "splits", "tail_tiles", "tail_splits", "tail_kbps", "group_m"), list(out)))


def bt_op_gemm_check(scratch, stream=None):
    _check(lib().bt_op_gemm_check(_ptr(scratch), _stream(stream)))


def bt_op_attention_fwd(qkv, B, T, C, H, o, o_split, lse, flags=0, stream=None, qkv_split=None):
    _check(lib().bt_op_attention_fwd(_ptr(qkv), _ptr(qkv_split), B, T, C, H, _ptr(o), _ptr(o_split), _ptr(lse), flags,
                                     _stream(stream)))


def bt_op_attention_bwd(qkv, o, lse, d_o, B, T, C, H, dqkv, dqkv_split, scratch, scratch_bytes, flags=0, stream=None,
                        qkv_split=None, d_o_split=None):
    _check(lib().bt_op_attention_bwd(_ptr(qkv), _ptr(qkv_split), _ptr(o), _ptr(lse), _ptr(d_o), _ptr(d_o_split), B, T,
                                     C, H, _ptr(dqkv), _ptr(dqkv_split), _ptr(scratch), scratch_bytes, flags,
                                     _stream(stream)))


def bt_op_gelu_fwd(x, n, tanh_form, y, y_split, stream=None):
    _check(lib().bt_op_gelu_fwd(_ptr(x), n, tanh_form, _ptr(y), _ptr(y_split), _stream(stream)))


def bt_op_gelu_bwd(x, dy, n, tanh_form, dx, dx_split, stream=None):
    _check(lib().bt_op_gelu_bwd(_ptr(x), _ptr(dy), n, tanh_form, _ptr(dx), _ptr(dx_split), _stream(stream)))


def bt_op_gelu_bwd_colsum(x, dy, N, C, tanh_form, dx, dx_split, colsum, scratch, scratch_bytes, stream=None):
    _check(lib().bt_op_gelu_bwd_colsum(_ptr(x), _ptr(dy), N, C, tanh_form, _ptr(dx), _ptr(dx_split), _ptr(colsum),
                                       _ptr(scratch), scratch_bytes, _stream(stream)))


def bt_op_softmax_xent(logits, targets, N, Vp, inv_count, losses, loss_mean, dlogits, dlogits_split, d_bad=None,
                       stream=None):
    _check(lib().bt_op_softmax_xent(_ptr(logits), _ptr(targets), N, Vp, inv_count, _ptr(losses), _ptr(loss_mean),
                                    _ptr(dlogits), _ptr(dlogits_split), _ptr(d_bad), _stream(stream)))


def bt_op_colsum_scratch_bytes(N, C):
    return int(lib().bt_op_colsum_scratch_bytes(N, C))


def bt_op_colsum(x, N, C, out, scratch, scratch_bytes, stream=None):
    _check(lib().bt_op_colsum(_ptr(x), N, C, _ptr(out), _ptr(scratch), scratch_bytes, _stream(stream)))


def bt_op_colsum_static_max_floats():
    return int(lib().bt_op_colsum_static_max_floats())


def bt_op_colsum_static(x, N, C, out, stream=None):
    """Column sums with the library's built-in scratch: for callers that cannot allocate device memory."""
    _check(lib().bt_op_colsum_static(_ptr(x), N, C, _ptr(out), _stream(stream)))


def bt_op_grad_norm_scratch_bytes(n):
    return int(lib().bt_op_grad_norm_scratch_bytes(n))


def bt_op_grad_norm(g, n, clip, out2, scratch, scratch_bytes, stream=None):
    _check(lib().bt_op_grad_norm(_ptr(g), n, clip, _ptr(out2), _ptr(scratch), scratch_bytes, _stream(stream)))


def bt_op_adamw_multi(p, g, m, v, decay, opt, t, d_scale=None, stream=None):
    """p, g, m, v: lists of CUDA tensors; decay: list of 0/1."""
    n = len(p)
    arr = lambda ts: (_vp * n)(*[_ptr(t) for t in ts])
    numel = (_i64 * n)(*[t.numel() for t in p])
    dec = (_i32 * n)(*decay)
    _check(lib().bt_op_adamw_multi(n, arr(p), arr(g), arr(m), arr(v), numel, dec, ctypes.byref(opt), t, _ptr(d_scale),
                                   _stream(stream)))


# ------------------------------------------------------------------ convenience holder

class Model:
    """Owns the torch workspace tensor and the bt_model handle; every method is one C call."""

    def __init__(self, n_layers, d_model, n_heads, seq_len, vocab_size, padded_vocab_size, max_batch, flags=0,
                 device="cuda:0"):
        self.cfg = make_config(n_layers, d_model, n_heads, seq_len, vocab_size, padded_vocab_size, max_batch, flags)
        nbytes = bt_workspace_bytes(self.cfg)
        if nbytes == 0:
            raise BtError(1, (lib().bt_last_error() or b"").decode())
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        off = (-self.workspace.data_ptr()) % 256
        self._base = self.workspace.data_ptr() + off
        self.workspace_bytes = nbytes
        self.h = bt_model_create(self.cfg, self._base, nbytes)
        self.T, self.C = seq_len, d_model
        self.names = [bt_tensor_info(self.h, i) for i in range(bt_num_tensors(self.h))]

    def close(self):
        if getattr(self, "h", None):
            bt_model_destroy(self.h)
            self.h = None

    __del__ = close

    def _view(self, ptr, numel):
        off = ptr - self.workspace.data_ptr()
        return self.workspace[off:off + 4 * numel].view(torch.float32)

    def tensor(self, name, kind=0):
        numel = next(n for nm, n, _ in self.names if nm == name)
        return self._view(bt_tensor_ptr(self.h, name, kind), numel)

    def activation(self, name, layer=0, planes=1):
        ptr, numel = bt_activation_ptr(self.h, name, layer)
        return self._view(ptr, numel * planes)

    def arena(self, kind=0):
        """One of the four flat arenas (0 parameters, 1 gradients, 2 / 3 moments) as a float32 view."""
        ptr, n = bt_arena_ptr(self.h, kind)
        return self._view(ptr, n)

    def ddp_attach(self, allreduce, comm_stream, bucket_cap_bytes=25 * 1000 * 1000):
        """allreduce(buf, bucket): must enqueue, on comm_stream, an in-place all-reduce of the float32
        tensor view `buf` (a range of the gradient arena) that leaves the average over the ranks."""
        def trampoline(_user, d_buf, count, bucket, _stream):
            try:
                with torch.cuda.stream(comm_stream):
                    allreduce(self._view(d_buf, count), int(bucket))
                return 0
            except Exception as exc:          # an exception must not cross the C frames
                self._ddp_error = exc
                return 1
        self._ddp_cb = ALLREDUCE_FN(trampoline)     # kept alive with the model
        self._ddp_stream = comm_stream
        _check(lib().bt_ddp_attach(self.h, bucket_cap_bytes, ctypes.cast(self._ddp_cb, _vp), None,
                                   comm_stream.cuda_stream))

    def ddp_detach(self):
        _check(lib().bt_ddp_detach(self.h))
        self._ddp_cb = None

    def load_params(self, params):
        for name, a in params.items():
            self.tensor(name).copy_(torch.as_tensor(a, dtype=torch.float32).reshape(-1))

    def init(self, seed):
        bt_model_init(self.h, seed)

    def forward(self, tokens, targets, want_loss=True):
        return bt_forward(self.h, tokens, targets, tokens.shape[0], want_loss)

    def backward(self):
        bt_backward(self.h)

    def adamw_step(self, opt, want_norm=True):
        return bt_adamw_step(self.h, opt, want_norm)

    def train_step(self, tokens, targets, opt, want_loss=True):
        return bt_train_step(self.h, tokens, targets, tokens.shape[0], opt, want_loss)

    def micro_step(self, tokens, targets, micro_index, n_micro, want_loss=True):
        return bt_micro_step(self.h, tokens, targets, tokens.shape[0], micro_index, n_micro, want_loss)

    def train_step_accum(self, tokens, targets, n_micro, opt, want_loss=True):
        return bt_train_step_accum(self.h, tokens, targets, tokens.shape[0] // n_micro, n_micro, opt, want_loss)

    def train_step_host(self, h_tokens, h_targets, opt, want_loss=True):
        return bt_train_step_host(self.h, h_tokens, h_targets, h_tokens.shape[0], opt, want_loss)
