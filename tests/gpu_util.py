"""Helpers shared by the GPU parity tests (device staging and error metrics only)."""
import numpy as np
import torch

DEV = "cuda:0"


def dev(a, dtype=None):
    t = torch.as_tensor(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.to(DEV).contiguous()


def empty(*shape, dtype=torch.float32):
    return torch.empty(*shape, dtype=dtype, device=DEV)


def zeros(*shape, dtype=torch.float32):
    return torch.zeros(*shape, dtype=dtype, device=DEV)


def scratch(nbytes):
    """256-byte aligned device scratch of at least nbytes."""
    t = torch.empty(nbytes + 512, dtype=torch.uint8, device=DEV)
    off = (-t.data_ptr()) % 256
    return t[off:off + nbytes + 256]


def host(t):
    torch.cuda.synchronize()
    return t.detach().cpu().numpy().astype(np.float64)


def rel_l2(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    den = np.linalg.norm(ref.ravel())
    return np.linalg.norm((got - ref).ravel()) / (den if den > 0 else 1.0)


def rel_max(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    den = np.abs(ref).max()
    return np.abs(np.asarray(got, dtype=np.float64) - ref).max() / (den if den > 0 else 1.0)


def check_split(split_t, raw64):
    """A split array [2][...] must satisfy hi + lo == raw (in FP32) and hi has 13 low zero bits."""
    s = split_t.detach().cpu().numpy()
    hi, lo = s[0], s[1]
    assert not (hi.view(np.uint32) & 0x1FFF).any(), "hi plane keeps low mantissa bits"
    np.testing.assert_array_equal((hi + lo).astype(np.float32), np.asarray(raw64, dtype=np.float32))
