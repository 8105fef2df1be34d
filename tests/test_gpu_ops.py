"""GPU parity tests, one kernel at a time: every per-op C-ABI entry point against the CPU
float64 oracle on the same seeded FP32 inputs.

Tolerances: embedding gather bit-exact; plain-FP32 kernels (LayerNorm, GELU, softmax
cross-entropy, column sums, norm, AdamW) 1e-5 relative L2; 3xTF32 tensor-core GEMM and
attention outputs 1e-4 relative (max and L2).
"""
import numpy as np
import pytest
import torch

import oracle
import seeded_inputs as si
from paper_2606_24780_b200 import binding as b

from gpu_util import check_split, dev, empty, host, rel_l2, rel_max, scratch, zeros

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------ embedding

@pytest.mark.parametrize("B,T,C,V,zipf", [(4, 64, 64, 512, False), (3, 100, 768, 50257, True), (1, 1, 64, 8, False)])
def test_embedding_fwd_bit_exact(B, T, C, V, zipf):
    wte, wpe = si.normal_f32(1, (V, C), 0.02), si.normal_f32(2, (T, C), 0.02)
    tok = (si.zipf_tokens(3, B, T, V) if zipf else si.uniform_tokens(3, B, T, V))[0]
    x = empty(B * T, C)
    b.bt_op_embedding_fwd(dev(tok), dev(wte), dev(wpe), B * T, T, C, V, x)
    ref = oracle.embedding_fwd(tok, wte, wpe, T, round_fp32=True).astype(np.float32)
    got = x.cpu().numpy()
    assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))


@pytest.mark.parametrize("B,T,C,V,zipf", [(4, 64, 64, 512, False), (8, 300, 768, 50257, True), (2, 513, 128, 7, False),
                                          (32, 1024, 768, 50257, True), (1, 5, 2048, 3, False), (3, 128, 64, 1, False)])
def test_embedding_bwd(B, T, C, V, zipf):
    """Chunks of 128 positions with a ragged last chunk, ids that collide inside a chunk and across
    chunks (V = 7, 3, 1), more than 256 float4 columns (C = 2048), and BASELINE config 3's token
    count with Zipf ids (thousands of positions on the most frequent id's row)."""
    tok = (si.zipf_tokens(5, B, T, V) if zipf else si.uniform_tokens(5, B, T, V))[0]
    dx = si.normal_f32(6, (B * T, C), 1e-2)
    base = si.normal_f32(7, (V, C), 1e-2)          # the LM-head gradient already in dwte
    dwte, dwpe = dev(base), empty(T, C)
    nbytes = b.bt_op_embedding_bwd_scratch_bytes(B * T, C, V)
    sc = scratch(nbytes)
    sc.fill_(0xAB)                                  # the scratch's previous contents must not matter
    b.bt_op_embedding_bwd(dev(tok), dev(dx), B * T, T, C, V, dwte, dwpe, sc, nbytes)
    rw, rp = oracle.embedding_bwd(tok, dx, T, V)
    assert rel_l2(host(dwte), rw + base) < 1e-5
    assert rel_l2(host(dwpe), rp) < 1e-5
    untouched = np.setdiff1d(np.arange(V), np.unique(tok))
    if untouched.size:
        assert np.array_equal(dwte.cpu().numpy()[untouched], base[untouched])
    # deterministic: a second run gives identical bits
    dwte2, dwpe2 = dev(base), empty(T, C)
    b.bt_op_embedding_bwd(dev(tok), dev(dx), B * T, T, C, V, dwte2, dwpe2, sc, nbytes)
    assert torch.equal(dwte, dwte2) and torch.equal(dwpe, dwpe2)
    with pytest.raises(b.BtError) as e:
        b.bt_op_embedding_bwd(dev(tok), dev(dx), B * T, T, C, V, dwte2, dwpe2, sc, nbytes - 1)
    assert e.value.status == 3


def test_out_of_range_ids_are_reported_and_never_used_as_an_index():
    """Ids outside [0, V) (negative, V itself, far beyond) are read as id 0 by the gather, by its
    backward and by the loss, and their position is left in the caller's error word."""
    B, T, C, V = 2, 70, 64, 50
    wte, wpe = si.normal_f32(1, (V, C), 0.02), si.normal_f32(2, (T, C), 0.02)
    tok = si.uniform_tokens(3, B, T, V)[0]
    bad_tok = tok.copy().ravel()
    bad_tok[[5, 77, 139]] = [V, -1, 2 ** 30]
    clean = bad_tok.copy()
    clean[[5, 77, 139]] = 0
    x, x_ref = empty(B * T, C), empty(B * T, C)
    flag = zeros(4, dtype=torch.int32)
    b.bt_op_embedding_fwd(dev(bad_tok), dev(wte), dev(wpe), B * T, T, C, V, x, flag)
    b.bt_op_embedding_fwd(dev(clean), dev(wte), dev(wpe), B * T, T, C, V, x_ref, flag[1:])
    assert torch.equal(x, x_ref)
    assert int(flag[0]) - 1 in (5, 77, 139) and int(flag[1]) == 0
    dx = si.normal_f32(6, (B * T, C), 1e-2)
    nbytes = b.bt_op_embedding_bwd_scratch_bytes(B * T, C, V)
    outs = []
    for ids in (bad_tok, clean):
        dwte, dwpe = zeros(V, C), empty(T, C)
        b.bt_op_embedding_bwd(dev(ids), dev(dx), B * T, T, C, V, dwte, dwpe, scratch(nbytes), nbytes)
        outs.append(dwte)
    assert torch.equal(outs[0], outs[1])
    z = si.normal_f32(23, (4, 64), 3.0)
    y_bad, y_clean = np.array([3, 64, -7, 9], np.int32), np.array([3, 0, 0, 9], np.int32)
    res = []
    flag.zero_()
    for i, y in enumerate((y_bad, y_clean)):
        losses, dl = empty(4), empty(4, 64)
        b.bt_op_softmax_xent(dev(z), dev(y), 4, 64, 0.25, losses, None, dl, None, flag[i:])
        res.append((losses, dl))
    assert torch.equal(res[0][0], res[1][0]) and torch.equal(res[0][1], res[1][1])
    assert int(flag[0]) - 1 in (1, 2) and int(flag[1]) == 0


# ------------------------------------------------------------------ LayerNorm

@pytest.mark.parametrize("N,C", [(256, 64), (1000, 768), (37, 1024), (5, 128), (300, 2048)])
def test_layernorm_fwd(N, C):
    x = si.normal_f32(10, (N, C), 2.0) + 0.5
    g, be = si.normal_f32(11, (C,), 0.3) + 1.0, si.normal_f32(12, (C,), 0.3)
    y, ys, mean, rstd = empty(N, C), empty(2, N, C), empty(N), empty(N)
    b.bt_op_layernorm_fwd(dev(x), dev(g), dev(be), N, C, y, ys, mean, rstd)
    ry, rm, rr = oracle.layernorm_fwd(x, g, be)
    assert rel_l2(host(y), ry) < 1e-5 and rel_max(host(y), ry) < 1e-5
    assert rel_l2(host(mean), rm) < 1e-5 and rel_l2(host(rstd), rr) < 1e-5
    check_split(ys, host(y))


@pytest.mark.parametrize("N,C,res", [(256, 64, True), (1000, 768, True), (4100, 768, False), (37, 1024, True),
                                     (300, 3072, True), (9, 4096, False), (70, 1028, True)])
def test_layernorm_bwd(N, C, res):
    x = si.normal_f32(13, (N, C), 1.5) - 0.2
    g = si.normal_f32(14, (C,), 0.3) + 1.0
    dy = si.normal_f32(15, (N, C), 1e-2)
    dres = si.normal_f32(16, (N, C), 1e-2) if res else None
    _, rm, rr = oracle.layernorm_fwd(x, g, np.zeros(C))
    mean, rstd = dev(rm, torch.float32), dev(rr, torch.float32)
    dx, dxs, dg, db = empty(N, C), empty(2, N, C), empty(C), empty(C)
    nb = b.bt_op_layernorm_bwd_scratch_bytes(N, C)
    b.bt_op_layernorm_bwd(dev(dy), dev(x), dev(g), mean, rstd, dev(dres) if res else None, N, C, dx, dxs, dg, db,
                          scratch(nb), nb)
    rdx, rdg, rdb = oracle.layernorm_bwd(dy, x, g, host(mean), host(rstd))
    if res:
        rdx = rdx + dres
    assert rel_l2(host(dx), rdx) < 1e-5
    assert rel_l2(host(dg), rdg) < 1e-5 and rel_l2(host(db), rdb) < 1e-5
    check_split(dxs, host(dx))


def test_layernorm_bwd_in_place_residual():
    """The step updates the residual-stream gradient in place (dx aliases dres)."""
    N, C = 600, 768
    x, g = si.normal_f32(17, (N, C)), si.normal_f32(18, (C,), 0.2) + 1.0
    dy, dres = si.normal_f32(19, (N, C), 1e-2), si.normal_f32(20, (N, C), 1e-2)
    _, rm, rr = oracle.layernorm_fwd(x, g, np.zeros(C))
    buf = dev(dres)
    nb = b.bt_op_layernorm_bwd_scratch_bytes(N, C)
    b.bt_op_layernorm_bwd(dev(dy), dev(x), dev(g), dev(rm, torch.float32), dev(rr, torch.float32), buf, N, C, buf,
                          None, empty(C), empty(C), scratch(nb), nb)
    rdx, _, _ = oracle.layernorm_bwd(dy, x, g, rm.astype(np.float32), rr.astype(np.float32))
    assert rel_l2(host(buf), rdx + dres) < 1e-5


@pytest.mark.parametrize("N,C", [(1000, 768), (37, 132), (8192, 1024), (3, 4), (700, 3072), (5, 2052)])
def test_layernorm_bwd_colsum(N, C):
    """The variant with fused column sums: same dx / dgamma / dbeta, plus colsum(dx) incl. residual."""
    x, dy, dres = si.normal_f32(31, (N, C), 1.5), si.normal_f32(32, (N, C), 1e-2), si.normal_f32(33, (N, C), 1e-2)
    g = (1.0 + si.normal_f32(34, (C,), 0.1)).astype(np.float32)
    rm, rr = oracle.layernorm_fwd(x, g, np.zeros(C, np.float32))[1:3]
    mean, rstd = dev(rm, torch.float32), dev(rr, torch.float32)
    nb = b.bt_op_layernorm_bwd_scratch_bytes(N, C)
    dx0, dg0, db0 = empty(N, C), empty(C), empty(C)
    b.bt_op_layernorm_bwd(dev(dy), dev(x), dev(g), mean, rstd, dev(dres), N, C, dx0, None, dg0, db0, scratch(nb), nb)
    dx1, dxs, dg1, db1, cs = empty(N, C), empty(2, N, C), empty(C), empty(C), empty(C)
    b.bt_op_layernorm_bwd_colsum(dev(dy), dev(x), dev(g), mean, rstd, dev(dres), N, C, dx1, dxs, dg1, db1, cs,
                                 scratch(nb), nb)
    assert np.array_equal(host(dx0), host(dx1)) and np.array_equal(host(dg0), host(dg1))
    assert np.array_equal(host(db0), host(db1))
    check_split(dxs, host(dx1))
    rdx, _, _ = oracle.layernorm_bwd(dy, x, g, host(mean), host(rstd))
    ref = (rdx.astype(np.float64) + dres).sum(0)
    assert np.abs(host(cs) - ref).max() < 1e-5 * np.abs(rdx + dres).sum(0).max() + 1e-12


# ------------------------------------------------------------------ GELU

@pytest.mark.parametrize("tanh_form", [0, 1])
def test_gelu_fwd_bwd(tanh_form):
    n = 4 * 12345
    x = np.concatenate([si.normal_f32(21, (n - 8,), 2.0), np.array([0, -0.0, 10, -10, 30, -30, 1e-20, -5], np.float32)])
    dy = si.normal_f32(22, (n,), 1e-2)
    y, ys, dx, dxs = empty(n), empty(2, n), empty(n), empty(2, n)
    b.bt_op_gelu_fwd(dev(x), n, tanh_form, y, ys)
    b.bt_op_gelu_bwd(dev(x), dev(dy), n, tanh_form, dx, dxs)
    ry, rdx = oracle.gelu_fwd(x, tanh_form), oracle.gelu_bwd(x, dy, tanh_form)
    assert rel_l2(host(y), ry) < 1e-5 and np.abs(host(y) - ry).max() < 2e-6
    assert rel_l2(host(dx), rdx) < 1e-5
    check_split(ys, host(y))
    check_split(dxs, host(dx))


@pytest.mark.parametrize("N,C", [(1000, 3072), (37, 132), (1, 4), (8192, 768)])
def test_gelu_bwd_colsum(N, C):
    """The fused kernel gives the dx of the plain one and its column sums (the bias gradient)."""
    x, dy = si.normal_f32(25, (N, C), 2.0), si.normal_f32(26, (N, C), 1e-2) + np.float32(3e-3)
    dx, dxs, cs = empty(N, C), empty(2, N, C), empty(C)
    nb = b.bt_op_colsum_scratch_bytes(N, C)
    b.bt_op_gelu_bwd_colsum(dev(x), dev(dy), N, C, 0, dx, dxs, cs, scratch(nb), nb)
    rdx = oracle.gelu_bwd(x.ravel(), dy.ravel(), 0).reshape(N, C)
    assert rel_l2(host(dx), rdx) < 1e-5
    check_split(dxs, host(dx))
    ref = rdx.astype(np.float64).sum(0)
    assert np.abs(host(cs) - ref).max() < 1e-5 * np.abs(rdx).sum(0).max() + 1e-12
    # split-only output (the form the training step uses)
    cs2 = empty(C)
    b.bt_op_gelu_bwd_colsum(dev(x), dev(dy), N, C, 0, None, dxs, cs2, scratch(nb), nb)
    assert np.array_equal(host(cs2), host(cs))


# ------------------------------------------------------------------ softmax cross-entropy

@pytest.mark.parametrize("N,Vp", [(256, 512), (64, 50304), (7, 1000), (3, 131072), (5, 4)])
def test_softmax_xent(N, Vp):
    z = si.normal_f32(23, (N, Vp), 3.0)
    z[0, :] = 0.0
    if N > 1:
        z[1, 3 % Vp] = 80.0
    y = si.uniform_tokens(24, 1, N, Vp)[0].ravel()
    inv = 1.0 / (4 * N)                      # as if this were one chunk of a larger batch
    losses, lm, dl, dls = empty(N), empty(1), empty(N, Vp), empty(2, N, Vp)
    b.bt_op_softmax_xent(dev(z), dev(y), N, Vp, inv, losses, lm, dl, dls)
    rl, rdl = oracle.softmax_xent(z, y, inv)
    assert rel_l2(host(losses), rl) < 1e-5 and np.abs(host(losses) - rl).max() < 1e-4
    assert abs(float(host(lm)[0]) - rl.sum() * inv) < 1e-5 * abs(rl.sum() * inv)
    assert rel_l2(host(dl), rdl) < 1e-5
    assert np.abs(host(dl).sum(1)).max() < 1e-6 * inv * Vp ** 0.5 + 1e-9
    check_split(dls, host(dl))


@pytest.mark.parametrize("N,Vp", [(640, 50304), (1201, 33000)])
def test_softmax_xent_row_loop_kernel(N, Vp):
    """Long rows with at least four rows per SM run as a row loop that fetches the next row while the
    current one is reduced and stored.  Checked against the oracle, bit for bit against the
    grid-per-row kernel (which the same rows take when handed over in pieces of fewer rows), and in
    place (the gradient's hi plane written over the logits)."""
    z = si.normal_f32(26, (N, Vp), 3.0)
    z[1, 3] = 80.0
    y = si.uniform_tokens(27, 1, N, Vp)[0].ravel()
    inv = 1.0 / N
    losses, lm, dl, dls = empty(N), empty(1), empty(N, Vp), empty(2, N, Vp)
    b.bt_op_softmax_xent(dev(z), dev(y), N, Vp, inv, losses, lm, dl, dls)
    rl, rdl = oracle.softmax_xent(z, y, inv)
    assert rel_l2(host(losses), rl) < 1e-5 and np.abs(host(losses) - rl).max() < 1e-4
    assert rel_l2(host(dl), rdl) < 1e-5
    check_split(dls, host(dl))
    # the same rows in pieces small enough for the grid-per-row kernel
    zd, yd = dev(z), dev(y)
    losses2, dl2 = empty(N), empty(N, Vp)
    step = 300
    for r0 in range(0, N, step):
        n = min(step, N - r0)
        b.bt_op_softmax_xent(zd[r0:r0 + n], yd[r0:r0 + n], n, Vp, inv, losses2[r0:r0 + n], None, dl2[r0:r0 + n], None)
    assert np.array_equal(host(losses2), host(losses)) and np.array_equal(host(dl2), host(dl))
    # in place: the hi plane of the gradient over the logits
    buf = empty(2, N, Vp)
    buf[0].copy_(zd)
    losses3 = empty(N)
    b.bt_op_softmax_xent(buf[0], yd, N, Vp, inv, losses3, None, None, buf)
    assert np.array_equal(host(losses3), host(losses)) and np.array_equal(host(buf), host(dls))


# ------------------------------------------------------------------ reductions

@pytest.mark.parametrize("N,C", [(256, 64), (8192, 768), (1000, 3072), (33, 2304)])
def test_colsum(N, C):
    x = si.normal_f32(25, (N, C), 1e-2)
    out = empty(C)
    nb = b.bt_op_colsum_scratch_bytes(N, C)
    b.bt_op_colsum(dev(x), N, C, out, scratch(nb), nb)
    assert rel_l2(host(out), x.astype(np.float64).sum(0)) < 1e-5


@pytest.mark.parametrize("n,mag", [(136960, 1e-3), (5_000_003, 1.0), (4, 100.0)])
def test_grad_norm_and_clip(n, mag):
    g = si.normal_f32(26, (n,), mag)
    out = empty(2)
    nb = b.bt_op_grad_norm_scratch_bytes(n)
    b.bt_op_grad_norm(dev(g), n, 1.0, out, scratch(nb), nb)
    gn = oracle.grad_norm([g])
    got = host(out)
    assert abs(got[0] - gn) < 1e-6 * gn
    assert abs(got[1] - oracle.clip_scale(gn, 1.0)) < 1e-6
    b.bt_op_grad_norm(dev(g), n, 0.0, out, scratch(nb), nb)
    assert host(out)[1] == 1.0


# ------------------------------------------------------------------ AdamW

def test_adamw_multi_matches_oracle_at_step_seven():
    shapes = [(50304 * 8,), (768,), (4097,), (3,), (2304 * 64,)]
    decay = [1, 0, 1, 0, 1]
    hp = si.ADAMW
    opt = b.make_adamw(**hp)
    t, scale = 7, 0.37
    ps, gs, ms, vs = [], [], [], []
    for i, s in enumerate(shapes):
        ps.append(si.normal_f32(30 + i, s, 0.02))
        gs.append(si.normal_f32(40 + i, s, 10.0 ** -(i + 1)))
        ms.append(si.normal_f32(50 + i, s, 1e-3))
        vs.append(np.abs(si.normal_f32(60 + i, s, 1e-5)))
    dp, dg, dm, dv = [dev(a) for a in ps], [dev(a) for a in gs], [dev(a) for a in ms], [dev(a) for a in vs]
    b.bt_op_adamw_multi(dp, dg, dm, dv, decay, opt, t, d_scale=dev(np.array([scale], np.float32)))
    for i in range(len(shapes)):
        rp, rm, rv = oracle.adamw(ps[i], gs[i], ms[i], vs[i], hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                                  hp["weight_decay"], decay[i], t, np.float32(scale))
        assert np.abs(host(dp[i]) - rp).max() < 1e-6, i
        assert rel_l2(host(dm[i]), rm) < 1e-6 and rel_l2(host(dv[i]), rv) < 1e-6


# ------------------------------------------------------------------ GEMM

GEMM_SHAPES = [
    (0, 256, 192, 64), (1, 256, 64, 192), (2, 192, 64, 256),          # tiny model
    (0, 1000, 2304, 768), (0, 520, 768, 3072),                        # ragged M, both tile widths
    (1, 1000, 768, 2304), (1, 384, 3072, 768),
    (2, 768, 768, 4096), (2, 2304, 768, 2000), (2, 1056, 160, 520),   # split-K, ragged everything
    (0, 128, 1056, 128), (0, 4, 4, 4),
]


@pytest.mark.parametrize("flags", [0, b.BT_FLAG_GEMM_SIMT, b.BT_FLAG_GEMM_PAIR, b.BT_FLAG_GEMM_SINGLE])
@pytest.mark.parametrize("layout,M,N,K", GEMM_SHAPES)
def test_gemm(layout, M, N, K, flags):
    """flags 0: the planner picks the tile; PAIR / SINGLE force the cta_group::2 (256-row tiles on
    CTA pairs) or the single-CTA kernel; SIMT is the FP32 FMA reference kernel."""
    if flags != b.BT_FLAG_GEMM_SIMT and ((layout == 2 and M % 32) or (layout != 0 and N % 32)):
        pytest.skip("transposed extents must be multiples of 32 on the tensor-core path")
    a_shape = (K, M) if layout == 2 else (M, K)
    b_shape = (N, K) if layout == 0 else (K, N)
    A, Bm = si.normal_f32(70, a_shape), si.normal_f32(71, b_shape, 0.05)
    bias, res = si.normal_f32(72, (N,)), si.normal_f32(73, (M, N))
    A64 = A.astype(np.float64).T if layout == 2 else A.astype(np.float64)
    B64 = Bm.astype(np.float64).T if layout == 0 else Bm.astype(np.float64)
    nb = b.bt_op_gemm_scratch_bytes(layout, M, N, K)
    sc = scratch(nb)
    for use_epi in (False, True):
        D = zeros(M, N)
        b.bt_op_gemm(layout, M, N, K, dev(A), dev(Bm), D, dev(bias) if use_epi else None,
                     dev(res) if use_epi else None, sc, nb, flags)
        ref = A64 @ B64
        if use_epi:
            ref = ref + bias + res
        assert rel_l2(host(D), ref) < (1e-5 if flags == b.BT_FLAG_GEMM_SIMT else 1e-4), (layout, M, N, K, use_epi)
        assert rel_max(host(D), ref) < 1e-4


@pytest.mark.parametrize("layout,M,N,K", [(1, 4864, 1024, 1024), (0, 4860, 1000, 1028), (2, 4864, 1024, 1040),
                                          (1, 8192, 768, 3072)])
def test_gemm_tail_split(layout, M, N, K):
    """Pair tiles whose last round is cut along K (76 tiles of 256 x 256 for 74 CTA pairs; 96 for the
    MLP down-projection's shape): the reduction pass adds the K ranges and applies bias, residual and the
    hi/lo planes; ragged rows, columns and k-blocks included."""
    flags = b.BT_FLAG_GEMM_PAIR
    plan = b.bt_op_gemm_plan(M, N, K, True, flags)
    assert plan["pair"] == 1 and plan["tail_splits"] > 1 and plan["tail_tiles"] > 0, plan
    a_shape = (K, M) if layout == 2 else (M, K)
    b_shape = (N, K) if layout == 0 else (K, N)
    A, Bm = si.normal_f32(170, a_shape), si.normal_f32(171, b_shape, 0.05)
    bias, res = si.normal_f32(172, (N,)), si.normal_f32(173, (M, N))
    A64 = A.astype(np.float64).T if layout == 2 else A.astype(np.float64)
    B64 = Bm.astype(np.float64).T if layout == 0 else Bm.astype(np.float64)
    As, Bs = empty(2, *a_shape), empty(2, *b_shape)
    b.bt_op_split(dev(A), A.size, As)
    b.bt_op_split(dev(Bm), Bm.size, Bs)
    nb = b.bt_op_gemm_split_scratch_bytes()
    sc = scratch(nb)
    for use_epi in (False, True):
        D, Ds = zeros(M, N), zeros(2, M, N)
        b.bt_op_gemm_split_act(layout, M, N, K, As, Bs, D, Ds, 0, dev(bias) if use_epi else None,
                               dev(res) if use_epi else None, sc, nb, flags)
        b.bt_op_gemm_check(sc)
        ref = A64 @ B64
        if use_epi:
            ref = ref + bias + res
        assert rel_l2(host(D), ref) < 1e-4 and rel_max(host(D), ref) < 1e-4, (layout, M, N, K, use_epi)
        check_split(Ds, host(D))


@pytest.mark.parametrize("act", [1, 4])
def test_gemm_tail_split_with_gelu_epilogue(act):
    """The forward GELU modes through the tail split: the reduction pass evaluates GELU (planes) and, in
    modes 3 / 4, GELU' (D) for the tiles of the last round."""
    M, N, K, flags = 4864, 1024, 1024, b.BT_FLAG_GEMM_PAIR
    assert b.bt_op_gemm_plan(M, N, K, True, flags)["tail_splits"] > 1
    x, w, bias = si.normal_f32(174, (M, K)), si.normal_f32(175, (K, N), 0.05), si.normal_f32(176, (N,), 0.5)
    xs, ws = empty(2, M, K), empty(2, K, N)
    b.bt_op_split(dev(x), M * K, xs)
    b.bt_op_split(dev(w), K * N, ws)
    D, Ds = empty(M, N), empty(2, M, N)
    nb = b.bt_op_gemm_split_scratch_bytes()
    sc = scratch(nb)
    b.bt_op_gemm_split_act(1, M, N, K, xs, ws, D, Ds, act, dev(bias), None, sc, nb, flags)
    b.bt_op_gemm_check(sc)
    rh = x.astype(np.float64) @ w.astype(np.float64) + bias
    tanh_form = act in (2, 4)
    got = host(Ds)
    assert rel_l2(got[0].astype(np.float64) + got[1], oracle.gelu_fwd(rh.ravel(), tanh_form).reshape(M, N)) < 1e-4
    want_d = rh if act <= 2 else oracle.gelu_bwd(rh.ravel(), np.ones(rh.size), tanh_form).reshape(M, N)
    assert rel_l2(host(D), want_d) < 1e-4


def _planner_sweep_shapes():
    """Seeded shapes whose tile counts land on every side of the planner's choices: fewer tiles than
    slots (K splits), one full round plus a small tail (tail split), several rounds, ragged edges."""
    rng = np.random.RandomState(20240607)
    shapes = []
    for _ in range(14):
        layout = int(rng.randint(0, 3))
        M = int(rng.choice([256, 1280, 4864, 9472, 12800, 19200])) - 4 * int(rng.randint(0, 3)) * (layout != 2)
        N = int(rng.choice([128, 768, 1024, 1536, 2304])) - 4 * int(rng.randint(0, 3)) * (layout == 0)
        K = int(rng.choice([256, 768, 1024, 2304, 3072])) + 4 * int(rng.randint(0, 3))
        shapes.append((layout, M, N, K))
    return shapes


@pytest.mark.parametrize("layout,M,N,K", _planner_sweep_shapes())
def test_gemm_planner_sweep(layout, M, N, K):
    """Whatever the planner picks for a shape (tile width, pair tiles, K split, tail split), the product
    with bias and residual matches the FP64 product; the plan itself is reported on failure."""
    plan = b.bt_op_gemm_plan(M, N, K, True)
    a_shape = (K, M) if layout == 2 else (M, K)
    b_shape = (N, K) if layout == 0 else (K, N)
    A, Bm = si.normal_f32(180, a_shape), si.normal_f32(181, b_shape, 0.05)
    bias, res = si.normal_f32(182, (N,)), si.normal_f32(183, (M, N))
    A64 = A.astype(np.float64).T if layout == 2 else A.astype(np.float64)
    B64 = Bm.astype(np.float64).T if layout == 0 else Bm.astype(np.float64)
    nb = b.bt_op_gemm_scratch_bytes(layout, M, N, K)
    sc = scratch(nb)
    for use_epi in (True, False):
        D = zeros(M, N)
        b.bt_op_gemm(layout, M, N, K, dev(A), dev(Bm), D, dev(bias) if use_epi else None, dev(res) if use_epi else None,
                     sc, nb, 0)
        ref = A64 @ B64 + ((bias + res) if use_epi else 0.0)
        assert rel_l2(host(D), ref) < 1e-4 and rel_max(host(D), ref) < 1e-4, (layout, M, N, K, use_epi, plan)


@pytest.mark.parametrize("layout,M,N,K", [(0, 4600, 5120, 264), (1, 4608, 4864, 512), (2, 4640, 5120, 1032),
                                          (0, 2300, 772, 3080)])
def test_gemm_tile_raster_groups(layout, M, N, K):
    """The tiles are walked in groups of row tiles (4, or 16 with many tile columns) with a shorter last
    group; every tile of the output must come out, whatever the order."""
    plan = b.bt_op_gemm_plan(M, N, K, False)
    tiles_m = -(-M // (256 if plan["pair"] else 128))
    assert 1 < plan["group_m"] < tiles_m and tiles_m % plan["group_m"] != 0, plan
    a_shape = (K, M) if layout == 2 else (M, K)
    b_shape = (N, K) if layout == 0 else (K, N)
    A, Bm = si.normal_f32(184, a_shape), si.normal_f32(185, b_shape, 0.05)
    A64 = A.astype(np.float64).T if layout == 2 else A.astype(np.float64)
    B64 = Bm.astype(np.float64).T if layout == 0 else Bm.astype(np.float64)
    nb = b.bt_op_gemm_scratch_bytes(layout, M, N, K)
    D = empty(M, N)
    D.fill_(float("nan"))
    b.bt_op_gemm(layout, M, N, K, dev(A), dev(Bm), D, None, None, scratch(nb), nb, 0)
    ref = A64 @ B64
    assert np.isfinite(host(D)).all()
    assert rel_l2(host(D), ref) < 1e-4 and rel_max(host(D), ref) < 1e-4, plan


def test_gemm_matches_oracle_linear_layer():
    """The three layouts are the forward, input-gradient and weight-gradient of a linear layer."""
    N, cin, cout = 640, 768, 1024
    x, w, bias = si.normal_f32(74, (N, cin)), si.normal_f32(75, (cout, cin), 0.02), si.normal_f32(76, (cout,), 0.1)
    dy = si.normal_f32(77, (N, cout), 1e-2)
    y, dx, dw = empty(N, cout), empty(N, cin), empty(cout, cin)
    for lay, M, Nn, K, A, Bm, D, bi in [(0, N, cout, cin, x, w, y, bias), (1, N, cin, cout, dy, w, dx, None),
                                       (2, cout, cin, N, dy, x, dw, None)]:
        nb = b.bt_op_gemm_scratch_bytes(lay, M, Nn, K)
        b.bt_op_gemm(lay, M, Nn, K, dev(A), dev(Bm), D, dev(bi) if bi is not None else None, None, scratch(nb), nb)
    ry = oracle.linear_fwd(x, w, bias)
    rdx, rdw, _ = oracle.linear_bwd(dy, x, w)
    assert rel_l2(host(y), ry) < 1e-4 and rel_l2(host(dx), rdx) < 1e-4 and rel_l2(host(dw), rdw) < 1e-4


# ------------------------------------------------------------------ attention

@pytest.mark.parametrize("flags", [0, b.BT_FLAG_ATTN_SIMT])
@pytest.mark.parametrize("B,T,H,d", [(4, 64, 4, 16), (2, 200, 3, 64), (1, 1, 2, 64), (1, 129, 2, 32), (1, 96, 1, 128)])
def test_attention_fwd_bwd(B, T, H, d, flags):
    C = H * d
    qkv = si.normal_f32(80, (B * T, 3 * C))
    d_o = si.normal_f32(81, (B * T, C), 1e-2)
    o, os_, lse = empty(B * T, C), empty(2, B * T, C), empty(B, H, T)
    b.bt_op_attention_fwd(dev(qkv), B, T, C, H, o, os_, lse, flags)
    ro, rlse = oracle.attention_fwd(qkv, B, T, H)
    assert rel_l2(host(o), ro) < 1e-4 and rel_max(host(o), ro) < 1e-4
    assert np.abs(host(lse) - rlse).max() < 1e-4
    check_split(os_, host(o))
    dqkv, dqs = empty(B * T, 3 * C), empty(2, B * T, 3 * C)
    nb = B * H * T * 4
    b.bt_op_attention_bwd(dev(qkv), o, lse, dev(d_o), B, T, C, H, dqkv, dqs, scratch(nb), nb, flags)
    rd = oracle.attention_bwd(qkv, d_o, B, T, H)
    for part in range(3):
        assert rel_l2(host(dqkv)[:, part * C:(part + 1) * C], rd[:, part * C:(part + 1) * C]) < 1e-4, part
    check_split(dqs, host(dqkv))


TC_ATTN_SHAPES = [(2, 200, 3, 64), (1, 1024, 2, 64), (1, 1, 2, 64), (3, 129, 1, 64), (1, 130, 12, 64), (2, 64, 1, 64),
                  (1, 65, 1, 64), (1, 33, 1, 64),
                  (28, 200, 8, 64),   # 224 heads x 2 blocks: the CTA order in two groups of 112 heads
                  (2, 200, 2, 128), (1, 1024, 1, 128), (1, 1, 2, 128), (2, 129, 1, 128), (1, 130, 3, 128),
                  (2, 64, 1, 128), (1, 33, 1, 128), (1, 300, 2, 128)]


@pytest.mark.parametrize("B,T,H,d", TC_ATTN_SHAPES)
def test_attention_fwd_tcgen05_kernel(B, T, H, d):
    """head_dim 64 / 128 with the qkv array given as hi/lo planes: the TMA + tcgen05 + TMEM kernels."""
    C = H * d
    qkv = si.normal_f32(82, (B * T, 3 * C))
    dq = dev(qkv)
    qs = empty(2, B * T, 3 * C)
    b.bt_op_split(dq, dq.numel(), qs)
    o, os_, lse = empty(B * T, C), empty(2, B * T, C), empty(B, H, T)
    b.bt_op_attention_fwd(None, B, T, C, H, o, os_, lse, 0, qkv_split=qs)
    ro, rlse = oracle.attention_fwd(qkv, B, T, H)
    assert rel_l2(host(o), ro) < 1e-4 and rel_max(host(o), ro) < 1e-4
    assert np.abs(host(lse) - rlse).max() < 1e-4
    check_split(os_, host(o))
    # and it agrees with the kernel that takes the raw array (warp-MMA; FMA for head_dim 128)
    o2, lse2 = empty(B * T, C), empty(B, H, T)
    b.bt_op_attention_fwd(dq, B, T, C, H, o2, None, lse2, 0)
    assert rel_max(host(o), host(o2)) < 1e-5


@pytest.mark.parametrize("B,T,H,d", TC_ATTN_SHAPES)
def test_attention_bwd_tcgen05_kernels(B, T, H, d):
    """head_dim 64 / 128, qkv and d_o given as hi/lo planes, only the split gradient requested."""
    C = H * d
    qkv = si.normal_f32(83, (B * T, 3 * C))
    d_o = si.normal_f32(84, (B * T, C), 1e-2)
    dq, ddo = dev(qkv), dev(d_o)
    qs, dos = empty(2, B * T, 3 * C), empty(2, B * T, C)
    b.bt_op_split(dq, dq.numel(), qs)
    b.bt_op_split(ddo, ddo.numel(), dos)
    o, lse = empty(B * T, C), empty(B, H, T)
    b.bt_op_attention_fwd(None, B, T, C, H, o, None, lse, 0, qkv_split=qs)
    dqs = zeros(2, B * T, 3 * C)
    nb = B * H * T * 4
    b.bt_op_attention_bwd(None, o, lse, None, B, T, C, H, None, dqs, scratch(nb), nb, 0, qkv_split=qs, d_o_split=dos)
    got = host(dqs)
    got = got[0] + got[1]
    rd = oracle.attention_bwd(qkv, d_o, B, T, H)
    for part in range(3):
        assert rel_l2(got[:, part * C:(part + 1) * C], rd[:, part * C:(part + 1) * C]) < 1e-4, part
    assert not (dqs[0].cpu().numpy().view(np.uint32) & 0x1FFF).any()


def test_attention_long_context_16k():
    """The long-context shape (T = 16,384, head_dim 64): 128 key tiles per query block in the forward,
    512 query tiles per key block in the backward.  Two heads of one sequence against the
    matrix-form float64 oracle."""
    B, T, H, d = 1, 16384, 2, 64
    C = H * d
    qkv = si.normal_f32(85, (B * T, 3 * C))
    d_o = si.normal_f32(86, (B * T, C), 1e-2)
    dq, ddo = dev(qkv), dev(d_o)
    qs, dos = empty(2, B * T, 3 * C), empty(2, B * T, C)
    b.bt_op_split(dq, dq.numel(), qs)
    b.bt_op_split(ddo, ddo.numel(), dos)
    o, lse = empty(B * T, C), empty(B, H, T)
    b.bt_op_attention_fwd(None, B, T, C, H, o, None, lse, 0, qkv_split=qs)
    dqs = zeros(2, B * T, 3 * C)
    nb = B * H * T * 4
    b.bt_op_attention_bwd(None, o, lse, None, B, T, C, H, None, dqs, scratch(nb), nb, 0, qkv_split=qs, d_o_split=dos)
    ro, rlse, rd = oracle.attention_dense(qkv, d_o, B, T, H)
    assert rel_l2(host(o), ro) < 1e-4 and rel_max(host(o), ro) < 1e-4
    assert np.abs(host(lse) - rlse).max() < 1e-4
    got = host(dqs)
    got = got[0] + got[1]
    errs = [rel_l2(got[:, part * C:(part + 1) * C], rd[:, part * C:(part + 1) * C]) for part in range(3)]
    print("T = 16384: o %.1e, dq %.1e, dk %.1e, dv %.1e (relative L2)" % (rel_l2(host(o), ro), *errs))
    assert max(errs) < 1e-4, errs


@pytest.mark.parametrize("act,flags", [(a, f) for a in (0, 1, 2, 3, 4)
                                       for f in (b.BT_FLAG_GEMM_PAIR, b.BT_FLAG_GEMM_SINGLE, b.BT_FLAG_GEMM_SIMT)
                                       if not (a > 2 and f == b.BT_FLAG_GEMM_SIMT)])
def test_gemm_epilogue_activation_planes(act, flags):
    """The MLP up-projection as the step runs it: weight given transposed (layout NN), bias in the
    epilogue, the raw output kept and GELU(output) emitted as TF32 hi/lo planes by the same kernel."""
    N, cin, cout = 520, 256, 768
    x, w, bias = si.normal_f32(91, (N, cin)), si.normal_f32(92, (cout, cin), 0.1), si.normal_f32(93, (cout,), 0.5)
    xs, wts = empty(2, N, cin), empty(2, cin, cout)
    b.bt_op_split(dev(x), N * cin, xs)
    b.bt_op_split(dev(np.ascontiguousarray(w.T)), cin * cout, wts)
    h, gs = empty(N, cout), empty(2, N, cout)
    nb = b.bt_op_gemm_split_scratch_bytes()
    b.bt_op_gemm_split_act(1, N, cout, cin, xs, wts, h, gs, act, dev(bias), None, scratch(nb), nb, flags)
    rh = oracle.linear_fwd(x, w, bias)
    tanh_form = act in (2, 4)
    want = rh if act == 0 else oracle.gelu_fwd(rh.ravel(), tanh_form).reshape(N, cout)
    got = host(gs)
    assert rel_l2(got[0] + got[1], want) < 1e-4
    assert not (gs[0].cpu().numpy().view(np.uint32) & 0x1FFF).any()
    if act >= 3:   # D holds GELU'(h): the derivative the oracle's backward applies to a gradient of ones
        want_d = oracle.gelu_bwd(rh.ravel(), np.ones(rh.size), tanh_form).reshape(N, cout)
        assert rel_l2(host(h), want_d) < 1e-4
        return
    assert rel_l2(host(h), rh) < 1e-4
    # the planes are the split of the kernel's own FP32 value of act(h)
    ref32 = host(h) if act == 0 else oracle.gelu_fwd(host(h).ravel(), tanh_form).reshape(N, cout)
    assert np.abs((got[0].astype(np.float64) + got[1]) - ref32).max() < 1e-5 * np.abs(ref32).max()


_GELU_BWD_CASES = [(M, N, K, t, f) for (M, N, K) in [(520, 768, 256), (8, 32, 4), (1000, 352, 132)] for t in (0, 1)
                   for f in (0, b.BT_FLAG_GEMM_SINGLE, b.BT_FLAG_GEMM_PAIR)] + [(4096, 3072, 768, 0, 0)] + \
                  [(4864, 1024, 1024, t, b.BT_FLAG_GEMM_PAIR) for t in (0, 1)]   # 76 pair tiles: two rounds


@pytest.mark.parametrize("M,N,K,tanh_form,flags", _GELU_BWD_CASES)
def test_gemm_gelu_bwd_epilogue(M, N, K, tanh_form, flags):
    """The input-gradient product of the MLP down-projection with the GELU backward in its epilogue:
    dh = (dy W) o GELU'(h) as hi/lo planes, and the column sums of dh (ragged row and column tiles,
    rows that do not fill a 32-row group, several tiles per CTA)."""
    dy, w, h = si.normal_f32(95, (M, K), 1e-2), si.normal_f32(96, (K, N), 0.1), si.normal_f32(97, (M, N), 2.0)
    dys, ws = empty(2, M, K), empty(2, K, N)
    b.bt_op_split(dev(dy), M * K, dys)
    b.bt_op_split(dev(w), K * N, ws)
    dh, cs = empty(2, M, N), empty(N)
    nb = b.bt_op_gemm_gelu_bwd_scratch_bytes(M, N)
    sc = scratch(nb)
    b.bt_op_gemm_gelu_bwd(M, N, K, dys, ws, dev(h), tanh_form, dh, cs, sc, nb, flags)
    b.bt_op_gemm_check(sc)
    dg = dy.astype(np.float64) @ w.astype(np.float64)
    want = oracle.gelu_bwd(h.ravel(), dg.ravel(), tanh_form).reshape(M, N)
    got = host(dh)
    assert rel_l2(got[0].astype(np.float64) + got[1], want) < 1e-5
    assert not (dh[0].cpu().numpy().view(np.uint32) & 0x1FFF).any()
    assert np.abs(host(cs) - want.sum(0)).max() < 1e-5 * np.abs(want).sum(0).max() + 1e-12
    # the column sums are those of the planes the kernel wrote, group by group
    assert np.abs(host(cs) - (got[0].astype(np.float64) + got[1]).sum(0)).max() < 2e-6 * np.abs(want).sum(0).max() + 1e-12
    # the same with GELU'(h) handed over instead of h (what the forward epilogue leaves): bit-identical
    # when the derivative is the library's own FP32 value
    gp = empty(M, N)
    b.bt_op_gelu_bwd(dev(h), dev(np.ones((M, N), np.float32)), M * N, tanh_form, gp, None)
    dh2, cs2 = empty(2, M, N), empty(N)
    b.bt_op_gemm_gelu_bwd(M, N, K, dys, ws, gp, 2, dh2, cs2, sc, nb, flags)
    b.bt_op_gemm_check(sc)
    assert torch.equal(dh2, dh) and torch.equal(cs2, cs)


def test_gemm_gelu_bwd_rejects_bad_arguments():
    x = empty(64)
    nb = b.bt_op_gemm_gelu_bwd_scratch_bytes(8, 32)
    sc = scratch(nb)
    for args, status in [((8, 30, 4), 1), ((0, 32, 4), 1), ((8, 32, 6), 1)]:
        with pytest.raises(b.BtError) as e:
            b.bt_op_gemm_gelu_bwd(*args, x, x, x, 0, x, x, sc, nb)
        assert e.value.status == status
    with pytest.raises(b.BtError) as e:
        b.bt_op_gemm_gelu_bwd(8, 32, 4, x, x, x, 0, x, x, sc, 16)
    assert e.value.status == 3
    with pytest.raises(b.BtError) as e:
        b.bt_op_gemm_gelu_bwd(8, 32, 4, x, x, x, 0, x, x, sc, nb, b.BT_FLAG_GEMM_SIMT)
    assert e.value.status == 2


def test_empty_inputs_are_no_ops_or_rejected():
    """Zero-length calls: the element-wise entry points accept n = 0 and launch nothing; calls whose
    result is undefined for no rows (reductions, GEMM) refuse them on the host."""
    x = empty(4)
    b.bt_op_gelu_fwd(x, 0, 0, x, None)
    b.bt_op_gelu_bwd(x, x, 0, 0, x, None)
    b.bt_op_embedding_fwd(dev(np.zeros(1, np.int32)), x, x, 0, 1, 4, 1, x)
    b.bt_op_layernorm_fwd(x, x, x, 0, 4, x, None, x, x)
    for call in (lambda: b.bt_op_colsum(x, 0, 4, x, x, 1024),
                 lambda: b.bt_op_softmax_xent(x, dev(np.zeros(1, np.int32)), 0, 4, 1.0, x, None, None, None),
                 lambda: b.bt_op_grad_norm(x, 0, 1.0, x, x, 1024),
                 lambda: b.bt_op_gemm_split(0, 0, 4, 4, x, x, x, None, None, scratch(b.bt_op_gemm_split_scratch_bytes()),
                                            b.bt_op_gemm_split_scratch_bytes())):
        with pytest.raises(b.BtError) as e:
            call()
        assert e.value.status == 1
    torch.cuda.synchronize()


# ------------------------------------------------------------------ rate probes (measurement aids)

def test_mma_rate_probes_give_the_rates_the_kernels_are_planned_with():
    """The probes behind the roofline's TF32 peak and behind the attention kernels' division of their
    products among issuing threads: a 128 x 256 x 8 MMA occupies the pipe for 128 clocks (2048 MAC per
    clock and SM); one thread cannot issue N = 64 MMAs as fast as the pipe executes them with the A
    operand in tensor memory (32 clocks), two can; bad arguments are refused on the host."""
    lo, med, hi = b.bt_probe_tf32_mma_rate(8, 2000)
    assert 120.0 < med < 140.0 and hi < 160.0
    one = b.bt_probe_mma_issue_rate(64, True, 1, n_ctas=8, iters=2048)
    two = b.bt_probe_mma_issue_rate(64, True, 2, n_ctas=8, iters=2048)
    assert 45.0 < one < 75.0 and 30.0 < two < 40.0 and two < 0.75 * one
    assert 120.0 < b.bt_probe_mma_issue_rate(256, False, 2, n_ctas=8, iters=1024) < 140.0
    for args in [(96, 0, 1), (256, 1, 1), (64, 0, 0), (64, 0, 5)]:
        with pytest.raises(b.BtError) as e:
            b.bt_probe_mma_issue_rate(*args, n_ctas=1, iters=16)
        assert e.value.status == 1
