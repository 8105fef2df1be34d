"""Whole-step GPU parity: forward, backward and AdamW of the CUDA library against the CPU
float64 oracle on the same seeded parameters and tokens.

Tolerances (the target the build is held to): logits and loss 1e-4 relative; every gradient
tensor 1e-3 relative L2; post-AdamW parameters 1e-5 absolute.  "Relative" for a tensor means
max|diff| / max|reference| and ||diff||_2 / ||reference||_2.  A gradient that is
mathematically zero (the key bias: softmax is shift invariant) is held to an absolute bound
scaled by the neighbouring query-bias gradient instead.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import seeded_inputs as si
from paper_2606_24780_b200 import binding as b

from gpu_util import dev, host, rel_l2, rel_max

pytestmark = pytest.mark.gpu

TOL_LOGITS, TOL_LOSS, TOL_GRAD, TOL_PARAM = 1e-4, 1e-4, 1e-3, 1e-5


def make_pair(cfg, seed, flags, max_batch, jitter=0.02):
    params = si.init_params(cfg, seed, jitter=jitter)
    gm = b.Model(cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["seq_len"], cfg["vocab_size"],
                 cfg["padded_vocab_size"], max_batch, flags)
    gm.load_params(params)
    om = oracle.Model(cfg)
    om.set_params(params)
    return gm, om


def grad_error(got, ref, scale=0.0):
    """Relative L2 error of a gradient (part); a gradient that is mathematically zero (oracle norm
    below 1e-12 sqrt(numel)) is held to an absolute bound instead -- 1e-9 per element, or 1e-5 of
    `scale`, the size of a neighbouring non-zero gradient -- and counts as error 0."""
    if np.linalg.norm(ref) < 1e-12 * math.sqrt(ref.size):
        assert np.linalg.norm(got) <= max(1e-9, 1e-5 * scale) * math.sqrt(ref.size), np.linalg.norm(got)
        return 0.0
    return rel_l2(got, ref)


def compare_gradients(gm, om, cfg):
    C = cfg["d_model"]
    worst = 0.0
    for name in om.names():
        ref = om.get(name, 1)
        got = host(gm.tensor(name, 1))
        if name.endswith("attn.qkv.b"):
            # q and v parts relative; the k part is exactly zero in exact arithmetic
            vscale = np.abs(ref[2 * C:]).max()
            for lo, hi in ((0, C), (2 * C, 3 * C)):
                e = grad_error(got[lo:hi], ref[lo:hi], vscale)
                assert e < TOL_GRAD, (name, lo, e)
                worst = max(worst, e)
            assert np.abs(ref[C:2 * C]).max() < 1e-12
            assert np.abs(got[C:2 * C]).max() <= max(1e-3 * np.abs(ref[:C]).max(), 1e-5 * vscale) + 1e-9, name
            continue
        e = grad_error(got, ref)
        assert e < TOL_GRAD, (name, e)
        worst = max(worst, e)
    return worst


def adamw_step_and_compare(gm, om, step, max_outside=0.02):
    """One optimizer step on both sides from IDENTICAL state (p, m, v, t), two comparisons.

    (A) optimizer exactness: the oracle's AdamW applied to the GPU's own gradient must give the
        GPU's new parameters within 1e-5 absolute on EVERY element (and the moments within 1e-5
        relative L2).  This is the post-AdamW tolerance for the update itself.
    (B) end to end against the oracle's own gradient: the update lr * mhat / (sqrt(vhat) + eps)
        is ill-conditioned where an element's gradient history is ~0 (at t = 1 it is
        lr * g / (|g| + eps): slope lr / eps = 6e4 at g = 0, so an FP32-rounding-sized gradient
        error flips the whole +-lr step).  Elements outside 1e-5 must therefore be rare and
        bounded by 2.2 lr; their count is reported.
    """
    hp = si.ADAMW
    opt = b.make_adamw(**hp)
    names = om.names()
    g_gpu = {n: host(gm.tensor(n, 1)) for n in names}
    state = {n: (om.get(n, 0), om.get(n, 2), om.get(n, 3)) for n in names}
    gn_gpu_ref = oracle.grad_norm(list(g_gpu.values()))
    scale = oracle.clip_scale(gn_gpu_ref, hp["grad_clip"])
    gn = gm.adamw_step(opt)
    ref_gn = om.adamw_step(hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"], hp["grad_clip"])
    # the norm is a gradient quantity: held to the gradient tolerance against the oracle's own
    # gradient, and to FP32 accuracy against the norm of the GPU's gradient
    assert abs(gn - ref_gn) < TOL_GRAD * ref_gn and abs(gn - gn_gpu_ref) < 1e-5 * gn_gpu_ref
    print(f"grad norm {gn:.6f} (oracle {ref_gn:.6f}, rel diff {(gn - ref_gn) / ref_gn:+.2e})")
    total, outside, worst_a = 0, 0, 0.0
    for n in names:
        p0, m0, v0 = state[n]
        pb, mb, vb = oracle.adamw(p0, g_gpu[n], m0, v0, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                                  hp["weight_decay"], om.decay(n), step + 1, scale)
        got = host(gm.tensor(n))
        da = np.abs(got - pb).max()
        worst_a = max(worst_a, da)
        assert da < TOL_PARAM, (step, n, da)                                   # (A)
        assert rel_l2(host(gm.tensor(n, 2)), mb) < 1e-5 and rel_l2(host(gm.tensor(n, 3)), vb) < 1e-5, n
        db = np.abs(got - om.get(n))                                           # (B)
        total += db.size
        outside += int((db >= TOL_PARAM).sum())
        assert db.max() <= 2.2 * hp["lr"], (step, n, db.max())
    assert outside <= max_outside * total, (step, outside, total)
    # continue from identical state: the oracle adopts the GPU's FP32 parameters and moments
    for n in names:
        for kind in (0, 2, 3):
            om.set_tensor(n, host(gm.tensor(n, kind)), kind)
    return outside / total, worst_a


def run_steps(cfg, seed, flags, B, steps, chunk=0):
    gm, om = make_pair(cfg, seed, flags, B)
    Vp = cfg["padded_vocab_size"]
    for step in range(steps):
        tok, tgt = si.tokens_for(cfg, 1000 * seed + step, B)
        dtok, dtgt = dev(tok), dev(tgt)
        loss = gm.forward(dtok, dtgt)
        ref_loss = om.loss_and_grad(tok, tgt, chunk)
        assert abs(loss - ref_loss) < TOL_LOSS * abs(ref_loss), (step, loss, ref_loss)
        if chunk == 0:
            ref_logits = om.activation("logits")
            got_logits = host(gm.activation("logits")).reshape(-1, Vp)
            assert rel_max(got_logits, ref_logits) < TOL_LOGITS and rel_l2(got_logits, ref_logits) < TOL_LOGITS
        gm.backward()
        compare_gradients(gm, om, cfg)
        frac, worst = adamw_step_and_compare(gm, om, step)
        print(f"step {step}: loss {loss:.6f} (oracle {ref_loss:.6f}); AdamW exactness {worst:.2e}; "
              f"{100 * frac:.3f}% of parameters ill-conditioned")
        assert b.bt_get_step(gm.h) == step + 1
    launches = b.bt_launch_count(gm.h)
    gm.close()
    return launches


@pytest.mark.parametrize("flags", [b.BT_FLAG_GEMM_SIMT | b.BT_FLAG_ATTN_SIMT, b.BT_FLAG_ATTN_SIMT, 0])
def test_tiny_config_three_steps(flags):
    """BASELINE config 0, three consecutive optimizer steps (the first alone barely exercises
    the moments, the bias correction or the clip)."""
    cfg = si.config(0)
    launches = run_steps(cfg, seed=0, flags=flags, B=cfg["batch"], steps=3)
    assert launches > 3 * 50


def test_initial_loss_near_log_vocab():
    cfg = si.config(0)
    gm, _ = make_pair(cfg, 0, 0, cfg["batch"], jitter=0.0)
    tok, tgt = si.tokens_for(cfg, 0)
    loss = gm.forward(dev(tok), dev(tgt))
    assert abs(loss - (math.log(cfg["padded_vocab_size"]) + 0.5 * cfg["d_model"] * 0.02 ** 2)) < 0.05
    gm.close()


def test_medium_config_spans_tiles_and_ragged_tails():
    """GPT-2-small width with a short context and a small vocabulary: several GEMM tiles in every
    dimension, ragged M (B*T = 3*200 = 600 rows), Zipf tokens, head_dim 64."""
    cfg = si.make_config(n_layers=2, d_model=768, n_heads=12, seq_len=200, vocab_size=4000,
                         padded_vocab_size=4032, batch=3, tokens="zipf")
    run_steps(cfg, seed=3, flags=0, B=3, steps=2)


def test_gpt2_124m_full_size_step():
    """BASELINE config 2 at full size, in the launch configuration the benchmark times: 12 layers,
    d_model 768, vocabulary 50257 (padded 50304), batch 8 x 1024 Zipf tokens.  The oracle runs
    the eight sequences one at a time (about two minutes on 16 host cores) and supplies the loss,
    the logits of the last sequence, every gradient tensor and the AdamW update."""
    import time
    cfg = si.config(2)
    B = cfg["batch"]
    t0 = time.time()
    gm, om = make_pair(cfg, seed=2, flags=0, max_batch=B, jitter=0.0)
    tok, tgt = si.tokens_for(cfg, 2, B)
    loss = gm.forward(dev(tok), dev(tgt))
    gm.backward()
    ref_loss = om.loss_and_grad(tok, tgt, chunk=1)
    print(f"oracle forward+backward of {B} x {cfg['seq_len']} tokens: {time.time() - t0:.0f} s; "
          f"loss {loss:.6f} vs {ref_loss:.6f}")
    assert abs(loss - ref_loss) < TOL_LOSS * abs(ref_loss)
    # "initial loss ~ ln(vocab)": with tied embeddings and Zipf text a position whose target repeats
    # its input token sees a large target logit, which pulls the mean a little below
    # ln(Vp) + (logit variance) / 2 = 10.98
    assert abs(ref_loss - math.log(cfg["padded_vocab_size"])) < 0.2
    T, Vp = cfg["seq_len"], cfg["padded_vocab_size"]
    ref_logits = om.activation("logits")                      # last chunk = last sequence
    got_logits = host(gm.activation("logits")).reshape(-1, Vp)[(B - 1) * T:]
    assert rel_max(got_logits, ref_logits) < TOL_LOGITS and rel_l2(got_logits, ref_logits) < TOL_LOGITS
    worst = compare_gradients(gm, om, cfg)
    frac, exact = adamw_step_and_compare(gm, om, 0, max_outside=0.05)
    print(f"worst gradient rel-L2 {worst:.2e}; AdamW exactness {exact:.2e}; {100 * frac:.2f}% of parameters "
          f"ill-conditioned at t = 1")
    gm.close()


def test_partial_batch_and_host_tokens():
    """A batch smaller than max_batch, and the host-buffer entry point, give the same step."""
    cfg = si.config(0)
    params = si.init_params(cfg, 5, jitter=0.02)
    opt = b.make_adamw(**si.ADAMW)
    tok, tgt = si.tokens_for(cfg, 5, 3)
    results = []
    for host_path in (False, True):
        gm = b.Model(cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["seq_len"], cfg["vocab_size"],
                     cfg["padded_vocab_size"], 8)
        gm.load_params(params)
        if host_path:
            loss = gm.train_step_host(torch.as_tensor(tok).pin_memory(), torch.as_tensor(tgt).pin_memory(), opt)
        else:
            loss = gm.train_step(dev(tok), dev(tgt), opt)
        results.append((loss, host(gm.tensor("h1.mlp.fc.w")), host(gm.tensor("wte"))))
        gm.close()
    assert results[0][0] == results[1][0]
    assert np.array_equal(results[0][1], results[1][1]) and np.array_equal(results[0][2], results[1][2])
    om = oracle.Model(cfg)
    om.set_params(params)
    ref = om.loss_and_grad(tok, tgt)
    assert abs(results[0][0] - ref) < TOL_LOSS * ref


def test_step_is_deterministic():
    cfg = si.config(0)
    params = si.init_params(cfg, 6, jitter=0.02)
    opt = b.make_adamw(**si.ADAMW)
    tok, tgt = si.tokens_for(cfg, 6)
    outs = []
    for _ in range(2):
        gm = b.Model(cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["seq_len"], cfg["vocab_size"],
                     cfg["padded_vocab_size"], cfg["batch"])
        gm.load_params(params)
        gm.train_step(dev(tok), dev(tgt), opt)
        outs.append(torch.cat([gm.tensor(n).clone() for n, _, _ in gm.names]))
        gm.close()
    assert torch.equal(outs[0], outs[1])


def test_model_init_distribution():
    cfg = si.config(0)
    gm = b.Model(cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["seq_len"], cfg["vocab_size"],
                 cfg["padded_vocab_size"], 1)
    gm.init(1234)
    wte = host(gm.tensor("wte"))
    assert abs(wte.mean()) < 1e-3 and abs(wte.std() - 0.02) < 5e-4
    pr = host(gm.tensor("h1.mlp.proj.w"))
    assert abs(pr.std() - 0.02 / math.sqrt(2 * cfg["n_layers"])) < 5e-4
    assert np.all(host(gm.tensor("h0.ln1.g")) == 1.0) and not host(gm.tensor("h0.attn.qkv.b")).any()
    assert not host(gm.tensor("wte", 2)).any()
    gm.close()


def test_gradient_accumulation_matches_one_large_batch():
    """Algorithm 1's micro-step loop: n_micro micro-batches of B sequences accumulate to the gradient
    of the mean loss over all n_micro * B sequences, which the oracle computes as one batch.  Both
    the explicit bt_micro_step calls and bt_train_step_accum are checked, then the optimizer step."""
    cfg = si.make_config(n_layers=2, d_model=64, n_heads=1, seq_len=96, vocab_size=300, padded_vocab_size=320,
                         batch=2, tokens="zipf")          # head_dim 64: the tcgen05 attention path
    B, n_micro = 2, 3
    gm, om = make_pair(cfg, 5, 0, B)
    tok, tgt = si.tokens_for(cfg, 77, B * n_micro)
    dtok, dtgt = dev(tok), dev(tgt)
    micro_losses = []
    for i in range(n_micro):
        sl = slice(i * B, (i + 1) * B)
        micro_losses.append(gm.micro_step(dtok[sl], dtgt[sl], i, n_micro))
    ref_loss = om.loss_and_grad(tok, tgt, chunk=B)
    assert abs(micro_losses[-1] - ref_loss) < TOL_LOSS * ref_loss                    # last call: the mean
    ref_micro0 = oracle.Model(cfg)
    ref_micro0.set_params(si.init_params(cfg, 5, jitter=0.02))
    assert abs(micro_losses[0] - ref_micro0.loss(tok[:B], tgt[:B])) < TOL_LOSS * ref_loss
    worst = compare_gradients(gm, om, cfg)
    print(f"accumulated gradient: worst relative L2 error {worst:.2e}")
    adamw_step_and_compare(gm, om, 0)
    # the one-call form, from the state both sides now share
    tok2, tgt2 = si.tokens_for(cfg, 78, B * n_micro)
    opt = b.make_adamw(**si.ADAMW)
    p_before = {n: host(gm.tensor(n)) for n in om.names()}
    loss2 = gm.train_step_accum(dev(tok2), dev(tgt2), n_micro, opt)
    ref2 = om.loss_and_grad(tok2, tgt2, chunk=B)
    assert abs(loss2 - ref2) < TOL_LOSS * ref2
    compare_gradients(gm, om, cfg)
    assert b.bt_get_step(gm.h) == 2
    assert any(np.abs(host(gm.tensor(n)) - p_before[n]).max() > 0 for n in om.names())
    gm.close()


def test_training_trajectory_with_schedule_and_accumulation():
    """100 optimizer steps of a small model on Zipf tokens, two micro-batches per step, learning rate
    from the warmup + cosine schedule: the GPU and the oracle run independently from the same start
    (no re-synchronisation) and must report the same falling loss curve."""
    cfg = si.make_config(n_layers=2, d_model=64, n_heads=4, seq_len=64, vocab_size=512, padded_vocab_size=512,
                         batch=4, tokens="zipf")
    B, n_micro, steps = 4, 2, 100
    gm, om = make_pair(cfg, 9, 0, B, jitter=0.0)
    hp = dict(si.ADAMW)
    sched = b.bt_lr_schedule(6e-3, 6e-4, 10, steps)       # a short schedule with a larger peak, same shape
    gpu_curve, ref_curve = [], []
    for step in range(1, steps + 1):
        tok, tgt = si.tokens_for(cfg, 5000 + step, B * n_micro)
        lr = b.bt_lr_at(sched, step)
        assert abs(lr - oracle.lr_schedule(step, np.float32(6e-3), np.float32(6e-4), 10, steps)) < 1e-9
        hp["lr"] = lr
        gpu_curve.append(gm.train_step_accum(dev(tok), dev(tgt), n_micro, b.make_adamw(**hp)))
        ref_curve.append(om.loss_and_grad(tok, tgt, chunk=B))
        om.adamw_step(lr, hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"], hp["grad_clip"])
    gpu_curve, ref_curve = np.array(gpu_curve), np.array(ref_curve)
    print("loss: start %.4f, step 50 %.4f, end %.4f (oracle %.4f)" % (gpu_curve[0], gpu_curve[49], gpu_curve[-1],
                                                                   ref_curve[-1]))
    print("largest loss difference along the trajectory: %.2e relative" % (np.abs(gpu_curve - ref_curve).max() /
                                                                            ref_curve.max()))
    assert np.abs(gpu_curve - ref_curve).max() < 5e-4 * ref_curve.max()   # measured 2e-5 on a B200; both sides run free
    assert np.abs(gpu_curve[:10] - ref_curve[:10]).max() < TOL_LOSS * ref_curve.max()
    assert gpu_curve[-10:].mean() < gpu_curve[0] - 0.5          # it learns the token frequencies
    gm.close()


def test_wide_model_head_dim_128():
    """One layer at the width of the paper's 2.42B configuration (d_model 3072, 24 heads of 128):
    the wide LayerNorm backward, head_dim-128 attention and K = 12,288 GEMMs in one step."""
    cfg = si.make_config(n_layers=1, d_model=3072, n_heads=24, seq_len=64, vocab_size=1000, padded_vocab_size=1024,
                         batch=2, tokens="zipf")
    run_steps(cfg, seed=6, flags=0, B=2, steps=1)


def test_350m_width_two_layers():
    """The width of BASELINE config 4 (d_model 1024, 16 heads of 64, MLP 4096) at reduced depth and
    context: the VPL = 8 LayerNorm instantiations and the 1024 / 4096-wide GEMM tilings in a step."""
    cfg = si.make_config(n_layers=2, d_model=1024, n_heads=16, seq_len=256, vocab_size=3000, padded_vocab_size=3072,
                         batch=2, tokens="zipf")
    run_steps(cfg, seed=10, flags=0, B=2, steps=1)


def test_wide_model_full_width_full_context():
    """Two layers at the full width of the paper's 2.42B configuration (d_model 3072, 24 heads of
    128) and its full context (T = 1024, one sequence): eight query blocks per head in the
    head_dim-128 attention passes, K = 12,288 GEMMs, CTA-per-row LayerNorm.  About half a minute
    of oracle time."""
    cfg = si.make_config(n_layers=2, d_model=3072, n_heads=24, seq_len=1024, vocab_size=2000, padded_vocab_size=2048,
                         batch=1, tokens="zipf")
    run_steps(cfg, seed=9, flags=0, B=1, steps=1)


def test_head_dim_128_model_with_several_query_blocks():
    """Two layers with two heads of 128 at T = 200: the head_dim-128 attention passes walk several
    128-row blocks and a ragged last tile inside a whole training step (loss, every gradient, the
    AdamW update against the oracle)."""
    cfg = si.make_config(n_layers=2, d_model=256, n_heads=2, seq_len=200, vocab_size=500, padded_vocab_size=512,
                         batch=2, tokens="zipf")
    run_steps(cfg, seed=8, flags=0, B=2, steps=2)


@pytest.mark.parametrize("pinned", [True, False])
def test_double_buffered_loader_feeds_the_step(pinned):
    """Algorithm 2 on the GPU: batches arrive through the copy stream two channels deep; every batch
    is bit-identical to the window the oracle's cursor names, for two interleaved ranks over three
    shards with wrap-around, and the training step can consume them directly."""
    cfg = si.config(0)
    B, T, world = 2, cfg["seq_len"], 2
    bt_ = B * T
    rng = np.random.Generator(np.random.PCG64(11))
    lens = [bt_ * world * 3 + 1, bt_ * world + 7, bt_ * world * 2 + 1]
    shards = [rng.integers(0, cfg["vocab_size"], n).astype(np.int32) for n in lens]
    tshards = [torch.from_numpy(s) for s in shards]
    loaders = [b.Loader(tshards, B, T, rank=r, world=world, pinned=pinned) for r in range(world)]
    want = [oracle.loader_windows(lens, B, T, r, world, 14) for r in range(world)]
    gm, om = make_pair(cfg, 3, 0, B)
    opt = b.make_adamw(**si.ADAMW)
    for i in range(14):
        for r in range(world):
            x, y = loaders[r].next()
            s, p = want[r][i]
            assert np.array_equal(x.cpu().numpy().ravel(), shards[s][p:p + bt_])
            assert np.array_equal(y.cpu().numpy().ravel(), shards[s][p + 1:p + bt_ + 1])
            if r == 0 and i < 3:
                loss = gm.train_step(x, y, opt)
                ref = om.loss_and_grad(x.cpu().numpy(), y.cpu().numpy())
                assert abs(loss - ref) < TOL_LOSS * ref
                hp = si.ADAMW
                om.adamw_step(hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"], hp["grad_clip"])
                for n in om.names():
                    for kind in (0, 2, 3):
                        om.set_tensor(n, host(gm.tensor(n, kind)), kind)
    for L in loaders:
        L.close()
    gm.close()


@pytest.mark.parametrize("L,C,H,T,V,B", [(1, 64, 4, 5, 40, 3), (1, 64, 1, 7, 36, 1), (2, 128, 2, 1, 32, 2),
                                         (1, 64, 4, 64, 512, 1), (1, 32, 2, 3, 8, 1)])
def test_ragged_and_degenerate_shapes(L, C, H, T, V, B):
    """Token counts that are no multiple of anything (15, 7, 3 rows), a single sequence, and context
    length 1, where attention is the identity on v and the query / key gradients vanish exactly."""
    cfg = si.make_config(n_layers=L, d_model=C, n_heads=H, seq_len=T, vocab_size=V,
                         padded_vocab_size=(V + 31) // 32 * 32, batch=B, tokens="uniform")
    run_steps(cfg, seed=4, flags=0, B=B, steps=2)
