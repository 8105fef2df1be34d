"""Data-parallel gradient exchange (Algorithm 1, "Distributed Data Parallel Training Step").

CPU part (no GPU): the bucket plan and the in-order launch gate are host arithmetic of the C
library; two gloo ranks then run the step the way the algorithm states it -- every rank's own
gradient (the oracle on its shard of the batch), buckets all-reduced (average) in the order the
gate releases them, only on the last micro-step -- and must end with the gradient of the
concatenated batch on every rank.
GPU part: one GPU, so the second rank's gradient is produced beforehand and the all-reduce
callback averages with it in place; the library's own marks, events, per-bucket accumulation and
the wait before the optimizer step are exactly what a multi-GPU run executes.
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import seeded_inputs as si                                   # noqa: E402
from paper_2606_24780_b200 import binding as b               # noqa: E402
from paper_2606_24780_b200 import build as bt_build          # noqa: E402


def _cfg_struct(cfg, max_batch=4):
    return b.make_config(cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["seq_len"], cfg["vocab_size"],
                         cfg["padded_vocab_size"], max_batch)


def _ready_order(n_layers):
    """Registry indices in the order the backward pass finishes their gradients: final LayerNorm, then
    per block (last first) MLP down-projection, MLP up-projection, second LayerNorm, attention output
    projection, QKV, first LayerNorm; a block's down-projection bias falls out of the LayerNorm
    backward that follows it; the tied embedding and the position table come last."""
    n = 2 + 12 * n_layers + 2
    LN1G, LN1B, QKVW, QKVB, PROJW, PROJB, LN2G, LN2B, FCW, FCB, PRW, PRB = range(12)
    at = lambda l, k: 2 + 12 * l + k
    order = [n - 1, n - 2, at(n_layers - 1, PRB)]
    for l in range(n_layers - 1, -1, -1):
        order += [at(l, PRW), at(l, FCB), at(l, FCW), at(l, LN2B), at(l, LN2G), at(l, PROJB), at(l, PROJW),
                  at(l, QKVB), at(l, QKVW), at(l, LN1B), at(l, LN1G)]
        if l > 0:
            order.append(at(l - 1, PRB))
    return order + [1, 0]


@pytest.fixture(scope="module")
def lib():
    bt_build.build()
    return b.lib()


def test_bucket_plan_covers_the_arena_once_in_ready_order(lib):
    for cfg, cap in [(si.config(0), 64 * 1024), (si.config(0), 4096), (si.config(2), 25 * 1000 * 1000),
                     (si.config(4), 25 * 1000 * 1000), (si.config(2), 1 << 40)]:
        plan = b.DdpPlan(_cfg_struct(cfg), cap)
        reg = si.tensor_registry(cfg)
        # tensors: registry order, 1024-float alignment, padded lengths
        end = 0
        for i, (_, shape, _, _) in enumerate(reg):
            off, ln = plan.tensor(i)
            assert off == end and off % 1024 == 0 and ln >= int(np.prod(shape)) and ln % 1024 == 0
            end = off + ln
        # buckets: contiguous, from the arena's end to its start, each under the cap unless it is one tensor
        cap_floats = cap // 4 // 1024 * 1024
        hi = end
        waits = 0
        for k in range(plan.n_buckets):
            off, cnt, nt = plan.bucket(k)
            assert off + cnt == hi and cnt > 0 and nt >= 1
            assert cnt <= cap_floats
            hi = off
            waits += nt
        assert hi == 0
        split = sum(1 for i in range(len(reg)) if plan.tensor(i)[1] > cap_floats)
        assert waits >= len(reg) and (split > 0 or waits == len(reg))
        # the gate: in backward order every bucket is released exactly once, in order, and never early
        plan.reset()
        released = []
        for t in _ready_order(cfg["n_layers"]):
            now = plan.mark_ready(t)
            for k in now:
                off, cnt, _ = plan.bucket(k)
                t_off, t_len = plan.tensor(t)
                assert off <= t_off + t_len - 1          # a bucket is complete when its LOWEST tensor is ready
            released += now
        assert released == list(range(plan.n_buckets))
        with pytest.raises(b.BtError):
            plan.mark_ready(0)                            # twice
        plan.close()
    if True:
        plan = b.DdpPlan(_cfg_struct(si.config(2)))
        assert plan.n_buckets >= 20                        # 498 MB of gradients under a 25 MB cap
        plan.close()


def test_launch_gate_keeps_bucket_order_under_any_arrival_order(lib):
    cfg = si.config(0)
    plan = b.DdpPlan(_cfg_struct(cfg), 16 * 1024)
    n = len(si.tensor_registry(cfg))
    rng = np.random.Generator(np.random.PCG64(5))
    for _ in range(20):
        plan.reset()
        released = []
        ready = set()
        for t in rng.permutation(n):
            now = plan.mark_ready(int(t))
            ready.add(int(t))
            released += now
            assert released == list(range(len(released)))             # strictly in order
            for k in now:                                             # and only when every tensor inside is ready
                off, cnt, _ = plan.bucket(k)
                inside = [i for i in range(n) if plan.tensor(i)[0] < off + cnt and plan.tensor(i)[0] + plan.tensor(i)[1] > off]
                assert set(inside) <= ready
        assert released == list(range(plan.n_buckets))
    plan.close()


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _ddp_rank(rank, world, port, out):
    """One rank of Algorithm 1 on the CPU: the oracle stands for forward/backward on the rank's shard."""
    import torch.distributed as dist
    import oracle
    torch.set_num_threads(1)
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    cfg = si.config(0)
    B, n_micro = 2, 2                                       # per rank and micro-step
    plan = b.DdpPlan(_cfg_struct(cfg), 32 * 1024)
    reg = si.tensor_registry(cfg)
    P = sum(plan.tensor(i)[1] for i in range(len(reg)))
    # identical start weights: rank 0 draws them, everybody receives them (line 3 of the algorithm)
    params = si.init_params(cfg, 21 if rank == 0 else 999, jitter=0.02)
    flat = torch.zeros(P, dtype=torch.float64)
    for i, (name, _, _, _) in enumerate(reg):
        off, _ = plan.tensor(i)
        flat[off:off + params[name].size] = torch.from_numpy(params[name].astype(np.float64).ravel())
    dist.broadcast(flat, src=0)
    params = {name: flat[plan.tensor(i)[0]:plan.tensor(i)[0] + int(np.prod(shape))].numpy().reshape(shape).astype(np.float32)
              for i, (name, shape, _, _) in enumerate(reg)}
    om = oracle.Model(cfg)
    om.set_params(params)
    tok, tgt = si.tokens_for(cfg, 300, B * n_micro * world)   # the global batch; rank r takes rows r, r + world, ...
    grads = torch.zeros(P, dtype=torch.float64)
    launches = []
    for micro in range(n_micro):
        rows = [world * (micro * B + j) + rank for j in range(B)]
        om.loss_and_grad(tok[rows], tgt[rows])
        grad_sync = micro == n_micro - 1
        plan.reset()
        for t in _ready_order(cfg["n_layers"]):               # the backward pass "fires" the hooks in this order
            name = reg[t][0]
            off, _ = plan.tensor(t)
            g = torch.from_numpy(om.get(name, 1))
            grads[off:off + g.numel()] += g / n_micro          # local accumulation, no communication
            if not grad_sync:
                continue
            for k in plan.mark_ready(t):                       # in-order launch gate
                o, c, _ = plan.bucket(k)
                dist.all_reduce(grads[o:o + c], op=dist.ReduceOp.SUM)
                grads[o:o + c] /= world                        # average
                launches.append(k)
    out.put((rank, launches, grads.numpy().copy(), {n: p.copy() for n, p in params.items()}))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_average_to_the_gradient_of_the_whole_batch(lib):
    import oracle
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_ddp_rank, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted((out.get(timeout=300) for _ in range(world)), key=lambda r: r[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg = si.config(0)
    plan = b.DdpPlan(_cfg_struct(cfg), 32 * 1024)
    reg = si.tensor_registry(cfg)
    (_, l0, g0, p0), (_, l1, g1, p1) = results
    assert l0 == l1 == list(range(plan.n_buckets))             # every bucket once, in order, on the last micro-step only
    assert np.array_equal(g0, g1)                              # all ranks hold the same averaged gradient
    for n in p0:
        assert np.array_equal(p0[n], p1[n])                    # the broadcast gave both ranks rank 0's weights
    om = oracle.Model(cfg)
    om.set_params(p0)
    tok, tgt = si.tokens_for(cfg, 300, 2 * 2 * world)
    om.loss_and_grad(tok, tgt)                                 # the whole global batch at once
    for i, (name, shape, _, _) in enumerate(reg):
        off, _ = plan.tensor(i)
        ref = om.get(name, 1)
        got = g0[off:off + ref.size]
        assert np.abs(got - ref).max() <= 1e-12 * max(1.0, np.abs(ref).max()), name
    plan.close()


@pytest.mark.gpu
@pytest.mark.parametrize("n_micro", [1, 3])
def test_gpu_step_with_attached_all_reduce(n_micro):
    """Rank 0 of a two-rank job on one GPU.  Rank 1's gradient of its own shard is computed first by a
    second model; rank 0 then runs its step with the exchange attached, the callback averaging every
    bucket in place with rank 1's range on the communication stream.  The result must equal (a) a
    single replica that processes both shards with gradient accumulation (the same mean gradient) and
    (b) the oracle on the whole batch, and the callback must have seen every bucket once, in order,
    during the last micro-step only."""
    import oracle
    from gpu_util import dev, host, rel_l2
    cfg = si.make_config(n_layers=2, d_model=64, n_heads=1, seq_len=96, vocab_size=300, padded_vocab_size=320,
                         batch=2, tokens="zipf")                 # head_dim 64: the tcgen05 attention path
    B = 2
    params = si.init_params(cfg, 31, jitter=0.02)
    tok, tgt = si.tokens_for(cfg, 400, 2 * B * n_micro)           # rows [0, B n_micro): rank 0; the rest: rank 1
    half = B * n_micro
    opt = b.make_adamw(**si.ADAMW)

    def model():
        m = b.Model(cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["seq_len"], cfg["vocab_size"],
                    cfg["padded_vocab_size"], B)
        m.load_params(params)
        return m

    def local_grad(m, rows_tok, rows_tgt):
        for i in range(n_micro):
            sl = slice(i * B, (i + 1) * B)
            m.micro_step(dev(rows_tok[sl]), dev(rows_tgt[sl]), i, n_micro)

    r1 = model()
    local_grad(r1, tok[half:], tgt[half:])
    g1 = r1.arena(1).clone()
    torch.cuda.synchronize()

    r0 = model()
    comm = torch.cuda.Stream()
    seen = []

    def allreduce(buf, bucket):
        off = (buf.data_ptr() - r0.arena(1).data_ptr()) // 4
        seen.append((bucket, off, buf.numel(), b.bt_get_step(r0.h)))
        buf.add_(g1[off:off + buf.numel()]).mul_(0.5)           # what an averaging all-reduce leaves on every rank

    r0.ddp_attach(allreduce, comm, bucket_cap_bytes=64 * 1024)
    local_grad(r0, tok[:half], tgt[:half])
    plan = b.DdpPlan(r0.cfg, 64 * 1024)
    assert [s[0] for s in seen] == list(range(plan.n_buckets)) and plan.n_buckets > 3
    assert [(s[1], s[2]) for s in seen] == [plan.bucket(k)[:2] for k in range(plan.n_buckets)]
    gn0 = r0.adamw_step(opt)

    ref = model()                                                 # one replica, both shards, 2 n_micro micro-steps
    for i in range(2 * n_micro):                                  # every micro-batch weighs 1 / (2 n_micro)
        sl = slice(i * B, (i + 1) * B)
        ref.micro_step(dev(tok[sl]), dev(tgt[sl]), i, 2 * n_micro)
    assert rel_l2(host(r0.arena(1)), host(ref.arena(1))) < 1e-6
    gn_ref = ref.adamw_step(opt)
    assert abs(gn0 - gn_ref) < 1e-5 * gn_ref

    om = oracle.Model(cfg)
    om.set_params(params)
    om.loss_and_grad(tok, tgt, chunk=B)
    for name in om.names():
        if name.endswith("attn.qkv.b"):
            continue                                              # its key third is mathematically zero
        assert rel_l2(host(r0.tensor(name, 1)), om.get(name, 1)) < 1e-3, name

    # a second step: the exchange runs again (events and gate are reusable), nothing runs on other micro-steps
    seen.clear()
    local_grad(r0, tok[:half], tgt[:half])
    assert [s[0] for s in seen] == list(range(plan.n_buckets))
    r0.ddp_detach()
    seen.clear()
    r0.train_step(dev(tok[:B]), dev(tgt[:B]), opt)
    assert seen == []
    for m in (r0, r1, ref):
        m.close()
    plan.close()
