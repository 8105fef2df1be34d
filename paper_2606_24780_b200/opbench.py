"""Per-kernel micro-benchmarks through the per-op C-ABI entry points.

Default workload: one GPT-2-small decoder block in isolation (d_model 768, 12 heads, MLP
3072, batch 8 x 1024 tokens), forward and backward, plus the LM-head GEMMs, the fused
softmax cross-entropy and AdamW at GPT-2 124M sizes.  Methodology (the paper's appendix on
benchmarking): warm-up iterations, then timed runs with the L2 flushed (a buffer larger than
L2 is overwritten) between iterations, CUDA events on the launching stream, median reported.

    python -m paper_2606_24780_b200.opbench [--only NAME[,NAME]] [--iters 100] [--warmup 25]
                                            [--batch 8] [--seq 1024] [--no-flush] [--json out.json]

Each line: kernel, median microseconds, achieved TFLOP/s (model FLOPs) for the contractions or
GB/s (algorithmic bytes) for the memory-bound kernels.
"""
from __future__ import annotations

import argparse
import json
import sys

import torch

from . import binding as b


def _rand(*shape, std=1.0):
    return torch.randn(*shape, device="cuda", dtype=torch.float32) * std


def _split(x):
    s = torch.empty((2,) + tuple(x.shape), device="cuda", dtype=torch.float32)
    b.bt_op_split(x, x.numel(), s)
    return s


def build_cases(B, T, C, H, Vp, n_params):
    N, F = B * T, 4 * C
    cases = {}
    gsb = b.bt_op_gemm_split_scratch_bytes()
    gscratch = torch.empty(gsb + 512, dtype=torch.uint8, device="cuda")
    gscratch = gscratch[(-gscratch.data_ptr()) % 256:]

    def gemm_case(name, layout, M, Nn, K, bias=False, residual=False):
        a_shape = (K, M) if layout == 2 else (M, K)
        b_shape = (Nn, K) if layout == 0 else (K, Nn)
        A, Bm = _split(_rand(*a_shape)), _split(_rand(*b_shape, std=0.02))
        D = torch.empty(M, Nn, device="cuda")
        bi = _rand(Nn) if bias else None
        res = _rand(M, Nn) if residual else None

        def run():
            b.bt_op_gemm_split(layout, M, Nn, K, A, Bm, D, bi, res, gscratch, gsb)
        cases[name] = dict(run=run, flops=2.0 * M * Nn * K, bytes=8.0 * (M * K + Nn * K) + 4.0 * M * Nn,
                           bound="tensor", keep=(A, Bm, D, bi, res), check=lambda: b.bt_op_gemm_check(gscratch))

    def fused_gelu_cases():
        # the MLP up-projection with GELU in its epilogue (planes of GELU(h), GELU'(h) kept for the
        # backward) and the down-projection's input gradient with the GELU backward in its epilogue
        x_s, wt_s = _split(_rand(N, C)), _split(_rand(C, F, std=0.02))
        hD, g_s, bi = torch.empty(N, F, device="cuda"), torch.empty(2, N, F, device="cuda"), _rand(F)
        cases["gemm_fwd_fc_gelu"] = dict(
            run=lambda: b.bt_op_gemm_split_act(1, N, F, C, x_s, wt_s, hD, g_s, 3, bi, None, gscratch, gsb),
            flops=2.0 * N * F * C, bytes=8.0 * (N * C + F * C) + 12.0 * N * F, bound="tensor",
            keep=(x_s, wt_s, hD, g_s, bi), check=lambda: b.bt_op_gemm_check(gscratch))
        dy_s, w_s = _split(_rand(N, C)), _split(_rand(C, F, std=0.02))
        gp, dh_s, cs = _rand(N, F), torch.empty(2, N, F, device="cuda"), torch.empty(F, device="cuda")
        nb = b.bt_op_gemm_gelu_bwd_scratch_bytes(N, F)
        sc = torch.empty(nb + 512, dtype=torch.uint8, device="cuda")
        sc = sc[(-sc.data_ptr()) % 256:]
        cases["gemm_nn_dmlpproj_gelu_bwd"] = dict(
            run=lambda: b.bt_op_gemm_gelu_bwd(N, F, C, dy_s, w_s, gp, 2, dh_s, cs, sc, nb),
            flops=2.0 * N * F * C, bytes=8.0 * (N * C + F * C) + 12.0 * N * F, bound="tensor",
            keep=(dy_s, w_s, gp, dh_s, cs, sc), check=lambda: b.bt_op_gemm_check(sc))

    fused_gelu_cases()
    # forward GEMMs of the block as the training step runs them (weight read from its transposed
    # copy: layout NN, bias / residual in the epilogue), the same products in the NT layout, the two
    # backward layouts of each, and the LM head
    gemm_case("gemm_fwd_qkv", 1, N, 3 * C, C, bias=True)
    gemm_case("gemm_fwd_attnproj", 1, N, C, C, bias=True, residual=True)
    gemm_case("gemm_fwd_fc", 1, N, F, C, bias=True)
    gemm_case("gemm_fwd_mlpproj", 1, N, C, F, bias=True, residual=True)
    gemm_case("gemm_nt_qkv", 0, N, 3 * C, C, bias=True)
    gemm_case("gemm_nt_attnproj", 0, N, C, C, bias=True, residual=True)
    gemm_case("gemm_nt_fc", 0, N, F, C, bias=True)
    gemm_case("gemm_nt_mlpproj", 0, N, C, F, bias=True, residual=True)
    gemm_case("gemm_nn_dqkv", 1, N, C, 3 * C)
    gemm_case("gemm_nn_dattnproj", 1, N, C, C)
    gemm_case("gemm_nn_dfc", 1, N, C, F)
    gemm_case("gemm_nn_dmlpproj", 1, N, F, C)
    gemm_case("gemm_tn_wqkv", 2, 3 * C, C, N)
    gemm_case("gemm_tn_wattnproj", 2, C, C, N)
    gemm_case("gemm_tn_wfc", 2, F, C, N)
    gemm_case("gemm_tn_wmlpproj", 2, C, F, N)
    if Vp:
        gemm_case("gemm_fwd_lmhead", 1, N, Vp, C)
        gemm_case("gemm_nt_lmhead", 0, N, Vp, C)
        gemm_case("gemm_nn_dlmhead", 1, N, C, Vp)
        gemm_case("gemm_tn_wlmhead", 2, Vp, C, N)

    # LayerNorm
    x, g, be = _rand(N, C), _rand(C) * 0.1 + 1.0, _rand(C) * 0.1
    ys, mean, rstd = torch.empty(2, N, C, device="cuda"), torch.empty(N, device="cuda"), torch.empty(N, device="cuda")
    cases["layernorm_fwd"] = dict(run=lambda: b.bt_op_layernorm_fwd(x, g, be, N, C, None, ys, mean, rstd),
                                  bytes=12.0 * N * C, bound="hbm", keep=(x, g, be, ys, mean, rstd))
    b.bt_op_layernorm_fwd(x, g, be, N, C, None, ys, mean, rstd)
    dy, dres = _rand(N, C, std=1e-2), _rand(N, C, std=1e-2)
    dxs, dg, db = torch.empty(2, N, C, device="cuda"), torch.empty(C, device="cuda"), torch.empty(C, device="cuda")
    lnb = b.bt_op_layernorm_bwd_scratch_bytes(N, C)
    lscr = torch.empty(lnb + 256, dtype=torch.uint8, device="cuda")
    lscr = lscr[(-lscr.data_ptr()) % 256:]
    cases["layernorm_bwd"] = dict(
        run=lambda: b.bt_op_layernorm_bwd(dy, x, g, mean, rstd, dres, N, C, dres, dxs, dg, db, lscr, lnb),
        bytes=24.0 * N * C, bound="hbm", keep=(dy, dres, dxs, dg, db, lscr))

    dcs = torch.empty(C, device="cuda")
    cases["layernorm_bwd_colsum"] = dict(          # the variant the training step runs (projection bias sums fused)
        run=lambda: b.bt_op_layernorm_bwd_colsum(dy, x, g, mean, rstd, dres, N, C, dres, dxs, dg, db, dcs, lscr, lnb),
        bytes=24.0 * N * C, bound="hbm", keep=(dcs,))

    # embedding gather and its scatter-add backward on Zipf ids (the 124M vocabulary)
    if Vp:
        import seeded_inputs as si
        V = 50257 if Vp == 50304 else Vp
        tok = torch.as_tensor(si.zipf_tokens(7, B, T, V)[0].ravel()).cuda()
        wte, wpe = _rand(Vp, C, std=0.02), _rand(T, C, std=0.02)
        x0, dx0 = torch.empty(N, C, device="cuda"), _rand(N, C, std=1e-2)
        dwte, dwpe = torch.zeros(Vp, C, device="cuda"), torch.empty(T, C, device="cuda")
        esb = b.bt_op_embedding_bwd_scratch_bytes(N, C, Vp)
        escr = torch.empty(esb + 256, dtype=torch.uint8, device="cuda")
        escr = escr[(-escr.data_ptr()) % 256:]
        cases["embedding_fwd"] = dict(run=lambda: b.bt_op_embedding_fwd(tok, wte, wpe, N, T, C, Vp, x0),
                                      bytes=12.0 * N * C, bound="hbm", keep=(tok, wte, wpe, x0))
        cases["embedding_bwd"] = dict(
            run=lambda: b.bt_op_embedding_bwd(tok, dx0, N, T, C, Vp, dwte, dwpe, escr, esb),
            bytes=8.0 * N * C, bound="hbm", keep=(dx0, dwte, dwpe, escr))

    # GELU
    h, dgl = _rand(N, F), _rand(N, F, std=1e-2)
    gs, dhs = torch.empty(2, N, F, device="cuda"), torch.empty(2, N, F, device="cuda")
    cases["gelu_fwd"] = dict(run=lambda: b.bt_op_gelu_fwd(h, N * F, 0, None, gs), bytes=12.0 * N * F, bound="hbm",
                             keep=(h, gs))
    cases["gelu_bwd"] = dict(run=lambda: b.bt_op_gelu_bwd(h, dgl, N * F, 0, None, dhs), bytes=16.0 * N * F,
                             bound="hbm", keep=(dgl, dhs))

    gcb = b.bt_op_colsum_scratch_bytes(N, F)
    gscr, gcs = torch.empty(gcb // 4, device="cuda"), torch.empty(F, device="cuda")
    cases["gelu_bwd_colsum"] = dict(
        run=lambda: b.bt_op_gelu_bwd_colsum(h, dgl, N, F, 0, None, dhs, gcs, gscr, gcb), bytes=16.0 * N * F,
        bound="hbm", keep=(gscr, gcs))

    # attention
    qkv, d_o = _rand(N, 3 * C), _rand(N, C, std=1e-2)
    o, os_, lse = torch.empty(N, C, device="cuda"), torch.empty(2, N, C, device="cuda"), torch.empty(B, H, T, device="cuda")
    dqs = torch.empty(2, N, 3 * C, device="cuda")
    dv = torch.empty(B * H * T, device="cuda")
    afl = 4.0 * B * H * (C // H) * (T * (T + 1) / 2.0)
    cases["attention_fwd"] = dict(run=lambda: b.bt_op_attention_fwd(qkv, B, T, C, H, o, os_, lse), flops=afl,
                                  bytes=24.0 * N * C, bound="tensor", keep=(qkv, o, os_, lse))
    b.bt_op_attention_fwd(qkv, B, T, C, H, o, os_, lse)
    if C // H in (64, 128):
        qkv_s = _split(qkv)
        cases["attention_fwd_tcgen05"] = dict(
            run=lambda: b.bt_op_attention_fwd(None, B, T, C, H, None, os_, lse, qkv_split=qkv_s), flops=afl,
            bytes=32.0 * N * C, bound="tensor", keep=(qkv_s,))
    if C // H in (64, 128):
        do_s, dqs2 = _split(d_o), torch.empty(2, N, 3 * C, device="cuda")
        cases["attention_bwd_tcgen05"] = dict(
            run=lambda: b.bt_op_attention_bwd(None, o, lse, None, B, T, C, H, None, dqs2, dv, dv.numel() * 4,
                                              qkv_split=qkv_s, d_o_split=do_s),
            flops=2.5 * afl, bytes=64.0 * N * C, bound="tensor", keep=(do_s, dqs2))
    cases["attention_bwd"] = dict(
        run=lambda: b.bt_op_attention_bwd(qkv, o, lse, d_o, B, T, C, H, None, dqs, dv, dv.numel() * 4),
        flops=2.5 * afl, bytes=48.0 * N * C, bound="tensor", keep=(d_o, dqs, dv))

    # column sums (bias gradients)
    csb = b.bt_op_colsum_scratch_bytes(N, F)
    cscr = torch.empty(csb + 256, dtype=torch.uint8, device="cuda")
    cscr = cscr[(-cscr.data_ptr()) % 256:]
    cout = torch.empty(F, device="cuda")
    cases["colsum_fc"] = dict(run=lambda: b.bt_op_colsum(h, N, F, cout, cscr, csb), bytes=4.0 * N * F, bound="hbm",
                              keep=(cout, cscr))

    if Vp:
        rows = min(N, 2048)      # 2048 x 50304 logits = 412 MB: several times L2, still a small case
        z = _rand(rows, Vp, std=2.0)
        tg = torch.randint(0, Vp, (rows,), device="cuda", dtype=torch.int32)
        losses, lm = torch.empty(rows, device="cuda"), torch.empty(1, device="cuda")
        dls = torch.empty(2, rows, Vp, device="cuda")
        cases["softmax_xent"] = dict(
            run=lambda: b.bt_op_softmax_xent(z, tg, rows, Vp, 1.0 / rows, losses, lm, None, dls),
            bytes=12.0 * rows * Vp, bound="hbm", keep=(z, tg, losses, lm, dls))
    if n_params:
        shapes = [n_params // 8] * 8
        ps = [_rand(s, std=0.02) for s in shapes]
        gr = [_rand(s, std=1e-3) for s in shapes]
        ms = [torch.zeros(s, device="cuda") for s in shapes]
        vs = [torch.zeros(s, device="cuda") for s in shapes]
        opt = b.make_adamw()
        cases["adamw"] = dict(run=lambda: b.bt_op_adamw_multi(ps, gr, ms, vs, [1] * 8, opt, 3),
                              bytes=28.0 * sum(shapes), bound="hbm", keep=(ps, gr, ms, vs))
        gnb = b.bt_op_grad_norm_scratch_bytes(shapes[0])
        nscr = torch.empty(gnb + 256, dtype=torch.uint8, device="cuda")
        nscr = nscr[(-nscr.data_ptr()) % 256:]
        out2 = torch.empty(2, device="cuda")
        cases["grad_norm"] = dict(run=lambda: b.bt_op_grad_norm(gr[0], shapes[0], 1.0, out2, nscr, gnb),
                                  bytes=4.0 * shapes[0], bound="hbm", keep=(nscr, out2))
    if n_params:
        # the optimizer and the weight split as the training step runs them (flat arenas of a model):
        # one GPT-2-small layer plus the 50304-row embedding, 46 M parameters, batch 1 x 64 tokens so
        # that the activations stay small
        mdl = b.Model(1, C, H, 64, 50257 if Vp == 50304 else Vp, Vp, 1)
        mdl.init(7)
        opt2 = b.make_adamw()
        tk = torch.zeros(1, 64, dtype=torch.int32, device="cuda")
        mdl.train_step(tk, tk, opt2)
        P = sum(-(-n // 1024) * 1024 for _, n, _ in mdl.names)
        cases["model_adamw_step"] = dict(run=lambda: mdl.adamw_step(opt2, want_norm=False), bytes=(28.0 + 4.0) * P,
                                         bound="hbm", keep=(mdl, tk))
        cases["model_forward_64_tokens"] = dict(run=lambda: mdl.forward(tk, tk, want_loss=False), bytes=20.0 * P,
                                                bound="hbm", keep=())
    return cases


def tf32_rate(sm_mhz=None):
    """The tensor pipe's measured dense TF32 rate (one SM): clocks per 128 x 256 x 8 MMA and MAC per clock."""
    lo, med, hi = b.bt_probe_tf32_mma_rate(torch.cuda.get_device_properties(0).multi_processor_count, 4000)
    return {"clocks_per_mma_128x256x8": med, "clocks_min_max": [lo, hi], "mac_per_clk_per_sm": 128 * 256 * 8 / med}


def issue_rates():
    """Clocks per MMA (M = 128, K = 8) by width, operand source and number of issuing threads."""
    out = {}
    for n, tmem in ((64, 0), (64, 1), (128, 0), (256, 0)):
        out[f"n{n}_{'tmem' if tmem else 'smem'}"] = [round(b.bt_probe_mma_issue_rate(n, tmem, k), 1) for k in (1, 2, 3)]
    return out


def hbm_rates(n_bytes=1 << 30, iters=10):
    """Measured HBM rates for the roofline denominators of the memory-bound kernels (harness-side torch
    kernels, best of `iters`): a copy (read + write bytes), a pure write (fill) and a pure read (sum).
    A kernel that writes more than it reads is bound by the write rate, not by the copy rate."""
    a = torch.empty(n_bytes // 4, device="cuda")
    c = torch.empty_like(a)
    a.fill_(1.0)
    out = {}
    for name, fn, moved in (("copy", lambda: c.copy_(a), 2 * n_bytes), ("write", lambda: c.fill_(2.0), n_bytes),
                            ("read", lambda: a.sum(), n_bytes)):
        best = 1e30
        for _ in range(iters):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        out[name + "_gbs"] = moved / best / 1e6
    return out


def time_case(case, iters, warmup, flush_buf):
    for _ in range(warmup):
        case["run"]()
    times = []
    for _ in range(iters):
        if flush_buf is not None:
            flush_buf.add_(1.0)          # rewrite a buffer larger than L2
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        case["run"]()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    if "check" in case:
        case["check"]()
    times.sort()
    return times[len(times) // 2] * 1e3  # microseconds


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--only", default="")
    ap.add_argument("--iters", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=25)
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--seq", type=int, default=1024)
    ap.add_argument("--d-model", type=int, default=768)
    ap.add_argument("--heads", type=int, default=12)
    ap.add_argument("--vocab", type=int, default=50304)
    ap.add_argument("--params", type=int, default=124_475_904)
    ap.add_argument("--no-flush", action="store_true")
    ap.add_argument("--json", default="")
    args = ap.parse_args(argv)
    torch.cuda.set_device(0)
    only = [s for s in args.only.split(",") if s]
    need_big = not only or any(s.startswith(("gemm_fwd_lm", "gemm_nt_lm", "gemm_nn_dlm", "gemm_tn_wlm", "softmax", "embedding"))
                               for s in only)
    need_params = not only or any(s.startswith(("adamw", "grad", "model_")) for s in only)
    cases = build_cases(args.batch, args.seq, args.d_model, args.heads, args.vocab if (need_big or need_params) else 0,
                        args.params if need_params else 0)
    flush = None if args.no_flush else torch.zeros(64 * 1024 * 1024, device="cuda")  # 256 MB > 126 MB L2
    results = {}
    if not only or "tf32_rate" in only:
        r = tf32_rate()
        sms = torch.cuda.get_device_properties(0).multi_processor_count
        r["tf32_tflops_at_1965_mhz"] = r["mac_per_clk_per_sm"] * 2 * sms * 1.965e9 / 1e12
        results["tf32_rate"] = r
        print(f"tf32_rate              {r['clocks_per_mma_128x256x8']:10.1f} clk per 128x256x8 MMA  "
              f"{r['mac_per_clk_per_sm']:7.0f} MAC/clk/SM  (x 2 x {sms} SMs x clock = dense TF32 peak; / 3 for 3xTF32)",
              flush=True)
    if not only or "issue_rates" in only:
        r = issue_rates()
        results["issue_rates"] = r
        print("issue_rates            clocks per 128 x N x 8 MMA with 1 / 2 / 3 issuing threads: " +
              ", ".join(f"{k} {v[0]} / {v[1]} / {v[2]}" for k, v in r.items()), flush=True)
    if not only or "hbm_rates" in only:
        r = hbm_rates()
        results["hbm_rates"] = r
        print(f"hbm_rates              copy {r['copy_gbs']:.0f} GB/s (read + write bytes), write only {r['write_gbs']:.0f} GB/s, "
              f"read only {r['read_gbs']:.0f} GB/s  (1 GiB each, best of 10)", flush=True)
    for name, case in cases.items():
        if only and name not in only:
            continue
        us = time_case(case, args.iters, args.warmup, flush)
        r = {"us": us, "bound": case["bound"]}
        if "flops" in case:
            r["tflops"] = case["flops"] / us / 1e6
        r["gbs"] = case["bytes"] / us / 1e3
        results[name] = r
        print(f"{name:22s} {us:10.1f} us  " + (f"{r['tflops']:8.1f} TFLOP/s  " if "tflops" in r else " " * 19) +
              f"{r['gbs']:8.0f} GB/s", flush=True)
    if args.json:
        with open(args.json, "w") as f:
            json.dump({"config": vars(args), "results": results}, f, indent=1)
    return 0


if __name__ == "__main__":
    sys.exit(main())
