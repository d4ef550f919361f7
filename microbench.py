"""Kernel-level micro-benchmarks of the rollout library, one JSON line per case.

    python microbench.py accept   # verification step at a paper-like commit length
    python microbench.py probs    # probability pipeline on 4096 rows
    python microbench.py gemm     # decoder GEMM shapes of a workload, each timed alone
    python microbench.py gemm_tiles  # the same shapes with every tile shape forced, over --row-list
    python microbench.py gemm_floor  # cost of a small GEMM launch with and without the host's launch rate in it
    python microbench.py bikl     # bidirectional-KL reduction (Eq. 3) on 4096 row pairs
    python microbench.py score    # teacher/student scoring of a batch of trajectories (Eq. 3)
    python microbench.py attention  # ragged attention at fixed context lengths (--workload L|XL, --contexts a,b,..)

The rollouts of bench.py run random-weight models whose acceptance pattern is not the paper's; `accept` feeds
the verification kernels synthetic (p, q) pairs instead: targets p = softmax(l), proposals q = softmax(l + sigma *
noise), drafts drawn from q, sigma tuned so that the mean number of committed tokens per image matches the
paper's probabilistic mode (2.3 tokens per forward, Table 10), at the L workload's sizes (batch 128, guidance,
window 32, V = 16384, top-k 1000).  Inputs are made with torch on the GPU; every timed step runs in the library.
Times are CUDA events around single calls (each call ends with a stream synchronise, so a launch gap of a few
microseconds is inside the figure); bandwidths divide the algorithmic bytes by that time.  `gemm` times bursts of
20 back-to-back launches instead (the way the decoder issues them).
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))


def _median_us(torch, fn, reset=None, reps=9, warm=3):
    ts = []
    for i in range(warm + reps):
        if reset is not None:
            reset()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        if i >= warm:
            ts.append(e0.elapsed_time(e1) * 1e3)
    return float(np.median(ts))


def _small_context(binding, synth, vocab, max_batch, max_window):
    """A context whose model is irrelevant here (one thin layer): the stand-alone entry points only use its
    stream, limits and scratch."""
    sh = synth.ModelShape(1, 64, 1, 64, vocab, 4, 4, 3, "bf16")
    return binding.Context(sh, synth.make_weights(sh, 3, target_entropy=None), max_batch, max_window)


def verify_inputs(torch, B, W, T, V, branches, cfg_scale, top_k, sigma, seed, sampled_frac=0.85, logit_std=2.5):
    """Device tensors of one verification step: ragged cursors, a previous round that committed 1..3 tokens,
    sampled drafts (with their proposal rows in q) and history drafts (point-mass proposals).  The proposals
    are the guided, top-k filtered targets perturbed by sigma * noise in the logits."""
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    base = torch.randn(B, W, V, device="cuda", generator=g) * logit_std
    if branches == 2:
        unc = base * 0.5 + torch.randn(B, W, V, device="cuda", generator=g)
        logits = torch.stack([base, unc]).contiguous()
        guided = unc + cfg_scale * (base - unc)
    else:
        logits = base[None].contiguous()
        guided = base
    cursor = torch.randint(0, T - W, (B,), device="cuda", generator=g, dtype=torch.int32)
    back = torch.randint(1, 4, (B,), device="cuda", generator=g, dtype=torch.int32)
    qbase = torch.clamp(cursor - back, min=0)
    seq = torch.randint(0, V, (B, T + 1), device="cuda", generator=g, dtype=torch.int32)
    delta = torch.ones(B, T + 1, device="cuda", dtype=torch.uint8)
    q = torch.empty(B, W, V, device="cuda")
    cur, qb = cursor.tolist(), qbase.tolist()
    i = torch.arange(0, W - 1, device="cuda")
    for b in range(B):
        shift = cur[b] - qb[b]
        noisy = guided[b] + sigma * torch.randn(W, V, device="cuda", generator=g)
        if 0 < top_k < V:
            kth = torch.topk(noisy, top_k, dim=-1).values[:, -1:]
            noisy = torch.where(noisy >= kth, noisy, torch.full_like(noisy, float("-inf")))
        # the proposal of the draft verified at window position i sits in row i + shift of the previous
        # round's probabilities
        q[b] = torch.softmax(torch.roll(noisy, shift, dims=0), dim=-1)
        draws = torch.multinomial(q[b], 1, generator=g).squeeze(1).to(torch.int32)  # one draw per proposal row
        qi = i + shift
        ok = (qi < W) & (torch.rand(W - 1, device="cuda", generator=g) < sampled_frac)
        t = cur[b] + 1 + i[ok]
        seq[b, t] = draws[qi[ok]]
        delta[b, t] = 0
    return logits, q, cursor, seq, delta, qbase


def bench_accept(args):
    import torch
    from paper_2608_18183_b200 import binding, synth
    B, W, T, V, branches, top_k = args.batch or 128, args.window, 256, args.vocab, 2 if args.cfg_scale != 1.0 else 1, args.top_k
    ctx = _small_context(binding, synth, V, B, W)

    def run_case(sigma, timed):
        logits, q, cursor, seq, delta, qbase = verify_inputs(torch, B, W, T, V, branches, args.cfg_scale, top_k, sigma, args.seed)
        p_out = torch.zeros(B, W, V, device="cuda")
        m_out = torch.zeros(B, dtype=torch.int32, device="cuda")
        desc = binding.hbsjd_verify_desc(B, W, T, V, branches, 16, 0, top_k, args.cfg_scale, 1.0, args.seed, 7, 0)
        st = [cursor.clone(), seq.clone(), delta.clone(), qbase.clone()]

        def reset():
            st[0].copy_(cursor); st[1].copy_(seq); st[2].copy_(delta); st[3].copy_(qbase)

        def call():
            ctx.hbsjd_verify(desc, logits, q, p_out, st[0], st[1], st[2], st[3], m_out)

        reset()
        call()
        m = m_out.float().mean().item()
        us = _median_us(torch, call, reset) if timed else None
        return m, us, (m_out < W).float().mean().item()

    # sigma by bisection on the mean commit length (monotone decreasing in sigma)
    lo, hi = 0.0, 8.0
    for _ in range(10):
        mid = 0.5 * (lo + hi)
        m, _, _ = run_case(mid, False)
        if m > args.target_commit:
            lo = mid
        else:
            hi = mid
    sigma = 0.5 * (lo + hi)
    m, us, rej = run_case(sigma, True)
    rows = B * W
    # logits of every branch read + probabilities written; proposal rows are read only at a reject (one per
    # image) and for the accept ratio (single elements), so they are left out of the algorithmic figure
    alg = rows * V * 4.0 * (branches + 1)
    print(json.dumps({"case": "accept", "batch": B, "window": W, "V": V, "branches": branches, "top_k": top_k,
                      "sigma": round(sigma, 4), "mean_committed_per_image": round(m, 3),
                      "images_with_reject": round(rej, 3), "us": round(us, 1),
                      "algorithmic_bytes": alg, "GB_s": round(alg / us / 1e3, 1)}))
    ctx.hbsjd_destroy()


def bench_probs(args):
    import torch
    from paper_2608_18183_b200 import binding, synth
    V, rows = args.vocab, args.rows
    ctx = _small_context(binding, synth, V, 2, 4)
    g = torch.Generator(device="cuda")
    g.manual_seed(args.seed)
    lc = torch.randn(rows, V, device="cuda", generator=g) * 3.5
    lu = torch.randn(rows, V, device="cuda", generator=g) * 3.5
    out = torch.empty_like(lc)
    for name, (u, s, tau, k) in {"plain": (None, 1.0, 1.0, 0), "guidance": (lu, 4.0, 1.0, 0),
                                 "top_k": (None, 1.0, 1.0, 1000), "guidance+top_k": (lu, 4.0, 1.0, 1000),
                                 "guidance+top_k+temperature": (lu, 4.0, 0.7, 1000)}.items():
        def call():
            ctx._check(ctx.lib.hbsjd_probs(ctx.h, lc.data_ptr(), None if u is None else u.data_ptr(), rows, s, tau, k,
                                           out.data_ptr()), "hbsjd_probs")
        us = _median_us(torch, call)
        alg = rows * V * 4.0 * ((2 if u is not None else 1) + 1)
        print(json.dumps({"case": "probs", "variant": name, "rows": rows, "V": V, "us": round(us, 1),
                          "algorithmic_bytes": alg, "GB_s": round(alg / us / 1e3, 1)}))
    ctx.hbsjd_destroy()


def bench_gemm(args):
    import torch
    from paper_2608_18183_b200 import binding, synth
    w = synth.WORKLOADS[args.workload]
    s = w.shape
    D, F, V = s.dim, s.ffn_hidden, s.vocab
    M = args.rows or w.batch * (2 if w.cfg_scale != 1.0 else 1) * w.window
    # a context of the workload's width (one thin layer): the residual-update form writes into its buffers
    sh = synth.ModelShape(1, D, s.n_heads, 64, 64, 4, 4, 3, "bf16")
    ctx = binding.Context(sh, synth.make_weights(sh, 3, target_entropy=None), (M + 63) // 64, 32)
    g = torch.Generator(device="cuda")
    g.manual_seed(args.seed)
    for name, N, K, acc in [("qkv", 3 * D, D, 0), ("attention out (+=)", D, D, 1),
                            ("attention out (+=, bf16 copy, sums of squares)", D, D, 2), ("gate|up", 2 * F, D, 0),
                            ("down (+=)", D, F, 1), ("down (+=, bf16 copy, sums of squares)", D, F, 2),
                            ("head", V, D, 0)]:
        if args.only and not name.startswith(args.only):
            continue
        A = torch.randn(M, K, device="cuda", generator=g).bfloat16()
        Wt = (torch.randn(N, K, device="cuda", generator=g) * 0.05).bfloat16()
        Cm = torch.zeros(M, N, device="cuda")
        def burst():
            ctx.hbsjd_debug_gemm(A, Wt, Cm, accumulate=acc, reps=20)  # 20 launches back to back, one sync
        us = _median_us(torch, burst, reps=5, warm=2) / 20
        print(json.dumps({"case": "gemm", "name": name, "M": M, "N": N, "K": K, "accumulate": acc,
                          "us": round(us, 1), "TFLOP_s": round(2.0 * M * N * K / us / 1e6, 1)}))
    ctx.hbsjd_destroy()


def _gemm_context(binding, synth, s, rows):
    sh = synth.ModelShape(1, s.dim, s.n_heads, 64, 64, 4, 4, 3, "bf16")
    return binding.Context(sh, synth.make_weights(sh, 3, target_entropy=None), (rows + 63) // 64, 32)


def bench_gemm_tiles(args):
    """Every tile shape of the GEMM kernel on the decoder's shapes, over a range of activation rows M."""
    import torch
    from paper_2608_18183_b200 import binding, synth
    s = synth.WORKLOADS[args.workload].shape
    D, F, V = s.dim, s.ffn_hidden, s.vocab
    ms = [int(x) for x in args.row_list.split(",")]
    ctx = _gemm_context(binding, synth, s, max(ms))
    g = torch.Generator(device="cuda")
    g.manual_seed(args.seed)
    for name, N, K, acc in [("qkv", 3 * D, D, 0), ("attention out (+=)", D, D, 1), ("gate|up", 2 * F, D, 0),
                            ("down (+=)", D, F, 1), ("head", V, D, 0)]:
        Wt = (torch.randn(N, K, device="cuda", generator=g) * 0.05).bfloat16()
        for M in ms:
            A = torch.randn(M, K, device="cuda", generator=g).bfloat16()
            Cm = torch.zeros(M, N, device="cuda")
            us = {}
            # 0: the library's choice; 512 / 640: 256 x 256 / 256 x 128 tiles on CTA pairs
            for tile in (0, 32, 64, 128, 256, 512, 640):
                if tile and N % (tile if tile < 512 else 768 - tile):
                    continue
                def burst():
                    ctx.hbsjd_debug_gemm(A, Wt, Cm, accumulate=acc, reps=20, tile=tile)
                us[str(tile)] = round(_median_us(torch, burst, reps=5, warm=2) / 20, 1)
            print(json.dumps({"case": "gemm_tiles", "name": name, "M": M, "N": N, "K": K, "us_by_tile": us}))
    ctx.hbsjd_destroy()


def bench_gemm_floor(args):
    """What a GEMM launch costs however small it is: 800 launches queued behind a spin of about 10 ms, so that the
    host's launch rate is outside the figure (and the same without the spin, where it is inside)."""
    import time
    import torch
    from paper_2608_18183_b200 import binding, synth
    s = synth.WORKLOADS[args.workload].shape
    ctx = _gemm_context(binding, synth, s, 256)
    g = torch.Generator(device="cuda")
    g.manual_seed(args.seed)
    for M, N, K in ((256, s.dim, 64), (256, s.dim, s.dim), (256, 3 * s.dim, s.dim), (64, s.dim, s.ffn_hidden)):
        A = torch.randn(M, K, device="cuda", generator=g).bfloat16()
        Wt = (torch.randn(N, K, device="cuda", generator=g) * 0.05).bfloat16()
        Cm = torch.zeros(M, N, device="cuda")
        ctx.hbsjd_debug_gemm(A, Wt, Cm, reps=50)
        out = {}
        for label, spin in (("host_in_figure", 0), ("queued_behind_spin", 20_000_000)):
            torch.cuda.synchronize()
            e1, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if spin:
                torch.cuda._sleep(spin)
            e1.record()
            ctx.hbsjd_debug_gemm(A, Wt, Cm, reps=800)
            e2.record()
            torch.cuda.synchronize()
            out[label] = round(e1.elapsed_time(e2) * 1e3 / 800, 2)
        print(json.dumps({"case": "gemm_floor", "M": M, "N": N, "K": K, "us_per_launch": out}))
    ctx.hbsjd_destroy()


def bench_bikl(args):
    import torch
    from paper_2608_18183_b200 import binding, synth
    V, rows = args.vocab, args.rows
    ctx = _small_context(binding, synth, V, 2, 4)
    g = torch.Generator(device="cuda")
    g.manual_seed(args.seed)
    ls = torch.randn(rows, V, device="cuda", generator=g) * 3.0
    lt = 0.6 * ls + torch.randn(rows, V, device="cuda", generator=g) * 2.0
    out = torch.empty(rows, device="cuda")

    def call():
        ctx._check(ctx.lib.hbsjd_bikl(ctx.h, ls.data_ptr(), lt.data_ptr(), rows, out.data_ptr()), "hbsjd_bikl")
    us = _median_us(torch, call)
    alg = rows * V * 4.0 * 2
    print(json.dumps({"case": "bikl", "rows": rows, "V": V, "us": round(us, 1), "algorithmic_bytes": alg,
                      "GB_s": round(alg / us / 1e3, 1)}))
    ctx.hbsjd_destroy()


def teacher_shape(synth, s):
    """The scoring benchmark's teacher: the XL decoder's width and depth on the student's grid and vocabulary."""
    x = synth.WORKLOADS["XL"].shape
    return synth.ModelShape(x.n_layers, x.dim, x.n_heads, x.ffn_hidden, s.vocab, s.grid_h, s.grid_w, s.n_classes,
                            s.dtype)


def bench_score(args):
    import torch
    from paper_2608_18183_b200 import binding, synth
    w = synth.WORKLOADS[args.workload]
    s = w.shape
    tsh = teacher_shape(synth, s)
    B = args.batch or w.batch
    stu = binding.Context(s, synth.make_weights(s, w.weight_seed), B, w.window)
    tea = binding.Context(tsh, synth.make_weights(tsh, 77, target_entropy=None), B, w.window)
    _, k, lab = synth.make_inputs(w, batch=B)
    rng = np.random.default_rng(args.seed)
    toks = torch.from_numpy(rng.integers(0, s.vocab, size=(B, s.T)).astype(np.int32)).cuda()
    kd, ld = torch.from_numpy(k).cuda(), torch.from_numpy(lab).cuda()

    def call():
        stu.hbsjd_score(tea, toks, kd, ld)
    ms = _median_us(torch, call, reps=5, warm=2) / 1e3
    for c in (stu, tea):
        c.lib.hbsjd_profile(c.h, 1)
    call()
    prof = {}
    for name, c in (("student", stu), ("teacher", tea)):
        pr = binding.hbsjd_kernel_profile()
        c.lib.hbsjd_profile_read(c.h, C.byref(pr))
        c.lib.hbsjd_profile(c.h, 0)
        prof[name] = {"gemm_ms": round(pr.ms[0], 2), "gemm_TFLOP_s": round(pr.work[0] / max(pr.ms[0], 1e-9) / 1e9, 1),
                      "attention_ms": round(pr.ms[1], 2),
                      "attention_GB_s": round(pr.work[1] / max(pr.ms[1], 1e-9) / 1e6, 1),
                      "vocab_reduce_ms": round(pr.ms[2], 2),
                      "vocab_reduce_GB_s": round(pr.work[2] / max(pr.ms[2], 1e-9) / 1e6, 1)}
    flops = 0.0
    for sh in (s, tsh):
        D, F, V = sh.dim, sh.ffn_hidden, sh.vocab
        flops += 2.0 * (sh.n_layers * (4 * D * D + 3 * D * F) + D * V) * B * s.T
    print(json.dumps({"case": "score", "student": args.workload, "teacher": "XL width/depth on the student's grid",
                      "batch": B, "T": s.T, "chunk": min(64, 2 * w.window, s.T), "ms": round(ms, 2),
                      "positions_per_s": round(B * s.T / ms * 1e3), "gemm_flops": flops,
                      "gemm_TFLOP_s_over_the_call": round(flops / ms / 1e9, 1), "profiled_pass": prof}))
    stu.hbsjd_destroy()
    tea.hbsjd_destroy()


def bench_attention(args):
    """The ragged attention kernel at fixed context lengths: every image of the workload's batch gets the same
    prefix, the prefix is pre-filled, then the verifier forward runs once under the library's per-class event
    timing.  Bytes: K and V rows 0..c+n-1 read per physical row, q read and output written per input."""
    import torch
    from paper_2608_18183_b200 import binding, synth
    w = synth.WORKLOADS[args.workload]
    s = w.shape
    B = args.batch or w.batch
    ctx = binding.Context(s, synth.make_weights(s, w.weight_seed), B, w.window)
    toks, _, lab = synth.make_inputs(w, batch=B)
    floor_us = ctx.hbsjd_profile_launch_floor(200)
    for c in [int(x) for x in args.contexts.split(",")]:
        k = np.full(B, min(c, s.T - 1), dtype=np.int32)
        p = binding.make_params(w.window, w.history_offset, w.cfg_scale, w.temperature, w.top_k, binding.VERIFY_PROB,
                                binding.EXEC_FULL, 0, 1, 0)
        ctx.hbsjd_rollout(torch.from_numpy(toks).cuda(), torch.from_numpy(k).cuda(), torch.from_numpy(lab).cuda(), p)
        ctx.hbsjd_debug_forward(s.n_layers - 1, 0)  # warm
        ctx.hbsjd_profile(True)
        for _ in range(3):
            ctx.hbsjd_debug_forward(s.n_layers - 1, 0)
        pr = ctx.hbsjd_profile_read()["attention"]
        ctx.hbsjd_profile(False)
        us = pr["ms"] * 1e3 / pr["launches"]
        alg = pr["work"] / pr["launches"]
        print(json.dumps({"case": "attention", "workload": args.workload, "batch": B, "window": w.window,
                          "context": int(k[0]), "us_per_launch": round(us, 2), "launches": pr["launches"],
                          "algorithmic_bytes": alg, "GB_s": round(alg / us / 1e3, 1),
                          "GB_s_net_of_launch_floor": round(alg / (us - floor_us) / 1e3, 1),
                          "event_pair_launch_floor_us": round(floor_us, 2)}))
    ctx.hbsjd_destroy()


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("case", choices=["accept", "probs", "gemm", "gemm_tiles", "gemm_floor", "bikl", "score",
                                     "attention"])
    ap.add_argument("--contexts", default="0,32,64,128,192,223")
    ap.add_argument("--workload", default="L")
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--window", type=int, default=32)
    ap.add_argument("--vocab", type=int, default=16384)
    ap.add_argument("--top-k", type=int, default=1000)
    ap.add_argument("--cfg-scale", type=float, default=4.0)
    ap.add_argument("--target-commit", type=float, default=2.3)
    ap.add_argument("--rows", type=int, default=0)
    ap.add_argument("--row-list", default="512,2048,4096,5120,8192", help="gemm_tiles: activation row counts")
    ap.add_argument("--only", default="", help="gemm: only the shapes whose name starts with this")
    ap.add_argument("--seed", type=int, default=1)
    args = ap.parse_args(argv)
    if args.case in ("probs", "bikl") and not args.rows:
        args.rows = 4096
    {"accept": bench_accept, "probs": bench_probs, "gemm": bench_gemm, "gemm_tiles": bench_gemm_tiles, "gemm_floor": bench_gemm_floor, "bikl": bench_bikl,
     "score": bench_score, "attention": bench_attention}[args.case](args)


if __name__ == "__main__":
    sys.exit(main())
