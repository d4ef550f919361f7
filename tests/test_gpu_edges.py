"""Edge and degenerate cases of the rollout on the GPU: nothing to generate, one token to generate, one image,
one kept token, no-op guidance, temperature and history offsets the standard workloads do not use, the largest
vocabulary of the verification kernels."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2608_18183_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _ctx(w, **kw):
    return binding.Context(w.shape, G.weights_for(w), kw.get("max_batch", w.batch), kw.get("max_window", w.window))


def test_nothing_or_one_token_to_generate():
    w = synth.WORKLOADS["tiny"]
    T = w.shape.T
    toks, k, lab = synth.make_inputs(w)
    ctx = _ctx(w)
    # every image already complete: no round runs, the prefix is the result
    kk = np.full_like(k, T)
    out, st = ctx.hbsjd_rollout(G.dev(toks), G.dev(kk), G.dev(lab), G.gpu_params(w, 0))
    assert st["rounds"] == 0 and st["committed"] == 0 and st["image_forwards"] == 0
    np.testing.assert_array_equal(out.cpu().numpy(), toks)
    assert ctx.hbsjd_round() == 0                     # stepping a finished rollout is a no-op
    # one token left, a complete image and an empty prefix side by side: one round finishes the short ones
    kk = np.array([T - 1, T, 0, T - 1], dtype=np.int32)
    out, st = ctx.hbsjd_rollout(G.dev(toks), G.dev(kk), G.dev(lab), G.gpu_params(w, 3, max_rounds=1))
    cur = ctx.hbsjd_get_state()[1]
    assert cur[0] == T and cur[1] == T and cur[3] == T and 1 <= cur[2] <= w.window
    model = O.Model(w.shape, G.weights_for(w))
    r = O.Rollout(model, toks, kk, lab, G.orc_params(w, 3))
    r.round()
    np.testing.assert_array_equal(cur, r.state()[1])
    # the last token of an image is the bonus sample of a window of one input
    full, _ = ctx.hbsjd_rollout(G.dev(toks), G.dev(kk), G.dev(lab), G.gpu_params(w, 3))
    r.run()
    np.testing.assert_array_equal(full.cpu().numpy(), r.tokens())
    ctx.hbsjd_destroy()


def test_single_image_and_context_larger_than_the_call():
    w = synth.WORKLOADS["tiny"]
    toks, k, lab = synth.make_inputs(w)
    big = _ctx(w, max_batch=7, max_window=16)        # limits above the call's batch and window
    one = _ctx(w, max_batch=1)
    model = O.Model(w.shape, G.weights_for(w))
    for b in range(2):
        a, _ = one.hbsjd_rollout(G.dev(toks[b:b + 1]), G.dev(k[b:b + 1]), G.dev(lab[b:b + 1]), G.gpu_params(w, 5))
        c, _ = big.hbsjd_rollout(G.dev(toks[b:b + 1]), G.dev(k[b:b + 1]), G.dev(lab[b:b + 1]), G.gpu_params(w, 5))
        np.testing.assert_array_equal(a.cpu().numpy(), c.cpu().numpy())
        r = O.Rollout(model, toks[b:b + 1], k[b:b + 1], lab[b:b + 1], G.orc_params(w, 5))
        r.run()
        np.testing.assert_array_equal(a.cpu().numpy(), r.tokens())
    one.hbsjd_destroy()
    big.hbsjd_destroy()


def test_one_kept_token_makes_sampling_greedy():
    """top-k = 1 leaves a one-hot distribution: every sample is the argmax, so the probabilistic rollout commits
    the greedy rollout's tokens (ties of the top logit aside: none in these models)."""
    w = synth.WORKLOADS["tiny_bf16"]
    toks, k, lab = synth.make_inputs(w)
    ctx = _ctx(w)
    a, sa = ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab), G.gpu_params(w, 9, top_k=1))
    g, sg = ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab), G.gpu_params(w, 9, top_k=1,
                                                                               verify_mode=binding.VERIFY_GREEDY))
    np.testing.assert_array_equal(a.cpu().numpy(), g.cpu().numpy())
    assert sa["rounds"] == sg["rounds"]
    # top-k >= V is no filter
    x, _ = ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab), G.gpu_params(w, 9, top_k=0))
    y, _ = ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab), G.gpu_params(w, 9, top_k=w.shape.vocab + 5))
    np.testing.assert_array_equal(x.cpu().numpy(), y.cpu().numpy())
    ctx.hbsjd_destroy()


def test_guidance_with_the_null_class_is_no_guidance():
    """With the null class as the label both branches compute the same logits, so l_u + s (l_c - l_u) = l_c bit
    for bit and the guided rollout equals the unguided one."""
    w = synth.WORKLOADS["tiny_bf16"]
    toks, k, lab = synth.make_inputs(w)
    null = np.full_like(lab, w.shape.n_classes)
    ctx = _ctx(w)
    a, _ = ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(null), G.gpu_params(w, 2, cfg_scale=3.5))
    b, _ = ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(null), G.gpu_params(w, 2, cfg_scale=1.0))
    np.testing.assert_array_equal(a.cpu().numpy(), b.cpu().numpy())
    ctx.hbsjd_destroy()


@pytest.mark.parametrize("temperature,history", [(0.7, 8), (1.6, 100), (1.0, 1)])
def test_temperature_and_history_offsets_in_lockstep(temperature, history):
    """Temperature other than 1, a history offset beyond the sequence (every history draft falls back to the
    keyed uniform token) and the shortest offset (a draft copies its left neighbour), fp32 model, every round
    compared with the oracle."""
    w = synth.with_shape(synth.WORKLOADS["tiny"], temperature=temperature, history_offset=history)
    toks, k, lab = synth.make_inputs(synth.with_shape(w, prefix=("uniform", 0, 30)))
    model = O.Model(w.shape, G.weights_for(w))
    ctx = _ctx(w)
    rep = G.lockstep(ctx, model, w, toks, k, lab, 11)
    assert rep["max_logit_err"] <= 1e-4 and rep["max_p_err"] <= 1e-6 and rep["replay_mismatch"] == 0
    assert rep["tokens"] == int((w.shape.T - k).sum()) and rep["same"] == rep["tokens"]
    ctx.hbsjd_destroy()


def test_largest_vocabulary_of_the_verification_kernels():
    """V = 32768 (128 KB of probabilities per CTA): probability pipeline against the oracle and one bit-exact
    verification step."""
    import torch
    V = 32768
    sh = synth.ModelShape(1, 64, 1, 64, V, 4, 4, 3, "bf16")
    ctx = binding.Context(sh, synth.make_weights(sh, 3, target_entropy=None), 6, 8)
    rng = np.random.default_rng(0)
    lc = (rng.normal(size=(3, V)) * 3).astype(np.float32)
    lu = (rng.normal(size=(3, V)) * 3).astype(np.float32)
    for kk in (0, 500):
        p = ctx.hbsjd_probs(G.dev(lc), G.dev(lu), 2.0, 0.9, kk).cpu().numpy()
        for r in range(3):
            ref = O.probs(lc[r], lu[r], s=2.0, tau=0.9, k=kk)
            np.testing.assert_array_equal(p[r] > 0, ref > 1e-37)
            assert np.all(np.abs(p[r] - ref) <= 1e-6 + 1e-5 * ref)
    case = G.verify_case(5, B=6, W=8, T=32, V=V, top_k=200)
    d = {n: G.dev(case[n]) for n in ("logits", "q", "cursor", "seq", "delta", "qbase")}
    p_out = torch.zeros_like(d["q"])
    m_out = torch.zeros(6, dtype=torch.int32, device="cuda")
    ctx.hbsjd_verify(G.verify_desc(case, 4, 2), d["logits"], d["q"], p_out, d["cursor"], d["seq"], d["delta"],
                     d["qbase"], m_out)
    p_gpu = p_out.cpu().numpy()
    for b in range(6):
        c = int(case["cursor"][b])
        if c >= case["T"]:
            continue
        n = min(case["W"], case["T"] - c)
        seq, dl = case["seq"][b].copy(), case["delta"][b].copy()
        nc, m, j = O.replay_round(V, case["T"], case["W"], case["H"], False, 4, b, 2, c, seq, dl, p_gpu[b][:n],
                                  case["q"][b], int(case["qbase"][b]))
        assert nc == int(d["cursor"][b]) and m == int(m_out[b])
        np.testing.assert_array_equal(seq[:nc + 1], d["seq"][b].cpu().numpy()[:nc + 1])
    ctx.hbsjd_destroy()


def test_batch_synchronous_progress_matches_the_oracle():
    """Execution mode SYNC (the baseline of the Table 2 ablation): every live image advances by the batch's
    smallest commit.  fp32 model, every round compared with the oracle's synchronous rollout; greedy verification
    still gives the greedy AR tokens."""
    w = synth.WORKLOADS["tiny"]
    T = w.shape.T
    toks, k, lab = synth.make_inputs(synth.with_shape(w, prefix=("uniform", 0, 30)), seed=3)
    model = O.Model(w.shape, G.weights_for(w))
    ctx = _ctx(w)
    for seed in (5, 6):
        orc = O.Rollout(model, toks, k, lab, G.orc_params(w, seed, exec_mode=3))
        ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab),
                          G.gpu_params(w, seed, exec_mode=binding.EXEC_SYNC, max_rounds=0))
        rounds = 0
        while orc.live():
            before = ctx.hbsjd_get_state()[1].copy()
            ctx.hbsjd_round()
            _, m_o, _ = orc.round()
            _, cur, seq, _, _ = ctx.hbsjd_get_state()
            _, o_cur, o_seq, _, _ = orc.state()
            live = before < T
            assert len(set((cur - before)[live].tolist())) == 1        # one pace for the whole batch
            np.testing.assert_array_equal(cur, o_cur)
            for b in range(len(k)):
                np.testing.assert_array_equal(seq[b, :cur[b] + 1], o_seq[b, :o_cur[b] + 1])
            rounds += 1
        out_sync, st_sync = ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab),
                                              G.gpu_params(w, seed, exec_mode=binding.EXEC_SYNC))
        out_free, st_free = ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab),
                                              G.gpu_params(w, seed, exec_mode=binding.EXEC_FULL))
        assert st_sync["rounds"] == rounds            # (more rounds than independent progress on average, not per seed)
        assert st_sync["committed"] == st_free["committed"] == int((T - k).sum())
        assert st_sync["compact_rounds"] == 0
    g, _ = ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab),
                             G.gpu_params(w, 0, exec_mode=binding.EXEC_SYNC, verify_mode=binding.VERIFY_GREEDY))
    ar = model.ar_rollout(toks, k, lab, G.orc_params(w, 0, greedy=True, window=1))
    np.testing.assert_array_equal(g.cpu().numpy(), ar)
    ctx.hbsjd_destroy()


def test_bf16_model_with_head_size_32_and_unsupported_head_sizes():
    """Head size 32 in bf16 runs the fused QKV epilogue with half a rotation table per head and the plain attention
    kernel; head size 128 is refused for bf16 models at creation."""
    sh = synth.ModelShape(2, 128, 4, 256, 512, 6, 6, 5, "bf16")          # dh = 32
    w = synth.Workload("dh32", sh, 3, 8, 2.0, 40, 1.0, 6, ("uniform", 0, 12))
    img = synth.make_weights(sh, 9)
    toks, k, lab = synth.make_inputs(w)
    ctx = binding.Context(sh, img, w.batch, w.window)
    model = O.Model(sh, img)
    rep = G.lockstep(ctx, model, w, toks, k, lab, 3, floor_every_round=True)
    # logits against the noise floor measured on the same windows (the context folds its RMSNorm: factor 1.5 on the
    # mean, measured 1.25; the maximum over these few thousand logits measured 1.43 x the floor's)
    G.check_logits_against_floor(rep, rep["floor_max"], rep["floor_sum"] / rep["floor_n"], "head size 32",
                                 max_factor=1.8, mean_factor=1.5)
    assert rep["max_p_err"] <= 1e-6
    G.check_flips_explained(rep)
    assert rep["same"] >= 0.9 * rep["tokens"]
    ctx.hbsjd_destroy()
    bad = synth.ModelShape(1, 256, 2, 256, 512, 4, 4, 5, "bf16")         # dh = 128
    with pytest.raises(binding.HbsjdError):
        binding.Context(bad, synth.make_weights(bad, 9, target_entropy=None), 2, 4)


def test_images_do_not_depend_on_their_batch_mates():
    """Each image advances on its own: replacing the other images of the batch (here: marking them complete, or
    giving them other prefixes and labels) leaves an image's tokens unchanged (bf16 model, guidance, top-k)."""
    w = synth.WORKLOADS["tiny_bf16"]
    T = w.shape.T
    toks, k, lab = synth.make_inputs(w)
    ctx = _ctx(w)
    ref, _ = ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab), G.gpu_params(w, 4))
    ref = ref.cpu().numpy()
    keep = [0, 2]
    k2, lab2, toks2 = k.copy(), lab.copy(), toks.copy()
    for b in range(w.batch):
        if b not in keep:
            k2[b] = T if b % 2 else max(0, int(k[b]) - 3)
            lab2[b] = (lab[b] + 1) % w.shape.n_classes
            toks2[b] = (toks[b] + 7) % w.shape.vocab
    for mode in (binding.EXEC_FULL, binding.EXEC_COMPACT):
        out, _ = ctx.hbsjd_rollout(G.dev(toks2), G.dev(k2), G.dev(lab2), G.gpu_params(w, 4, exec_mode=mode))
        out = out.cpu().numpy()
        for b in keep:
            np.testing.assert_array_equal(out[b], ref[b])
    ctx.hbsjd_destroy()


def test_kernel_profile_bins_add_up():
    """Per-class event timing: the GEMM class split by activation rows adds up to the class, every bin that has
    launches has time, FLOPs and algorithmic bytes, and switching the profile off stops the accounting."""
    w = synth.WORKLOADS["small_bf16"]
    toks, k, lab = synth.make_inputs(w)
    ctx = binding.Context(w.shape, G.weights_for(w), w.batch, w.window)
    ctx.hbsjd_profile(True)
    _, st = ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab), G.gpu_params(w, 3))
    p = ctx.hbsjd_profile_read()
    ctx.hbsjd_profile(False)
    g, bins = p["gemm"], p["gemm_by_rows"]
    assert g["launches"] > 0 and p["attention"]["launches"] > 0 and p["accept"]["launches"] == st["rounds"]
    assert sum(b["launches"] for b in bins.values()) == g["launches"]
    assert abs(sum(b["ms"] for b in bins.values()) - g["ms"]) <= 1e-6 * g["ms"]
    assert abs(sum(b["work"] for b in bins.values()) - g["work"]) <= 1e-9 * g["work"]
    for b in bins.values():
        assert (b["launches"] > 0) == (b["ms"] > 0) == (b["work"] > 0) == (b["bytes"] > 0)
    assert bins["rows>6144"]["launches"] == 0                  # this context has at most 2 x batch x window rows
    ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab), G.gpu_params(w, 3))
    assert ctx.hbsjd_profile_read()["gemm"]["launches"] == g["launches"]
    ctx.hbsjd_destroy()

