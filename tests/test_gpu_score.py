"""Distillation score on the GPU (Eq. 3) against the oracle, through the C ABI."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2608_18183_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _teacher_shape(s, dtype=None):
    """A wider, deeper model over the same vocabulary, grid and classes."""
    return synth.ModelShape(s.n_layers + 1, s.dim * 2, s.n_heads * 2, s.ffn_hidden * 2, s.vocab, s.grid_h, s.grid_w,
                            s.n_classes, dtype or s.dtype)


def test_bikl_rows_match_the_definition():
    import torch
    sh = synth.ModelShape(1, 64, 1, 64, 16384, 4, 4, 3, "bf16")
    ctx = binding.Context(sh, synth.make_weights(sh, 3, target_entropy=None), 2, 4)
    rng = np.random.default_rng(0)
    rows = 37
    s = (rng.normal(size=(rows, sh.vocab)) * 3.0).astype(np.float32)
    t = (0.6 * s + rng.normal(size=(rows, sh.vocab)) * 2.0).astype(np.float32)
    s[1], t[1] = s[1] + 50.0, t[1] - 70.0          # shifted rows: the normalisers cancel
    t[2] = s[2]                                     # equal distributions
    s[3, 5], t[3, 9] = 90.0, 90.0                   # two nearly one-hot rows that disagree
    got = ctx.hbsjd_bikl(G.dev(s), G.dev(t)).cpu().numpy()
    want = O.bikl(s, t)
    # fp32 sums of V terms with ex2.approx exponentials: a few 1e-6 relative on each of the two halves
    assert np.abs(got - want).max() <= 2e-5 * max(1.0, np.abs(want).max()), np.abs(got - want).max()
    np.testing.assert_allclose(got, want, rtol=2e-4, atol=2e-5)
    assert got[2] == 0.0 and want[3] > 40.0
    ctx.hbsjd_destroy()
    # a small vocabulary (fewer entries than threads x 4) and one that needs several chunks per thread
    for V in (256, 32768):
        sh = synth.ModelShape(1, 64, 1, 64, V, 4, 4, 3, "bf16")
        ctx = binding.Context(sh, synth.make_weights(sh, 3, target_entropy=None), 2, 4)
        s = (rng.normal(size=(5, V)) * 2.0).astype(np.float32)
        t = (rng.normal(size=(5, V)) * 2.0).astype(np.float32)
        np.testing.assert_allclose(ctx.hbsjd_bikl(G.dev(s), G.dev(t)).cpu().numpy(), O.bikl(s, t), rtol=2e-4)
        ctx.hbsjd_destroy()


def _score_both(w, tsh, toks, k, lab, max_batch=None):
    timg = synth.make_weights(tsh, 77)
    stu = binding.Context(w.shape, G.weights_for(w), max_batch or len(k), w.window)
    tea = binding.Context(tsh, timg, max_batch or len(k), w.window)
    pos, per, loss = stu.hbsjd_score(tea, G.dev(toks), G.dev(k), G.dev(lab))
    want = O.score(O.Model(w.shape, G.weights_for(w)), O.Model(tsh, timg), toks, k, lab)
    out = (pos.cpu().numpy(), per.cpu().numpy(), loss), want
    stu.hbsjd_destroy()
    tea.hbsjd_destroy()
    return out


def test_score_fp32_models_match_the_oracle():
    w = synth.WORKLOADS["tiny"]
    T, V = w.shape.T, w.shape.vocab
    rng = np.random.default_rng(2)
    B = 5
    toks = rng.integers(0, V, size=(B, T)).astype(np.int32)
    k = np.array([0, 13, T - 1, T, 40], dtype=np.int32)     # T is not a multiple of the chunk for some rows only
    lab = rng.integers(0, w.shape.n_classes, size=B).astype(np.int32)
    (pos, per, loss), (opos, oper, oloss) = _score_both(w, _teacher_shape(w.shape), toks, k, lab)
    assert opos.max() > 0.05                                    # the comparison is not vacuous
    np.testing.assert_allclose(pos, opos, rtol=2e-3, atol=2e-5)
    for b in range(B):
        assert (pos[b, :k[b]] == 0).all()
    np.testing.assert_allclose(per, oper, rtol=5e-4, atol=1e-6)
    assert per[3] == 0.0
    assert abs(loss - oloss) <= 5e-4 * oloss


def test_score_window_that_does_not_divide_the_sequence():
    w = synth.with_shape(synth.WORKLOADS["tiny"], window=7)      # 64 = 9 chunks of 7 + 1
    T, V = w.shape.T, w.shape.vocab
    rng = np.random.default_rng(3)
    toks = rng.integers(0, V, size=(3, T)).astype(np.int32)
    k = np.array([5, 0, 62], dtype=np.int32)
    lab = np.array([1, 2, 3], dtype=np.int32)
    (pos, per, loss), (opos, oper, oloss) = _score_both(w, _teacher_shape(w.shape), toks, k, lab, max_batch=4)
    np.testing.assert_allclose(pos, opos, rtol=2e-3, atol=2e-5)
    assert abs(loss - oloss) <= 5e-4 * oloss


def test_score_bf16_models_within_the_derived_tolerance():
    """bf16 models: each model's logits carry the rounding noise the forward parity tests bound (mean s per logit,
    max tol: the measured noise floor).  With d = s - t, D = 1/2 sum (p - q) d moves under logit noise e_s, e_t by
    1/2 sum (p - q)(e_s - e_t) + 1/2 (Cov_p(e_s, d) - Cov_q(e_t, d)): the first part has rms <= s (|p - q|_2 <=
    sqrt 2), the second rms <= s std(d) (|p|_2, |q|_2 <= 1).  So a position's error has rms <= s (1 + std d); the
    maximum over the positions is held to the same expression with the max-abs logit bound tol in place of s."""
    w = synth.WORKLOADS["small_bf16"]
    tsh = _teacher_shape(w.shape)
    timg = synth.make_weights(tsh, 77)
    T, V = w.shape.T, w.shape.vocab
    rng = np.random.default_rng(4)
    B = 3
    toks = rng.integers(0, V, size=(B, T)).astype(np.int32)
    k = np.array([0, 50, 100], dtype=np.int32)
    lab = rng.integers(0, w.shape.n_classes, size=B).astype(np.int32)
    (pos, per, loss), (opos, oper, oloss) = _score_both(w, tsh, toks, k, lab)
    seq0 = np.concatenate([[0], toks[0, :T - 1]]).astype(np.int32)
    m_s, m_t = O.Model(w.shape, G.weights_for(w)), O.Model(tsh, timg)
    l_s, l_t = m_s.forward_full(int(lab[0]), seq0), m_t.forward_full(int(lab[0]), seq0)
    # s, tol: mean and maximum of the logit noise floor, measured as the oracle against its own diagnostic form (fp32
    # sums, bf16 attention weights, the RMSNorm form both contexts use) on the same sequence, with the factors of
    # the forward parity tests (1.5 on the mean, 2 on a maximum taken over fewer logits than the GPU's)
    s = tol = 0.0
    for m, ref in ((m_s, l_s), (m_t, l_t)):
        m.set_diag(acc_f32=True, attn_w_bf16=True, norm_folded=True)
        try:
            d = np.abs(m.forward_full(int(lab[0]), seq0).astype(np.float64) - ref)
        finally:
            m.set_diag()
        s, tol = max(s, 1.5 * float(d.mean())), max(tol, 2.0 * float(d.max()))
    spread = 1.0 + float((l_s - l_t).std(axis=1).max())
    live = opos > 0
    assert live.sum() == int((T - k).sum())
    err = np.abs(pos - opos)[live]
    assert err.max() <= tol * spread, (err.max(), tol * spread)
    assert err.mean() <= s * spread, (err.mean(), s * spread)
    assert (pos[~live] == 0).all()
    assert abs(loss - oloss) <= s * spread
    # regression guard, looser than what is measured (3e-5 on the loss, 0.13 % mean per position)
    assert abs(loss - oloss) <= 2e-3 * oloss and err.mean() <= 5e-3 * opos[live].mean()
    np.testing.assert_allclose(per, [pos[b, k[b]:].mean() for b in range(B)], rtol=1e-5)


def test_score_of_a_model_against_itself_is_zero_and_the_call_is_repeatable():
    w = synth.WORKLOADS["tiny_bf16"]
    T, V = w.shape.T, w.shape.vocab
    toks, k, lab = synth.make_inputs(w)
    toks = np.random.default_rng(0).integers(0, V, size=toks.shape).astype(np.int32)
    a = binding.Context(w.shape, G.weights_for(w), w.batch, w.window)
    b = binding.Context(w.shape, G.weights_for(w), w.batch, w.window)
    pos, per, loss = a.hbsjd_score(b, G.dev(toks), G.dev(k), G.dev(lab))
    assert float(pos.abs().max()) == 0.0 and loss == 0.0       # same kernels, same inputs: bit-identical logits
    # scoring follows a rollout on the same context and leaves it usable for the next rollout
    out, st = a.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab), G.gpu_params(w, 1))
    tsh = _teacher_shape(w.shape)
    tea = binding.Context(tsh, synth.make_weights(tsh, 77), w.batch, w.window)
    r1 = a.hbsjd_score(tea, out, G.dev(k), G.dev(lab))
    out2, _ = a.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab), G.gpu_params(w, 1))
    assert bool((out2 == out).all())
    r2 = a.hbsjd_score(tea, out, G.dev(k), G.dev(lab))
    assert bool((r1[0] == r2[0]).all()) and r1[2] == r2[2] and r1[2] > 0
    # misuse is refused before any launch
    with pytest.raises(binding.HbsjdError) as e:
        a.hbsjd_score(a, out, G.dev(k), G.dev(lab))
    assert e.value.code == -1
    bad = out.clone()
    bad[0, 3] = V
    with pytest.raises(binding.HbsjdError) as e:
        a.hbsjd_score(tea, bad, G.dev(k), G.dev(lab))
    assert e.value.code == -1
    for c in (a, b, tea):
        c.hbsjd_destroy()
