"""Pins for the oracle's distillation score (Eq. 3): the bidirectional KL and the trajectory scoring."""
import math

import numpy as np
from scipy.special import rel_entr, softmax

from oracle import oracle as O
from paper_2608_18183_b200 import synth
from tests import torch_restatement as TR


def test_bikl_two_classes_closed_form():
    # p = (sigmoid(a), .), q = (sigmoid(b), .): D = 1/2 (p0 - q0)(a - b)
    for a, b in [(0.3, -1.2), (2.0, 2.0), (-4.0, 5.0), (0.0, 1e-3)]:
        p0, q0 = 1 / (1 + math.exp(-a)), 1 / (1 + math.exp(-b))
        want = 0.5 * (p0 - q0) * (a - b)
        got = O.bikl(np.array([[a, 0.0]]), np.array([[b, 0.0]]))[0]
        assert abs(got - want) < 1e-7 * max(1.0, abs(want)), (a, b, got, want)
        # written as the two KL terms
        kl = lambda x, y: x * math.log(x / y) + (1 - x) * math.log((1 - x) / (1 - y))
        assert abs(got - 0.5 * (kl(p0, q0) + kl(q0, p0))) < 1e-7


def test_bikl_uniform_against_one_raised_logit():
    # s uniform over V, t raises entry 0 by L: D = 1/2 L (q0 - 1/V), q0 = e^L / (e^L + V - 1)
    V, L = 64, 3.0
    s = np.zeros((1, V), dtype=np.float32)
    t = s.copy()
    t[0, 0] = L
    q0 = math.exp(L) / (math.exp(L) + V - 1)
    assert abs(O.bikl(s, t)[0] - 0.5 * L * (q0 - 1.0 / V)) < 1e-9


def test_bikl_invariants_and_library_cross_check():
    rng = np.random.default_rng(0)
    s = (rng.normal(size=(6, 97)) * 3).astype(np.float32)
    t = (rng.normal(size=(6, 97)) * 2).astype(np.float32)
    d = O.bikl(s, t)
    assert (d > 0).all()
    np.testing.assert_allclose(O.bikl(t, s), d, rtol=1e-12)                      # symmetric
    np.testing.assert_allclose(O.bikl(s, s), 0.0, atol=1e-12)                    # equal distributions
    np.testing.assert_allclose(O.bikl(s + np.float32(2.0), t - np.float32(4.0)), d, rtol=1e-5)  # shift invariant
    p, q = softmax(s.astype(np.float64), axis=1), softmax(t.astype(np.float64), axis=1)
    np.testing.assert_allclose(d, 0.5 * rel_entr(p, q).sum(1) + 0.5 * rel_entr(q, p).sum(1), rtol=1e-9)
    # the normalisers cancel: D = 1/2 sum_v (p_v - q_v)(s_v - t_v)
    np.testing.assert_allclose(d, 0.5 * ((p - q) * (s.astype(np.float64) - t)).sum(1), rtol=1e-9)
    # far-apart logits do not overflow or lose the small side
    big = np.array([[80.0, 0.0, -80.0]], dtype=np.float32)
    assert np.isfinite(O.bikl(big, -big)[0]) and O.bikl(big, -big)[0] > 79.0


def _teacher_of(w):
    """A second, wider model over the same vocabulary and grid (the paper distils a larger teacher)."""
    s = w.shape
    sh = synth.ModelShape(s.n_layers + 1, s.dim * 2, s.n_heads * 2, s.ffn_hidden * 2, s.vocab, s.grid_h, s.grid_w,
                          s.n_classes, s.dtype)
    return sh, synth.make_weights(sh, 77)


def test_score_against_restated_forward_and_definition(tiny):
    w, img = tiny
    tsh, timg = _teacher_of(w)
    stu, tea = O.Model(w.shape, img), O.Model(tsh, timg)
    T, V = w.shape.T, w.shape.vocab
    rng = np.random.default_rng(4)
    B = 4
    toks = rng.integers(0, V, size=(B, T)).astype(np.int32)
    k = np.array([0, 17, T - 1, T], dtype=np.int32)
    lab = rng.integers(0, w.shape.n_classes, size=B).astype(np.int32)
    pos, per, loss = O.score(stu, tea, toks, k, lab)
    Ps, Pt = TR.load(w.shape, img), TR.load(tsh, timg)
    for b in range(B):
        seq = np.concatenate([[0], toks[b, :T - 1]]).astype(np.int32)  # inputs: class token, x_1 .. x_{T-1}
        p = softmax(TR.forward(w.shape, Ps, int(lab[b]), seq).astype(np.float64), axis=1)
        q = softmax(TR.forward(tsh, Pt, int(lab[b]), seq).astype(np.float64), axis=1)
        d = 0.5 * rel_entr(p, q).sum(1) + 0.5 * rel_entr(q, p).sum(1)  # row i: the term of position i + 1
        want = np.where(np.arange(1, T + 1) >= k[b] + 1, d, 0.0)
        np.testing.assert_allclose(pos[b], want, rtol=2e-4, atol=1e-7)
        assert (pos[b, :k[b]] == 0).all()
        if k[b] < T:
            assert abs(per[b] - want.sum() / (T - k[b])) < 2e-4 * per[b]
    assert per[3] == 0.0                                  # nothing generated: no term
    assert abs(loss - per[:3].mean()) < 1e-12             # and the image is left out of the mean
    assert per[2] == pos[2, T - 1]                        # one generated token: its own term
    # a model against itself scores zero everywhere
    pos0, per0, loss0 = O.score(stu, stu, toks, k, lab)
    assert np.abs(pos0).max() < 1e-12 and loss0 == 0.0


def test_score_terms_are_causal_in_the_trajectory(tiny):
    # the term of position t conditions on x_<t only: changing x_t moves the terms after t and none up to t
    w, img = tiny
    tsh, timg = _teacher_of(w)
    stu, tea = O.Model(w.shape, img), O.Model(tsh, timg)
    T, V = w.shape.T, w.shape.vocab
    rng = np.random.default_rng(5)
    toks = rng.integers(0, V, size=(1, T)).astype(np.int32)
    k, lab = np.array([0], dtype=np.int32), np.array([2], dtype=np.int32)
    pos, _, _ = O.score(stu, tea, toks, k, lab)
    t = 20
    toks2 = toks.copy()
    toks2[0, t - 1] = (toks[0, t - 1] + 1) % V
    pos2, _, _ = O.score(stu, tea, toks2, k, lab)
    np.testing.assert_array_equal(pos2[0, :t], pos[0, :t])
    assert pos2[0, t] != pos[0, t]
    # the class label enters every term
    pos3, _, _ = O.score(stu, tea, toks, k, np.array([3], dtype=np.int32))
    assert (pos3[0] != pos[0]).all()
