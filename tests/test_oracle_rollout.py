"""Pins for the oracle's rollout: special cases and invariants the method fixes."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2608_18183_b200 import synth


@pytest.fixture(scope="module")
def small():
    """A reduced tiny model (T = 4x4) so that the quadratic-cost AR sampler stays fast."""
    w = synth.WORKLOADS["tiny"]
    sh = synth.ModelShape(2, 32, 2, 64, 48, 4, 4, 5, "fp32")
    img = synth.make_weights(sh, 11, target_entropy=2.0)
    return synth.with_shape(w, shape=sh, batch=5, history_offset=4), img, O.Model(sh, img)


def _inputs(w, seed, kmax):
    toks, k, lab = synth.make_inputs(synth.with_shape(w, prefix=("uniform", 0, kmax)), seed=seed)
    return toks, k, lab


@pytest.mark.parametrize("cfg,topk", [(1.0, 0), (2.5, 7)])
def test_window_one_is_plain_ar_sampling(small, cfg, topk):
    """A window of one input (the last committed token, no drafts) commits one token per round,
    sampled from the model's next-token distribution: exactly the AR sampler of Eq. 2."""
    w, img, m = small
    toks, k, lab = _inputs(w, 3, 6)
    P = O.make_params(1, 4, cfg_scale=cfg, top_k=topk, seed=77)
    r = O.Rollout(m, toks, k, lab, P)
    r.run()
    ar = m.ar_rollout(toks, k, lab, P)
    np.testing.assert_array_equal(r.tokens(), ar)
    st = r.stats()
    assert st["committed"] == int((w.shape.T - k).sum()) and st["rejects"] == 0
    # the prefix is passed through untouched
    for b in range(len(k)):
        np.testing.assert_array_equal(ar[b, :k[b]], toks[b, :k[b]])


@pytest.mark.parametrize("W", [1, 2, 3, 8, 16])
@pytest.mark.parametrize("H", [1, 4, 9])
def test_greedy_sjd_equals_greedy_ar(small, W, H):
    """Greedy verification (Eq. 4) commits the student's argmax chain whatever the window and
    history offset: the Jacobi fixed point is the greedy AR sequence."""
    w, img, m = small
    toks, k, lab = _inputs(w, 4, 5)
    P = O.make_params(W, H, greedy=True, seed=1)
    r = O.Rollout(m, toks, k, lab, P)
    r.run()
    np.testing.assert_array_equal(r.tokens(), m.ar_rollout(toks, k, lab, P))
    if W > 1:
        assert r.stats()["rounds"] <= w.shape.T  # never slower than one token per round


def test_modes_do_not_change_values_and_follow_eq6(small):
    w, img, m = small
    toks, k, lab = _inputs(w, 5, 12)
    outs, traces = [], []
    for mode, gamma in [(0, 0), (1, 0), (2, 0), (2, 2), (2, 3), (2, 100)]:
        P = O.make_params(4, 4, cfg_scale=2.0, exec_mode=mode, gamma=gamma, seed=5)
        r = O.Rollout(m, toks, k, lab, P)
        ms = []
        while r.live():
            ms.append(r.round()[1])
        outs.append((r.tokens(), np.array(ms)))
        st = r.stats()
        traces.append(st)
        if mode == 2:  # Eq. 6: Full iff A > gamma
            np.testing.assert_array_equal(st["mode_trace"], (st["live_trace"] <= gamma).astype(np.int32))
        else:
            assert (st["mode_trace"] == mode).all()
        assert (np.diff(st["live_trace"]) <= 0).all()  # the live set only shrinks
    for t, ms in outs[1:]:
        np.testing.assert_array_equal(t, outs[0][0])
        np.testing.assert_array_equal(ms, outs[0][1])


def test_images_are_independent(small):
    """Any subset of the batch, run alone under its original image indices, yields the same tokens."""
    w, img, m = small
    toks, k, lab = _inputs(w, 6, 10)
    P = O.make_params(4, 4, cfg_scale=1.5, top_k=20, seed=9)
    r = O.Rollout(m, toks, k, lab, P)
    r.run()
    full = r.tokens()
    for sub in ([0], [3, 1], [4, 2, 0]):
        rs = O.Rollout(m, toks[sub], k[sub], lab[sub], P, image_ids=sub)
        rs.run()
        np.testing.assert_array_equal(rs.tokens(), full[sub])
    # under different indices the draws differ
    rs = O.Rollout(m, toks[[3]], k[[3]], lab[[3]], P)
    rs.run()
    assert not np.array_equal(rs.tokens()[0], full[3])


def test_guidance_special_cases(small):
    w, img, m = small
    toks, k, lab = _inputs(w, 7, 6)
    null = np.full_like(lab, w.shape.n_classes)
    base = O.Rollout(m, toks, k, null, O.make_params(4, 4, seed=2))
    base.run()
    # conditional branch already on the null class: guidance at any scale changes nothing
    g = O.Rollout(m, toks, k, null, O.make_params(4, 4, cfg_scale=4.0, seed=2))
    g.run()
    np.testing.assert_array_equal(g.tokens(), base.tokens())


def test_rollout_bookkeeping(small):
    w, img, m = small
    T = w.shape.T
    toks, k, lab = _inputs(w, 8, T)
    k[0] = T       # finished from the start
    k[1] = T - 1   # a single token to generate
    k[2] = 0       # empty prefix: the anchor is the class token
    P = O.make_params(8, 4, seed=3)
    r = O.Rollout(m, toks, k, lab, P)
    assert r.live() == int((k < T).sum())
    total_m = np.zeros(len(k), dtype=np.int64)
    rounds = 0
    while r.live():
        _, cur_before, *_ = r.state()
        live_after, mm, jj = r.round()
        _, cur_after, *_ = r.state()
        np.testing.assert_array_equal(cur_after - cur_before, mm)
        act = cur_before < T
        assert (mm[act] >= 1).all() and (mm[~act] == 0).all()
        assert (mm <= np.minimum(8, T - cur_before)).all()
        # a reject at j commits j+1 tokens; no reject commits the whole window
        for b in np.nonzero(act)[0]:
            n = min(8, T - cur_before[b])
            assert mm[b] == (jj[b] + 1 if jj[b] >= 0 else n)
        total_m += mm
        rounds += 1
    np.testing.assert_array_equal(total_m, T - k)
    out = r.tokens()
    for b in range(len(k)):
        np.testing.assert_array_equal(out[b, :k[b]], toks[b, :k[b]])
    st = r.stats()
    assert st["rounds"] == rounds and st["committed"] == int((T - k).sum())
    assert st["image_forwards"] == int(st["live_trace"].sum())
    assert (out >= 0).all() and (out < w.shape.vocab).all()


def test_history_fill_of_initial_window(small):
    """Before the first round every draft is the token H positions back (Sec. 4.2), or a keyed
    uniform token where that position does not exist; all are point-mass proposals."""
    w, img, m = small
    toks, k, lab = _inputs(w, 9, 8)
    k[:] = [0, 1, 3, 6, 8]
    H, W = 3, 6
    P = O.make_params(W, H, seed=4)
    r = O.Rollout(m, toks, k, lab, P)
    _, cur, seq, delta, _ = r.state()
    for b in range(len(k)):
        c = k[b]
        for t in range(c + 1, c + min(W, w.shape.T - c)):
            assert delta[b, t] == 1
            if t - H >= 1:
                assert seq[b, t] == seq[b, t - H]
            else:
                w3 = int(O.philox([b, t, 0xFFFFFFFF, 0], [4, 0])[3])
                assert seq[b, t] == (w3 * w.shape.vocab) >> 32


def test_round_matches_replay_on_exported_probabilities(small):
    """The verify / commit / refresh step is a pure function of (p, q, state, words)."""
    w, img, m = small
    toks, k, lab = _inputs(w, 10, 6)
    P = O.make_params(5, 4, cfg_scale=2.0, seed=6)
    r = O.Rollout(m, toks, k, lab, P)
    V, T = w.shape.vocab, w.shape.T
    qprev = [np.zeros((5, V), dtype=np.float32) for _ in k]
    while r.live():
        rnd, cur, seq, delta, qbase = r.state()
        r.round()
        _, cur2, seq2, delta2, qbase2 = r.state()
        for b in range(len(k)):
            if cur[b] >= T:
                continue
            p = r.last_probs(b)
            s, d = seq[b].copy(), delta[b].copy()
            qp = np.zeros((5, V), dtype=np.float32)
            qp[:qprev[b].shape[0]] = qprev[b]
            nc, mm, j = O.replay_round(V, T, 5, 4, False, 6, b, rnd, int(cur[b]), s, d, p, qp, int(qbase[b]))
            assert nc == cur2[b]
            np.testing.assert_array_equal(s, seq2[b])
            np.testing.assert_array_equal(d[nc + 1:nc + 5], delta2[b][nc + 1:nc + 5])
            qprev[b] = p
