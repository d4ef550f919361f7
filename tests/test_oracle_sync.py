"""Pins for the oracle's batch-synchronous progress (execution mode 3): the baseline of the paper's "Is
independent progress necessary" ablation, in which every live image advances by the smallest commit of the batch."""
import numpy as np
import pytest
from scipy import stats

from oracle import oracle as O
from paper_2608_18183_b200 import synth
from tests import test_oracle_distribution as D

SYNC = 3


def _rollout(model, w, toks, k, lab, seed, mode, greedy=False, ids=None):
    P = O.make_params(w.window, w.history_offset, cfg_scale=w.cfg_scale, temperature=w.temperature, top_k=w.top_k,
                      greedy=greedy, exec_mode=mode, seed=seed)
    return O.Rollout(model, toks, k, lab, P, image_ids=ids)


def test_every_live_image_advances_by_the_batch_minimum(tiny):
    w, img = tiny
    model = O.Model(w.shape, img)
    toks, k, lab = synth.make_inputs(synth.with_shape(w, prefix=("uniform", 0, 30)), seed=3)
    T = w.shape.T
    r = _rollout(model, w, toks, k, lab, 5, SYNC)
    free = _rollout(model, w, toks, k, lab, 5, 0)
    first = True
    while r.live():
        cur = r.state()[1].copy()
        _, m, j = r.round()
        live = cur < T
        assert len(set(m[live].tolist())) == 1 and (m[~live] == 0).all()   # one pace for the whole batch
        assert (m[live] <= np.minimum(w.window, T - cur[live])).all()
        if first:
            # the first round starts from the same state as independent progress: the pace is its smallest commit,
            # and an image held back keeps exactly the first tokens it would have committed
            _, m_free, _ = free.round()
            assert m[live][0] == m_free[live].min()
            s_sync, s_free = r.state()[2], free.state()[2]
            for b in np.nonzero(live)[0]:
                np.testing.assert_array_equal(s_sync[b, :cur[b] + m[b] + (m[b] == m_free[b])],
                                              s_free[b, :cur[b] + m[b] + (m[b] == m_free[b])])
            first = False
    assert (r.state()[1] == T).all()


def test_synchronous_progress_needs_more_rounds_and_keeps_greedy_exact(tiny):
    w, img = tiny
    model = O.Model(w.shape, img)
    toks, k, lab = synth.make_inputs(w)
    rounds_sync = rounds_free = 0
    for seed in range(4):
        a, b = _rollout(model, w, toks, k, lab, seed, SYNC), _rollout(model, w, toks, k, lab, seed, 0)
        a.run()
        b.run()
        rounds_sync += a.stats()["rounds"]
        rounds_free += b.stats()["rounds"]
        assert a.stats()["committed"] == b.stats()["committed"] == int((w.shape.T - k).sum())
    assert rounds_sync > rounds_free                       # the paper's Table 2: 241 against 176 rounds
    # greedy verification is exact under either pace: the greedy AR tokens
    g = _rollout(model, w, toks, k, lab, 0, SYNC, greedy=True)
    g.run()
    ar = model.ar_rollout(toks, k, lab, O.make_params(1, w.history_offset, greedy=True))
    np.testing.assert_array_equal(g.tokens(), ar)
    # a batch of one has nobody to wait for
    one_s, one_f = _rollout(model, w, toks[:1], k[:1], lab[:1], 9, SYNC), _rollout(model, w, toks[:1], k[:1], lab[:1], 9, 0)
    one_s.run()
    one_f.run()
    np.testing.assert_array_equal(one_s.tokens(), one_f.tokens())


def test_truncated_commit_keeps_accepted_drafts_only():
    # hand-made round: point-mass proposals whose drafts all carry probability 1 -> every draft is accepted;
    # the image's own commit is the whole window (3 drafts + bonus), a limit of 2 keeps the first two drafts
    V, T, W, H = 5, 8, 4, 2
    seq = np.array([0, 3, 1, 4, 2, 0, 0, 0, 0], dtype=np.int32)     # cursor 1: drafts x_2..x_4 = 1, 4, 2
    delta = np.array([0, 0, 1, 1, 1, 0, 0, 0, 0], dtype=np.uint8)
    p = np.zeros((W, V), dtype=np.float32)
    for i, z in enumerate([1, 4, 2, 3]):
        p[i, z] = 1.0
    q = np.zeros((W, V), dtype=np.float32)
    s1, d1 = seq.copy(), delta.copy()
    c1, m1, j1 = O.replay_round(V, T, W, H, False, 7, 0, 0, 1, s1, d1, p, q, 0)
    assert (c1, m1, j1) == (5, 4, -1) and s1[2:6].tolist() == [1, 4, 2, 3]
    s2, d2 = seq.copy(), delta.copy()
    c2, m2, j2 = O.replay_round(V, T, W, H, False, 7, 0, 0, 1, s2, d2, p, q, 0, m_limit=2)
    assert (c2, m2, j2) == (3, 2, -1) and s2[2:4].tolist() == [1, 4] and d2[3] == 0
    # the positions after the new cursor are drafts again: resampled from this round's distributions
    assert s2[4] == 2 and s2[5] == 3 and d2[4] == 0 and d2[5] == 0
    # a limit at or above the image's own commit changes nothing
    s3, d3 = seq.copy(), delta.copy()
    assert O.replay_round(V, T, W, H, False, 7, 0, 0, 1, s3, d3, p, q, 0, m_limit=4)[:2] == (5, 4)
    np.testing.assert_array_equal(s3, s1)


def test_synchronous_rollouts_follow_the_ar_joint(micro_model):
    """Holding an image back to the batch's pace depends on the other images only, so its tokens keep the AR
    distribution: chi-square of batches of three against the enumerated joint."""
    sh, img = micro_model
    joint, _ = D._exact_joint(sh, img, 1, 1.0, ())
    m = O.Model(sh, img)
    batches, B = 12_000, 3
    toks = np.zeros((B, sh.T), dtype=np.int32)
    k = np.zeros(B, dtype=np.int32)
    lab = np.full(B, 1, dtype=np.int32)
    P = O.make_params(3, 2, exec_mode=SYNC, seed=11)
    counts, forwards = {}, 0
    for i in range(batches):
        r = O.Rollout(m, toks, k, lab, P, image_ids=[3 * i, 3 * i + 1, 3 * i + 2])
        r.run()
        forwards += r.stats()["image_forwards"]
        for row in r.tokens():
            key = tuple(int(x) for x in row)
            counts[key] = counts.get(key, 0) + 1
    n = batches * B
    keys = sorted(joint)
    exp = np.array([joint[x] for x in keys]) * n
    obs = np.array([counts.get(x, 0) for x in keys], dtype=np.float64)
    order = np.argsort(exp)
    exp, obs = exp[order], obs[order]
    cut = int(np.searchsorted(np.cumsum(exp), 8.0)) + 1
    e2 = np.concatenate([[exp[:cut].sum()], exp[cut:]])
    o2 = np.concatenate([[obs[:cut].sum()], obs[cut:]])
    assert stats.chisquare(o2, e2 * o2.sum() / e2.sum()).pvalue > 1e-3
    assert forwards < n * sh.T                                  # speculation still happened


@pytest.fixture(scope="module")
def micro_model():
    sh = synth.WORKLOADS["micro"].shape
    return sh, synth.make_weights(sh, 21, target_entropy=1.25, std=0.6)
