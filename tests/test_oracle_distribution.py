"""Distributional pin: probabilistic SJD rollouts are distributed exactly as AR sampling (Eq. 1 / Eq. 2).

The exact joint over all V^T sequences is enumerated with the independent torch restatement of
the forward; the oracle's rollouts (one image index per sample, so each has its own keyed random
stream) are compared against it with a chi-square goodness-of-fit test."""
import itertools

import numpy as np
import pytest
from scipy import stats

from oracle import oracle as O
from paper_2608_18183_b200 import synth
from tests import torch_restatement as TR

N = 200_000


@pytest.fixture(scope="module")
def micro():
    sh = synth.WORKLOADS["micro"].shape  # 1 layer, D=16, V=6, T=2x2
    img = synth.make_weights(sh, 21, target_entropy=1.25, std=0.6)  # strong context dependence
    return sh, img


def _softmax(l):
    e = np.exp(l - l.max())
    return e / e.sum()


def _exact_joint(sh, img, label, cfg, prefix):
    """P(x_{k+1..T} | prefix) for every completion, from the restated forward."""
    P = TR.load(sh, img)
    V, T, k = sh.vocab, sh.T, len(prefix)
    joint = {}
    cond = {}
    for comp in itertools.product(range(V), repeat=T - k):
        seq = [0] + list(prefix) + list(comp)
        lc = TR.forward(sh, P, label, seq[:T])
        lg = lc if cfg == 1.0 else None
        if lg is None:
            lu = TR.forward(sh, P, sh.n_classes, seq[:T])
            lg = lu + cfg * (lc - lu)
        pr = 1.0
        for t in range(k + 1, T + 1):
            pt = _softmax(lg[t - 1])
            cond[tuple(seq[1:t])] = pt
            pr *= pt[seq[t]]
        joint[comp] = pr
    return joint, cond


def _chi2(counts, joint):
    keys = sorted(joint)
    exp = np.array([joint[k] for k in keys]) * N
    obs = np.array([counts.get(k, 0) for k in keys], dtype=np.float64)
    order = np.argsort(exp)
    exp, obs = exp[order], obs[order]
    # merge the smallest cells until each expectation is >= 8
    cut = int(np.searchsorted(np.cumsum(exp), 8.0)) + 1
    e2 = np.concatenate([[exp[:cut].sum()], exp[cut:]])
    o2 = np.concatenate([[obs[:cut].sum()], obs[cut:]])
    e2 *= o2.sum() / e2.sum()
    return stats.chisquare(o2, e2).pvalue


def _rollouts(sh, img, label, cfg, prefix, W, H, seed):
    m = O.Model(sh, img)
    k = len(prefix)
    toks = np.zeros((N, sh.T), dtype=np.int32)
    toks[:, :k] = prefix
    P = O.make_params(W, H, cfg_scale=cfg, seed=seed)
    r = O.Rollout(m, toks, np.full(N, k, dtype=np.int32), np.full(N, label, dtype=np.int32), P)
    r.run()
    out = r.tokens()
    assert (out[:, :k] == np.asarray(prefix, dtype=np.int32)).all()
    vals, cnt = np.unique(out[:, k:], axis=0, return_counts=True)
    return {tuple(int(x) for x in v): int(c) for v, c in zip(vals, cnt)}, r.stats()


def test_model_is_context_sensitive(micro):
    sh, img = micro
    joint, cond = _exact_joint(sh, img, 1, 1.0, ())
    tv = max(0.5 * np.abs(cond[(a,)] - cond[(b,)]).sum() for a in range(6) for b in range(6))
    assert tv > 0.25  # a wrong context or a wrong position would be visible in the joint
    assert abs(sum(joint.values()) - 1) < 1e-9


@pytest.mark.parametrize("W,H,cfg,prefix,seed", [
    (2, 2, 1.0, (), 1), (3, 2, 1.0, (), 2), (4, 2, 1.0, (), 3), (4, 1, 1.0, (), 4),
    (3, 2, 2.0, (), 5), (4, 3, 1.0, (4,), 6), (1, 2, 1.0, (), 7)])
def test_sjd_rollouts_follow_the_ar_joint(micro, W, H, cfg, prefix, seed):
    sh, img = micro
    joint, _ = _exact_joint(sh, img, 1, cfg, prefix)
    counts, st = _rollouts(sh, img, 1, cfg, prefix, W, H, seed)
    p = _chi2(counts, joint)
    assert p > 1e-3, p
    if W > 1:  # speculation happened: some rounds committed several tokens, some rejected
        assert st["image_forwards"] < N * (sh.T - len(prefix)) and st["rejects"] > 0


def test_chi_square_detects_a_wrong_sampler(micro):
    """Sensitivity of the test above: rollouts at another guidance scale fail against the joint."""
    sh, img = micro
    joint, _ = _exact_joint(sh, img, 1, 1.0, ())
    counts, _ = _rollouts(sh, img, 1, 1.15, (), 3, 2, 8)
    assert _chi2(counts, joint) < 1e-6
