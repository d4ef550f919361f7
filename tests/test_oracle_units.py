"""Pins for the oracle's building blocks: the keyed generator, the probability
pipeline, the fixed-point sampler, and the accept / resample decision."""
import itertools
import os

import numpy as np
import pytest

from oracle import oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLD, "philox4x32_10_kat.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r if x != "->"]
        out = O.philox(v[0:4], v[4:6])
        assert [int(x) for x in out] == v[6:10]


def test_bf16_round_ties_to_even():
    # 1 + 2^-8 is exactly halfway between bf16 neighbours 1 and 1 + 2^-7: goes to even (1.0)
    assert O.bf16_round(1.0 + 2.0 ** -8) == 1.0
    assert O.bf16_round(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6
    assert O.bf16_round(1.0 + 2.0 ** -8 + 2.0 ** -20) == 1.0 + 2.0 ** -7
    assert O.bf16_round(-3.0) == -3.0


def test_probs_is_softmax_and_topk_keeps_ties():
    rng = np.random.default_rng(0)
    l = rng.normal(size=97).astype(np.float32) * 3
    p = O.probs(l)
    e = np.exp(l.astype(np.float64) - l.max())
    np.testing.assert_allclose(p, (e / e.sum()).astype(np.float32), rtol=1e-6, atol=0)
    assert abs(p.astype(np.float64).sum() - 1) < 1e-6
    # top-k without ties keeps exactly k
    for k in (1, 5, 96):
        pk = O.probs(l, k=k)
        assert (pk > 0).sum() == k
        kept = np.argsort(-l)[:k]
        assert set(np.nonzero(pk)[0]) == set(kept)
        ek = np.exp(l[kept].astype(np.float64) - l.max())
        np.testing.assert_allclose(pk[kept], ek / ek.sum(), rtol=1e-6)
    # k >= V and k == 0 mean "off"
    np.testing.assert_array_equal(O.probs(l, k=97), p)
    np.testing.assert_array_equal(O.probs(l, k=1000), p)
    # ties at the k-th value are all kept
    lt = np.array([3, 1, 2, 2, 2, 0], dtype=np.float32)
    assert (O.probs(lt, k=2) > 0).sum() == 4
    assert (O.probs(lt, k=4) > 0).sum() == 4
    assert (O.probs(lt, k=5) > 0).sum() == 5
    # temperature divides the logits
    np.testing.assert_allclose(O.probs(l, tau=0.5), O.probs((l.astype(np.float64) * 2).astype(np.float32)), rtol=2e-6,
                               atol=1e-12)


def test_probs_guidance_formula():
    rng = np.random.default_rng(1)
    lc = rng.normal(size=33).astype(np.float32)
    lu = rng.normal(size=33).astype(np.float32)
    for s in (0.0, 1.0, 2.0, 4.0):
        g = lu.astype(np.float64) + s * (lc.astype(np.float64) - lu)
        e = np.exp(g - g.max())
        np.testing.assert_allclose(O.probs(lc, lu, s=s), e / e.sum(), rtol=3e-6)
    # s = 1 with both branches given is the conditional distribution
    np.testing.assert_allclose(O.probs(lc, lu, s=1.0), O.probs(lc), rtol=2e-6)
    # identical branches: guidance has no effect, whatever the scale
    np.testing.assert_allclose(O.probs(lc, lc, s=4.0), O.probs(lc), rtol=2e-6)


def test_sampler_definition_by_brute_force():
    # every 32-bit word maps to the bin of its fixed-point target; check on a word lattice
    a = np.array([0.25, 0.0, 0.5, 0.125, 0.125], dtype=np.float32)
    w = np.floor(a.astype(np.float64) * 2 ** 30).astype(np.int64)
    S = int(w.sum())
    cum = np.cumsum(w)
    for word in list(range(0, 2 ** 32, 2 ** 32 // 997)) + [2 ** 32 - 1, 2 ** 30, 2 ** 30 - 1, 2 ** 31, 3 * 2 ** 30]:
        target = (word * S) >> 32
        assert O.sample(a, word) == int(np.searchsorted(cum, target, side="right"))
    # exact bin edges: the word range of bin v is [ceil(cum[v-1] 2^32 / S), ceil(cum[v] 2^32 / S))
    assert O.sample(a, 2 ** 30 - 1) == 0 and O.sample(a, 2 ** 30) == 2
    assert O.sample(a, 3 * 2 ** 30 - 1) == 2 and O.sample(a, 3 * 2 ** 30) == 3
    # zero total weight is reported, a zero-weight bin is never returned
    assert O.sample(np.zeros(4, dtype=np.float32), 12345) == -1
    assert all(O.sample(a, wd) != 1 for wd in range(0, 2 ** 32, 2 ** 32 // 4099))


def test_sampler_frequencies_match_weights():
    rng = np.random.default_rng(3)
    a = rng.random(7).astype(np.float32)
    a /= a.sum()
    N = 1 << 16
    counts = np.zeros(7)
    for i in range(N):
        counts[O.sample(a, (i << 16) + 0x8000)] += 1
    np.testing.assert_allclose(counts / N, a, atol=2.0 / N * 7 + 1e-6)


def _decide_once(V, p, q, z, is_delta, w0, w1, n=2, W=2, T=4, c=0, greedy=False):
    """Two-input window (anchor + one draft z at position c+1).  Returns the token committed at c+1."""
    seq = np.zeros(T + 1, dtype=np.int32)
    delta = np.zeros(T + 1, dtype=np.uint8)
    seq[c + 1] = z
    delta[c + 1] = 1 if is_delta else 0
    pp = np.stack([p, p]).astype(np.float32)  # p_0 (verifies z) and p_1 (bonus)
    qprev = np.stack([q, q]).astype(np.float32)
    words = np.zeros((n, 4), dtype=np.uint32)
    words[0, 0] = w0
    words[0, 1] = w1
    words[1, 1] = w1
    nc, m, j = O.decide(V, T, W, 2, greedy, c, seq, delta, pp, qprev, c, words, np.zeros(W, dtype=np.uint32))
    assert nc == c + m and m == (1 if j == 0 else 2)
    return int(seq[c + 1]), j


@pytest.mark.parametrize("V", [3, 5, 8])
def test_accept_resample_identity_by_enumeration(V):
    """Eq. 5 with residual resampling leaves the target distribution unchanged:
    sum_z q(z) [ min(1, p(z)/q(z)) 1{v=z} + (1 - min(1, p(z)/q(z))) r(v) ] = p(v),
    r = [p-q]+ / |[p-q]+|.  Checked by enumerating the draft z, a lattice of the
    accept uniform and a lattice of the resampling word through the oracle's decision."""
    rng = np.random.default_rng(V)
    p = rng.random(V) ** 2
    q = rng.random(V) ** 2
    p /= p.sum()
    q /= q.sum()
    p = p.astype(np.float32)
    q = q.astype(np.float32)
    NU, NW = 256, 256
    out = np.zeros(V)
    for z in range(V):
        for iu in range(NU):
            w0 = ((iu << 24) // NU + (1 << 23) // NU) << 8  # u = (iu + 0.5)/NU on the 24-bit lattice
            tok, j = _decide_once(V, p, q, z, False, w0, 0)
            if j < 0:
                assert tok == z
                out[z] += q[z] / NU
            else:
                for iw in range(NW):
                    tok, _ = _decide_once(V, p, q, z, False, w0, ((iw << 32) // NW + (1 << 31) // NW))
                    out[tok] += q[z] / NU / NW
    np.testing.assert_allclose(out, p, atol=2.5 / NU)


def test_accept_rule_special_cases():
    V = 6
    rng = np.random.default_rng(9)
    p = rng.random(V).astype(np.float32)
    p /= p.sum()
    top = 0xFFFFFF00  # u = 1 - 2^-24
    for z in range(V):
        # p == q: always accepted, even at the largest uniform
        assert _decide_once(V, p, p, z, False, top, 0)[1] == -1
        # point-mass proposal: accepted iff u < p(z)
        u_lo = int(np.floor(float(p[z]) * 2 ** 24)) - 1
        assert _decide_once(V, p, p, z, True, max(u_lo, 0) << 8, 0)[1] == -1
        assert _decide_once(V, p, p, z, True, (u_lo + 2) << 8, 0)[1] == 0
        # ... and a rejected point-mass draft is never resampled to itself
        for w1 in range(0, 2 ** 32, 2 ** 32 // 64):
            tok, j = _decide_once(V, p, p, z, True, top, w1)
            assert j == 0 and tok != z
    # u = 0 accepts whenever alpha > 0; alpha = 0 (p(z) = 0) always rejects
    pz = p.copy()
    pz[2] = 0
    assert _decide_once(V, pz, p, 2, False, 0, 0)[1] == 0
    assert _decide_once(V, p, p, 2, False, 0, 0)[1] == -1


def test_point_mass_proposal_identity():
    """Deterministic (history) draft z: accept with p(z), else sample p with z removed -> marginal p."""
    V = 5
    rng = np.random.default_rng(4)
    p = rng.random(V).astype(np.float32)
    p /= p.sum()
    NU, NW = 128, 128
    for z in range(V):
        out = np.zeros(V)
        for iu in range(NU):
            w0 = ((iu << 24) // NU + (1 << 23) // NU) << 8
            tok, j = _decide_once(V, p, p, z, True, w0, 0)
            if j < 0:
                out[z] += 1.0 / NU
            else:
                for iw in range(NW):
                    tok, _ = _decide_once(V, p, p, z, True, w0, ((iw << 32) // NW + (1 << 31) // NW))
                    out[tok] += 1.0 / NU / NW
        np.testing.assert_allclose(out, p, atol=2.5 / NU)


def test_greedy_decision():
    V = 4
    p = np.array([0.1, 0.4, 0.4, 0.1], dtype=np.float32)  # tie: lowest index wins
    assert _decide_once(V, p, p, 1, False, 0, 0, greedy=True) == (1, -1)
    assert _decide_once(V, p, p, 2, False, 0, 0, greedy=True) == (1, 0)
