"""The verification kernels (probabilities, accept test, residual resampling, commit, refresh) on synthetic
proposal / target pairs with a paper-like reject rate, replayed by the oracle on the GPU's own probabilities:
bit-exact."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2608_18183_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    w = synth.WORKLOADS["tiny_bf16"]
    c = binding.Context(w.shape, G.weights_for(w), 32, 16)
    yield c
    c.hbsjd_destroy()


@pytest.mark.parametrize("greedy,branches,top_k,sigma", [(False, 1, 0, 0.6), (False, 2, 100, 0.4), (True, 1, 0, 0.6),
                                                         (False, 1, 0, 0.0)])
def test_verify_step_is_bit_exact_against_the_oracle(ctx, greedy, branches, top_k, sigma):
    case = G.verify_case(3, branches=branches, cfg_scale=2.0 if branches == 2 else 1.0, top_k=top_k, sigma=sigma)
    B, W, T, V, H = (case[k] for k in "BWTVH")
    seed, rnd = 0x1234567890, 7
    d = {k: G.dev(case[k]) for k in ("logits", "q", "cursor", "seq", "delta", "qbase")}
    import torch
    p_out = torch.zeros((B, W, V), device="cuda")
    m_out = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    ctx.hbsjd_verify(G.verify_desc(case, seed, rnd, greedy), d["logits"], d["q"], p_out, d["cursor"], d["seq"],
                     d["delta"], d["qbase"], m_out)
    p = p_out.cpu().numpy()
    cur2, seq2, dl2, qb2 = (d[k].cpu().numpy() for k in ("cursor", "seq", "delta", "qbase"))
    m = m_out.cpu().numpy()
    rejects = tested = 0
    for b in range(B):
        c = int(case["cursor"][b])
        if c >= T:
            assert m[b] == -1 and cur2[b] == T and np.array_equal(seq2[b], case["seq"][b])
            continue
        n = min(W, T - c)
        # probabilities against the oracle's pipeline on the same logits
        for i in range(n):
            ref = O.probs(case["logits"][0, b, i], case["logits"][1, b, i] if branches == 2 else None,
                          s=case["cfg_scale"], k=top_k)
            assert np.all(np.abs(p[b, i] - ref) <= 1e-6 + 1e-5 * ref)
        # decision replayed on the GPU's probabilities
        s2, d2 = case["seq"][b].copy(), case["delta"][b].copy()
        nc, mm, jj = O.replay_round(V, T, W, H, greedy, seed, b, rnd, c, s2, d2, p[b, :n], case["q"][b],
                                    int(case["qbase"][b]))
        assert nc == cur2[b] and mm == m[b] and qb2[b] == c
        np.testing.assert_array_equal(s2, seq2[b])
        np.testing.assert_array_equal(d2[nc + 1:nc + W], dl2[b][nc + 1:nc + W])
        rejects += jj >= 0
        tested += n > 1
    live = case["cursor"] < T
    if not greedy:
        # a real mix: rejections happened, and accepted drafts too (more than one token per window on average)
        assert rejects > 0 and m[live].mean() > 1.5, (rejects, m[live].mean())


def test_verify_rejects_bad_arguments(ctx):
    import torch
    case = G.verify_case(1, B=4, W=8, T=16, V=64)
    d = {k: G.dev(case[k]) for k in ("logits", "q", "cursor", "seq", "delta", "qbase")}
    p_out = torch.zeros((4, 8, 64), device="cuda")
    m_out = torch.zeros(4, dtype=torch.int32, device="cuda")
    for field, val in (("batch", 33), ("window", 17), ("V", 66), ("branches", 3), ("temperature", 0.0)):
        desc = G.verify_desc(case, 1, 0)
        setattr(desc, field, val)
        with pytest.raises(binding.HbsjdError) as e:
            ctx.hbsjd_verify(desc, d["logits"], d["q"], p_out, d["cursor"], d["seq"], d["delta"], d["qbase"], m_out)
        assert e.value.code == -1


@pytest.mark.parametrize("what", ["token_high", "token_negative", "cursor_negative", "cursor_high", "qbase", "cfg_nan"])
def test_verify_reports_invalid_state_arrays_instead_of_touching_memory(ctx, what):
    """The state arrays of hbsjd_verify live on the device and cannot be checked on the host before the launch:
    the kernels bound every index they derive from them.  A draft token outside the vocabulary, a cursor outside
    0..T or a proposal row outside the window is recorded, its access skipped, and the call returns
    HBSJD_EINVAL; the context stays usable."""
    import torch
    case = G.verify_case(5, B=8, W=8, T=32, V=256)
    b = 4
    c = int(case["cursor"][b])
    assert c + 2 < case["T"]
    case["delta"][b, c + 1] = 0  # a sampled draft: its proposal row is read
    if what == "token_high":
        case["seq"][b, c + 1] = case["V"] + 5
    elif what == "token_negative":
        case["seq"][b, c + 1] = -3
    elif what == "cursor_negative":
        case["cursor"][b] = -2
    elif what == "cursor_high":
        case["cursor"][b] = case["T"] + 7
    elif what == "qbase":
        case["qbase"][b] = c - 200  # row t - qbase - 1 far outside the window
    desc = G.verify_desc(case, 1, 0)
    if what == "cfg_nan":
        desc.cfg_scale = float("nan")
    d = {k: G.dev(case[k]) for k in ("logits", "q", "cursor", "seq", "delta", "qbase")}
    p_out = torch.zeros((8, 8, 256), device="cuda")
    m_out = torch.zeros(8, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()
    for call in (lambda: ctx.hbsjd_verify(desc, d["logits"], d["q"], p_out, d["cursor"], d["seq"], d["delta"],
                                          d["qbase"], m_out),
                 lambda: binding.hbsjd_verify_static(stream, desc, d["logits"], d["q"], p_out, d["cursor"], d["seq"],
                                                     d["delta"], d["qbase"], m_out)):
        for k in ("cursor", "seq", "delta", "qbase"):
            d[k].copy_(G.dev(case[k]))
        with pytest.raises(binding.HbsjdError) as e:
            call()
        assert e.value.code == -1
    torch.cuda.synchronize()
    # a valid call right after succeeds
    good = G.verify_case(6, B=8, W=8, T=32, V=256)
    dg = {k: G.dev(good[k]) for k in ("logits", "q", "cursor", "seq", "delta", "qbase")}
    ctx.hbsjd_verify(G.verify_desc(good, 1, 0), dg["logits"], dg["q"], p_out, dg["cursor"], dg["seq"], dg["delta"],
                     dg["qbase"], m_out)
    assert int(m_out.cpu().numpy()[good["cursor"] < good["T"]].min()) >= 1
