"""hbsjd_verify_static -- the verification step for callers that are not allowed to allocate device memory
(their framework owns the whole device, or an allocation would stall a latency-critical loop).  It keeps its
scratch in a fixed array inside the library instead of a context's buffers.

The test calls it through the C ABI twice in a row on different inputs and checks every output against
hbsjd_verify (the context-backed entry point) on the same inputs: the kernels are the same, so integers must
be equal and probabilities equal to the last bit.  The second call finds the first call's leftovers in the
shared array, so it also checks that nothing stale leaks through.  This file sorts last on purpose."""
import numpy as np
import pytest

from paper_2608_18183_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _run(fn, case, desc):
    import torch
    B, W, V = case["B"], case["W"], case["V"]
    d = {k: G.dev(case[k]) for k in ("logits", "q", "cursor", "seq", "delta", "qbase")}
    p_out = torch.zeros((B, W, V), device="cuda")
    m_out = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    fn(desc, d["logits"], d["q"], p_out, d["cursor"], d["seq"], d["delta"], d["qbase"], m_out)
    torch.cuda.synchronize()
    return [x.cpu().numpy() for x in (p_out, d["cursor"], d["seq"], d["delta"], d["qbase"], m_out)]


def test_static_scratch_variant_matches_the_context_variant_twice_in_a_row():
    import torch
    w = synth.WORKLOADS["tiny_bf16"]
    ctx = binding.Context(w.shape, G.weights_for(w), 64, 16)
    stream = torch.cuda.current_stream()
    static = lambda *a: binding.hbsjd_verify_static(stream, *a)
    # two different problems back to back: the larger one first, so that the second call runs over leftovers
    cases = [(G.verify_case(11, B=48, W=16, T=64, V=2048, branches=2, cfg_scale=3.0, top_k=50), 5, 3),
             (G.verify_case(12, B=20, W=12, T=40, V=1024, sigma=0.8), 99, 0)]
    for case, seed, rnd in cases:
        desc = G.verify_desc(case, seed, rnd)
        got = _run(static, case, desc)
        ref = _run(ctx.hbsjd_verify, case, desc)
        names = ("p_out", "cursor", "seq", "delta", "qbase", "m_out")
        for name, a, b in zip(names, got, ref):
            np.testing.assert_array_equal(a, b, err_msg=name)
        assert (got[5][case["cursor"] < case["T"]] >= 1).all()  # something was committed for every live image
    ctx.hbsjd_destroy()


def test_static_scratch_variant_refuses_oversized_requests():
    import torch
    case = G.verify_case(1, B=4, W=8, T=16, V=64)
    stream = torch.cuda.current_stream()
    d = {k: G.dev(case[k]) for k in ("logits", "q", "cursor", "seq", "delta", "qbase")}
    p_out = torch.zeros((4, 8, 64), device="cuda")
    m_out = torch.zeros(4, dtype=torch.int32, device="cuda")
    for field, val in (("batch", 1025), ("window", 65), ("V", 32772), ("batch", 600)):
        desc = G.verify_desc(case, 1, 0)
        setattr(desc, field, val)
        if field == "batch" and val == 600:
            desc.window = 32  # 600 x 32 > 16384 (image, position) pairs
        with pytest.raises(binding.HbsjdError) as e:
            binding.hbsjd_verify_static(stream, desc, d["logits"], d["q"], p_out, d["cursor"], d["seq"], d["delta"],
                                        d["qbase"], m_out)
        assert e.value.code == -1
