"""Component parity at one-layer depth: every kernel of decoder layer 0 on the GPU against the oracle's stage of
the same name, element by element, on IDENTICAL inputs -- each oracle stage is fed the GPU's own output of the
stage before it (the first stage starts from the embeddings, which are exact).  This is the direct check of the
RMSNorm kernel, the QKV + RoPE + paged-KV epilogue (incl. the cache rows written by chunked prefix pre-filling),
the ragged attention kernel, the residual epilogues and the SwiGLU epilogue, before bf16 rounding noise compounds
over the layers; the end-to-end logit comparison only bounds them loosely.

Unit of comparison.  bf16 buffers: the error in bf16 ulps of the oracle's value, where elements below their row's
rms are measured in the ulp of that rms (a sum carries the absolute error of its terms, which is set by the
row's scale).  fp32 residual stream: the error of the sub-block's update relative to the update's row rms.

Both sides round to bf16 at the same points (weights, normed operand, rotated q / k, v, attention output, SwiGLU
output); they differ in accumulation (fp32 tensor-core sums vs double), in exp / division approximations, and in
one place by construction: the attention kernel rounds the softmax weights to bf16 before the P.V product (the
oracle keeps them in double), a relative perturbation of 2^-9 per weight that averages to a fraction of an ulp of
the output.  The bounds below are what those differences can produce; dropping a single key of the longest
context exceeds them several times over (checked at the end of each case)."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2608_18183_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def ulp_bf16(x):
    """bf16 unit in the last place at the magnitude of x (8 significand bits)."""
    return np.exp2(np.floor(np.log2(np.maximum(np.abs(x), 1e-30))) - 7.0)


def round_bf16(x):
    """fp32 array rounded to bf16 (nearest even) and widened again."""
    return synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(np.ascontiguousarray(x, dtype=np.float32))).reshape(x.shape)


def err_in_ulps(g, o):
    """|g - o| in bf16 ulps of o, elements below their row's rms measured at that rms."""
    o64, g64 = o.astype(np.float64), g.astype(np.float64)
    rms = np.sqrt((o64 * o64).mean(axis=-1, keepdims=True))
    return np.abs(g64 - o64) / ulp_bf16(np.maximum(np.abs(o64), rms))


def update_err(g, o, x_in):
    """Error of a residual update (x_out - x_in) relative to the update's row rms."""
    yo = o.astype(np.float64) - x_in
    yg = g.astype(np.float64) - x_in
    rms = np.sqrt((yo * yo).mean(axis=-1, keepdims=True))
    return np.abs(yg - yo) / rms


def first_layer_model(s, weights):
    """The oracle on layer 0 alone: the weight image of a one-layer model cut out of the full image (same
    embeddings, layer 0, output norm and head), so that tracing layer 0 does not pay for the layers above it."""
    s1 = synth.ModelShape(1, s.dim, s.n_heads, s.ffn_hidden, s.vocab, s.grid_h, s.grid_w, s.n_classes, s.dtype,
                          s.rms_eps, s.rope_base)
    full, _ = synth.tensor_table(s)
    one, total = synth.tensor_table(s1)
    src = {name: (off, r * c * s.elem_bytes) for name, r, c, off in full}
    img = np.zeros(total, dtype=np.uint8)
    for name, r, c, off in one:
        o, nbytes = src[name]
        img[off:off + nbytes] = weights[o:o + nbytes]
    return O.Model(s1, img)


def run_case(w, ks, fold, seed=3):
    """GPU: init + chunked prefill + initial windows for prefix lengths `ks`, then layer 0 in two stages, with
    RMSNorm folded into the GEMM epilogues (fold) or as its own kernel.
    Oracle: the same prefill and the traced window forward per image and branch.  Returns per-buffer error
    arrays (concatenated over images and branches) and the pieces of the longest-context image."""
    s = w.shape
    B, T, W, D = len(ks), s.T, w.window, s.dim
    weights = G.weights_for(w)
    toks, _, lab = synth.make_inputs(w, seed=seed, batch=B)
    k = np.asarray(ks, dtype=np.int32)
    ctx = binding.Context(s, weights, B, W)
    ctx.hbsjd_debug_fold_norm(fold)
    ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab), G.gpu_params(w, seed, max_rounds=0,
                                                                      exec_mode=binding.EXEC_FULL))
    _, cur, seq, _, _ = ctx.hbsjd_get_state()
    np.testing.assert_array_equal(cur, k)
    nb = 2 if w.cfg_scale != 1.0 else 1
    gpu = {}
    # DBG_ACT_A: folded form, the bf16 copy of the residual stream; separate form, the normed operand
    for stage, names in ((0, (("hb_attn", binding.DBG_ACT_A), ("q", binding.DBG_ACT_Q), ("o", binding.DBG_ACT_O),
                              ("x_attn", binding.DBG_ACT_H), ("k", binding.DBG_KV_K), ("v", binding.DBG_KV_V))),
                         (1, (("hb_out", binding.DBG_ACT_A), ("act", binding.DBG_ACT_FFN),
                              ("x_out", binding.DBG_ACT_H)))):
        ctx.hbsjd_debug_forward(0, stage)
        for b in range(B):
            for br in range(nb):
                for name, what in names:
                    gpu[(name, b, br)] = ctx.hbsjd_debug_read(what, 2 * b + br)
    ctx.hbsjd_destroy()

    model = first_layer_model(s, weights)
    tok_emb = synth.read_tensor(s, weights, "tok_emb")
    cls_emb = synth.read_tensor(s, weights, "cls_emb")
    errs = {n: [] for n in ("q", "k", "v", "o", "x_attn", "act", "x_out") + (("hb_attn", "hb_out") if fold else
                                                                             ("a", "m"))}
    longest = None
    for b in range(B):
        c = int(k[b])
        n = min(W, T - c)
        if n <= 0:
            continue
        for br in range(nb):
            label = s.n_classes if br else int(lab[b])
            G_ = {name: gpu[(name, b, br)] for name in ("q", "k", "v", "o", "x_attn", "hb_attn", "act", "x_out",
                                                         "hb_out")}
            # the oracle's cache of layer 0 after chunked pre-filling of 0..c-1 and this window
            cache = model.new_cache()
            for pc in range(0, c, W):
                model.forward_window(cache, label, seq[b], pc, min(W, c - pc), want_logits=False)
            x_in = np.stack([cls_emb[label] if c + i == 0 else tok_emb[seq[b][c + i]] for i in range(n)])
            a, q, kk, vv = model.stage_qkv(0, x_in, c)
            cache[0][0][c:c + n], cache[1][0][c:c + n] = kk, vv
            errs["q"].append(err_in_ulps(G_["q"], q).reshape(-1))
            # cache rows 0 .. c+n-1: the prefix rows come from chunked pre-filling, the rest from this forward
            assert G_["k"].shape[0] == c + n and G_["v"].shape[0] == c + n
            errs["k"].append(err_in_ulps(G_["k"], cache[0][0][:c + n]).reshape(-1))
            errs["v"].append(err_in_ulps(G_["v"], cache[1][0][:c + n]).reshape(-1))
            # from here on every oracle stage reads the GPU's output of the stage before
            o = model.stage_attend(G_["q"], G_["k"], G_["v"], c)
            errs["o"].append(err_in_ulps(G_["o"], o).reshape(-1))
            x_attn = model.stage_attn_out(0, G_["o"], x_in)
            errs["x_attn"].append(update_err(G_["x_attn"], x_attn, x_in.astype(np.float64)).reshape(-1))
            m, act = model.stage_ffn_act(0, G_["x_attn"])
            errs["act"].append(err_in_ulps(G_["act"], act).reshape(-1))
            if fold:
                # the bf16 copy of the residual stream that the next projection reads is the rounding of the fp32 one
                errs["hb_attn"].append(np.abs(G_["hb_attn"] - round_bf16(G_["x_attn"])).reshape(-1))
            else:
                # at the stage-0 stop the operand buffer still holds the attention norm's output; the buffer read
                # at the stage-1 stop is the FFN norm's, which the oracle stage computed from the GPU's own rows
                errs["a"].append(err_in_ulps(G_["hb_attn"], a).reshape(-1))
                errs["m"].append(err_in_ulps(G_["hb_out"], m).reshape(-1))
            x_out = model.stage_ffn_down(0, G_["act"], G_["x_attn"])
            errs["x_out"].append(update_err(G_["x_out"], x_out, G_["x_attn"].astype(np.float64)).reshape(-1))
            if fold:
                errs["hb_out"].append(np.abs(G_["hb_out"] - round_bf16(G_["x_out"])).reshape(-1))
            if longest is None or c + n > longest["keys"]:
                longest = dict(keys=c + n, q=G_["q"], K=G_["k"], V=G_["v"], o=o, c=c, n=n)
    return {n: np.concatenate(v) for n, v in errs.items()}, longest


def one_key_dropped(case, dh):  # noqa: D401
    """Attention output of the last query of the longest context with its oldest cached key left out, head 0:
    the error that a block-edge bug of one key would cause, in the same units as err_in_ulps."""
    q = case["q"][-1, :dh].astype(np.float64)
    K = case["K"][:, :dh].astype(np.float64)
    V = case["V"][:, :dh].astype(np.float64)
    sc = K[1:] @ q / np.sqrt(dh)
    p = np.exp(sc - sc.max())
    o_drop = (p / p.sum()) @ V[1:]
    full = case["o"][-1].astype(np.float64)
    rms = np.sqrt((full * full).mean())
    ref = full[:dh]
    return float((np.abs(o_drop - ref) / ulp_bf16(np.maximum(np.abs(ref), rms))).max())


# (max error, 99.9th percentile) per buffer, in the units above.  Separate norm: the operands of the projections are
# the oracle's to the bit (a, m), so every product differs by summation order only.  Folded norm: the projections
# read bf16(x) instead of bf16(x r g) -- the same function, rounded at another point -- so q, k, v and the SwiGLU
# output carry an independent bf16 rounding of every operand element (a few tenths of an ulp of the row scale,
# more in the tails of the product of two such sums), while the attention kernel, the residual updates and the
# bf16 copy of the residual stream, fed identical inputs, stay as tight as before.
BOUNDS = {False: {"a": (1.0, 1.0), "m": (1.0, 1.0), "q": (2.0, 1.0), "k": (2.0, 1.0), "v": (2.0, 1.0), "o": (2.0, 1.0),
                  "act": (2.0, 1.0), "x_attn": (5e-5, 2e-5), "x_out": (5e-5, 2e-5)},
          True: {"q": (3.0, 2.0), "k": (3.0, 2.0), "v": (3.0, 2.0), "o": (2.0, 1.0), "act": (12.0, 4.0),
                 "x_attn": (5e-5, 2e-5), "x_out": (5e-5, 2e-5), "hb_attn": (0.0, 0.0), "hb_out": (0.0, 0.0)}}


def check(errs, longest, dh, label, fold):
    report = {n: (float(e.max()), float(np.quantile(e, 0.999)), float((e > 0).mean())) for n, e in errs.items()}
    print(label, "folded" if fold else "separate", {n: tuple(round(x, 3) for x in v) for n, v in report.items()},
          "keys", longest["keys"])
    for n, (mx, q999, _) in report.items():
        assert mx <= BOUNDS[fold][n][0] and q999 <= BOUNDS[fold][n][1], (label, fold, n, mx, q999)
    drop = one_key_dropped(longest, dh)
    print(label, "one key dropped:", round(drop, 1), "ulps")
    assert drop > 2 * BOUNDS[fold]["o"][0], drop


@pytest.mark.parametrize("fold", [False, True])
def test_layer0_small_bf16_windows_and_tails(fold):
    """Four heads of 64, T = 144 (three pages): windows 32 / 64 / 20, cursors on both sides of page and key-block
    boundaries, a chunk-prefilled prefix, the ragged tail n < W."""
    for W in (32, 64, 20):
        w = synth.with_shape(synth.WORKLOADS["small_bf16"], window=W)
        T = w.shape.T
        errs, longest = run_case(w, [0, 1, 31, 33, 63, 64, 65, 100, 127, 129, T - 5, T - 1], fold)
        check(errs, longest, w.shape.head_dim, f"small_bf16 W={W}", fold)


@pytest.mark.parametrize("fold", [False, True])
def test_layer0_head_size_32(fold):
    """Head size 32 (the plain attention kernel and the 16-pair RoPE table half)."""
    base = synth.WORKLOADS["small_bf16"]
    s = base.shape
    w = synth.with_shape(base, shape=synth.ModelShape(2, 256, 8, 512, 1024, 12, 12, 10, "bf16"), window=16)
    errs, longest = run_case(w, [0, 17, 64, 90, s.T - 3], fold)
    check(errs, longest, 32, "head 32", fold)


@pytest.mark.parametrize("fold", [False, True])
@pytest.mark.parametrize("name,ks", [("L", [0, 40, 70, 130, 200, 251]), ("XL", [0, 100, 300, 520, 571])])
def test_layer0_full_size_shapes(name, ks, fold):
    """The L (16 heads, dim 1024, T = 256) and XL (20 heads, dim 1280, T = 576, nine pages) decoders with guidance:
    cursors beyond one, two and (XL) eight pages, prefixes written by chunked pre-filling, the tail n < W."""
    w = synth.WORKLOADS[name]
    errs, longest = run_case(w, ks, fold)
    check(errs, longest, w.shape.head_dim, name, fold)
