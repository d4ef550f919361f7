"""An independent fp64 restatement of the decoder forward with torch CPU library
ops (matmul, softmax, complex multiplication for the rotary embedding).  It shares
no code with the C++ oracle or with the CUDA library; tests use it to pin the
oracle's forward."""
import numpy as np
import torch

from paper_2608_18183_b200 import synth


def load(shape, img):
    g = lambda n: torch.from_numpy(synth.read_tensor(shape, img, n).astype(np.float64))
    P = dict(tok=g("tok_emb"), cls=g("cls_emb"), g_out=g("g_out")[0], head=g("w_head"), layers=[])
    for l in range(shape.n_layers):
        P["layers"].append(dict(g_attn=g(f"l{l}.g_attn")[0], qkv=g(f"l{l}.w_qkv"), o=g(f"l{l}.w_o"),
                                g_ffn=g(f"l{l}.g_ffn")[0], w13=g(f"l{l}.w_13"), w2=g(f"l{l}.w_2")))
    return P


def _norm(x, g, eps):
    return x * torch.rsqrt((x * x).mean(-1, keepdim=True) + eps) * g


def _rope_factors(shape, n):
    dh = shape.head_dim
    quarter = dh // 4
    idx = torch.arange(n)
    row = torch.where(idx > 0, (idx - 1) // shape.grid_w, torch.zeros_like(idx)).double()
    col = torch.where(idx > 0, (idx - 1) % shape.grid_w, torch.zeros_like(idx)).double()
    freq = torch.tensor(shape.rope_base, dtype=torch.float64) ** (-torch.arange(quarter).double() / quarter)
    ang = torch.cat([row[:, None] * freq[None, :], col[:, None] * freq[None, :]], dim=1)  # [n, dh/2]
    ang[0] = 0.0
    return torch.polar(torch.ones_like(ang), ang)  # e^{i ang}


BF16_POINTS = ("norm", "q", "k", "v", "o", "act")


def _bf16(t):
    """double -> float -> bfloat16 (round to nearest even) -> double, with torch's own casts."""
    return t.to(torch.float32).to(torch.bfloat16).to(torch.float64)


def forward(shape, P, label, seq, bf16_points=()):
    """seq: int array [n], seq[0] ignored.  Returns fp64 logits [n, V].  bf16_points: the activations that are
    rounded to bf16 -- any of "norm" (every RMSNorm output), "q", "k" (after the rotation), "v", "o" (attention
    output), "act" (SwiGLU output); extra names "resid" (the residual stream) and "gu" (gate / up pre-activations)
    exist so that a test can show that rounding at a point that is NOT on the list is detected."""
    r = lambda name, t: _bf16(t) if name in bf16_points else t
    n = len(seq)
    Hh, dh, D = shape.n_heads, shape.head_dim, shape.dim
    x = torch.cat([P["cls"][label][None, :], P["tok"][torch.as_tensor(np.asarray(seq[1:], dtype=np.int64))]], 0)
    rot = _rope_factors(shape, n)[:, None, :]  # [n,1,dh/2]
    mask = torch.full((n, n), float("-inf"), dtype=torch.float64).triu(1)
    for Ly in P["layers"]:
        a = r("norm", _norm(x, Ly["g_attn"], shape.rms_eps))
        qkv = a @ Ly["qkv"].T
        q, k, v = [t.reshape(n, Hh, dh) for t in qkv.split(D, dim=1)]
        qc = torch.view_as_real(torch.view_as_complex(q.reshape(n, Hh, dh // 2, 2).contiguous()) * rot).reshape(n, Hh, dh)
        kc = torch.view_as_real(torch.view_as_complex(k.reshape(n, Hh, dh // 2, 2).contiguous()) * rot).reshape(n, Hh, dh)
        qc, kc, v = r("q", qc), r("k", kc), r("v", v)
        sc = torch.einsum("ihd,jhd->hij", qc, kc) / np.sqrt(dh) + mask[None]
        o = r("o", torch.einsum("hij,jhd->ihd", torch.softmax(sc, -1), v).reshape(n, D))
        x = r("resid", x + o @ Ly["o"].T)
        m = r("norm", _norm(x, Ly["g_ffn"], shape.rms_eps))
        gu = r("gu", m @ Ly["w13"].T)
        F = shape.ffn_hidden
        x = r("resid", x + r("act", torch.nn.functional.silu(gu[:, :F]) * gu[:, F:]) @ Ly["w2"].T)
    return (r("norm", _norm(x, P["g_out"], shape.rms_eps)) @ P["head"].T).numpy()
