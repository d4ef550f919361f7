"""Seeded synthetic workloads for the HB-SJD rollout path (numpy only).

This module holds data generation only: model shapes, random weight images,
prefix / label draws.  It contains none of the rollout method's arithmetic and
imports neither the CUDA binding nor the CPU oracle; both sides consume its
outputs as plain arrays.

The paper measures on ImageNet-trained LlamaGen students (Sec. 5.1,
"Experimental Setup"); neither the weights nor the data exist here, so these
workloads stand in for them with the same layer counts, widths, vocabulary,
token grids, batch sizes and prefix-length spreads (Tables 4-6, 8).

Weight image layout (one flat byte buffer, every tensor start aligned to 256
bytes, element type fp32 or bf16, matrices row-major [out, in]):

    tok_emb [V, D]
    cls_emb [C+1, D]          row C is the null class of the unconditional branch
    per layer l = 0..L-1:
        g_attn [D]
        w_qkv  [3D, D]        rows 0..D-1 = Wq, D..2D-1 = Wk, 2D..3D-1 = Wv
        w_o    [D, D]
        g_ffn  [D]
        w_13   [2F, D]        rows 0..F-1 = W1 (gate), F..2F-1 = W3 (up)
        w_2    [D, F]
    g_out  [D]
    w_head [V, D]
"""
from __future__ import annotations

import dataclasses
import numpy as np

ALIGN = 256


@dataclasses.dataclass(frozen=True)
class ModelShape:
    n_layers: int
    dim: int
    n_heads: int
    ffn_hidden: int
    vocab: int
    grid_h: int
    grid_w: int
    n_classes: int
    dtype: str  # "fp32" | "bf16"
    rms_eps: float = 1e-5
    rope_base: float = 10000.0

    @property
    def T(self) -> int:
        return self.grid_h * self.grid_w

    @property
    def head_dim(self) -> int:
        return self.dim // self.n_heads

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "fp32" else 2


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    shape: ModelShape
    batch: int
    window: int
    cfg_scale: float      # 1.0 = no classifier-free guidance
    top_k: int            # 0 = off
    temperature: float
    history_offset: int
    prefix: tuple         # ("const", k) | ("uniform", lo, hi) | ("bimodal", lo0, hi0, lo1, hi1)
    weight_seed: int = 1
    input_seed: int = 2


def _shape(L, D, Hh, F, V, g, C, dtype):
    return ModelShape(L, D, Hh, F, V, g, g, C, dtype)


WORKLOADS = {
    # the five configurations of the benchmark description; H defaults to the grid width
    "tiny": Workload("tiny", _shape(2, 64, 4, 192, 256, 8, 10, "fp32"), 4, 8, 1.0, 0, 1.0, 8, ("const", 0)),
    "B": Workload("B", _shape(12, 768, 12, 2048, 16384, 16, 1000, "bf16"), 64, 16, 1.0, 1000, 1.0, 16,
                  ("uniform", 0, 64)),
    "L": Workload("L", _shape(24, 1024, 16, 2816, 16384, 16, 1000, "bf16"), 128, 32, 4.0, 1000, 1.0, 16,
                  ("uniform", 0, 128)),
    "XL": Workload("XL", _shape(36, 1280, 20, 3456, 16384, 24, 1000, "bf16"), 64, 32, 4.0, 1000, 1.0, 24,
                   ("uniform", 0, 288)),
    "stress": Workload("stress", _shape(24, 1024, 16, 2816, 16384, 16, 1000, "bf16"), 256, 32, 4.0, 1000, 1.0,
                       16, ("bimodal", 0, 16, 192, 240)),
    # small shapes for tests: same structure, sizes the CPU oracle finishes quickly
    "tiny_bf16": Workload("tiny_bf16", _shape(2, 128, 2, 384, 512, 8, 10, "bf16"), 6, 8, 3.0, 50, 1.0, 8,
                          ("uniform", 0, 20)),
    "small_bf16": Workload("small_bf16", ModelShape(2, 256, 4, 512, 1024, 12, 12, 10, "bf16"), 6, 32, 2.0, 100, 1.0,
                           12, ("uniform", 0, 100)),
    "micro": Workload("micro", _shape(1, 16, 1, 32, 6, 2, 3, "fp32"), 1, 2, 1.0, 0, 1.0, 2, ("const", 0)),
}


def with_shape(w: Workload, **kw) -> Workload:
    return dataclasses.replace(w, **kw)


def tensor_table(s: ModelShape):
    """[(name, rows, cols, byte_offset)] in file order, and the total byte size."""
    out = []
    off = 0

    def add(name, r, c):
        nonlocal off
        out.append((name, r, c, off))
        nbytes = r * c * s.elem_bytes
        off += (nbytes + ALIGN - 1) // ALIGN * ALIGN

    D, F, V = s.dim, s.ffn_hidden, s.vocab
    add("tok_emb", V, D)
    add("cls_emb", s.n_classes + 1, D)
    for l in range(s.n_layers):
        add(f"l{l}.g_attn", 1, D)
        add(f"l{l}.w_qkv", 3 * D, D)
        add(f"l{l}.w_o", D, D)
        add(f"l{l}.g_ffn", 1, D)
        add(f"l{l}.w_13", 2 * F, D)
        add(f"l{l}.w_2", D, F)
    add("g_out", 1, D)
    add("w_head", V, D)
    return out, off


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _head_scale(w_head: np.ndarray, D: int, rng: np.random.Generator, target_nats: float) -> float:
    """Scalar a such that softmax(a * w_head @ g) has mean entropy `target_nats` over
    64 seeded unit-RMS Gaussian directions g (stand-ins for final-normed hiddens,
    whose RMS is 1 when the output gain is 1)."""
    g = rng.standard_normal((64, D))
    g /= np.sqrt((g * g).mean(axis=1, keepdims=True))
    base = g @ w_head.astype(np.float64).T  # [64, V]

    def mean_entropy(a):
        z = a * base
        z -= z.max(axis=1, keepdims=True)
        e = np.exp(z)
        p = e / e.sum(axis=1, keepdims=True)
        return float(-(p * np.log(np.maximum(p, 1e-300))).sum(axis=1).mean())

    lo, hi = 0.0, 1.0
    while mean_entropy(hi) > target_nats:
        hi *= 2.0
        if hi > 1e6:
            raise RuntimeError("entropy target unreachable")
    for _ in range(60):
        mid = 0.5 * (lo + hi)
        if mean_entropy(mid) > target_nats:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def make_weights(s: ModelShape, seed: int = 1, target_entropy: float = 3.0, std: float = 0.02) -> np.ndarray:
    """Flat weight image (uint8) for shape `s`: every matrix N(0, std) (0.02 in every benchmark
    workload), gains 1, LM head rescaled for a mean next-token entropy of about `target_entropy` nats."""
    table, total = tensor_table(s)
    img = np.zeros(total, dtype=np.uint8)
    rng = np.random.Generator(np.random.Philox(seed))
    for name, r, c, off in table:
        if name.endswith("g_attn") or name.endswith("g_ffn") or name == "g_out":
            t = np.ones((r, c), dtype=np.float32)
        else:
            t = (rng.standard_normal((r, c), dtype=np.float32) * np.float32(std)).astype(np.float32)
            if name == "w_head" and target_entropy is not None and target_entropy < np.log(s.vocab):
                a = _head_scale(t, s.dim, rng, target_entropy)
                t = (t.astype(np.float64) * a).astype(np.float32)
        nbytes = r * c * s.elem_bytes
        if s.dtype == "fp32":
            img[off:off + nbytes] = t.reshape(-1).view(np.uint8)
        else:
            img[off:off + nbytes] = f32_to_bf16_bits(t).reshape(-1).view(np.uint8)
    return img


def read_tensor(s: ModelShape, img: np.ndarray, name: str) -> np.ndarray:
    """Tensor `name` of a weight image widened to fp32 (for tests that restate the model)."""
    table, _ = tensor_table(s)
    for n, r, c, off in table:
        if n == name:
            nbytes = r * c * s.elem_bytes
            raw = img[off:off + nbytes]
            if s.dtype == "fp32":
                return raw.view(np.float32).reshape(r, c).copy()
            return bf16_bits_to_f32(raw.view(np.uint16)).reshape(r, c)
    raise KeyError(name)


def make_inputs(w: Workload, seed: int | None = None, batch: int | None = None):
    """(prefix_tokens int32[B,T], prefix_len int32[B], labels int32[B]) for workload `w`."""
    s = w.shape
    B = w.batch if batch is None else batch
    rng = np.random.Generator(np.random.Philox(w.input_seed if seed is None else seed))
    kind = w.prefix[0]
    if kind == "const":
        k = np.full(B, w.prefix[1], dtype=np.int32)
    elif kind == "uniform":
        k = rng.integers(w.prefix[1], w.prefix[2] + 1, size=B, dtype=np.int32)
    elif kind == "bimodal":
        half = B // 2
        a = rng.integers(w.prefix[1], w.prefix[2] + 1, size=half, dtype=np.int32)
        b = rng.integers(w.prefix[3], w.prefix[4] + 1, size=B - half, dtype=np.int32)
        k = np.concatenate([a, b])
        rng.shuffle(k)
    else:
        raise ValueError(kind)
    k = np.minimum(k, s.T).astype(np.int32)
    toks = rng.integers(0, s.vocab, size=(B, s.T), dtype=np.int32)
    labels = rng.integers(0, s.n_classes, size=B, dtype=np.int32)
    return toks, k, labels
