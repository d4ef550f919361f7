"""ctypes front end of the CPU oracle (oracle/hbsjd_oracle.cpp).

TEST INFRASTRUCTURE: imported only by tests/, the smoke check and the
benchmark's cpu_baseline / reference legs.  Never imported by the product
package, and it imports nothing from the CUDA binding.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hbsjd_oracle.cpp")
_LIB = os.path.join(_HERE, "liborc.so")


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", _SRC, "-o", _LIB]
        subprocess.run(cmd, check=True)
    return _LIB


class Desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("L", "D", "Hh", "F", "V", "gh", "gw", "C", "dtype")] + [
        ("eps", C.c_float), ("rope_base", C.c_float)]


class Params(C.Structure):
    _fields_ = [("window", C.c_int32), ("history", C.c_int32), ("top_k", C.c_int32), ("verify_mode", C.c_int32),
                ("exec_mode", C.c_int32), ("gamma", C.c_int32), ("cfg_scale", C.c_float),
                ("temperature", C.c_float), ("seed", C.c_uint64)]


class Trace(C.Structure):
    _fields_ = [("layer", C.c_int32)] + [(n, C.POINTER(C.c_float)) for n in
                                         ("a", "q", "k", "v", "o", "x_attn", "m", "act", "x_out")]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, i32p, u32p, u8p, f32p = C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_uint32), C.POINTER(
            C.c_uint8), C.POINTER(C.c_float)
        L.orc_philox.argtypes = [u32p, u32p, u32p]
        L.orc_bf16_round.argtypes = [C.c_float]
        L.orc_bf16_round.restype = C.c_float
        L.orc_model_create.argtypes = [C.POINTER(Desc), vp, C.c_size_t, C.c_int]
        L.orc_model_create.restype = vp
        L.orc_model_destroy.argtypes = [vp]
        L.orc_forward_full.argtypes = [vp, C.c_int, i32p, C.c_int, f32p]
        L.orc_forward_window.argtypes = [vp, f32p, f32p, C.c_int, i32p, C.c_int, C.c_int, f32p]
        L.orc_forward_window_trace.argtypes = [vp, f32p, f32p, C.c_int, i32p, C.c_int, C.c_int, f32p,
                                               C.POINTER(Trace)]
        L.orc_model_set_diag.argtypes = [vp, C.c_int, C.c_int, C.c_int]
        L.orc_stage_qkv.argtypes = [vp, C.c_int, f32p, C.c_int, C.c_int, f32p, f32p]
        L.orc_stage_attend.argtypes = [vp, f32p, f32p, f32p, C.c_int, C.c_int, f32p]
        L.orc_stage_attn_out.argtypes = [vp, C.c_int, f32p, C.c_int, f32p]
        L.orc_stage_ffn_act.argtypes = [vp, C.c_int, f32p, C.c_int, f32p, f32p]
        L.orc_stage_ffn_down.argtypes = [vp, C.c_int, f32p, C.c_int, f32p]
        L.orc_probs.argtypes = [f32p, f32p, C.c_float, C.c_float, C.c_int, C.c_int, f32p]
        L.orc_sample.argtypes = [f32p, C.c_int, C.c_uint32]
        L.orc_sample.restype = C.c_int
        L.orc_decide.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, i32p, i32p, u8p, f32p, C.c_int, f32p,
                                 C.c_int, u32p, u32p, i32p]
        L.orc_decide.restype = C.c_int
        L.orc_replay_round.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_uint64, C.c_int, C.c_uint32,
                                       i32p, i32p, u8p, f32p, f32p, C.c_int, i32p, C.c_int]
        L.orc_replay_round.restype = C.c_int
        L.orc_rollout_create.argtypes = [vp, C.c_int, i32p, i32p, i32p, i32p, C.POINTER(Params)]
        L.orc_rollout_create.restype = vp
        L.orc_rollout_destroy.argtypes = [vp]
        L.orc_rollout_live.argtypes = [vp]
        L.orc_rollout_round.argtypes = [vp, i32p, i32p]
        L.orc_rollout_run.argtypes = [vp, C.c_int]
        L.orc_rollout_tokens.argtypes = [vp, i32p]
        L.orc_rollout_get_state.argtypes = [vp, i32p, i32p, u8p, i32p]
        L.orc_rollout_probs.argtypes = [vp, C.c_int, f32p]
        L.orc_rollout_logits.argtypes = [vp, C.c_int, C.c_int, f32p]
        L.orc_rollout_stats.argtypes = [vp, C.POINTER(C.c_int64), i32p, i32p, C.c_int]
        L.orc_ar_rollout.argtypes = [vp, C.c_int, i32p, i32p, i32p, i32p, C.POINTER(Params), i32p]
        L.orc_bikl.argtypes = [f32p, f32p, C.c_int, C.c_int, C.POINTER(C.c_double)]
        L.orc_score.argtypes = [vp, vp, C.c_int, i32p, i32p, i32p, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                C.POINTER(C.c_double)]
        L.orc_num_threads.restype = C.c_int
        _lib = L
    return _lib


def _p(a, t):
    return None if a is None else a.ctypes.data_as(C.POINTER(t))


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def philox(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    o = np.zeros(4, dtype=np.uint32)
    lib().orc_philox(_p(c, C.c_uint32), _p(k, C.c_uint32), _p(o, C.c_uint32))
    return o


def bf16_round(x: float) -> float:
    return float(lib().orc_bf16_round(C.c_float(x)))


def probs(lc, lu=None, s=1.0, tau=1.0, k=0):
    lc = np.ascontiguousarray(lc, dtype=np.float32)
    lu = None if lu is None else np.ascontiguousarray(lu, dtype=np.float32)
    p = np.zeros_like(lc)
    lib().orc_probs(_p(lc, C.c_float), _p(lu, C.c_float), s, tau, k, lc.shape[-1], _p(p, C.c_float))
    return p


def sample(a, word: int) -> int:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return int(lib().orc_sample(_p(a, C.c_float), a.shape[0], C.c_uint32(word)))


def make_params(window, history, cfg_scale=1.0, temperature=1.0, top_k=0, greedy=False, exec_mode=0, gamma=0,
                seed=0) -> Params:
    return Params(window, history, top_k, 1 if greedy else 0, exec_mode, gamma, cfg_scale, temperature, seed)


def decide(V, T, W, H, greedy, c, seq, delta, p, qprev, qbase, words, w3_beyond):
    """One image's verify / commit / refresh on given probabilities and words.
    seq, delta are modified in place.  Returns (new_cursor, m, j)."""
    n = p.shape[0]
    cc = C.c_int32(c)
    j = C.c_int32(-1)
    p = np.ascontiguousarray(p, dtype=np.float32)
    qprev = np.ascontiguousarray(qprev, dtype=np.float32)
    words = np.ascontiguousarray(words, dtype=np.uint32)
    w3 = np.ascontiguousarray(w3_beyond, dtype=np.uint32)
    assert seq.dtype == np.int32 and delta.dtype == np.uint8 and w3.shape[0] >= W
    m = lib().orc_decide(V, T, W, H, int(greedy), C.byref(cc), _p(seq, C.c_int32), _p(delta, C.c_uint8),
                         _p(p, C.c_float), n, _p(qprev, C.c_float), qbase, _p(words, C.c_uint32),
                         _p(w3, C.c_uint32), C.byref(j))
    return cc.value, m, j.value


def replay_round(V, T, W, H, greedy, seed, image_id, rnd, c, seq, delta, p, qprev, qbase, m_limit=0):
    """As decide(), words drawn from the keyed generator.  m_limit > 0: commit at most that many tokens
    (batch-synchronous progress).  Returns (new_cursor, m, j)."""
    cc = C.c_int32(c)
    j = C.c_int32(-1)
    p = np.ascontiguousarray(p, dtype=np.float32)
    qprev = np.ascontiguousarray(qprev, dtype=np.float32)
    assert seq.dtype == np.int32 and delta.dtype == np.uint8
    m = lib().orc_replay_round(V, T, W, H, int(greedy), C.c_uint64(seed), image_id, C.c_uint32(rnd), C.byref(cc),
                               _p(seq, C.c_int32), _p(delta, C.c_uint8), _p(p, C.c_float), _p(qprev, C.c_float),
                               qbase, C.byref(j), int(m_limit))
    return cc.value, m, j.value


def bikl(s, t) -> np.ndarray:
    """Eq. 3's divergence per row: D_biKL(softmax(s), softmax(t)) for fp32 logits [rows, V] -> float64 [rows]."""
    s = np.ascontiguousarray(np.atleast_2d(s), dtype=np.float32)
    t = np.ascontiguousarray(np.atleast_2d(t), dtype=np.float32)
    assert s.shape == t.shape
    out = np.zeros(s.shape[0], dtype=np.float64)
    lib().orc_bikl(_p(s, C.c_float), _p(t, C.c_float), s.shape[0], s.shape[1], _p(out, C.c_double))
    return out


def score(student: "Model", teacher: "Model", tokens, prefix_len, labels):
    """Eq. 3 on completed trajectories.  Returns (pos float64 [B, T], per_image float64 [B], loss)."""
    tk, pl, lb = _i32(tokens), _i32(prefix_len), _i32(labels)
    assert student.shape.T == teacher.shape.T and student.shape.vocab == teacher.shape.vocab
    B, T = tk.shape
    pos = np.zeros((B, T), dtype=np.float64)
    per = np.zeros(B, dtype=np.float64)
    loss = C.c_double(0.0)
    lib().orc_score(student.h, teacher.h, B, _p(tk, C.c_int32), _p(pl, C.c_int32), _p(lb, C.c_int32),
                    _p(pos, C.c_double), _p(per, C.c_double), C.byref(loss))
    return pos, per, loss.value


class Model:
    """The decoder of the rollout, loaded from a flat weight image (see the synthetic
    workload module for the layout).  act_bf16 defaults to the image's dtype."""

    def __init__(self, shape, weights: np.ndarray, act_bf16: bool | None = None):
        self.shape = shape
        self.desc = Desc(shape.n_layers, shape.dim, shape.n_heads, shape.ffn_hidden, shape.vocab, shape.grid_h,
                         shape.grid_w, shape.n_classes, 0 if shape.dtype == "fp32" else 1, shape.rms_eps,
                         shape.rope_base)
        w = np.ascontiguousarray(weights, dtype=np.uint8)
        if act_bf16 is None:
            act_bf16 = shape.dtype == "bf16"
        self.h = lib().orc_model_create(C.byref(self.desc), w.ctypes.data, w.nbytes, int(act_bf16))
        if not self.h:
            raise RuntimeError("orc_model_create failed")

    def __del__(self):
        if getattr(self, "h", None):
            lib().orc_model_destroy(self.h)
            self.h = None

    def forward_full(self, label: int, seq: np.ndarray) -> np.ndarray:
        """seq: int32[len], seq[0] ignored (class token).  Returns logits [len, V]."""
        seq = _i32(seq)
        out = np.zeros((seq.shape[0], self.shape.vocab), dtype=np.float32)
        lib().orc_forward_full(self.h, label, _p(seq, C.c_int32), seq.shape[0], _p(out, C.c_float))
        return out

    def new_cache(self):
        s = self.shape
        return (np.zeros((s.n_layers, s.T, s.dim), dtype=np.float32), np.zeros((s.n_layers, s.T, s.dim),
                                                                               dtype=np.float32))

    def forward_window(self, cache, label, seq, c, n, want_logits=True):
        seq = _i32(seq)
        out = np.zeros((n, self.shape.vocab), dtype=np.float32) if want_logits else None
        lib().orc_forward_window(self.h, _p(cache[0], C.c_float), _p(cache[1], C.c_float), label,
                                 _p(seq, C.c_int32), c, n, _p(out, C.c_float))
        return out

    def forward_window_trace(self, cache, label, seq, c, n, layer, want_logits=False):
        """forward_window that also returns the intermediates of `layer` as a dict of fp32 arrays (row i =
        sequence index c + i): a, q, k, v, o, x_attn, m [n, D]; act [n, F]; x_out [n, D]."""
        seq = _i32(seq)
        s = self.shape
        out = np.zeros((n, s.vocab), dtype=np.float32) if want_logits else None
        bufs = {name: np.zeros((n, s.ffn_hidden if name == "act" else s.dim), dtype=np.float32)
                for name in ("a", "q", "k", "v", "o", "x_attn", "m", "act", "x_out")}
        tr = Trace(layer, *[_p(bufs[name], C.c_float) for name in ("a", "q", "k", "v", "o", "x_attn", "m", "act",
                                                                    "x_out")])
        lib().orc_forward_window_trace(self.h, _p(cache[0], C.c_float), _p(cache[1], C.c_float), label,
                                       _p(seq, C.c_int32), c, n, _p(out, C.c_float), C.byref(tr))
        return bufs, out

    # ---- single stages of one block on given inputs (the functions forward_window is made of)
    def stage_qkv(self, layer, x, c):
        """x fp32 [n, D] residual rows at sequence indices c.. -> (a, q, k, v) each [n, D]."""
        x = np.ascontiguousarray(x, dtype=np.float32)
        n, D = x.shape
        a = np.zeros((n, D), dtype=np.float32)
        qkv = np.zeros((n, 3 * D), dtype=np.float32)
        lib().orc_stage_qkv(self.h, layer, _p(x, C.c_float), n, c, _p(a, C.c_float), _p(qkv, C.c_float))
        return a, qkv[:, :D].copy(), qkv[:, D:2 * D].copy(), qkv[:, 2 * D:].copy()

    def stage_attend(self, q, K, V, c):
        """q [n, D] at sequence indices c..; K, V [>= c+n, D] cache rows of one layer -> o [n, D]."""
        q, K, V = (np.ascontiguousarray(t, dtype=np.float32) for t in (q, K, V))
        n = q.shape[0]
        assert K.shape[0] >= c + n and V.shape[0] >= c + n
        o = np.zeros_like(q)
        lib().orc_stage_attend(self.h, _p(q, C.c_float), _p(K, C.c_float), _p(V, C.c_float), c, n, _p(o, C.c_float))
        return o

    def stage_attn_out(self, layer, o, x):
        """x + W_o o, fp32 [n, D]."""
        o = np.ascontiguousarray(o, dtype=np.float32)
        x = np.array(x, dtype=np.float32, copy=True, order="C")
        lib().orc_stage_attn_out(self.h, layer, _p(o, C.c_float), o.shape[0], _p(x, C.c_float))
        return x

    def stage_ffn_act(self, layer, x):
        """x fp32 [n, D] -> (m [n, D], act [n, F])."""
        x = np.ascontiguousarray(x, dtype=np.float32)
        n = x.shape[0]
        m = np.zeros_like(x)
        act = np.zeros((n, self.shape.ffn_hidden), dtype=np.float32)
        lib().orc_stage_ffn_act(self.h, layer, _p(x, C.c_float), n, _p(m, C.c_float), _p(act, C.c_float))
        return m, act

    def stage_ffn_down(self, layer, act, x):
        """x + W_2 act, fp32 [n, D]."""
        act = np.ascontiguousarray(act, dtype=np.float32)
        x = np.array(x, dtype=np.float32, copy=True, order="C")
        lib().orc_stage_ffn_down(self.h, layer, _p(act, C.c_float), act.shape[0], _p(x, C.c_float))
        return x

    def set_diag(self, acc_f32: bool = False, attn_w_bf16: bool = False, norm_folded: bool = False):
        """Diagnostics of the noise-floor calibration, never a comparison target: accumulate dot products in fp32
        instead of double; round the unnormalised attention weights to bf16 before they multiply the values;
        apply RMSNorm's row factor after the projection (operand bf16(x) instead of bf16(x r g)).
        set_diag() restores the oracle proper."""
        lib().orc_model_set_diag(self.h, int(acc_f32), int(attn_w_bf16), int(norm_folded))

    def ar_rollout(self, prefix_tokens, prefix_len, labels, params: Params, image_ids=None) -> np.ndarray:
        pt, pl, lb = _i32(prefix_tokens), _i32(prefix_len), _i32(labels)
        ids = None if image_ids is None else _i32(image_ids)
        out = np.zeros_like(pt)
        lib().orc_ar_rollout(self.h, pt.shape[0], _p(pt, C.c_int32), _p(pl, C.c_int32), _p(lb, C.c_int32),
                             _p(ids, C.c_int32), C.byref(params), _p(out, C.c_int32))
        return out


class Rollout:
    """Rollout state of a batch: created after prefix pre-filling with the initial windows built."""

    def __init__(self, model: Model, prefix_tokens, prefix_len, labels, params: Params, image_ids=None):
        self.model = model
        self.params = params
        pt, pl, lb = _i32(prefix_tokens), _i32(prefix_len), _i32(labels)
        ids = None if image_ids is None else _i32(image_ids)
        self.B = pt.shape[0]
        self.T = model.shape.T
        self.V = model.shape.vocab
        self.h = lib().orc_rollout_create(model.h, self.B, _p(pt, C.c_int32), _p(pl, C.c_int32), _p(lb, C.c_int32),
                                          _p(ids, C.c_int32), C.byref(params))

    def __del__(self):
        if getattr(self, "h", None):
            lib().orc_rollout_destroy(self.h)
            self.h = None

    def live(self) -> int:
        return lib().orc_rollout_live(self.h)

    def round(self):
        """Runs one round.  Returns (live_after, m[B], j[B])."""
        m = np.zeros(self.B, dtype=np.int32)
        j = np.zeros(self.B, dtype=np.int32)
        live = lib().orc_rollout_round(self.h, _p(m, C.c_int32), _p(j, C.c_int32))
        return live, m, j

    def run(self, max_rounds: int = 0) -> int:
        return lib().orc_rollout_run(self.h, max_rounds)

    def tokens(self) -> np.ndarray:
        out = np.zeros((self.B, self.T), dtype=np.int32)
        lib().orc_rollout_tokens(self.h, _p(out, C.c_int32))
        return out

    def state(self):
        """(round, cursor[B], seq[B,T+1], delta[B,T+1], qbase[B])"""
        cur = np.zeros(self.B, dtype=np.int32)
        seq = np.zeros((self.B, self.T + 1), dtype=np.int32)
        dl = np.zeros((self.B, self.T + 1), dtype=np.uint8)
        qb = np.zeros(self.B, dtype=np.int32)
        r = lib().orc_rollout_get_state(self.h, _p(cur, C.c_int32), _p(seq, C.c_int32), _p(dl, C.c_uint8),
                                        _p(qb, C.c_int32))
        return r, cur, seq, dl, qb

    def last_probs(self, b: int) -> np.ndarray:
        out = np.zeros((self.params.window, self.V), dtype=np.float32)
        n = lib().orc_rollout_probs(self.h, b, _p(out, C.c_float))
        return out[:n]

    def last_logits(self, b: int, branch: int = 0) -> np.ndarray:
        out = np.zeros((self.params.window, self.V), dtype=np.float32)
        n = lib().orc_rollout_logits(self.h, b, branch, _p(out, C.c_float))
        return out[:n]

    def stats(self):
        s4 = (C.c_int64 * 4)()
        cap = 4096
        live = np.zeros(cap, dtype=np.int32)
        mode = np.zeros(cap, dtype=np.int32)
        n = lib().orc_rollout_stats(self.h, s4, _p(live, C.c_int32), _p(mode, C.c_int32), cap)
        n = min(n, cap)
        return dict(rounds=int(s4[0]), image_forwards=int(s4[1]), committed=int(s4[2]), rejects=int(s4[3]),
                    live_trace=live[:n].copy(), mode_trace=mode[:n].copy())


def num_threads() -> int:
    return int(lib().orc_num_threads())
