"""Thin ctypes binding of libhbsjd.so: same names as the C ABI (include/hbsjd.h), argument
marshalling only.  Every step of the rollout runs inside the CUDA library; torch supplies device
memory and the stream.  There is no fallback: a missing library or GPU raises."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "libhbsjd.so")

DTYPE_FP32, DTYPE_BF16 = 0, 1
VERIFY_PROB, VERIFY_GREEDY = 0, 1
EXEC_FULL, EXEC_COMPACT, EXEC_HYBRID, EXEC_SYNC = 0, 1, 2, 3
DBG_PROBS, DBG_LOGITS, DBG_SLOTS = 0, 1, 2
DBG_ACT_A, DBG_ACT_Q, DBG_ACT_O, DBG_ACT_FFN, DBG_ACT_H, DBG_KV_K, DBG_KV_V = 3, 4, 5, 6, 7, 8, 9

EXPORTS = ["hbsjd_create", "hbsjd_rollout", "hbsjd_rollout_host", "hbsjd_profile", "hbsjd_profile_read", "hbsjd_profile_launch_floor", "hbsjd_probs", "hbsjd_verify", "hbsjd_verify_static", "hbsjd_calibrate_gamma", "hbsjd_round", "hbsjd_tokens", "hbsjd_destroy", "hbsjd_get_state",
           "hbsjd_set_state", "hbsjd_debug_read", "hbsjd_debug_forward", "hbsjd_debug_gemm",
           "hbsjd_debug_shuffle_pages", "hbsjd_debug_fold_norm", "hbsjd_gemm", "hbsjd_bikl", "hbsjd_score", "hbsjd_strerror",
           "hbsjd_last_error"]


class hbsjd_model_desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_layers", "dim", "n_heads", "ffn_hidden", "vocab", "grid_h", "grid_w", "n_classes", "dtype")] + [
                   ("rms_eps", C.c_float), ("rope_base", C.c_float)]


class hbsjd_params(C.Structure):
    _fields_ = [("window", C.c_int32), ("history_offset", C.c_int32), ("cfg_scale", C.c_float),
                ("temperature", C.c_float), ("top_k", C.c_int32), ("verify_mode", C.c_int32),
                ("exec_mode", C.c_int32), ("gamma", C.c_int32), ("seed", C.c_uint64), ("max_rounds", C.c_int32),
                ("reserved", C.c_int32)]


class hbsjd_stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in
                ("rounds", "image_forwards", "committed", "rejects", "full_rounds", "compact_rounds",
                 "prefill_forwards", "kernel_launches")] + [("ms_total", C.c_float), ("ms_prefill", C.c_float)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class hbsjd_kernel_profile(C.Structure):
    _fields_ = [("ms", C.c_double * 4), ("work", C.c_double * 4), ("launches", C.c_int64 * 4),
                ("dropped", C.c_int64), ("gemm_ms_by_rows", C.c_double * 4), ("gemm_work_by_rows", C.c_double * 4),
                ("gemm_launches_by_rows", C.c_int64 * 4), ("gemm_bytes_by_rows", C.c_double * 4)]


PROF_CLASSES = ("gemm", "attention", "accept", "other")
PROF_GEMM_ROW_BINS = ("rows<=512", "rows<=2048", "rows<=6144", "rows>6144")


class hbsjd_verify_desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("batch", "window", "T", "V", "branches", "history_offset", "greedy", "top_k")] + [
                   ("cfg_scale", C.c_float), ("temperature", C.c_float), ("seed", C.c_uint64),
                   ("round", C.c_uint32), ("reserved", C.c_uint32)]


class HbsjdError(RuntimeError):
    def __init__(self, code, what, detail=""):
        super().__init__(f"{what}: {code} ({detail})")
        self.code = code


_lib = None


def load():
    """Loads the library (no CUDA call is made); compiles it first if it has not been built.  Raises if that fails."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            # a fresh checkout: compile in-tree (nvcc, sm_100a); there is no other implementation to fall back to
            from . import build
            build.build()
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} is missing: run paper_2608_18183_b200/build.py (nvcc, sm_100a)")
        L = C.CDLL(LIB_PATH)
        vp = C.c_void_p
        L.hbsjd_create.argtypes = [C.POINTER(vp), C.POINTER(hbsjd_model_desc), vp, C.c_size_t, C.c_int, C.c_int, vp]
        L.hbsjd_rollout.argtypes = [vp, C.c_int, vp, vp, vp, C.POINTER(hbsjd_params), vp, C.POINTER(hbsjd_stats)]
        L.hbsjd_rollout_host.argtypes = [vp, C.c_int, vp, vp, vp, C.POINTER(hbsjd_params), vp,
                                         C.POINTER(hbsjd_stats)]
        L.hbsjd_profile.argtypes = [vp, C.c_int]
        L.hbsjd_profile_read.argtypes = [vp, C.POINTER(hbsjd_kernel_profile)]
        L.hbsjd_profile_launch_floor.argtypes = [vp, C.c_int, C.POINTER(C.c_float)]
        L.hbsjd_probs.argtypes = [vp, vp, vp, C.c_int, C.c_float, C.c_float, C.c_int, vp]
        L.hbsjd_verify.argtypes = [vp, C.POINTER(hbsjd_verify_desc)] + [vp] * 8
        L.hbsjd_verify_static.argtypes = [vp, C.POINTER(hbsjd_verify_desc)] + [vp] * 8
        L.hbsjd_calibrate_gamma.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int),
                                            C.POINTER(C.c_float), C.POINTER(C.c_float)]
        L.hbsjd_round.argtypes = [vp, C.POINTER(C.c_int)]
        L.hbsjd_tokens.argtypes = [vp, vp]
        L.hbsjd_destroy.argtypes = [vp]
        L.hbsjd_destroy.restype = None
        L.hbsjd_get_state.argtypes = [vp, vp, vp, vp, vp, C.POINTER(C.c_int32)]
        L.hbsjd_set_state.argtypes = [vp, vp, vp, vp, vp, C.c_int32]
        L.hbsjd_debug_read.argtypes = [vp, C.c_int, C.c_int, vp, C.c_size_t]
        L.hbsjd_debug_forward.argtypes = [vp, C.c_int, C.c_int]
        L.hbsjd_gemm.argtypes = [vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, C.c_int]
        L.hbsjd_debug_gemm.argtypes = [vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_uint, C.c_int]
        L.hbsjd_debug_shuffle_pages.argtypes = [vp, C.c_uint64]
        L.hbsjd_debug_fold_norm.argtypes = [vp, C.c_int]
        L.hbsjd_bikl.argtypes = [vp, vp, vp, C.c_int, vp]
        L.hbsjd_score.argtypes = [vp, vp, C.c_int, vp, vp, vp, vp, vp, C.POINTER(C.c_float)]
        L.hbsjd_strerror.argtypes = [C.c_int]
        L.hbsjd_strerror.restype = C.c_char_p
        L.hbsjd_last_error.argtypes = [vp]
        L.hbsjd_last_error.restype = C.c_char_p
        _lib = L
    return _lib


def make_desc(shape) -> hbsjd_model_desc:
    return hbsjd_model_desc(shape.n_layers, shape.dim, shape.n_heads, shape.ffn_hidden, shape.vocab, shape.grid_h,
                            shape.grid_w, shape.n_classes, DTYPE_FP32 if shape.dtype == "fp32" else DTYPE_BF16,
                            shape.rms_eps, shape.rope_base)


def make_params(window, history_offset, cfg_scale=1.0, temperature=1.0, top_k=0, verify_mode=VERIFY_PROB,
                exec_mode=EXEC_HYBRID, gamma=0, seed=0, max_rounds=-1) -> hbsjd_params:
    return hbsjd_params(window, history_offset, cfg_scale, temperature, top_k, verify_mode, exec_mode, gamma, seed,
                        max_rounds, 0)


def hbsjd_verify_static(stream, desc, logits, q_prev, p_out, cursor, seq, delta, qbase, m_out):
    """The allocation-free verification step: no context, scratch inside the library image.
    `stream` is a torch.cuda.Stream; tensors are device tensors, state updated in place."""
    rc = load().hbsjd_verify_static(C.c_void_p(stream.cuda_stream), C.byref(desc), logits.data_ptr(),
                                    q_prev.data_ptr(), p_out.data_ptr(), cursor.data_ptr(), seq.data_ptr(),
                                    delta.data_ptr(), qbase.data_ptr(), m_out.data_ptr())
    if rc != 0:
        raise HbsjdError(rc, "hbsjd_verify_static", load().hbsjd_strerror(rc).decode())


class Context:
    """Owner of one hbsjd_ctx.  Methods carry the names of the C entry points."""

    def __init__(self, shape, weights: np.ndarray, max_batch: int, max_window: int, stream=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("hbsjd needs a CUDA device; there is no CPU path")
        self._torch = torch
        self.shape = shape
        self.lib = load()
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        w = np.ascontiguousarray(weights, dtype=np.uint8)
        self.h = C.c_void_p()
        desc = make_desc(shape)
        rc = self.lib.hbsjd_create(C.byref(self.h), C.byref(desc), w.ctypes.data, w.nbytes, max_batch, max_window,
                                   C.c_void_p(self.stream.cuda_stream))
        if rc != 0:
            raise HbsjdError(rc, "hbsjd_create", self.lib.hbsjd_strerror(rc).decode())
        self.max_batch, self.max_window = max_batch, max_window
        # the library's rule for the form of RMSNorm of a bf16 context (see hbsjd_debug_fold_norm)
        self.fold_norm = shape.dtype == "bf16" and 2 * max_batch * max_window <= 2048
        self.batch = 0
        self.window = 0

    def _check(self, rc, what):
        if rc < 0:
            raise HbsjdError(rc, what, self.lib.hbsjd_last_error(self.h).decode())
        return rc

    def hbsjd_rollout(self, prefix_tokens, prefix_len, class_labels, params: hbsjd_params, out_tokens=None):
        """Device int32 tensors in, device int32 [batch, T] out.  Returns (out_tokens, stats dict)."""
        torch = self._torch
        assert prefix_tokens.is_cuda and prefix_tokens.dtype == torch.int32 and prefix_tokens.is_contiguous()
        assert prefix_len.is_cuda and prefix_len.dtype == torch.int32
        assert class_labels.is_cuda and class_labels.dtype == torch.int32
        B = prefix_tokens.shape[0]
        if out_tokens is None:
            out_tokens = torch.empty((B, self.shape.T), dtype=torch.int32, device=prefix_tokens.device)
        st = hbsjd_stats()
        rc = self.lib.hbsjd_rollout(self.h, B, prefix_tokens.data_ptr(), prefix_len.data_ptr(),
                                    class_labels.data_ptr(), C.byref(params), out_tokens.data_ptr(), C.byref(st))
        self._check(rc, "hbsjd_rollout")
        self.batch, self.window = B, params.window
        return out_tokens, st.as_dict()

    def hbsjd_rollout_host(self, prefix_tokens, prefix_len, class_labels, params: hbsjd_params, out_tokens):
        """Host int32 buffers in (numpy arrays or pinned torch CPU tensors), host int32 [batch, T] out."""
        def ptr(x):
            return x.ctypes.data if isinstance(x, np.ndarray) else x.data_ptr()
        B = prefix_tokens.shape[0]
        st = hbsjd_stats()
        rc = self.lib.hbsjd_rollout_host(self.h, B, ptr(prefix_tokens), ptr(prefix_len), ptr(class_labels),
                                         C.byref(params), ptr(out_tokens), C.byref(st))
        self._check(rc, "hbsjd_rollout_host")
        self.batch, self.window = B, params.window
        return out_tokens, st.as_dict()

    def hbsjd_profile(self, enable: bool):
        self._check(self.lib.hbsjd_profile(self.h, 1 if enable else 0), "hbsjd_profile")

    def hbsjd_profile_read(self):
        p = hbsjd_kernel_profile()
        self._check(self.lib.hbsjd_profile_read(self.h, C.byref(p)), "hbsjd_profile_read")
        return {n: dict(ms=p.ms[i], work=p.work[i], launches=p.launches[i]) for i, n in enumerate(PROF_CLASSES)} | {
            "dropped": p.dropped,
            "gemm_by_rows": {n: dict(ms=p.gemm_ms_by_rows[i], work=p.gemm_work_by_rows[i],
                                     launches=p.gemm_launches_by_rows[i], bytes=p.gemm_bytes_by_rows[i])
                             for i, n in enumerate(PROF_GEMM_ROW_BINS)}}

    def hbsjd_profile_launch_floor(self, reps=200) -> float:
        """Median event bracket of an empty kernel launch, microseconds."""
        us = C.c_float(0.0)
        self._check(self.lib.hbsjd_profile_launch_floor(self.h, reps, C.byref(us)), "hbsjd_profile_launch_floor")
        return us.value

    def hbsjd_probs(self, logits_c, logits_u=None, cfg_scale=1.0, temperature=1.0, top_k=0):
        """Device fp32 [rows, V] logits -> device fp32 [rows, V] probabilities."""
        out = self._torch.empty_like(logits_c)
        self._check(self.lib.hbsjd_probs(self.h, logits_c.data_ptr(), None if logits_u is None else logits_u.data_ptr(),
                                         logits_c.shape[0], cfg_scale, temperature, top_k, out.data_ptr()),
                    "hbsjd_probs")
        return out

    def hbsjd_verify(self, desc: hbsjd_verify_desc, logits, q_prev, p_out, cursor, seq, delta, qbase, m_out):
        """Verification step on device tensors; state tensors are updated in place."""
        self._check(self.lib.hbsjd_verify(self.h, C.byref(desc), logits.data_ptr(), q_prev.data_ptr(),
                                          p_out.data_ptr(), cursor.data_ptr(), seq.data_ptr(), delta.data_ptr(),
                                          qbase.data_ptr(), m_out.data_ptr()), "hbsjd_verify")

    def hbsjd_calibrate_gamma(self, batch, window, guidance):
        """Returns (gamma, ms_full[5], ms_compact[5]) for live = batch, 3/4, 1/2, 1/4, 1/8 of the batch."""
        g = C.c_int(0)
        mf, mc = (C.c_float * 5)(), (C.c_float * 5)()
        self._check(self.lib.hbsjd_calibrate_gamma(self.h, batch, window, 1 if guidance else 0, C.byref(g), mf, mc),
                    "hbsjd_calibrate_gamma")
        self.batch = 0
        return g.value, list(mf), list(mc)

    def hbsjd_round(self) -> int:
        live = C.c_int(0)
        self._check(self.lib.hbsjd_round(self.h, C.byref(live)), "hbsjd_round")
        return live.value

    def hbsjd_tokens(self):
        out = self._torch.empty((self.batch, self.shape.T), dtype=self._torch.int32, device="cuda")
        self._check(self.lib.hbsjd_tokens(self.h, out.data_ptr()), "hbsjd_tokens")
        return out

    def hbsjd_get_state(self):
        """(round, cursor[B], seq[B,T+1], delta[B,T+1], qbase[B]) as numpy arrays."""
        B, T1 = self.batch, self.shape.T + 1
        cur = np.zeros(B, dtype=np.int32)
        seq = np.zeros((B, T1), dtype=np.int32)
        dl = np.zeros((B, T1), dtype=np.uint8)
        qb = np.zeros(B, dtype=np.int32)
        rnd = C.c_int32(0)
        self._check(self.lib.hbsjd_get_state(self.h, cur.ctypes.data, seq.ctypes.data, dl.ctypes.data,
                                             qb.ctypes.data, C.byref(rnd)), "hbsjd_get_state")
        return rnd.value, cur, seq, dl, qb

    def hbsjd_set_state(self, rnd, cursor, seq, delta, qbase):
        cur = np.ascontiguousarray(cursor, dtype=np.int32)
        seq = np.ascontiguousarray(seq, dtype=np.int32)
        dl = np.ascontiguousarray(delta, dtype=np.uint8)
        qb = np.ascontiguousarray(qbase, dtype=np.int32)
        self._check(self.lib.hbsjd_set_state(self.h, cur.ctypes.data, seq.ctypes.data, dl.ctypes.data,
                                             qb.ctypes.data, int(rnd)), "hbsjd_set_state")

    def hbsjd_debug_read(self, what, index):
        V = self.shape.vocab
        if what == DBG_SLOTS:
            buf = np.zeros((3, self.max_batch), dtype=np.int32)
            n = self._check(self.lib.hbsjd_debug_read(self.h, what, 0, buf.ctypes.data, buf.nbytes), "debug_read")
            return buf.reshape(-1)[:3 * n].reshape(3, n)
        if what >= DBG_ACT_A:
            # activation rows / cache rows in the context's element type, returned widened to fp32
            s = self.shape
            width = s.ffn_hidden if what == DBG_ACT_FFN else s.dim
            rows = s.T + 1 if what in (DBG_KV_K, DBG_KV_V) else self.window
            raw16 = s.dtype == "bf16" and what != DBG_ACT_H
            buf = np.zeros((rows, width), dtype=np.uint16 if raw16 else np.float32)
            n = self._check(self.lib.hbsjd_debug_read(self.h, what, index, buf.ctypes.data, buf.nbytes), "debug_read")
            out = buf[:n]
            return (out.astype(np.uint32) << np.uint32(16)).view(np.float32) if raw16 else out
        buf = np.zeros((self.window, V), dtype=np.float32)
        n = self._check(self.lib.hbsjd_debug_read(self.h, what, index, buf.ctypes.data, buf.nbytes), "debug_read")
        return buf[:n]

    def hbsjd_debug_forward(self, layer: int, stage: int):
        """Partial verifier forward of the current state up to `layer` (stage 0: attention sub-block, 1: whole block)."""
        self._check(self.lib.hbsjd_debug_forward(self.h, layer, stage), "hbsjd_debug_forward")

    def hbsjd_gemm(self, A, W, Cout, accumulate=False):
        """Cout[M,N] fp32 (+)= A[M,K] . W[N,K]^T, tensors of the context's element type on the GPU."""
        M, K = A.shape
        N = W.shape[0]
        assert W.shape[1] == K and tuple(Cout.shape) == (M, N) and Cout.dtype == self._torch.float32
        assert A.is_contiguous() and W.is_contiguous() and Cout.is_contiguous()
        self._check(self.lib.hbsjd_gemm(self.h, A.data_ptr(), W.data_ptr(), Cout.data_ptr(), M, N, K,
                                        1 if accumulate else 0), "hbsjd_gemm")
        return Cout

    def hbsjd_debug_gemm(self, A, W, Cout, accumulate=False, reps=1, acc_wait_ns=0, tile=0):
        """hbsjd_gemm `reps` times back to back; acc_wait_ns > 0 shortens the epilogue's bounded wait (time-out test)."""
        M, K = A.shape
        N = W.shape[0]
        assert W.shape[1] == K and tuple(Cout.shape) == (M, N) and Cout.dtype == self._torch.float32
        self._check(self.lib.hbsjd_debug_gemm(self.h, A.data_ptr(), W.data_ptr(), Cout.data_ptr(), M, N, K,
                                              int(accumulate), reps, acc_wait_ns, tile), "hbsjd_debug_gemm")
        return Cout

    def hbsjd_debug_fold_norm(self, on: bool):
        """RMSNorm folded into the GEMM epilogues (True) or as its own kernel (False); before the first rollout."""
        self._check(self.lib.hbsjd_debug_fold_norm(self.h, 1 if on else 0), "hbsjd_debug_fold_norm")
        self.fold_norm = bool(on)

    def hbsjd_debug_shuffle_pages(self, seed: int):
        self._check(self.lib.hbsjd_debug_shuffle_pages(self.h, seed), "hbsjd_debug_shuffle_pages")

    def hbsjd_bikl(self, logits_s, logits_t):
        """Device fp32 [rows, V] logits of two models -> device fp32 [rows] bidirectional KL (Eq. 3)."""
        out = self._torch.empty(logits_s.shape[0], dtype=self._torch.float32, device="cuda")
        assert logits_s.shape == logits_t.shape and logits_s.is_contiguous() and logits_t.is_contiguous()
        self._check(self.lib.hbsjd_bikl(self.h, logits_s.data_ptr(), logits_t.data_ptr(), logits_s.shape[0],
                                        out.data_ptr()), "hbsjd_bikl")
        return out

    def hbsjd_score(self, teacher: "Context", tokens, prefix_len, class_labels):
        """Eq. 3 on completed trajectories, this context the student.  Device int32 tensors in; returns
        (bikl_pos device fp32 [batch, T], per_image device fp32 [batch], loss float)."""
        torch = self._torch
        batch = tokens.shape[0]
        assert tokens.is_cuda and tokens.dtype == torch.int32 and tokens.is_contiguous()
        assert tuple(tokens.shape) == (batch, self.shape.T)
        assert prefix_len.dtype == torch.int32 and class_labels.dtype == torch.int32
        pos = torch.empty((batch, self.shape.T), dtype=torch.float32, device="cuda")
        per = torch.empty(batch, dtype=torch.float32, device="cuda")
        loss = C.c_float(0.0)
        self._check(self.lib.hbsjd_score(self.h, teacher.h, batch, tokens.data_ptr(), prefix_len.data_ptr(),
                                         class_labels.data_ptr(), pos.data_ptr(), per.data_ptr(), C.byref(loss)),
                    "hbsjd_score")
        self.batch = 0
        teacher.batch = 0
        return pos, per, loss.value

    def hbsjd_destroy(self):
        if self.h:
            self.lib.hbsjd_destroy(self.h)
            self.h = C.c_void_p()

    def __del__(self):
        try:
            self.hbsjd_destroy()
        except Exception:
            pass
