"""Python face of the CPU fp64 oracle (``ll_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library never imports this package and
this package never imports the CUDA library; the two share no code.

All tensors cross this boundary as ``numpy.float64`` arrays in the token-major
layout ``[tokens, heads, head_dim]``; bf16 inputs are widened exactly by the
caller before they get here.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ll_oracle.c")
_LIB = os.path.join(_HERE, "libll_oracle.so")
_lock = threading.Lock()
_lib = None

OK = 0
ERR_ARG = -1
ERR_POSITION = -2
ERR_NOT_RESIDENT = -3


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, OpenMP over query rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _dp(a):
    return a.ctypes.data_as(C.POINTER(C.c_double)) if a is not None else None


def _ip(a):
    return a.ctypes.data_as(C.POINTER(C.c_int64)) if a is not None else None


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = C.CDLL(build())
            L.llo_create.restype = C.c_void_p
            L.llo_create.argtypes = [C.c_int] * 8
            L.llo_destroy.argtypes = [C.c_void_p]
            L.llo_reset.argtypes = [C.c_void_p]
            L.llo_seek.argtypes = [C.c_void_p, C.c_int, C.c_int64]
            L.llo_get_state.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int64),
                                        C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
            L.llo_slot_of.argtypes = [C.c_void_p, C.c_int64]
            L.llo_visible.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64]
            L.llo_rope_split.argtypes = [C.c_int] + [C.POINTER(C.c_int)] * 3
            L.llo_rope_split.restype = None
            L.llo_round_bf16.restype = C.c_double
            L.llo_round_bf16.argtypes = [C.c_double]
            L.llo_round_e4m3.restype = C.c_double
            L.llo_round_e4m3.argtypes = [C.c_double]
            L.llo_set_kv_e4m3.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.POINTER(C.c_float)]
            L.llo_rope.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_double), C.c_int64,
                                   C.c_int, C.c_int, C.c_int64, C.c_int, C.c_int, C.c_double, C.c_int]
            L.llo_append.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                     C.c_int64, C.c_int, C.c_int, C.c_int, C.c_double]
            L.llo_attn.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_double), C.c_int64, C.c_int,
                                   C.c_int64, C.POINTER(C.c_int64), C.c_int64,
                                   C.POINTER(C.c_double), C.POINTER(C.c_double)]
            L.llo_attn_probs.restype = C.c_int64
            L.llo_attn_probs.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_double), C.c_int64,
                                         C.c_int64, C.c_int64, C.c_int, C.POINTER(C.c_double),
                                         C.POINTER(C.c_int64), C.c_int64]
            L.llo_recache.argtypes = [C.c_void_p, C.c_int] + [C.POINTER(C.c_double)] * 3 + \
                                     [C.c_int, C.c_int, C.c_int, C.c_double, C.POINTER(C.c_int64), C.c_int64] + \
                                     [C.POINTER(C.c_double)] * 3
            L.llo_visible_window.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int]
            L.llo_clip.argtypes = [C.c_void_p, C.c_int] + [C.POINTER(C.c_double)] * 3 + \
                                  [C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_double,
                                   C.POINTER(C.c_int64), C.c_int64] + [C.POINTER(C.c_double)] * 3
            L.llo_clip_backward.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                            C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_double] + \
                                           [C.POINTER(C.c_double)] * 6
            L.llo_rms_norm.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_double), C.c_double, C.c_int64, C.c_int,
                                       C.POINTER(C.c_double)]
            L.llo_dense_attn.argtypes = [C.POINTER(C.c_double)] * 3 + [C.c_int64, C.c_int64, C.c_int, C.c_int,
                                                                       C.POINTER(C.c_int64), C.c_int64,
                                                                       C.POINTER(C.c_double), C.POINTER(C.c_double)]
            L.llo_read_row.argtypes = [C.c_void_p, C.c_int, C.c_int64,
                                       C.POINTER(C.c_double), C.POINTER(C.c_double)]
            L.llo_read_layer.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double)]
            _lib = L
    return _lib


class OracleError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__("%s: oracle status %d" % (what, code))
        self.code = code


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def rope_split(D: int):
    a, b, c = C.c_int(), C.c_int(), C.c_int()
    lib().llo_rope_split(D, C.byref(a), C.byref(b), C.byref(c))
    return a.value, b.value, c.value


def round_bf16(x):
    """Nearest-bf16 (ties to even) of float64 values, returned as float64."""
    f = np.vectorize(lambda t: lib().llo_round_bf16(float(t)), otypes=[np.float64])
    return f(np.asarray(x, dtype=np.float64))


def round_e4m3(x):
    """Nearest E4M3 value (ties to even, saturating at 448) of float64 values, as float64."""
    f = np.vectorize(lambda t: lib().llo_round_e4m3(float(t)), otypes=[np.float64])
    return f(np.asarray(x, dtype=np.float64))


def rope(x, frame_start: int, gh: int, gw: int, theta: float = 10000.0, round_bf16: bool = False):
    """3-D RoPE of a token-major tensor [n_frames*gh*gw, H, D]."""
    x = _f64(x)
    n, H, D = x.shape
    out = np.empty_like(x)
    st = lib().llo_rope(_dp(x), _dp(out), n, H, D, frame_start, gh, gw, theta, int(round_bf16))
    if st != OK:
        raise OracleError(st, "rope")
    return out


def rms_norm(x, gain, eps: float):
    """RMS norm of every token's whole row: x [tokens, H, D], gain [H, D] (or flat [H*D])."""
    x = _f64(x)
    g = _f64(gain).reshape(-1)
    n = int(np.prod(x.shape[1:]))
    if g.shape[0] != n:
        raise OracleError(ERR_ARG, "rms_norm shape")
    y = np.empty_like(x)
    st = lib().llo_rms_norm(_dp(x), _dp(g), eps, x.shape[0], n, _dp(y))
    if st != OK:
        raise OracleError(st, "rms_norm")
    return y


def qkv_proj(x, w, bias=None):
    """The layer's QKV projection (upstream of the path; Sec. 3.1 names the block, the base
    model defines the projection): y = x W^T + b in fp64 with the library matrix product.
    x [tokens, d_model], w [3*H*D, d_model] (q features, then k, then v), bias [3*H*D] or None.
    Returns (q, k, v), each [tokens, H*D]."""
    x, w = _f64(x), _f64(w)
    y = x @ w.T
    if bias is not None:
        y = y + _f64(bias)[None, :]
    n = w.shape[0] // 3
    return y[:, :n], y[:, n:2 * n], y[:, 2 * n:]


def dense_attn(q, k, v, rows=None):
    """Plain softmax attention, every query over every key (cross-attention, Sec. 3.1).
    q [n_q, H, D], k and v [n_k, H, D].  Returns (out [n_rows, H, D], lse [n_rows, H])."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    n_q, H, D = q.shape
    if k.shape != v.shape or k.shape[1:] != (H, D):
        raise OracleError(ERR_ARG, "dense_attn shape")
    r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n_rows = n_q if r is None else r.shape[0]
    out = np.empty((n_rows, H, D), dtype=np.float64)
    lse = np.empty((n_rows, H), dtype=np.float64)
    st = lib().llo_dense_attn(_dp(q), _dp(k), _dp(v), n_q, k.shape[0], H, D, _ip(r), n_rows, _dp(out), _dp(lse))
    if st != OK:
        raise OracleError(st, "dense_attn")
    return out, lse


class Oracle:
    """One stream's cache state and fp64 storage; mirrors the five library calls."""

    def __init__(self, layers, heads, head_dim, tokens_per_frame, chunk_frames,
                 sink_frames, window_frames, faithful: bool = False):
        self.L, self.H, self.D, self.P = layers, heads, head_dim, tokens_per_frame
        self.C, self.S, self.W = chunk_frames, sink_frames, window_frames
        self.faithful = bool(faithful)
        self._h = lib().llo_create(layers, heads, head_dim, tokens_per_frame, chunk_frames,
                                   sink_frames, window_frames, int(faithful))
        if not self._h:
            raise OracleError(ERR_ARG, "create")

    def close(self):
        if self._h:
            lib().llo_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- integer state ----------------------------------------------------
    def state(self, layer: int = 0):
        end, ev = C.c_int64(), C.c_int64()
        sf = np.empty(self.S + self.W, dtype=np.int32)
        st = lib().llo_get_state(self._h, layer, C.byref(end),
                                 sf.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(ev))
        if st != OK:
            raise OracleError(st, "get_state")
        return {"end": end.value, "slot_frame": sf, "evictions": ev.value}

    def slot_of(self, frame: int) -> int:
        return lib().llo_slot_of(self._h, frame)

    def visible(self, fq: int, fk: int, lo_floor: int = 0) -> bool:
        return bool(lib().llo_visible(self._h, fq, fk, lo_floor))

    def set_kv_e4m3(self, k_scale, v_scale):
        """8-bit storage from now on: rows hold scale * E4M3(x / scale), scales [L, H] fp32."""
        ks = np.ascontiguousarray(k_scale, dtype=np.float32).reshape(-1)
        vs = np.ascontiguousarray(v_scale, dtype=np.float32).reshape(-1)
        if ks.shape[0] != self.L * self.H or vs.shape[0] != self.L * self.H:
            raise OracleError(ERR_ARG, "set_kv_e4m3 shape")
        fp = C.POINTER(C.c_float)
        st = lib().llo_set_kv_e4m3(self._h, ks.ctypes.data_as(fp), vs.ctypes.data_as(fp))
        if st != OK:
            raise OracleError(st, "set_kv_e4m3")

    def reset(self):
        st = lib().llo_reset(self._h)
        if st != OK:
            raise OracleError(st, "reset")

    def seek(self, layer: int, end: int):
        """Continue the stream at frame ``end`` with an empty window (sink kept)."""
        st = lib().llo_seek(self._h, layer, end)
        if st != OK:
            raise OracleError(st, "seek")

    # -- the path ---------------------------------------------------------
    def append(self, layer, k, v, frame_start, gh, gw, theta=10000.0, n_frames=None):
        k, v = _f64(k), _f64(v)
        nf = self.C if n_frames is None else n_frames
        if k.shape != (nf * gh * gw, self.H, self.D) or v.shape != k.shape:
            raise OracleError(ERR_ARG, "append shape")
        st = lib().llo_append(self._h, layer, _dp(k), _dp(v), frame_start, nf, gh, gw, theta)
        if st != OK:
            raise OracleError(st, "append")

    def rope_q(self, q, frame_start, gh, gw, theta=10000.0):
        return rope(q, frame_start, gh, gw, theta, round_bf16=self.faithful)

    def attn(self, layer, q_roped, q_frame_start, n_q_frames=None, rows=None, lo_floor=0):
        """Returns (out [n_rows, H, D], lse [n_rows, H]) for the chosen query rows."""
        q = _f64(q_roped)
        nqf = self.C if n_q_frames is None else n_q_frames
        if q.shape != (nqf * self.P, self.H, self.D):
            raise OracleError(ERR_ARG, "attn shape")
        r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
        n_rows = q.shape[0] if r is None else r.shape[0]
        out = np.empty((n_rows, self.H, self.D), dtype=np.float64)
        lse = np.empty((n_rows, self.H), dtype=np.float64)
        st = lib().llo_attn(self._h, layer, _dp(q), q_frame_start, nqf, lo_floor,
                            _ip(r), n_rows, _dp(out), _dp(lse))
        if st != OK:
            raise OracleError(st, "attn")
        return out, lse

    def attn_probs(self, layer, q_roped, q_frame_start, row, head, lo_floor=0):
        q = _f64(q_roped)
        cap = (self.S + self.W) * self.P
        p = np.empty(cap, dtype=np.float64)
        kr = np.empty(cap, dtype=np.int64)
        n = lib().llo_attn_probs(self._h, layer, _dp(q), q_frame_start, lo_floor, row, head,
                                 _dp(p), _ip(kr), cap)
        if n < 0:
            raise OracleError(int(n), "attn_probs")
        return p[:n].copy(), kr[:n].copy()

    def recache(self, layer, q, k, v, n_frames, gh, gw, theta=10000.0, rows=None):
        """Returns (q_roped, out, lse); empty arrays when there is nothing to rebuild."""
        q, k, v = _f64(q), _f64(k), _f64(v)
        r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
        n_rows = q.shape[0] if r is None else r.shape[0]
        qr = np.empty_like(q)
        out = np.empty((n_rows, self.H, self.D), dtype=np.float64)
        lse = np.empty((n_rows, self.H), dtype=np.float64)
        st = lib().llo_recache(self._h, layer, _dp(q), _dp(k), _dp(v), n_frames, gh, gw, theta,
                               _ip(r), n_rows, _dp(qr), _dp(out), _dp(lse))
        if st != OK:
            raise OracleError(st, "recache")
        return qr, out, lse

    def clip(self, layer, q, k, v, frame_start, n_frames, window, gh, gw, theta=10000.0, rows=None):
        """A clip of whole chunks appended and attended in one step under a local window of
        ``window`` frames (Sec. 3.3, training/inference consistency).  Returns (q_roped, out, lse)."""
        q, k, v = _f64(q), _f64(k), _f64(v)
        if q.shape != (n_frames * gh * gw, self.H, self.D) or k.shape != q.shape or v.shape != q.shape:
            raise OracleError(ERR_ARG, "clip shape")
        r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
        n_rows = q.shape[0] if r is None else r.shape[0]
        qr = np.empty_like(q)
        out = np.empty((n_rows, self.H, self.D), dtype=np.float64)
        lse = np.empty((n_rows, self.H), dtype=np.float64)
        st = lib().llo_clip(self._h, layer, _dp(q), _dp(k), _dp(v), frame_start, n_frames, window, gh, gw,
                            theta, _ip(r), n_rows, _dp(qr), _dp(out), _dp(lse))
        if st != OK:
            raise OracleError(st, "clip")
        return qr, out, lse

    def clip_backward(self, layer, q, d_out, frame_start, n_frames, window, gh, gw, theta=10000.0):
        """Gradients of a scalar loss through the clip step that was just run (the cache is as
        ``clip`` left it): q is the clip's unrotated query tensor, d_out the loss gradient with
        respect to the clip's attention output.  Returns (dq, dk, dv, mag_q, mag_k, mag_v), all
        [n_frames*P, H, D]: gradients with respect to the q, k, v handed to ``clip`` and the
        sums of absolute values of the terms each element adds up."""
        q, g = _f64(q), _f64(d_out)
        if q.shape != (n_frames * gh * gw, self.H, self.D) or g.shape != q.shape:
            raise OracleError(ERR_ARG, "clip_backward shape")
        outs = [np.empty_like(q) for _ in range(6)]
        st = lib().llo_clip_backward(self._h, layer, _dp(q), _dp(g), frame_start, n_frames, window, gh, gw, theta,
                                     *[_dp(a) for a in outs])
        if st != OK:
            raise OracleError(st, "clip_backward")
        return tuple(outs)

    def visible_window(self, fq: int, fk: int, window: int) -> bool:
        return bool(lib().llo_visible_window(self._h, fq, fk, window))

    # -- storage ------------------------------------------------------------
    def read_row(self, layer, cache_row):
        k = np.empty((self.H, self.D), dtype=np.float64)
        v = np.empty((self.H, self.D), dtype=np.float64)
        st = lib().llo_read_row(self._h, layer, cache_row, _dp(k), _dp(v))
        if st != OK:
            raise OracleError(st, "read_row")
        return k, v

    def read_layer(self, layer=0):
        """(K, V), each [S+W, P, H, D]."""
        shp = (self.S + self.W, self.P, self.H, self.D)
        k = np.empty(shp, dtype=np.float64)
        v = np.empty(shp, dtype=np.float64)
        st = lib().llo_read_layer(self._h, layer, _dp(k), _dp(v))
        if st != OK:
            raise OracleError(st, "read_layer")
        return k, v
