"""ctypes binding of ``libllattn.so``: same names as the C ABI, argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  PyTorch is used
for device memory and streams; nothing here computes.  If the shared library
has not been built, importing the binding's functions raises: there is no
fallback.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libllattn.so")

LL_OK = 0
LL_ERR_INVALID_ARG = -1
LL_ERR_BAD_POSITION = -2
LL_ERR_UNSUPPORTED_SHAPE = -3
LL_ERR_NO_STORAGE = -4
LL_ERR_CUDA = -5
LL_ERR_DEVICE_TIMEOUT = -6
LL_ERR_DEVICE_CHECK = -7
LL_MAX_SLOTS = 64
LL_KV_BF16, LL_KV_E4M3 = 0, 1
LL_MAX_RANGES = 4
LL_STATIC_MAX_FRAMES = 64
LL_STATIC_MAX_GRID_SUM = 1024


class ll_state(C.Structure):
    _fields_ = [
        ("end", C.c_int64),
        ("n_slots", C.c_int32),
        ("ring_valid", C.c_int32),
        ("slot_frame", C.c_int32 * LL_MAX_SLOTS),
        ("n_appends", C.c_int64),
        ("n_overwrites", C.c_int64),
        ("n_evictions", C.c_int64),
        ("n_recaches", C.c_int64),
        ("n_attn_calls", C.c_int64),
    ]


LL_MAX_GROUPS = 24
LL_MAX_CTAS = 160


class ll_attn_plan(C.Structure):
    _fields_ = [
        ("n_ctas", C.c_int32),
        ("n_groups", C.c_int32),
        ("heads", C.c_int32),
        ("n_waves", C.c_int32),
        ("n_shares", C.c_int32),
        ("all_cols", C.c_int32),
        ("shared_steps", C.c_int64),
        ("tiles", C.c_int32 * LL_MAX_GROUPS),
        ("n_kt", C.c_int32 * LL_MAX_GROUPS),
        ("col_begin", C.c_int32 * LL_MAX_GROUPS),
        ("wave_cols", C.c_int32 * LL_MAX_GROUPS),
        ("step_begin", C.c_int64 * LL_MAX_GROUPS),
        ("share_begin", C.c_int32 * (LL_MAX_CTAS + 1)),
        ("share_of_cta", C.c_int32 * LL_MAX_CTAS),
    ]


LL_MAX_BATCH = 8


class ll_attn_item(C.Structure):
    _fields_ = [
        ("cache", C.c_void_p),
        ("layer", C.c_int32),
        ("n_q_frames", C.c_int32),
        ("q_roped", C.c_void_p),
        ("q_frame_start", C.c_int64),
        ("out", C.c_void_p),
        ("lse_out", C.c_void_p),
    ]


class LLError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__("llattn error %d: %s" % (code, message))
        self.code = code


_lib = None

# name -> (restype, argtypes); also the list of symbols include/llattn.h and include/llattn_debug.h declare
SIGNATURES = {
    "ll_cache_create": (C.c_int, [C.c_int] * 7 + [C.POINTER(C.c_void_p)]),
    "ll_cache_destroy": (None, [C.c_void_p]),
    "ll_cache_storage_bytes": (C.c_size_t, [C.c_void_p]),
    "ll_cache_bind_storage": (C.c_int, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "ll_cache_set_kv_format": (C.c_int, [C.c_void_p, C.c_int]),
    "ll_cache_set_kv_scales": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_float), C.POINTER(C.c_float), C.c_void_p]),
    "ll_cache_kv_offset": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_size_t)]),
    "ll_rope_append_kv": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                    C.c_int, C.c_int, C.c_int, C.c_float, C.c_void_p, C.c_void_p]),
    "ll_norm_rope_append_kv": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_float, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_float,
                                         C.c_void_p, C.c_void_p]),
    "ll_sink_window_attn": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_int64, C.c_int, C.c_void_p,
                                      C.c_void_p, C.c_void_p]),
    "ll_sink_window_attn_scaled": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_void_p,
                                             C.c_void_p, C.c_void_p]),
    "ll_qkv_proj_workspace_bytes": (C.c_size_t, [C.c_void_p]),
    "ll_qkv_proj_append": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                     C.c_float, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_float, C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.c_size_t, C.c_void_p]),
    "ll_sink_window_attn_batched": (C.c_int, [C.POINTER(ll_attn_item), C.c_int, C.c_void_p]),
    "ll_cross_attn": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                C.c_void_p, C.c_void_p]),
    "ll_clip_append_attn": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int,
                                      C.c_int, C.c_int, C.c_int, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.c_void_p]),
    "ll_clip_backward_workspace_bytes": (C.c_size_t, [C.c_void_p, C.c_int]),
    "ll_clip_attn_backward": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int,
                                        C.c_int, C.c_int, C.c_int, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_size_t, C.c_void_p]),
    "ll_recache": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                             C.c_int, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ll_rope_q_static": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int64, C.c_int, C.c_int, C.c_int,
                                   C.c_float, C.c_void_p]),
    "ll_cache_reset": (C.c_int, [C.c_void_p]),
    "ll_cache_get_state": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(ll_state)]),
    "ll_cache_set_state": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(ll_state)]),
    "ll_cache_visible_ranges": (C.c_int, [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.POINTER(C.c_int64),
                                          C.POINTER(C.c_int64), C.POINTER(C.c_int)]),
    "ll_cache_set_dry_run": (C.c_int, [C.c_void_p, C.c_int]),
    "ll_cache_device_status": (C.c_int, [C.c_void_p, C.c_void_p]),
    "ll_debug_attn_simt": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_int64, C.c_int, C.c_void_p,
                                     C.c_void_p, C.c_void_p]),
    "ll_debug_wait_timeout": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p]),
    "ll_debug_attn_plan": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(ll_attn_plan)]),
    "ll_debug_attn_plan_batched": (C.c_int, [C.POINTER(ll_attn_item), C.c_int, C.c_int, C.POINTER(ll_attn_plan)]),
    "ll_debug_aux_layout": (C.c_int, [C.c_void_p] + [C.POINTER(C.c_size_t)] * 4),
    "ll_debug_guard_layout": (C.c_int, [C.c_void_p] + [C.POINTER(C.c_size_t)] * 3),
    "ll_launch_count": (C.c_int64, []),
    "ll_last_error": (C.c_char_p, []),
    "ll_version": (C.c_char_p, []),
}


def lib():
    """Load the shared library (fails loudly when it is missing)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "%s is missing: build it with `python -m paper_2509_22622_b200.build` "
                "(there is no CPU or PyTorch fallback)" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _check(code: int):
    if code != LL_OK:
        raise LLError(code, lib().ll_last_error().decode())


def _ptr(t):
    """Device (or host) address of a torch tensor, None -> NULL."""
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        if not torch.cuda.is_available():      # bookkeeping-only handles never launch
            return C.c_void_p(0)
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)
    return C.c_void_p(stream if isinstance(stream, int) else stream.cuda_stream)


# ---- the C ABI, one Python function per entry point -----------------------------

def ll_cache_create(layers, heads, head_dim, tokens_per_frame, chunk_frames, sink_frames, window_frames):
    h = C.c_void_p()
    _check(lib().ll_cache_create(layers, heads, head_dim, tokens_per_frame, chunk_frames, sink_frames,
                                 window_frames, C.byref(h)))
    return h


def ll_cache_destroy(h):
    lib().ll_cache_destroy(h)


def ll_cache_storage_bytes(h) -> int:
    return lib().ll_cache_storage_bytes(h)


def ll_cache_bind_storage(h, storage, stream=None):
    _check(lib().ll_cache_bind_storage(h, _ptr(storage), storage.numel() * storage.element_size(), _stream(stream)))


def ll_cache_set_kv_format(h, fmt: int):
    _check(lib().ll_cache_set_kv_format(h, fmt))


def ll_cache_set_kv_scales(h, layer, k_scale, v_scale, stream=None):
    """k_scale, v_scale: sequences of `heads` floats (host)."""
    n = len(k_scale)
    ks = (C.c_float * n)(*[float(x) for x in k_scale])
    vs = (C.c_float * n)(*[float(x) for x in v_scale])
    _check(lib().ll_cache_set_kv_scales(h, layer, ks, vs, _stream(stream)))


def ll_cache_kv_offset(h, layer, which, head) -> int:
    off = C.c_size_t()
    _check(lib().ll_cache_kv_offset(h, layer, which, head, C.byref(off)))
    return off.value


def ll_rope_append_kv(h, layer, q, k, v, frame_start, n_frames, grid_h, grid_w, rope_theta=10000.0,
                      q_out=None, stream=None):
    _check(lib().ll_rope_append_kv(h, layer, _ptr(q), _ptr(k), _ptr(v), frame_start, n_frames, grid_h, grid_w,
                                   rope_theta, _ptr(q_out), _stream(stream)))


def ll_norm_rope_append_kv(h, layer, q, k, v, gain_q, gain_k, eps, frame_start, n_frames, grid_h, grid_w,
                           rope_theta=10000.0, q_out=None, stream=None):
    _check(lib().ll_norm_rope_append_kv(h, layer, _ptr(q), _ptr(k), _ptr(v), _ptr(gain_q), _ptr(gain_k), eps,
                                        frame_start, n_frames, grid_h, grid_w, rope_theta, _ptr(q_out),
                                        _stream(stream)))


def ll_sink_window_attn(h, layer, q_roped, q_frame_start, n_q_frames, out, lse_out=None, stream=None):
    _check(lib().ll_sink_window_attn(h, layer, _ptr(q_roped), q_frame_start, n_q_frames, _ptr(out),
                                     _ptr(lse_out), _stream(stream)))


def ll_sink_window_attn_scaled(h, layer, q_roped, q_row_scale, q_frame_start, n_q_frames, out, lse_out=None,
                               stream=None):
    _check(lib().ll_sink_window_attn_scaled(h, layer, _ptr(q_roped), _ptr(q_row_scale), q_frame_start, n_q_frames,
                                            _ptr(out), _ptr(lse_out), _stream(stream)))


def ll_qkv_proj_workspace_bytes(h) -> int:
    return lib().ll_qkv_proj_workspace_bytes(h)


def ll_qkv_proj_append(h, layer, x, w_qkv, bias, gain_q, gain_k, eps, frame_start, n_frames, grid_h, grid_w,
                       rope_theta, q_out, q_row_scale=None, workspace=None, stream=None):
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().ll_qkv_proj_append(h, layer, _ptr(x), x.shape[-1], _ptr(w_qkv), _ptr(bias), _ptr(gain_q), _ptr(gain_k),
                                    eps, frame_start, n_frames, grid_h, grid_w, rope_theta, _ptr(q_out),
                                    _ptr(q_row_scale), _ptr(workspace), nbytes, _stream(stream)))


def ll_sink_window_attn_batched(items, stream=None):
    """items: sequence of (handle, layer, q_roped, q_frame_start, n_q_frames, out, lse_out or None)."""
    def addr(t):
        return None if t is None else t.data_ptr()
    arr = (ll_attn_item * max(len(items), 1))()
    for i, (h, layer, q_roped, q_frame_start, n_q_frames, out, lse_out) in enumerate(items):
        arr[i] = ll_attn_item(h.value if isinstance(h, C.c_void_p) else h, layer, n_q_frames, addr(q_roped),
                              q_frame_start, addr(out), addr(lse_out))
    _check(lib().ll_sink_window_attn_batched(arr, len(items), _stream(stream)))


def ll_debug_attn_simt(h, layer, q_roped, q_frame_start, n_q_frames, out, lse_out=None, stream=None):
    _check(lib().ll_debug_attn_simt(h, layer, _ptr(q_roped), q_frame_start, n_q_frames, _ptr(out),
                                    _ptr(lse_out), _stream(stream)))


def ll_cross_attn(h, q, k, v, out, lse_out=None, stream=None, n_q=None, n_k=None):
    n_q = q.shape[0] if n_q is None else n_q
    n_k = k.shape[0] if n_k is None else n_k
    _check(lib().ll_cross_attn(h, _ptr(q), n_q, _ptr(k), _ptr(v), n_k, _ptr(out), _ptr(lse_out), _stream(stream)))


def ll_clip_append_attn(h, layer, q, k, v, frame_start, n_frames, attn_window_frames, grid_h, grid_w,
                        rope_theta, q_out, out, lse_out=None, stream=None):
    _check(lib().ll_clip_append_attn(h, layer, _ptr(q), _ptr(k), _ptr(v), frame_start, n_frames, attn_window_frames,
                                     grid_h, grid_w, rope_theta, _ptr(q_out), _ptr(out), _ptr(lse_out),
                                     _stream(stream)))


def ll_clip_backward_workspace_bytes(h, n_frames) -> int:
    return lib().ll_clip_backward_workspace_bytes(h, n_frames)


def ll_clip_attn_backward(h, layer, q_roped, out, d_out, lse, frame_start, n_frames, attn_window_frames, grid_h, grid_w,
                          rope_theta, dq, dk, dv, workspace, stream=None):
    _check(lib().ll_clip_attn_backward(h, layer, _ptr(q_roped), _ptr(out), _ptr(d_out), _ptr(lse), frame_start, n_frames,
                                       attn_window_frames, grid_h, grid_w, rope_theta, _ptr(dq), _ptr(dk), _ptr(dv),
                                       _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))


def ll_recache(h, layer, q, k, v, n_frames, grid_h, grid_w, rope_theta, q_out, out, lse_out=None, stream=None):
    _check(lib().ll_recache(h, layer, _ptr(q), _ptr(k), _ptr(v), n_frames, grid_h, grid_w, rope_theta,
                            _ptr(q_out), _ptr(out), _ptr(lse_out), _stream(stream)))


def ll_rope_q_static(q, q_out, heads, head_dim, frame_start, n_frames, grid_h, grid_w, rope_theta=10000.0,
                     stream=None):
    """RoPE(q) -> q_out through the entry point that allocates nothing (tables in a fixed array)."""
    _check(lib().ll_rope_q_static(_ptr(q), _ptr(q_out), heads, head_dim, frame_start, n_frames, grid_h, grid_w,
                                  rope_theta, _stream(stream)))


def ll_cache_reset(h):
    _check(lib().ll_cache_reset(h))


def ll_cache_get_state(h, layer=0) -> ll_state:
    st = ll_state()
    _check(lib().ll_cache_get_state(h, layer, C.byref(st)))
    return st


def ll_cache_set_state(h, layer, st: ll_state):
    _check(lib().ll_cache_set_state(h, layer, C.byref(st)))


def ll_cache_visible_ranges(h, layer, q_frame_start, lo_floor=0):
    starts = (C.c_int64 * LL_MAX_RANGES)()
    lens = (C.c_int64 * LL_MAX_RANGES)()
    n = C.c_int()
    _check(lib().ll_cache_visible_ranges(h, layer, q_frame_start, lo_floor, starts, lens, C.byref(n)))
    return [(starts[i], lens[i]) for i in range(n.value)]


def ll_cache_set_dry_run(h, on: bool):
    _check(lib().ll_cache_set_dry_run(h, int(on)))


def ll_cache_device_status(h, stream=None):
    _check(lib().ll_cache_device_status(h, _stream(stream)))


def ll_debug_wait_timeout(h, limit_ms=20, stream=None):
    _check(lib().ll_debug_wait_timeout(h, limit_ms, _stream(stream)))


def ll_debug_attn_plan(h, layer=0, recache=False, sm_count=0) -> ll_attn_plan:
    plan = ll_attn_plan()
    _check(lib().ll_debug_attn_plan(h, layer, int(recache), sm_count, C.byref(plan)))
    return plan


def ll_debug_attn_plan_batched(handles_and_layers, sm_count=0) -> ll_attn_plan:
    arr = (ll_attn_item * len(handles_and_layers))()
    for i, (h, layer) in enumerate(handles_and_layers):
        arr[i].cache = h.value if isinstance(h, C.c_void_p) else h
        arr[i].layer = layer
    plan = ll_attn_plan()
    _check(lib().ll_debug_attn_plan_batched(arr, len(handles_and_layers), sm_count, C.byref(plan)))
    return plan


def ll_debug_aux_layout(h):
    """(status_offset, status_bytes, counters_offset, counters_bytes) inside the bound storage."""
    v = [C.c_size_t() for _ in range(4)]
    _check(lib().ll_debug_aux_layout(h, *[C.byref(x) for x in v]))
    return tuple(x.value for x in v)


def ll_debug_guard_layout(h):
    """(front_offset, back_offset, bytes) of the guard bands of a handle created under LL_DEBUG."""
    v = [C.c_size_t() for _ in range(3)]
    _check(lib().ll_debug_guard_layout(h, *[C.byref(x) for x in v]))
    return tuple(x.value for x in v)


def ll_launch_count() -> int:
    return lib().ll_launch_count()


def ll_version() -> str:
    return lib().ll_version().decode()


# ---- a small convenience owner ---------------------------------------------------

class Cache:
    """Owns a handle plus the torch tensor that backs it.  Marshalling only."""

    def __init__(self, layers, heads, head_dim, tokens_per_frame, chunk_frames, sink_frames, window_frames,
                 device="cuda:0", dry_run=False, kv_format=0):
        self.L, self.H, self.D, self.P = layers, heads, head_dim, tokens_per_frame
        self.C, self.S, self.W = chunk_frames, sink_frames, window_frames
        self.h = ll_cache_create(layers, heads, head_dim, tokens_per_frame, chunk_frames, sink_frames,
                                 window_frames)
        self.storage = None
        self.kv_format = kv_format
        if kv_format:
            ll_cache_set_kv_format(self.h, kv_format)
        if dry_run:
            ll_cache_set_dry_run(self.h, True)
        else:
            import torch
            if not torch.cuda.is_available():
                raise RuntimeError("llattn needs a CUDA device; there is no CPU fallback")
            nbytes = ll_cache_storage_bytes(self.h)
            # over-allocate so the bound address can be rounded up to 1024 bytes
            self._raw = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
            shift = (-self._raw.data_ptr()) % 1024
            self.storage = self._raw[shift:shift + nbytes]
            ll_cache_bind_storage(self.h, self.storage)

    def close(self):
        if self.h is not None:
            ll_cache_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def state(self, layer=0):
        st = ll_cache_get_state(self.h, layer)
        return {"end": st.end, "slot_frame": list(st.slot_frame[:st.n_slots]), "ring_valid": st.ring_valid,
                "evictions": st.n_evictions, "appends": st.n_appends, "overwrites": st.n_overwrites,
                "recaches": st.n_recaches, "attn_calls": st.n_attn_calls}

    def kv_view(self, layer, which):
        """View [H, rows, D] of a layer's K (which=0) or V (which=1) matrix: bf16, or the
        E4M3 codes as uint8 for an 8-bit cache."""
        import torch
        rows = (self.S + self.W) * self.P
        off = ll_cache_kv_offset(self.h, layer, which, 0)
        if self.kv_format == LL_KV_E4M3:
            n = self.H * rows * self.D
            return self.storage[off:off + n].view(self.H, rows, self.D)
        n = self.H * rows * self.D * 2
        return self.storage[off:off + n].view(torch.bfloat16).view(self.H, rows, self.D)

    def set_kv_scales(self, layer, k_scale, v_scale, stream=None):
        ll_cache_set_kv_scales(self.h, layer, k_scale, v_scale, stream)

    def rope_append_kv(self, layer, q, k, v, frame_start, grid_h, grid_w, theta=10000.0, q_out=None, stream=None):
        ll_rope_append_kv(self.h, layer, q, k, v, frame_start, self.C, grid_h, grid_w, theta, q_out, stream)

    def norm_rope_append_kv(self, layer, q, k, v, gain_q, gain_k, eps, frame_start, grid_h, grid_w, theta=10000.0,
                            q_out=None, stream=None):
        ll_norm_rope_append_kv(self.h, layer, q, k, v, gain_q, gain_k, eps, frame_start, self.C, grid_h, grid_w,
                               theta, q_out, stream)

    def sink_window_attn(self, layer, q_roped, q_frame_start, out, lse_out=None, stream=None):
        ll_sink_window_attn(self.h, layer, q_roped, q_frame_start, self.C, out, lse_out, stream)

    @staticmethod
    def sink_window_attn_batched(items, stream=None):
        """items: (Cache, layer, q_roped, q_frame_start, out, lse_out or None) per stream, one launch."""
        ll_sink_window_attn_batched([(c.h, layer, q, f0, c.C, out, lse) for c, layer, q, f0, out, lse in items],
                                    stream)

    def cross_attn(self, q, k, v, out, lse_out=None, stream=None):
        ll_cross_attn(self.h, q, k, v, out, lse_out, stream)

    def clip_append_attn(self, layer, q, k, v, frame_start, n_frames, attn_window_frames, grid_h, grid_w, theta,
                         q_out, out, lse_out=None, stream=None):
        ll_clip_append_attn(self.h, layer, q, k, v, frame_start, n_frames, attn_window_frames, grid_h, grid_w,
                            theta, q_out, out, lse_out, stream)

    def recache(self, layer, q, k, v, n_frames, grid_h, grid_w, theta, q_out, out, lse_out=None, stream=None):
        ll_recache(self.h, layer, q, k, v, n_frames, grid_h, grid_w, theta, q_out, out, lse_out, stream)

    def reset(self):
        ll_cache_reset(self.h)

    def check_device(self, stream=None):
        ll_cache_device_status(self.h, stream)
