"""CPU-only tests of the library's host side: exported symbols, argument
checks, and the integer cache state against the oracle (bit-exact).  No kernel
is launched: handles run in bookkeeping-only mode."""
import ctypes
import os
import re

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from paper_2509_22622_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="session", autouse=True)
def built():
    from paper_2509_22622_b200 import build
    build.build()


def test_library_exports_every_declared_symbol():
    text = "".join(open(os.path.join(ROOT, "include", name)).read()
                   for name in sorted(os.listdir(os.path.join(ROOT, "include"))) if name.endswith(".h"))
    declared = set(re.findall(r"\b(ll_[a-z_0-9]+)\s*\(", text))
    assert declared == set(B.SIGNATURES), declared ^ set(B.SIGNATURES)
    L = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(L, name), name
    assert "sm_100a" in B.ll_version()


def test_create_rejects_unsupported_shapes():
    for args in [(1, 2, 96, 16, 1, 1, 2), (1, 2, 64, 16, 2, 1, 2), (1, 2, 64, 16, 2, 2, 3),
                 (1, 2, 64, 16, 1, 40, 40), (1, 2, 64, 16, 4, 0, 2)]:
        with pytest.raises(B.LLError) as e:
            B.ll_cache_create(*args)
        assert e.value.code == B.LL_ERR_UNSUPPORTED_SHAPE
    with pytest.raises(B.LLError) as e:
        B.ll_cache_create(0, 2, 64, 16, 1, 1, 2)
    assert e.value.code == B.LL_ERR_INVALID_ARG


def test_storage_bytes_and_offsets():
    h = B.ll_cache_create(2, 12, 128, 1560, 3, 3, 9)
    total = B.ll_cache_storage_bytes(h)
    kv = 12 * 12 * 1560 * 128 * 2
    aux = B.ll_cache_kv_offset(h, 0, 0, 0)
    assert aux % 1024 == 0 and total == aux + 2 * 2 * kv
    assert B.ll_cache_kv_offset(h, 0, 1, 0) == aux + kv
    assert B.ll_cache_kv_offset(h, 1, 0, 0) == aux + 2 * kv
    assert B.ll_cache_kv_offset(h, 0, 0, 5) == aux + 5 * 12 * 1560 * 128 * 2
    B.ll_cache_destroy(h)


def test_compute_calls_need_storage_and_fail_loudly():
    h = B.ll_cache_create(1, 2, 64, 16, 1, 1, 2)
    buf = np.zeros(16 * 2 * 64, dtype=np.uint16)
    ptr = ctypes.c_void_p(buf.ctypes.data)
    rc = B.lib().ll_rope_append_kv(h, 0, None, ptr, ptr, 0, 1, 4, 4, 10000.0, None, None)
    assert rc == B.LL_ERR_NO_STORAGE
    assert b"storage" in B.lib().ll_last_error()
    assert B.ll_cache_get_state(h).end == 0          # state unchanged on error
    rc = B.lib().ll_rope_append_kv(h, 0, None, ptr, ptr, 0, 1, 4, 5, 10000.0, None, None)
    assert rc == B.LL_ERR_INVALID_ARG
    rc = B.lib().ll_rope_append_kv(h, 3, None, ptr, ptr, 0, 1, 4, 4, 10000.0, None, None)
    assert rc == B.LL_ERR_INVALID_ARG
    B.ll_cache_destroy(h)


def drive(cache, orc, schedule, gh, gw):
    """Replay a schedule on a dry-run handle and on the oracle; compare states."""
    C = cache.C
    x = np.zeros((C * gh * gw, cache.H, cache.D))
    for op in schedule:
        end = cache.state()["end"]
        if op == "new":
            B.ll_rope_append_kv(cache.h, 0, None, None, None, end, C, gh, gw)
            orc.append(0, x, x, end, gh, gw)
        elif op == "over":
            if end < C:
                with pytest.raises(B.LLError) as e:
                    B.ll_rope_append_kv(cache.h, 0, None, None, None, end - C, C, gh, gw)
                assert e.value.code == B.LL_ERR_BAD_POSITION
                continue
            B.ll_rope_append_kv(cache.h, 0, None, None, None, end - C, C, gh, gw)
            orc.append(0, x, x, end - C, gh, gw)
        elif op == "recache":
            n = max(0, end - max(cache.S, end - cache.W))
            B.ll_recache(cache.h, 0, None, None, None, n, gh, gw, 10000.0, None, None)
            e = np.zeros((n * gh * gw, cache.H, cache.D))
            orc.recache(0, e, e, e, n, gh, gw)
        elif op == "reset":
            B.ll_cache_reset(cache.h)
            orc.reset()
        elif op == "bad":
            with pytest.raises(B.LLError) as e:
                B.ll_rope_append_kv(cache.h, 0, None, None, None, end + C, C, gh, gw)
            assert e.value.code == B.LL_ERR_BAD_POSITION
        got, want = cache.state(), orc.state()
        assert got["end"] == want["end"]
        assert got["slot_frame"] == list(want["slot_frame"])
        assert got["evictions"] == want["evictions"]


shapes = st.sampled_from([(1, 1, 2), (3, 3, 9), (2, 2, 4), (1, 0, 3), (2, 4, 6), (3, 3, 3), (3, 3, 18), (1, 2, 5)])
ops = st.lists(st.sampled_from(["new"] * 6 + ["over", "over", "recache", "bad", "reset"]), min_size=1, max_size=60)


@settings(max_examples=60, deadline=None)
@given(shape=shapes, schedule=ops)
def test_state_bit_exact_vs_oracle(oracle_mod, shape, schedule):
    C, S, W = shape
    cache = B.Cache(1, 1, 64, 2, C, S, W, dry_run=True)
    orc = oracle_mod.Oracle(1, 1, 64, 2, C, S, W)
    drive(cache, orc, schedule, 1, 2)
    cache.close()


@pytest.mark.parametrize("C,S,W", [(1, 1, 2), (3, 3, 9), (2, 2, 4), (1, 0, 3), (3, 3, 18)])
def test_visible_ranges_cover_exactly_the_oracle_visible_rows(oracle_mod, C, S, W):
    P = 5
    cache = B.Cache(1, 1, 64, P, C, S, W, dry_run=True)
    orc = oracle_mod.Oracle(1, 1, 64, P, C, S, W)
    for chunk in range(14):
        B.ll_rope_append_kv(cache.h, 0, None, None, None, chunk * C, C, 1, P)
        end = (chunk + 1) * C
        # decode: newest chunk
        ranges = B.ll_cache_visible_ranges(cache.h, 0, chunk * C)
        rows = sorted(r for s, n in ranges for r in range(s, s + n))
        want = sorted(orc.slot_of(f) * P + t for f in range(end) if orc.visible(chunk * C, f) for t in range(P))
        assert rows == want and len(ranges) <= 2
        assert ranges == [(0, len(want))]            # decode always sees one contiguous run
        # recache groups
        r0 = max(S, end - W)
        for fq in range(r0, end, C):
            ranges = B.ll_cache_visible_ranges(cache.h, 0, fq, r0)
            rows = sorted(r for s, n in ranges for r in range(s, s + n))
            want = sorted(orc.slot_of(f) * P + t for f in range(end) if orc.visible(fq, f, r0) for t in range(P))
            assert rows == want and len(ranges) <= 3
    cache.close()


def test_state_roundtrip_and_validation():
    a = B.Cache(2, 1, 64, 2, 3, 3, 9, dry_run=True)
    for chunk in range(7):
        B.ll_rope_append_kv(a.h, 1, None, None, None, chunk * 3, 3, 1, 2)
    saved = B.ll_cache_get_state(a.h, 1)
    b = B.Cache(2, 1, 64, 2, 3, 3, 9, dry_run=True)
    B.ll_cache_set_state(b.h, 1, saved)
    assert a.state(1) == b.state(1) and b.state(0)["end"] == 0
    B.ll_rope_append_kv(b.h, 1, None, None, None, 21, 3, 1, 2)     # resumes where it left off
    bad = B.ll_cache_get_state(a.h, 1)
    bad.slot_frame[4] = 17                                         # frame 17 belongs in slot 5
    with pytest.raises(B.LLError):
        B.ll_cache_set_state(b.h, 1, bad)
    other = B.Cache(1, 1, 64, 2, 3, 3, 6, dry_run=True)
    with pytest.raises(B.LLError):
        B.ll_cache_set_state(other.h, 0, saved)


def test_attention_position_checks():
    c = B.Cache(1, 1, 64, 2, 3, 3, 9, dry_run=True)
    with pytest.raises(B.LLError) as e:
        B.ll_sink_window_attn(c.h, 0, None, 0, 3, None)
    assert e.value.code == B.LL_ERR_BAD_POSITION                   # nothing appended yet
    B.ll_rope_append_kv(c.h, 0, None, None, None, 0, 3, 1, 2)
    B.ll_rope_append_kv(c.h, 0, None, None, None, 3, 3, 1, 2)
    B.ll_sink_window_attn(c.h, 0, None, 3, 3, None)
    with pytest.raises(B.LLError):
        B.ll_sink_window_attn(c.h, 0, None, 0, 3, None)            # not the newest chunk
    with pytest.raises(B.LLError):
        B.ll_sink_window_attn(c.h, 0, None, 3, 2, None)
    assert c.state()["attn_calls"] == 1


def test_batched_attention_checks_every_item_before_anything_changes():
    a = B.Cache(2, 2, 64, 2, 3, 3, 9, dry_run=True)
    b = B.Cache(1, 2, 64, 5, 1, 0, 2, dry_run=True)            # other frame size, chunk, sink, window
    three_heads = B.Cache(1, 3, 64, 2, 3, 3, 9, dry_run=True)
    d128 = B.Cache(1, 2, 128, 2, 3, 3, 9, dry_run=True)
    for c in (a, three_heads, d128):
        for layer in range(c.L):
            B.ll_rope_append_kv(c.h, layer, None, None, None, 0, 3, 1, 2)
    B.ll_rope_append_kv(b.h, 0, None, None, None, 0, 1, 1, 5)
    B.ll_rope_append_kv(b.h, 0, None, None, None, 1, 1, 1, 5)

    def item(c, layer=0, start=0):
        return (c.h, layer, None, start, c.C, None, None)

    def calls():
        return [a.state(0)["attn_calls"], a.state(1)["attn_calls"], b.state()["attn_calls"]]

    B.ll_sink_window_attn_batched([item(a, 0), item(b, 0, 1), item(a, 1)])
    assert calls() == [1, 1, 1]
    for bad, code in [([], B.LL_ERR_INVALID_ARG),
                      ([item(a), item(three_heads)], B.LL_ERR_UNSUPPORTED_SHAPE),
                      ([item(a), item(d128)], B.LL_ERR_UNSUPPORTED_SHAPE),
                      ([item(a), item(b, 0, 1), item(a)], B.LL_ERR_INVALID_ARG),          # a layer twice
                      ([item(a), item(b, 0, 0)], B.LL_ERR_BAD_POSITION),                  # b's newest chunk is frame 1
                      ([item(a), item(a, 5)], B.LL_ERR_INVALID_ARG)]:                     # no such layer
        with pytest.raises(B.LLError) as e:
            B.ll_sink_window_attn_batched(bad)
        assert e.value.code == code, bad
        assert calls() == [1, 1, 1]
    many = [B.Cache(1, 2, 64, 2, 3, 3, 9, dry_run=True) for _ in range(B.LL_MAX_BATCH + 1)]
    for c in many:
        B.ll_rope_append_kv(c.h, 0, None, None, None, 0, 3, 1, 2)
    B.ll_sink_window_attn_batched([item(c) for c in many[:B.LL_MAX_BATCH]])
    with pytest.raises(B.LLError) as e:
        B.ll_sink_window_attn_batched([item(c) for c in many])
    assert e.value.code == B.LL_ERR_UNSUPPORTED_SHAPE
    assert [c.state()["attn_calls"] for c in many] == [1] * B.LL_MAX_BATCH + [0]


def test_clip_step_bookkeeping_matches_the_oracle_and_errors_change_nothing(oracle_mod):
    C, S, Wa, T = 2, 2, 4, 6
    ring = Wa + T - C
    c = B.Cache(1, 1, 64, 1, C, S, ring, dry_run=True)
    o = oracle_mod.Oracle(1, 1, 2, 1, C, S, ring)
    x = np.zeros((C, 1, 2))
    for chunk in range(3):
        B.ll_rope_append_kv(c.h, 0, None, None, None, chunk * C, C, 1, 1)
        o.append(0, x, x, chunk * C, 1, 1)
    before = c.state()
    for args, code in [((6, T + 1, Wa), B.LL_ERR_BAD_POSITION),            # not whole chunks
                       ((4, T, Wa), B.LL_ERR_BAD_POSITION),                # not at the end of the stream
                       ((6, T, Wa + C), B.LL_ERR_UNSUPPORTED_SHAPE),       # the ring cannot keep the first window
                       ((6, T + C, Wa), B.LL_ERR_UNSUPPORTED_SHAPE),
                       ((6, T, 3), B.LL_ERR_INVALID_ARG)]:                 # window not whole chunks
        with pytest.raises(B.LLError) as e:
            B.ll_clip_append_attn(c.h, 0, None, None, None, args[0], args[1], args[2], 1, 1, 10000.0, None, None)
        assert e.value.code == code, args
        assert c.state() == before
    for rep in range(3):                                                   # three clips in a row: the ring wraps
        f0 = 6 + rep * T
        B.ll_clip_append_attn(c.h, 0, None, None, None, f0, T, Wa, 1, 1, 10000.0, None, None)
        xs = np.zeros((T, 1, 2))
        o.clip(0, xs, xs, xs, f0, T, Wa, 1, 1)
        st, ost = c.state(), o.state()
        assert st["end"] == ost["end"] == f0 + T
        assert st["slot_frame"] == list(ost["slot_frame"]) and st["evictions"] == ost["evictions"]
    assert c.state()["appends"] == 3 + 3 * (T // C) and c.state()["attn_calls"] == 3
    # a shorter window than the ring allows is fine, and decoding goes on afterwards
    B.ll_clip_append_attn(c.h, 0, None, None, None, 24, C, C, 1, 1, 10000.0, None, None)
    B.ll_rope_append_kv(c.h, 0, None, None, None, 26, C, 1, 1)
    B.ll_sink_window_attn(c.h, 0, None, 26, C, None)


def test_cross_attention_argument_checks():
    c = B.Cache(1, 2, 64, 4, 1, 1, 2, dry_run=True)
    B.ll_cross_attn(c.h, None, None, None, None, n_q=10, n_k=3)
    for n_q, n_k in [(0, 3), (10, 0), (-1, 3), (1 << 31, 3)]:
        with pytest.raises(B.LLError):
            B.ll_cross_attn(c.h, None, None, None, None, n_q=n_q, n_k=n_k)
    with pytest.raises(B.LLError):
        B.ll_cross_attn(None, None, None, None, None, n_q=1, n_k=1)
    real = B.ll_cache_create(1, 2, 64, 4, 1, 1, 2)           # no storage bound: must refuse, not compute
    with pytest.raises(B.LLError) as e:
        B.ll_cross_attn(real, None, None, None, None, n_q=1, n_k=1)
    assert e.value.code in (B.LL_ERR_INVALID_ARG, B.LL_ERR_NO_STORAGE)
    B.ll_cache_destroy(real)
    assert c.state()["attn_calls"] == 0
