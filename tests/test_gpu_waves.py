"""GPU parity of the attention kernel's whole-column mode, on every row.

A launch with at least as many work columns (256 query rows of one head) as SMs
hands the first columns out whole, one per persistent CTA and wave, and cuts the
steps of the columns left over into levelled shares whose parts are merged
through scratch slots.  That is the mode the benchmark shapes run in (228 columns
on 148 SMs).  The shapes here have many heads and small frames, so that they
reach it with few enough keys for the oracle to evaluate EVERY query row of
every head: decode, recache and the several-streams launch are compared element
by element, not sampled.  The closed-form histogram check (K = 0, V = one-hot of
the frame) needs no oracle and runs at the benchmark's full layer shape over all
4680 x 12 rows, through the same three launches."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

from gpu_util import bits, check_attn, dev, f64, guarded, new_cache

pytestmark = pytest.mark.gpu

F64 = synth.bf16_bits_to_f64

# 80 heads x 64: 512 query rows per chunk = 2 tiles per head = 160 columns (one whole wave on
# 148 SMs plus 12 shared columns of 12 steps); 52 heads x 128: 640 rows = 3 tiles per head (the
# third one 128 rows: a single MMA lane) = 156 columns of up to 20 steps.
WIDE64 = synth.Workload("wide_d64", 1, 80, 64, 16, 16, 2, 2, 4, n_chunks=5, seed=41)
WIDE128 = synth.Workload("wide_d128", 1, 52, 128, 16, 20, 2, 2, 6, n_chunks=6, seed=42)


def oracle_for(oracle_mod, wl):
    return oracle_mod.Oracle(1, wl.heads, wl.head_dim, wl.tokens_per_frame, wl.chunk_frames,
                             wl.sink_frames, wl.window_frames)


def plan_is_waves_plus_shares(cache, recache=False):
    plan = B.ll_debug_attn_plan(cache.h, 0, recache, 148)
    return plan.n_waves >= 1 and plan.n_shares > 0


@pytest.mark.parametrize("wl", [WIDE64, WIDE128], ids=lambda w: w.name)
def test_decode_in_whole_column_mode_every_row(oracle_mod, wl):
    cache = new_cache(wl)
    orc = oracle_for(oracle_mod, wl)
    C, P = wl.chunk_frames, wl.tokens_per_frame
    nq = C * P
    saw_mode = 0
    worst = (0.0, 0.0)
    for chunk in range(wl.n_chunks):
        q, k, v = synth.chunk_qkv(wl, chunk)
        dq, dk, dv = dev(q), dev(k), dev(v)
        q_out, q_guard = guarded(dq.shape)
        out, out_guard = guarded(dq.shape, fill=float("nan"))
        lse = torch.full((wl.heads, nq), float("nan"), device="cuda", dtype=torch.float32)
        cache.rope_append_kv(0, dq, dk, dv, chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
        saw_mode += plan_is_waves_plus_shares(cache)
        cache.sink_window_attn(0, q_out, chunk * C, out, lse)
        cache.check_device()
        q_guard()
        out_guard()
        orc.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        want, want_lse = orc.attn(0, orc.rope_q(F64(q), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta), chunk * C)
        e = check_attn(f64(out), want)
        worst = (max(worst[0], e[0]), max(worst[1], e[1]))
        assert np.abs(lse.cpu().numpy().T - want_lse).max() <= 2e-2
        assert cache.state()["slot_frame"] == list(orc.state()["slot_frame"])
    # the launches were of the kind this file is about (whole waves and shared steps)
    assert saw_mode >= wl.n_chunks - 1
    print("parity %s, every row, whole-column mode: worst max-abs %.3e mean-abs %.3e" % (wl.name, worst[0], worst[1]))
    cache.close()


@pytest.mark.parametrize("wl", [WIDE64, WIDE128], ids=lambda w: w.name)
def test_recache_in_whole_column_mode_every_row(oracle_mod, wl):
    cache = new_cache(wl)
    orc = oracle_for(oracle_mod, wl)
    C, P, W = wl.chunk_frames, wl.tokens_per_frame, wl.window_frames
    for chunk in range(wl.n_chunks):                 # past the wrap-around of the ring
        q, k, v = synth.chunk_qkv(wl, chunk)
        cache.rope_append_kv(0, None, dev(k), dev(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        orc.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
    assert plan_is_waves_plus_shares(cache, recache=True)
    rq, rk, rv = synth.chunk_qkv(wl, wl.n_chunks, pass_id=synth.RECACHE_PASS, n_frames=W)
    drq = dev(rq)
    rq_out, q_guard = guarded(drq.shape)
    out, out_guard = guarded(drq.shape, fill=float("nan"))
    lse = torch.full((wl.heads, W * P), float("nan"), device="cuda", dtype=torch.float32)
    cache.recache(0, drq, dev(rk), dev(rv), W, wl.grid_h, wl.grid_w, wl.rope_theta, rq_out, out, lse)
    cache.check_device()
    q_guard()
    out_guard()
    _, want, want_lse = orc.recache(0, F64(rq), F64(rk), F64(rv), W, wl.grid_h, wl.grid_w, wl.rope_theta)
    e = check_attn(f64(out), want)
    assert np.abs(lse.cpu().numpy().T - want_lse).max() <= 2e-2
    print("parity %s recache, every row: max-abs %.3e mean-abs %.3e" % (wl.name, e[0], e[1]))
    cache.close()


def test_several_streams_in_whole_column_mode_every_row(oracle_mod):
    """Three streams of the wide shape at different positions (first chunk, filling ring,
    wrapped ring) in one launch: 468 columns, three whole waves and a shared remainder
    that straddles streams with different key counts."""
    wl = WIDE128
    C = wl.chunk_frames
    positions = (0, 2, 5)
    caches, items, wants = [], [], []
    for stream, pos in enumerate(positions):
        cache = new_cache(wl)
        orc = oracle_for(oracle_mod, wl)
        for chunk in range(pos + 1):
            q, k, v = synth.chunk_qkv(wl, chunk, stream=stream)
            dq = dev(q)
            q_out = torch.empty_like(dq)
            cache.rope_append_kv(0, dq, dev(k), dev(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
            orc.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        want, _ = orc.attn(0, orc.rope_q(F64(q), pos * C, wl.grid_h, wl.grid_w, wl.rope_theta), pos * C)
        out, guard = guarded(q_out.shape, fill=float("nan"))
        caches.append(cache)
        items.append((cache, 0, q_out, pos * C, out, None))
        wants.append((want, guard))
        orc.close()
    plan = B.ll_debug_attn_plan_batched([(c.h, 0) for c in caches], 148)
    assert plan.n_waves >= 3 and plan.n_shares > 0
    B.Cache.sink_window_attn_batched(items)
    for cache, item, (want, guard) in zip(caches, items, wants):
        cache.check_device()
        guard()
        check_attn(f64(item[4]), want)
        cache.close()


# ---------------------------------------------------------------------------
# closed form at the benchmark's layer shape, every row of every head
# ---------------------------------------------------------------------------

def one_hot_frames(wl, frame_start, n_frames):
    """V whose rows are the one-hot code of their frame (index = frame mod head_dim)."""
    P, D = wl.tokens_per_frame, wl.head_dim
    v = torch.zeros(n_frames * P, wl.heads, D, device="cuda", dtype=torch.bfloat16)
    for i in range(n_frames):
        v[i * P:(i + 1) * P, :, (frame_start + i) % D] = 1.0
    return v


def histogram(wl, frames):
    want = np.zeros(wl.head_dim)
    want[[f % wl.head_dim for f in frames]] = 1.0 / len(frames)
    return want


def assert_histogram(out, want):
    """Every row of every head equals `want` up to one rounding of the uniform weight
    to bf16 (for the PV product) and one of the result."""
    got = f64(out)
    assert np.abs(got - want).max() <= 2.0 ** -8 * want.max() + 1e-6, np.abs(got - want).max()


def visible_frames(wl, end, chunk_end=None, r0=0):
    hi = end if chunk_end is None else chunk_end
    return [f for f in range(hi) if f < wl.sink_frames or f >= max(r0, hi - wl.window_frames)]


def test_closed_form_histogram_at_the_benchmark_shape():
    """Config-1 layer shape (4680 query rows x 12 heads, up to 18720 keys, 228 columns):
    decode at every fill level and after wrap-around, then a recache of the full window."""
    wl = synth.CONFIGS[1]
    C, P, W = wl.chunk_frames, wl.tokens_per_frame, wl.window_frames
    cache = new_cache(wl)
    q, _, _ = synth.chunk_qkv(wl, 0)
    dq = dev(q)
    k0 = torch.zeros_like(dq)
    out, guard = guarded(dq.shape, fill=float("nan"))
    for chunk in range(7):
        cache.rope_append_kv(0, dq, k0, one_hot_frames(wl, chunk * C, C), chunk * C, wl.grid_h, wl.grid_w)
        out.fill_(float("nan"))
        cache.sink_window_attn(0, dq, chunk * C, out)
        cache.check_device()
        guard()
        assert_histogram(out, histogram(wl, visible_frames(wl, (chunk + 1) * C)))
    end = 7 * C
    r0 = end - W
    rq = torch.cat([dq] * (W // C))
    r_out, r_guard = guarded(rq.shape, fill=float("nan"))
    rq_out = torch.empty_like(rq)
    cache.recache(0, rq, torch.zeros_like(rq), one_hot_frames(wl, r0, W), W, wl.grid_h, wl.grid_w, wl.rope_theta,
                  rq_out, r_out)
    cache.check_device()
    r_guard()
    for g in range(W // C):
        rows = slice(g * C * P, (g + 1) * C * P)
        assert_histogram(r_out[rows], histogram(wl, visible_frames(wl, end, chunk_end=r0 + (g + 1) * C, r0=r0)))
    cache.close()


def test_closed_form_histogram_of_eight_streams_in_one_launch():
    """The benchmark's serving case: eight streams of the config-1 layer shape at the ragged
    positions of config 4, one launch; every row of every stream is its own histogram."""
    wl = synth.CONFIGS[1]
    C = wl.chunk_frames
    q, _, _ = synth.chunk_qkv(wl, 0)
    dq = dev(q)
    k0 = torch.zeros_like(dq)
    caches, items, checks = [], [], []
    for pos in synth.SWEEP_POSITIONS[:7] + (9,):
        cache = new_cache(wl)
        first = max(1, pos + 1 - wl.window_frames // C)
        chunks = [0] + list(range(first, pos + 1)) if pos > 0 else [0]
        for chunk in chunks:
            if chunk == first and pos > 0 and first > 1:
                st = B.ll_cache_get_state(cache.h, 0)       # jump over the chunks that were evicted anyway
                st.end = first * C
                B.ll_cache_set_state(cache.h, 0, st)
            cache.rope_append_kv(0, None, k0, one_hot_frames(wl, chunk * C, C), chunk * C, wl.grid_h, wl.grid_w)
        out, guard = guarded(dq.shape, fill=float("nan"))
        caches.append(cache)
        items.append((cache, 0, dq, pos * C, out, None))
        checks.append((guard, histogram(wl, visible_frames(wl, (pos + 1) * C))))
    B.Cache.sink_window_attn_batched(items)
    for cache, item, (guard, want) in zip(caches, items, checks):
        cache.check_device()
        guard()
        assert_histogram(item[4], want)
        cache.close()
