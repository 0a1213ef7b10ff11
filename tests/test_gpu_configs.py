"""GPU parity at the benchmark's full sizes (configs 1-4), in the launch
configuration bench.py times, on sampled query rows the oracle evaluates one by
one; integer state bit-exact for every chunk of every layer."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

from gpu_util import bits, check_attn, check_attn_outliers, dev, f64, new_cache

pytestmark = pytest.mark.gpu

F64 = synth.bf16_bits_to_f64


def make_oracle(oracle_mod, wl, faithful=False):
    return oracle_mod.Oracle(1, wl.heads, wl.head_dim, wl.tokens_per_frame, wl.chunk_frames,
                             wl.sink_frames, wl.window_frames, faithful=faithful)


def state_oracle(oracle_mod, wl):
    """A one-token oracle: the integer state does not depend on tensor sizes."""
    return oracle_mod.Oracle(1, 1, 2, 1, wl.chunk_frames, wl.sink_frames, wl.window_frames)


def same_state(cache, layer, orc):
    st, ost = cache.state(layer), orc.state()
    return st["end"] == ost["end"] and st["slot_frame"] == list(ost["slot_frame"]) and \
        st["evictions"] == ost["evictions"]


class DevicePool:
    def __init__(self, pool):
        self.pool = pool
        self.sets = [tuple(dev(t) for t in s) for s in pool.sets]

    def get(self, *key):
        return self.sets[self.pool.index(*key)]


# Rows the oracle evaluates per checked call: the first and last row of every 128-row
# query tile (74 of them at 4680 rows) plus random rows.
N_ROWS = 256


def check_rows(orc, cache_out, q_bits, frame_start, wl, seed, orc_abs=None, orc_truth=None, label=""):
    nq = wl.chunk_tokens
    rows = synth.sample_rows(nq, N_ROWS, seed=seed)
    qr = orc.rope_q(F64(q_bits), frame_start, wl.grid_h, wl.grid_w, wl.rope_theta)
    want, _ = orc.attn(0, qr, frame_start, rows=rows)
    got = f64(cache_out)[rows]
    if orc_abs is None:
        return check_attn(got, want)
    scale = orc_abs.attn(0, qr, frame_start, rows=rows)[0]
    q_true = orc_truth.rope_q(F64(q_bits), frame_start, wl.grid_h, wl.grid_w, wl.rope_theta)
    truth = orc_truth.attn(0, q_true, frame_start, rows=rows)[0]
    return check_attn_outliers(got, want, scale, truth, label=label)


# ---------------------------------------------------------------------------
# config 1: one Wan-1.3B-shaped layer, streamed
# ---------------------------------------------------------------------------

def test_config1_streamed_layer(oracle_mod):
    wl = synth.CONFIGS[1]
    C = wl.chunk_frames
    cache = new_cache(wl)
    orc = make_oracle(oracle_mod, wl)
    worst = (0.0, 0.0)
    for chunk in range(7):                      # ramp-up (1, 2, 3 ring chunks), steady state, wrapped ring
        q, k, v = synth.chunk_qkv(wl, chunk)
        dq, dk, dv = dev(q), dev(k), dev(v)
        q_out = torch.empty_like(dq)
        out = torch.full_like(dq, float("nan"))
        cache.rope_append_kv(0, dq, dk, dv, chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
        cache.sink_window_attn(0, q_out, chunk * C, out)
        cache.check_device()
        assert torch.isfinite(out.float()).all()
        orc.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        assert cache.state()["slot_frame"] == list(orc.state()["slot_frame"])
        if chunk in (0, 2, 3, 6):
            e = check_rows(orc, out, q, chunk * C, wl, chunk)
            worst = (max(worst[0], e[0]), max(worst[1], e[1]))
    print("parity config1: worst max-abs %.3e mean-abs %.3e" % worst)
    cache.close()


# ---------------------------------------------------------------------------
# config 2: 30 layers x (4 denoising passes + commit) x 7 chunks; sink+window vs full causal
# ---------------------------------------------------------------------------

def run_full_stack(oracle_mod, wl, dpool, check_layers, check_chunks):
    C, L = wl.chunk_frames, wl.layers
    passes = wl.steps_per_chunk + 1
    cache = new_cache(wl)
    orcs = {l: make_oracle(oracle_mod, wl) for l in check_layers}
    sorc = state_oracle(oracle_mod, wl)
    nq = wl.chunk_tokens
    q_out = torch.empty(nq, wl.heads, wl.head_dim, device="cuda", dtype=torch.bfloat16)
    out = torch.empty_like(q_out)
    kept = {}
    x = np.zeros((C, 1, 2))
    for chunk in range(wl.n_chunks):
        for p in range(passes):
            for layer in range(L):
                dq, dk, dv = dpool.get(chunk, layer, p)
                cache.rope_append_kv(layer, dq, dk, dv, chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
                cache.sink_window_attn(layer, q_out, chunk * C, out)
                if p == passes - 1 and layer in check_layers:
                    kept[(layer, chunk)] = out.clone()
        cache.check_device()
        sorc.append(0, x, x, chunk * C, 1, 1)
        assert all(same_state(cache, l, sorc) for l in range(L))
        for layer in check_layers:
            q, k, v = dpool.pool.get(chunk, layer, passes - 1)
            orcs[layer].append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
            if chunk in check_chunks:
                check_rows(orcs[layer], kept[(layer, chunk)], q, chunk * C, wl, chunk)
    assert cache.state(0)["overwrites"] == wl.n_chunks * (passes - 1)
    cache.close()
    return kept


def test_config2_full_stack_and_full_causal_equivalence(oracle_mod):
    wl = synth.CONFIGS[2]
    dpool = DevicePool(synth.InputPool(wl))
    a = run_full_stack(oracle_mod, wl, dpool, (3, 29), (0, 4, 6))
    b = run_full_stack(oracle_mod, synth.FULL_CAUSAL, dpool, (3, 29), (0, 6))
    # while the window still covers the whole history the two runs are the same computation
    n_same = (wl.sink_frames + wl.window_frames) // wl.chunk_frames
    for (layer, chunk), t in a.items():
        same = torch.equal(t, b[(layer, chunk)])
        assert same == (chunk < n_same), (layer, chunk)


# ---------------------------------------------------------------------------
# config 3: 320 chunks x 30 layers, recache every 40 chunks
# ---------------------------------------------------------------------------

def test_config3_long_stream(oracle_mod):
    wl = synth.CONFIGS[3]
    C, L, W, S = wl.chunk_frames, wl.layers, wl.window_frames, wl.sink_frames
    passes = wl.steps_per_chunk + 1
    pool = synth.InputPool(wl)
    dpool = DevicePool(pool)
    rpool = synth.InputPool(wl, n_sets=2, n_frames=W, pass_id=synth.RECACHE_PASS)
    drpool = DevicePool(rpool)
    cache = new_cache(wl)
    storage_bytes = B.ll_cache_storage_bytes(cache.h)
    sorc = state_oracle(oracle_mod, wl)
    nq = wl.chunk_tokens
    q_out = torch.empty(nq, wl.heads, wl.head_dim, device="cuda", dtype=torch.bfloat16)
    out = torch.empty_like(q_out)
    rq_out = torch.empty(W * wl.tokens_per_frame, wl.heads, wl.head_dim, device="cuda", dtype=torch.bfloat16)
    r_out = torch.empty_like(rq_out)
    x = np.zeros((C, 1, 2))
    e = np.zeros((W, 1, 2))
    probe_layer = 11
    kept, timing = {}, {}
    sink_before = None
    for chunk in range(wl.n_chunks):
        if chunk and chunk % synth.LONG_STREAM_SWITCH_EVERY == 0:
            for layer in range(L):
                dq, dk, dv = drpool.get(chunk, layer)
                cache.recache(layer, dq, dk, dv, W, wl.grid_h, wl.grid_w, wl.rope_theta, rq_out, r_out)
                if layer == probe_layer and chunk == 40:
                    kept["recache"] = r_out.clone()
            sorc.recache(0, e, e, e, W, 1, 1)
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for p in range(passes):
            for layer in range(L):
                dq, dk, dv = dpool.get(chunk, layer, p)
                cache.rope_append_kv(layer, dq, dk, dv, chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
                cache.sink_window_attn(layer, q_out, chunk * C, out)
                if p == passes - 1 and (layer, chunk) in ((probe_layer, 10), (probe_layer, 40), (29, 319)):
                    kept[(layer, chunk)] = out.clone()
        t1.record()
        sorc.append(0, x, x, chunk * C, 1, 1)
        if chunk % 16 == 0 or chunk in (39, 40, 41, 319):
            cache.check_device()
            assert all(same_state(cache, l, sorc) for l in (0, probe_layer, L - 1)), chunk
            timing[chunk] = t0.elapsed_time(t1)
        if chunk == 0:
            sink_before = bits(cache.kv_view(probe_layer, 0)[:, :S * wl.tokens_per_frame]).copy()
    cache.check_device()
    assert all(same_state(cache, l, sorc) for l in range(L))
    st = cache.state(0)
    assert st["end"] == 960 and st["recaches"] == 7 and st["slot_frame"][:S] == [0, 1, 2]
    assert B.ll_cache_storage_bytes(cache.h) == storage_bytes           # O(W+S), not O(video length)
    # sink bytes never change after chunk 0 (recaches included)
    assert np.array_equal(bits(cache.kv_view(probe_layer, 0)[:, :S * wl.tokens_per_frame]), sink_before)
    # per-chunk latency does not grow with the stream (ring full from chunk 3 on)
    early, late = timing[16], timing[304]
    print("config3 per-chunk latency: chunk 16 %.2f ms, chunk 304 %.2f ms" % (early, late))
    assert late < 1.25 * early

    last = passes - 1
    # (a) chunk 10: sink + chunks 7..10
    orc = make_oracle(oracle_mod, wl)
    _, k, v = pool.get(0, probe_layer, last)
    orc.append(0, F64(k), F64(v), 0, wl.grid_h, wl.grid_w, wl.rope_theta)
    orc.seek(0, 7 * C)
    for c in range(7, 11):
        q, k, v = pool.get(c, probe_layer, last)
        orc.append(0, F64(k), F64(v), c * C, wl.grid_h, wl.grid_w, wl.rope_theta)
    check_rows(orc, kept[(probe_layer, 10)], q, 10 * C, wl, 10)
    # (b) the recache before chunk 40 rebuilds chunks 37..39, then chunk 40 attends over them
    orc.seek(0, 37 * C)
    for c in range(37, 40):
        q, k, v = pool.get(c, probe_layer, last)
        orc.append(0, F64(k), F64(v), c * C, wl.grid_h, wl.grid_w, wl.rope_theta)
    rq, rk, rv = rpool.get(40, probe_layer)
    rows = synth.sample_rows(W * wl.tokens_per_frame, 384, seed=40)
    _, want, _ = orc.recache(0, F64(rq), F64(rk), F64(rv), W, wl.grid_h, wl.grid_w, wl.rope_theta, rows=rows)
    check_attn(f64(kept["recache"])[rows], want)
    q, k, v = pool.get(40, probe_layer, last)
    orc.append(0, F64(k), F64(v), 40 * C, wl.grid_h, wl.grid_w, wl.rope_theta)
    check_rows(orc, kept[(probe_layer, 40)], q, 40 * C, wl, 40)
    orc.close()
    # (c) the last chunk of the 240 s stream, last layer
    orc = make_oracle(oracle_mod, wl)
    _, k, v = pool.get(0, 29, last)
    orc.append(0, F64(k), F64(v), 0, wl.grid_h, wl.grid_w, wl.rope_theta)
    orc.seek(0, 316 * C)
    for c in range(316, 320):
        q, k, v = pool.get(c, 29, last)
        orc.append(0, F64(k), F64(v), c * C, wl.grid_h, wl.grid_w, wl.rope_theta)
    check_rows(orc, kept[(29, 319)], q, 319 * C, wl, 319)
    assert list(orc.state()["slot_frame"]) == cache.state(29)["slot_frame"]
    cache.close()


# ---------------------------------------------------------------------------
# config 4: ragged stream positions x window sweep, 1% outliers x20
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("batched", [False, True], ids=["per_stream", "one_launch"])
@pytest.mark.parametrize("W", synth.SWEEP_WINDOWS)
def test_config4_ragged_streams_window_sweep(oracle_mod, W, batched):
    """Each stream owns a cache and sits at its own position; the attention of the
    newest chunk runs either as one call per stream or as one launch for all."""
    wl = dataclasses.replace(synth.CONFIGS[4], window_frames=W)
    C, S = wl.chunk_frames, wl.sink_frames
    pool = synth.InputPool(wl)
    dpool = DevicePool(pool)
    positions = synth.SWEEP_POSITIONS if W == 9 else (0, 2, 6, 50)
    nq = wl.chunk_tokens
    caches, q_outs, outs = [], [], []
    for stream, pos in enumerate(positions):
        cache = new_cache(wl)
        q_out = torch.empty(nq, wl.heads, wl.head_dim, device="cuda", dtype=torch.bfloat16)
        for chunk in range(pos + 1):
            dq, dk, dv = dpool.get(chunk, 0, 0, stream)
            cache.rope_append_kv(0, dq, dk, dv, chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
        caches.append(cache)
        q_outs.append(q_out)
        outs.append(torch.full_like(q_out, float("nan")))
    if batched:
        B.Cache.sink_window_attn_batched([(cache, 0, q_out, pos * C, out, None)
                                          for cache, q_out, out, pos in zip(caches, q_outs, outs, positions)])
    else:
        for cache, q_out, out, pos in zip(caches, q_outs, outs, positions):
            cache.sink_window_attn(0, q_out, pos * C, out)
    worst = (0.0, 0.0)
    for stream, pos in enumerate(positions):
        cache, out = caches[stream], outs[stream]
        cache.check_device()
        assert cache.state()["attn_calls"] == 1
        # reference: storage-faithful oracle; a twin with |V| gives the error scale sum_j p_j |v_j|
        orc = make_oracle(oracle_mod, wl, faithful=True)
        orc_abs = make_oracle(oracle_mod, wl, faithful=True)
        orc_truth = make_oracle(oracle_mod, wl, faithful=False)       # unrounded rotations: the raw figure
        first = max(1, pos + 1 - W // C)
        for chunk in [0] + list(range(first, pos + 1)):
            if chunk == first and pos > 0:
                for o in (orc, orc_abs, orc_truth):
                    o.seek(0, first * C)
            _, k, v = pool.get(chunk, 0, 0, stream)
            orc.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
            orc_abs.append(0, F64(k), np.abs(F64(v)), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
            orc_truth.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        assert cache.state()["slot_frame"] == list(orc.state()["slot_frame"]), (W, pos)
        q, _, _ = pool.get(pos, 0, 0, stream)
        e = check_rows(orc, out, q, pos * C, wl, pos, orc_abs=orc_abs, orc_truth=orc_truth,
                       label="config4 W=%d stream %d (chunk %d)" % (W, stream, pos))
        worst = (max(worst[0], e[0]), max(worst[1], e[1]))
        orc.close()
        orc_abs.close()
        orc_truth.close()
        cache.close()
    print("parity config4 W=%d %s: worst scaled max %.3e mean %.3e"
          % (W, "one launch" if batched else "per stream", worst[0], worst[1]))
