"""GPU: clearing a live cache (Algorithm 2, "C <- []") and streaming again over the
stale bytes; what a reported time-out leaves behind; a replayed graph after the
handle's RoPE tables have moved."""
import numpy as np
import pytest
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

from gpu_util import bits, check_attn, dev, f64, guarded, new_cache, ulp_distance

pytestmark = pytest.mark.gpu

F64 = synth.bf16_bits_to_f64

# 133-token frames: no slot boundary falls on a 128-row tile boundary, so the ragged last
# tile of every key run fetches rows of the slot behind it - stale rows after a reset
ODD = synth.Workload("reset_odd", 1, 2, 128, 7, 19, 1, 1, 3, n_chunks=7, seed=51)
MED = synth.Workload("reset_medium", 2, 3, 64, 9, 14, 2, 2, 4, n_chunks=6, seed=52)


def stream_chunks(oracle_mod, cache, orc, wl, seed_shift, n_chunks, layer=0):
    C, P = wl.chunk_frames, wl.tokens_per_frame
    for chunk in range(n_chunks):
        q, k, v = synth.chunk_qkv(wl, chunk, layer=layer, stream=seed_shift)
        dq, dk, dv = dev(q), dev(k), dev(v)
        q_out = torch.empty_like(dq)
        out, guard = guarded(dq.shape, fill=float("nan"))
        cache.rope_append_kv(layer, dq, dk, dv, chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
        cache.sink_window_attn(layer, q_out, chunk * C, out)
        cache.check_device()
        guard()
        orc.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        want, _ = orc.attn(0, orc.rope_q(F64(q), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta), chunk * C)
        check_attn(f64(out), want)
        st, ost = cache.state(layer), orc.state()
        assert st["end"] == ost["end"] and st["slot_frame"] == list(ost["slot_frame"])
        # the resident rows hold this stream's K/V, not the previous stream's
        K, V = orc.read_layer()
        vc = cache.kv_view(layer, 1)
        kc = cache.kv_view(layer, 0)
        for slot, frame in enumerate(st["slot_frame"]):
            if frame < 0:
                continue
            got_v = bits(vc[:, slot * P:(slot + 1) * P, :]).transpose(1, 0, 2)
            assert np.array_equal(got_v, synth.f32_to_bf16_bits(V[slot].astype(np.float32)))
            got_k = bits(kc[:, slot * P:(slot + 1) * P, :]).transpose(1, 0, 2)
            assert ulp_distance(got_k, synth.f32_to_bf16_bits(K[slot].astype(np.float32))).max() <= 1


@pytest.mark.parametrize("wl", [ODD, MED], ids=lambda w: w.name)
def test_reset_then_stream_again_over_stale_bytes(oracle_mod, wl):
    """Stream past the ring's wrap-around, clear the cache, stream different inputs: state,
    cache rows and attention match an oracle that was cleared at the same point.  The bytes
    of the first stream stay in the storage (reset does not touch the device) and sit right
    behind the rows the second stream's first chunks attend over."""
    cache = new_cache(wl)
    orcs = [oracle_mod.Oracle(1, wl.heads, wl.head_dim, wl.tokens_per_frame, wl.chunk_frames, wl.sink_frames,
                              wl.window_frames) for _ in range(wl.layers)]
    for layer in range(wl.layers):
        stream_chunks(oracle_mod, cache, orcs[layer], wl, 0, wl.n_chunks, layer)
    before = [cache.state(layer) for layer in range(wl.layers)]
    stale_v = bits(cache.kv_view(0, 1)).copy()
    cache.reset()
    for orc in orcs:
        orc.reset()
    for layer in range(wl.layers):
        st, ost = cache.state(layer), orcs[layer].state()
        assert st["end"] == 0 and st["end"] == ost["end"]
        assert st["slot_frame"] == [-1] * (wl.sink_frames + wl.window_frames) == list(ost["slot_frame"])
        assert st["appends"] == before[layer]["appends"] and st["evictions"] == ost["evictions"]   # lifetime counters stay
    assert np.array_equal(bits(cache.kv_view(0, 1)), stale_v)       # the stored bytes were not cleared
    q, _, _ = synth.chunk_qkv(wl, 0)
    with pytest.raises(B.LLError) as e:                              # nothing to attend over any more
        cache.sink_window_attn(0, dev(q), 0, torch.empty_like(dev(q)))
    assert e.value.code == B.LL_ERR_BAD_POSITION
    for layer in range(wl.layers):
        stream_chunks(oracle_mod, cache, orcs[layer], wl, 1, wl.n_chunks - 2, layer)
    cache.close()


def test_a_reported_timeout_also_clears_the_merge_counters(oracle_mod):
    """A launch that is abandoned leaves the arrival counters of the split-column merge
    mid-count.  Here the counters are dirtied by hand (the memory is the caller's), the
    bounded-wait probe produces a time-out record, and reading the record must leave both
    regions zero; a split-column launch right after it matches the oracle."""
    wl = synth.Workload("recover", 1, 2, 128, 10, 20, 3, 3, 9, n_chunks=4, seed=53)
    cache = new_cache(wl)
    orc = oracle_mod.Oracle(1, wl.heads, wl.head_dim, wl.tokens_per_frame, wl.chunk_frames, wl.sink_frames,
                            wl.window_frames)
    C = wl.chunk_frames
    for chunk in range(wl.n_chunks):
        q, k, v = synth.chunk_qkv(wl, chunk)
        dq = dev(q)
        q_out = torch.empty_like(dq)
        cache.rope_append_kv(0, dq, dev(k), dev(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
        orc.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
    plan = B.ll_debug_attn_plan(cache.h, 0, False, 0)
    assert plan.n_shares > 0                                          # this launch merges split columns
    s_off, s_bytes, c_off, c_bytes = B.ll_debug_aux_layout(cache.h)
    counters = cache.storage[c_off:c_off + c_bytes].view(torch.int32)
    status = cache.storage[s_off:s_off + s_bytes].view(torch.int32)
    cache.check_device()
    assert int(counters.abs().sum()) == 0                             # clean between launches
    counters.fill_(1)                                                 # what an abandoned launch leaves
    B.ll_debug_wait_timeout(cache.h, 20)
    with pytest.raises(B.LLError) as e:
        cache.check_device()
    assert e.value.code == B.LL_ERR_DEVICE_TIMEOUT
    torch.cuda.synchronize()
    assert int(counters.abs().sum()) == 0 and int(status.abs().sum()) == 0
    out = torch.full_like(q_out, float("nan"))
    last = wl.n_chunks - 1
    cache.sink_window_attn(0, q_out, last * C, out)
    cache.check_device()
    want, _ = orc.attn(0, orc.rope_q(F64(q), last * C, wl.grid_h, wl.grid_w, wl.rope_theta), last * C)
    check_attn(f64(out), want)
    assert int(counters.abs().sum()) == 0
    cache.close()


def test_replayed_append_after_the_tables_moved(oracle_mod):
    """A captured overwrite pass is replayed after another layer of the same handle was
    appended at a far-away position (which moves the handle's sine/cosine tables): the
    replay must still rotate with the angles of its own frames."""
    wl = synth.Workload("graph_tables", 2, 2, 128, 10, 20, 3, 3, 9, n_chunks=2, seed=54)
    C = wl.chunk_frames
    cache = new_cache(wl)
    q, k, v = synth.chunk_qkv(wl, 0)
    sq, sk, sv = dev(q), dev(k), dev(v)
    s_qout = torch.empty_like(sq)
    cache.rope_append_kv(0, sq, sk, sv, 0, wl.grid_h, wl.grid_w, wl.rope_theta, s_qout)     # commit chunk 0, eager
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        cache.rope_append_kv(0, sq, sk, sv, 0, wl.grid_h, wl.grid_w, wl.rope_theta, s_qout)  # overwrite pass
    # layer 1 of the same handle jumps to frame 900 (another table window) and appends there
    st = B.ll_cache_get_state(cache.h, 1)
    st.end = 900
    B.ll_cache_set_state(cache.h, 1, st)
    cache.rope_append_kv(1, sq, sk, sv, 900, wl.grid_h, wl.grid_w, wl.rope_theta, s_qout)
    q2, k2, v2 = synth.chunk_qkv(wl, 1)
    sq.copy_(dev(q2)); sk.copy_(dev(k2)); sv.copy_(dev(v2))
    s_qout.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    cache.check_device()
    want_q = synth.f32_to_bf16_bits(oracle_mod.rope(F64(q2), 0, wl.grid_h, wl.grid_w, wl.rope_theta).astype(np.float32))
    d = ulp_distance(bits(s_qout), want_q)
    assert d.max() <= 1 and (d == 0).mean() >= 0.99
    want_k = synth.f32_to_bf16_bits(oracle_mod.rope(F64(k2), 0, wl.grid_h, wl.grid_w, wl.rope_theta).astype(np.float32))
    P = wl.tokens_per_frame
    got_k = bits(cache.kv_view(0, 0)[:, :C * P, :]).transpose(1, 0, 2)
    assert ulp_distance(got_k, want_k).max() <= 1
    # and an eager call after the replay does not trust stale table state either
    cache.rope_append_kv(1, sq, sk, sv, 900, wl.grid_h, wl.grid_w, wl.rope_theta, s_qout)
    cache.check_device()
    want_q = synth.f32_to_bf16_bits(oracle_mod.rope(F64(q2), 900, wl.grid_h, wl.grid_w, wl.rope_theta).astype(np.float32))
    assert ulp_distance(bits(s_qout), want_q).max() <= 1
    cache.close()


def test_debug_handle_guard_bands_and_nvtx_ranges(oracle_mod, monkeypatch):
    """A handle created under LL_DEBUG keeps a 4 KB band of a fixed pattern in front of and
    behind its K/V region: a stream with wrap-around, a recache and a clip leave both intact
    (no kernel writes outside the layers' rows), and a band overwritten from the host is
    reported.  The calls run inside NVTX ranges (LL_NVTX) without changing any result."""
    monkeypatch.setenv("LL_DEBUG", "1")
    monkeypatch.setenv("LL_NVTX", "1")
    wl = synth.Workload("debug", 2, 2, 128, 7, 19, 1, 1, 4, n_chunks=7, seed=55)
    plain_bytes = None
    monkeypatch.delenv("LL_DEBUG")
    h = B.ll_cache_create(*wl.cache_args)
    plain_bytes = B.ll_cache_storage_bytes(h)
    B.ll_cache_destroy(h)
    monkeypatch.setenv("LL_DEBUG", "1")
    cache = B.Cache(*wl.cache_args)
    front, back, nbytes = B.ll_debug_guard_layout(cache.h)
    assert B.ll_cache_storage_bytes(cache.h) == plain_bytes + 2 * nbytes and back + nbytes == plain_bytes + 2 * nbytes
    orc = oracle_mod.Oracle(*wl.cache_args)
    C = wl.chunk_frames
    for layer in (0, 1):                                   # layer 0 touches the front band's neighbour rows, layer 1 the back's
        for chunk in range(wl.n_chunks):
            q, k, v = synth.chunk_qkv(wl, chunk, layer=layer)
            dq = dev(q)
            q_out, out = torch.empty_like(dq), torch.empty_like(dq)
            cache.rope_append_kv(layer, dq, dev(k), dev(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
            cache.sink_window_attn(layer, q_out, chunk * C, out)
            orc.append(layer, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        cache.check_device()
        want, _ = orc.attn(layer, orc.rope_q(F64(q), (wl.n_chunks - 1) * C, wl.grid_h, wl.grid_w, wl.rope_theta),
                           (wl.n_chunks - 1) * C)
        check_attn(f64(out), want)
        n = wl.window_frames
        rq, rk, rv = (dev(t) for t in synth.chunk_qkv(wl, 99, layer=layer, n_frames=n))
        cache.recache(layer, rq, rk, rv, n, wl.grid_h, wl.grid_w, wl.rope_theta, torch.empty_like(rq), torch.empty_like(rq))
        cache.check_device()
    band = cache.storage[back:back + nbytes]
    assert bool((band == 0xA5).all())
    band[17] = 0
    with pytest.raises(B.LLError) as e:
        cache.check_device()
    assert e.value.code == B.LL_ERR_DEVICE_CHECK and "behind" in str(e.value) and "byte 17" in str(e.value)
    band[17] = 0xA5
    cache.check_device()
    cache.close()
