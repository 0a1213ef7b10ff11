"""GPU parity at the limits the header states: 64 slots, 24 query groups in one
launch (recache of a 24-chunk window, a 24-chunk clip), one-token frames, and a
window of a single chunk."""
import numpy as np
import pytest
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

from gpu_util import check_attn, dev, f64

pytestmark = pytest.mark.gpu

F64 = synth.bf16_bits_to_f64


def stream_chunks(cache, orc, wl, chunks):
    C = wl.chunk_frames
    for chunk in chunks:
        _, k, v = synth.chunk_qkv(wl, chunk)
        cache.rope_append_kv(0, None, dev(k), dev(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        orc.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)


def test_recache_of_24_chunks_in_64_slots(oracle_mod):
    """S + W = 16 + 48 = 64 slots, chunks of 2 frames: the recache launches 24 query groups, and
    after 40 chunks the ring has wrapped, so most groups see three runs of cache rows."""
    wl = synth.Workload("limits", 1, 2, 64, 5, 7, 2, 16, 48, n_chunks=40, seed=61)
    P, C, W = wl.tokens_per_frame, wl.chunk_frames, wl.window_frames
    cache = B.Cache(1, wl.heads, wl.head_dim, P, C, wl.sink_frames, W)
    orc = oracle_mod.Oracle(1, wl.heads, wl.head_dim, P, C, wl.sink_frames, W)
    stream_chunks(cache, orc, wl, range(40))
    plan = B.ll_debug_attn_plan(cache.h, recache=True)
    assert plan.n_groups == 24
    q, k, v = synth.chunk_qkv(wl, 100, pass_id=synth.RECACHE_PASS, n_frames=W)
    dq = dev(q)
    q_out, out = torch.empty_like(dq), torch.full_like(dq, float("nan"))
    lse = torch.full((wl.heads, W * P), float("nan"), device="cuda")
    cache.recache(0, dq, dev(k), dev(v), W, wl.grid_h, wl.grid_w, wl.rope_theta, q_out, out, lse)
    cache.check_device()
    _, want, want_lse = orc.recache(0, F64(q), F64(k), F64(v), W, wl.grid_h, wl.grid_w, wl.rope_theta)
    check_attn(f64(out), want)
    assert np.abs(lse.cpu().numpy().T - want_lse).max() <= 2e-2
    # decoding goes on over the rebuilt ring
    q, k, v = synth.chunk_qkv(wl, 40)
    qo = torch.empty_like(dev(q))
    o1 = torch.empty_like(qo)
    cache.rope_append_kv(0, dev(q), dev(k), dev(v), 80, wl.grid_h, wl.grid_w, wl.rope_theta, qo)
    cache.sink_window_attn(0, qo, 80, o1)
    cache.check_device()
    orc.append(0, F64(k), F64(v), 80, wl.grid_h, wl.grid_w, wl.rope_theta)
    want, _ = orc.attn(0, orc.rope_q(F64(q), 80, wl.grid_h, wl.grid_w, wl.rope_theta), 80)
    check_attn(f64(o1), want)
    st, ost = cache.state(), orc.state()
    assert st["end"] == ost["end"] == 82 and st["slot_frame"] == list(ost["slot_frame"])
    cache.close()


def test_longest_clip_a_ring_takes(oracle_mod):
    """A ring is at most 24 chunks long; with a window of 4 one-frame chunks that leaves room for a
    clip of 21 chunks (4 + 21 - 1 = 24), all attended in one launch of 21 query groups."""
    C, S, Wa, n = 1, 2, 4, 21
    wl = synth.Workload("clip21", 1, 3, 128, 6, 9, C, S, Wa + n - C, n_chunks=0, seed=62)
    P = wl.tokens_per_frame
    cache = B.Cache(1, wl.heads, wl.head_dim, P, C, S, wl.window_frames)
    orc = oracle_mod.Oracle(1, wl.heads, wl.head_dim, P, C, S, wl.window_frames)
    stream_chunks(cache, orc, wl, range(7))
    parts = [synth.chunk_qkv(wl, 7 + i) for i in range(n)]
    q, k, v = (np.concatenate([p[i] for p in parts]) for i in range(3))
    dq = dev(q)
    q_out, out = torch.empty_like(dq), torch.full_like(dq, float("nan"))
    cache.clip_append_attn(0, dq, dev(k), dev(v), 7, n, Wa, wl.grid_h, wl.grid_w, wl.rope_theta, q_out, out)
    cache.check_device()
    _, want, _ = orc.clip(0, F64(q), F64(k), F64(v), 7, n, Wa, wl.grid_h, wl.grid_w, wl.rope_theta)
    check_attn(f64(out), want)
    assert cache.state()["slot_frame"] == list(orc.state()["slot_frame"])
    before = cache.state()
    with pytest.raises(B.LLError) as e:                  # one chunk more does not fit the ring: refused, nothing launched
        cache.clip_append_attn(0, dq, dev(k), dev(v), 28, n + 1, Wa, wl.grid_h, wl.grid_w, wl.rope_theta, q_out, out)
    assert e.value.code == B.LL_ERR_UNSUPPORTED_SHAPE and cache.state() == before
    cache.close()


def test_one_token_frames_and_a_window_of_one_chunk(oracle_mod):
    """P = 1: every tile is ragged (3 query rows, at most 6 keys); W = C: a chunk sees the sink and itself."""
    wl = synth.Workload("one_token", 1, 2, 64, 1, 1, 3, 3, 3, n_chunks=6, seed=63)
    cache = B.Cache(1, wl.heads, wl.head_dim, 1, 3, 3, 3)
    orc = oracle_mod.Oracle(1, wl.heads, wl.head_dim, 1, 3, 3, 3)
    for chunk in range(wl.n_chunks):
        q, k, v = synth.chunk_qkv(wl, chunk)
        qo = torch.empty_like(dev(q))
        out = torch.full_like(qo, float("nan"))
        cache.rope_append_kv(0, dev(q), dev(k), dev(v), 3 * chunk, 1, 1, wl.rope_theta, qo)
        cache.sink_window_attn(0, qo, 3 * chunk, out)
        cache.check_device()
        orc.append(0, F64(k), F64(v), 3 * chunk, 1, 1, wl.rope_theta)
        want, _ = orc.attn(0, orc.rope_q(F64(q), 3 * chunk, 1, 1, wl.rope_theta), 3 * chunk)
        check_attn(f64(out), want)
    cache.close()
