"""GPU parity of the one-launch attention over several streams: caches that
differ in frame size, chunk length, sink, window, fill and layer share a launch,
and every stream's output is checked against the CPU oracle of that stream
alone.  Also the work division when a launch has fewer shared steps than CTAs."""
import numpy as np
import pytest
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

from gpu_util import bits, check_attn, dev, f64, new_cache

pytestmark = pytest.mark.gpu

F64 = synth.bf16_bits_to_f64

# heads and head_dim agree (a launch needs that); everything else differs
STREAMS = [
    (synth.Workload("a", 2, 2, 128, 10, 20, 3, 3, 9, n_chunks=7, seed=21), 6),     # wrapped ring, two layers
    (synth.Workload("b", 1, 2, 128, 7, 19, 1, 1, 3, n_chunks=6, seed=22), 2),       # 133-token frames, ragged tiles
    (synth.Workload("c", 1, 2, 128, 16, 20, 2, 2, 12, n_chunks=3, seed=23), 0),     # first chunk only: sees itself
    (synth.Workload("d", 1, 2, 128, 12, 12, 4, 0, 4, n_chunks=5, seed=24), 4),      # no sink
]


class Stream:
    """One cache advanced to `last` chunks, with an oracle fed the same inputs per layer."""

    def __init__(self, oracle_mod, wl, last):
        self.wl, self.last = wl, last
        self.cache = new_cache(wl)
        self.items = []
        C = wl.chunk_frames
        for layer in range(wl.layers):
            orc = oracle_mod.Oracle(1, wl.heads, wl.head_dim, wl.tokens_per_frame, wl.chunk_frames,
                                    wl.sink_frames, wl.window_frames)
            for chunk in range(last + 1):
                q, k, v = synth.chunk_qkv(wl, chunk, layer=layer)
                dq = dev(q)
                q_out = torch.empty_like(dq)
                self.cache.rope_append_kv(layer, dq, dev(k), dev(v), chunk * C, wl.grid_h, wl.grid_w,
                                          wl.rope_theta, q_out)
                orc.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
            qr = orc.rope_q(F64(q), last * C, wl.grid_h, wl.grid_w, wl.rope_theta)
            want, want_lse = orc.attn(0, qr, last * C)
            out = torch.full_like(q_out, float("nan"))
            lse = torch.full((wl.heads, C * wl.tokens_per_frame), float("nan"), device="cuda")
            self.items.append(dict(layer=layer, q=q_out, out=out, lse=lse, want=want, want_lse=want_lse))

    def launch_items(self, with_lse=True):
        C = self.wl.chunk_frames
        return [(self.cache, it["layer"], it["q"], self.last * C, it["out"], it["lse"] if with_lse else None)
                for it in self.items]

    def check(self):
        self.cache.check_device()
        for it in self.items:
            check_attn(f64(it["out"]), it["want"])
            got_lse = it["lse"].cpu().numpy().T.astype(np.float64)
            assert np.abs(got_lse - it["want_lse"]).max() <= 2e-2


def test_streams_of_different_shape_in_one_launch(oracle_mod):
    streams = [Stream(oracle_mod, wl, last) for wl, last in STREAMS]
    items = [it for s in streams for it in s.launch_items()]
    assert len(items) == 5
    B.Cache.sink_window_attn_batched(items)
    for s in streams:
        s.check()
        assert all(s.cache.state(layer)["attn_calls"] == 1 for layer in range(s.wl.layers))
    # the same launch again gives the same bits
    first = [bits(it[4]).copy() for it in items]
    for it in items:
        it[4].fill_(float("nan"))
    B.Cache.sink_window_attn_batched(items)
    for before, it in zip(first, items):
        assert np.array_equal(before, bits(it[4]))
    # and any order of the items gives results within the same bar
    for it in items:
        it[4].fill_(float("nan"))
    B.Cache.sink_window_attn_batched(items[::-1])
    for s in streams:
        s.check()
        s.cache.close()


def test_one_item_launch_equals_the_plain_call(oracle_mod):
    s = Stream(oracle_mod, *STREAMS[0])
    item = s.launch_items()[1]
    B.Cache.sink_window_attn_batched([item])
    got = bits(item[4]).copy()
    got_lse = item[5].clone()
    item[4].fill_(float("nan"))
    s.cache.sink_window_attn(item[1], item[2], item[3], item[4], item[5])
    assert np.array_equal(got, bits(item[4])) and torch.equal(got_lse, item[5])
    s.cache.check_device()
    s.cache.close()


def test_errors_launch_nothing(oracle_mod):
    a = Stream(oracle_mod, *STREAMS[1])
    item = a.launch_items()[0]
    other_wl = synth.Workload("e", 1, 3, 128, 4, 4, 1, 1, 3, n_chunks=1, seed=25)      # 3 heads
    other = new_cache(other_wl)
    q, k, v = (dev(t) for t in synth.chunk_qkv(other_wl, 0))
    q_out = torch.empty_like(q)
    other.rope_append_kv(0, q, k, v, 0, other_wl.grid_h, other_wl.grid_w, other_wl.rope_theta, q_out)
    out = torch.empty_like(q_out)
    with pytest.raises(B.LLError) as e:
        B.Cache.sink_window_attn_batched([item, (other, 0, q_out, 0, out, None)])
    assert e.value.code == B.LL_ERR_UNSUPPORTED_SHAPE
    with pytest.raises(B.LLError):
        B.Cache.sink_window_attn_batched([item, item])                       # the same layer twice
    with pytest.raises(B.LLError):
        B.Cache.sink_window_attn_batched([item[:3] + (0,) + item[4:]])       # not the newest chunk
    assert torch.isnan(item[4].float()).all()
    assert a.cache.state()["attn_calls"] == 0 and other.state()["attn_calls"] == 0
    a.cache.check_device()
    a.cache.close()
    other.close()


def test_split_column_with_fewer_shared_steps_than_ctas(oracle_mod):
    """150 columns on a 148-SM device: 148 go out whole and the 58 steps of the last
    two are fewer than the CTAs, so most CTAs take no share; the parts of each
    split column must still be found and merged."""
    wl = synth.Workload("few_shared", 1, 10, 128, 50, 74, 1, 0, 1, n_chunks=1, seed=26)
    assert wl.tokens_per_frame == 3700
    cache = new_cache(wl)
    orc = oracle_mod.Oracle(1, wl.heads, wl.head_dim, wl.tokens_per_frame, 1, 0, 1)
    q, k, v = synth.chunk_qkv(wl, 0)
    dq = dev(q)
    q_out = torch.empty_like(dq)
    out = torch.full_like(dq, float("nan"))
    cache.rope_append_kv(0, dq, dev(k), dev(v), 0, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
    cache.sink_window_attn(0, q_out, 0, out)
    cache.check_device()
    plan = B.ll_debug_attn_plan(cache.h)
    if plan.n_ctas == 148:
        assert plan.wave_cols[0] == 148 and plan.shared_steps == 58 and plan.n_shares == 58
    assert torch.isfinite(out.float()).all()
    orc.append(0, F64(k), F64(v), 0, wl.grid_h, wl.grid_w, wl.rope_theta)
    qr = orc.rope_q(F64(q), 0, wl.grid_h, wl.grid_w, wl.rope_theta)
    # every row of the two split columns (head 9, the last two query tiles) and a sample of the rest
    rows = np.concatenate([np.arange(13 * 256, 3700), synth.sample_rows(13 * 256, 64, seed=1)])
    want, _ = orc.attn(0, qr, 0, rows=rows)
    check_attn(f64(out)[rows], want)
    cache.close()
