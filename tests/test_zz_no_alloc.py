"""The allocation-free RoPE entry point against the regular one.

``ll_rope_q_static`` serves callers that have no way to hand the library a
storage block (everything on the GPU is already owned by someone else, or
allocating at call time is forbidden).  Its tables sit in a fixed array inside
the library, shared by every call, so the interesting failure is a call that
reads what an earlier call left behind.  The test therefore makes two calls in a
row with different frame positions and grids and compares each with the
rotated queries that ``ll_rope_append_kv`` produces for the same inputs, and
with the CPU oracle's rotation, under the bar every other RoPE test uses.

This file sorts last on purpose: a run that stops at the first failure has
already been through every other test when it gets here.
"""
import numpy as np
import pytest
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

from gpu_util import bits, dev, new_cache, ulp_distance

pytestmark = pytest.mark.gpu

# (workload, chunk whose queries are rotated): different grids, head sizes and frame offsets
CASES = [
    (synth.Workload("static_a", 1, 3, 128, 9, 14, 2, 2, 4, n_chunks=4, seed=21), 3),
    (synth.Workload("static_b", 1, 2, 64, 5, 31, 3, 3, 6, n_chunks=2, seed=22), 1),
]


def regular_q_out(wl, upto_chunk):
    """Rotated queries of chunk `upto_chunk` from ll_rope_append_kv (the existing entry point)."""
    cache = new_cache(wl)
    C = wl.chunk_frames
    q_out = None
    for chunk in range(upto_chunk + 1):
        q, k, v = synth.chunk_qkv(wl, chunk)
        dq, dk, dv = dev(q), dev(k), dev(v)
        q_out = torch.empty_like(dq)
        cache.rope_append_kv(0, dq, dk, dv, chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
    cache.check_device()
    cache.close()
    return bits(q_out)


def test_static_rope_matches_regular_entry_point_twice_in_a_row(oracle_mod):
    want = [regular_q_out(wl, chunk) for wl, chunk in CASES]
    want_oracle = [synth.f32_to_bf16_bits(
        oracle_mod.rope(synth.bf16_bits_to_f64(synth.chunk_qkv(wl, chunk)[0]), chunk * wl.chunk_frames,
                        wl.grid_h, wl.grid_w, wl.rope_theta).astype(np.float32)) for wl, chunk in CASES]
    launches0 = B.ll_launch_count()
    got = []
    for wl, chunk in CASES:                      # back to back: the second call finds the first one's tables
        q, _, _ = synth.chunk_qkv(wl, chunk)
        dq = dev(q)
        out = torch.empty_like(dq)
        B.ll_rope_q_static(dq, out, wl.heads, wl.head_dim, chunk * wl.chunk_frames, wl.chunk_frames,
                           wl.grid_h, wl.grid_w, wl.rope_theta)
        got.append(out)
    torch.cuda.synchronize()
    assert B.ll_launch_count() - launches0 == 2 * len(CASES)     # table kernel + rotation kernel per call
    for g, w, wo in zip(got, want, want_oracle):
        d = ulp_distance(bits(g), w)
        # the same fp32 arithmetic on the same fp64-built tables: the parity tests allow one bf16 ulp
        assert d.max() <= 1 and (d == 0).mean() >= 0.99
        d = ulp_distance(bits(g), wo)                # and the fp64 definition, rounded once
        assert d.max() <= 1 and (d == 0).mean() >= 0.99
    # and once more in the opposite order, in place
    for (wl, chunk), w in reversed(list(zip(CASES, want))):
        q, _, _ = synth.chunk_qkv(wl, chunk)
        dq = dev(q)
        B.ll_rope_q_static(dq, dq, wl.heads, wl.head_dim, chunk * wl.chunk_frames, wl.chunk_frames,
                           wl.grid_h, wl.grid_w, wl.rope_theta)
        d = ulp_distance(bits(dq), w)
        assert d.max() <= 1 and (d == 0).mean() >= 0.99


def test_static_rope_refuses_what_the_fixed_table_cannot_hold():
    x = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    for kwargs in [dict(n_frames=B.LL_STATIC_MAX_FRAMES + 1, grid_h=1, grid_w=1),
                   dict(n_frames=1, grid_h=1000, grid_w=B.LL_STATIC_MAX_GRID_SUM - 999)]:
        with pytest.raises(B.LLError) as e:
            B.ll_rope_q_static(x, x, 1, 64, 0, kwargs["n_frames"], kwargs["grid_h"], kwargs["grid_w"])
        assert e.value.code == B.LL_ERR_UNSUPPORTED_SHAPE
        assert "LL_STATIC_MAX" in str(e.value)
