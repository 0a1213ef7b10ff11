"""GPU parity of the clip step (Sec. 3.3, "Consistency between Training and
Inference"): several chunks appended and attended in one call under a sink plus
a local window shorter than the resident ring, against the CPU oracle; and the
property the paper wants from it: every chunk gets what chunk-by-chunk decoding
with that window gives."""
import numpy as np
import pytest
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

from gpu_util import bits, check_attn, dev, f64

pytestmark = pytest.mark.gpu

F64 = synth.bf16_bits_to_f64

# (name, heads, D, grid, C, S, W_a, clip chunks, chunks streamed before each clip)
CASES = [
    ("d128", 2, 128, (10, 20), 3, 3, 9, 4, (0, 5)),          # first clip starts the stream: holds the sink itself
    ("d64", 3, 64, (9, 14), 2, 2, 4, 5, (1, 4)),
    ("odd", 1, 128, (7, 19), 1, 1, 3, 6, (2, 9)),           # 133 tokens per frame: ragged tiles
    ("no_sink", 2, 128, (12, 12), 2, 0, 2, 3, (3,)),        # window = one chunk: each chunk sees itself only
]


def clip_inputs(wl, first_chunk, n_chunks):
    parts = [synth.chunk_qkv(wl, first_chunk + i) for i in range(n_chunks)]
    return tuple(np.concatenate([p[i] for p in parts]) for i in range(3))


@pytest.mark.parametrize("case", CASES, ids=lambda c: c[0])
def test_clip_matches_oracle_and_chunkwise_decoding(oracle_mod, case):
    name, H, D, (gh, gw), C, S, Wa, clip_chunks, befores = case
    T = clip_chunks * C
    ring = Wa + T - C
    P = gh * gw
    wl = synth.Workload(name, 1, H, D, gh, gw, C, S, ring, n_chunks=0, seed=41)
    for before in befores:
        cache = B.Cache(1, H, D, P, C, S, ring)
        small = B.Cache(1, H, D, P, C, S, Wa)                  # chunk-by-chunk decoding with window W_a
        orc = oracle_mod.Oracle(1, H, D, P, C, S, ring)
        nq = C * P
        for chunk in range(before):
            q, k, v = synth.chunk_qkv(wl, chunk)
            cache.rope_append_kv(0, None, dev(k), dev(v), chunk * C, gh, gw, wl.rope_theta)
            small.rope_append_kv(0, None, dev(k), dev(v), chunk * C, gh, gw, wl.rope_theta)
            orc.append(0, F64(k), F64(v), chunk * C, gh, gw, wl.rope_theta)
        # two clips in a row, so that the second one finds a wrapped ring
        for rep in range(2):
            first = before + rep * clip_chunks
            q, k, v = clip_inputs(wl, first, clip_chunks)
            dq, dk, dv = dev(q), dev(k), dev(v)
            q_out = torch.full_like(dq, float("nan"))
            out = torch.full_like(dq, float("nan"))
            lse = torch.full((H, T * P), float("nan"), device="cuda")
            cache.clip_append_attn(0, dq, dk, dv, first * C, T, Wa, gh, gw, wl.rope_theta, q_out, out, lse)
            cache.check_device()
            _, want, want_lse = orc.clip(0, F64(q), F64(k), F64(v), first * C, T, Wa, gh, gw, wl.rope_theta)
            check_attn(f64(out), want)
            assert np.abs(lse.cpu().numpy().T - want_lse).max() <= 2e-2
            st, ost = cache.state(), orc.state()
            assert st["end"] == ost["end"] and st["slot_frame"] == list(ost["slot_frame"])
            assert st["evictions"] == ost["evictions"]
            # the same chunks one at a time on the short ring
            for i in range(clip_chunks):
                sl = slice(i * nq, (i + 1) * nq)
                qo = torch.empty_like(dq[sl])
                o1 = torch.empty_like(dq[sl])
                small.rope_append_kv(0, dq[sl], dk[sl], dv[sl], (first + i) * C, gh, gw, wl.rope_theta, qo)
                small.sink_window_attn(0, qo, (first + i) * C, o1)
                assert np.array_equal(bits(qo), bits(q_out[sl]))            # same rotation, bit for bit
                d = (o1.float() - out[sl].float()).abs()
                assert d.max().item() <= 1e-2 and d.mean().item() <= 1e-3
            small.check_device()
        # decoding goes on from the clip's cache: the next chunk under the ring's own window
        q, k, v = synth.chunk_qkv(wl, before + 2 * clip_chunks)
        f0 = (before + 2 * clip_chunks) * C
        qo = torch.empty_like(dev(q))
        o1 = torch.empty_like(qo)
        cache.rope_append_kv(0, dev(q), dev(k), dev(v), f0, gh, gw, wl.rope_theta, qo)
        cache.sink_window_attn(0, qo, f0, o1)
        cache.check_device()
        orc.append(0, F64(k), F64(v), f0, gh, gw, wl.rope_theta)
        want, _ = orc.attn(0, orc.rope_q(F64(q), f0, gh, gw, wl.rope_theta), f0)
        check_attn(f64(o1), want)
        cache.close()
        small.close()
        orc.close()


def test_clip_at_the_benchmark_layer_shape(oracle_mod):
    """A 21-frame clip (7 chunks) behind 5 streamed chunks at the Wan-1.3B layer shape,
    checked on sampled rows of every chunk."""
    H, D, gh, gw, C, S, Wa, clip_chunks, before = 12, 128, 30, 52, 3, 3, 9, 7, 5
    T, P = clip_chunks * C, gh * gw
    ring = Wa + T - C
    wl = synth.Workload("clip_wan", 1, H, D, gh, gw, C, S, ring, n_chunks=0, seed=42)
    cache = B.Cache(1, H, D, P, C, S, ring)
    orc = oracle_mod.Oracle(1, H, D, P, C, S, ring)
    for chunk in range(before):
        _, k, v = synth.chunk_qkv(wl, chunk)
        cache.rope_append_kv(0, None, dev(k), dev(v), chunk * C, gh, gw, wl.rope_theta)
        orc.append(0, F64(k), F64(v), chunk * C, gh, gw, wl.rope_theta)
    q, k, v = clip_inputs(wl, before, clip_chunks)
    dq = dev(q)
    q_out, out = torch.empty_like(dq), torch.full_like(dq, float("nan"))
    cache.clip_append_attn(0, dq, dev(k), dev(v), before * C, T, Wa, gh, gw, wl.rope_theta, q_out, out)
    cache.check_device()
    assert torch.isfinite(out.float()).all()
    rows = np.concatenate([g * C * P + synth.sample_rows(C * P, 10, seed=g) for g in range(clip_chunks)])
    _, want, _ = orc.clip(0, F64(q), F64(k), F64(v), before * C, T, Wa, gh, gw, wl.rope_theta, rows=rows)
    check_attn(f64(out)[rows], want)
    assert cache.state()["slot_frame"] == list(orc.state()["slot_frame"])
    cache.close()
