"""GPU: the denoising passes of a chunk as a captured CUDA graph.

After the pass that commits a chunk, every further pass over it re-appends the
chunk at the same frames (overwriting its K/V in place) and attends from the
same positions: the launches of such a pass have the same parameters each time,
only the contents of the input buffers differ (Algorithm 2's inner loop over
denoising steps).  So one pass over all layers is captured once and replayed
for the others.  The handle's call counters count calls made, not replays."""
import numpy as np
import pytest
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

from gpu_util import bits, check_attn, dev, f64, new_cache

pytestmark = pytest.mark.gpu

F64 = synth.bf16_bits_to_f64
WL = synth.Workload("graph", 3, 2, 128, 10, 20, 3, 3, 9, n_chunks=5, seed=31, steps_per_chunk=3)


def test_replayed_passes_equal_eager_passes_and_the_oracle(oracle_mod):
    wl = WL
    C, L, nq = wl.chunk_frames, wl.layers, wl.chunk_tokens
    passes = wl.steps_per_chunk + 1
    eager, graphed = new_cache(wl), new_cache(wl)
    shape = (nq, wl.heads, wl.head_dim)
    # static buffers of the captured pass, per layer
    sq, sk, sv = (torch.empty((L,) + shape, device="cuda", dtype=torch.bfloat16) for _ in range(3))
    s_qout = torch.empty_like(sq)
    s_out = torch.empty_like(sq)
    e_qout = torch.empty(shape, device="cuda", dtype=torch.bfloat16)
    e_out = torch.empty((L,) + shape, device="cuda", dtype=torch.bfloat16)
    orc = oracle_mod.Oracle(1, wl.heads, wl.head_dim, wl.tokens_per_frame, C, wl.sink_frames, wl.window_frames)
    probe = L - 1

    def one_pass(cache, chunk, q, k, v, q_out_of, out):
        for layer in range(L):
            cache.rope_append_kv(layer, q[layer], k[layer], v[layer], chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta,
                                 q_out_of(layer))
            cache.sink_window_attn(layer, q_out_of(layer), chunk * C, out[layer])

    for chunk in range(wl.n_chunks):
        graph = None
        for p in range(passes):
            host = [synth.chunk_qkv(wl, chunk, layer=layer, pass_id=p) for layer in range(L)]
            q, k, v = (torch.stack([dev(h[i]) for h in host]) for i in range(3))
            one_pass(eager, chunk, q, k, v, lambda layer: e_qout, e_out)
            sq.copy_(q); sk.copy_(k); sv.copy_(v)
            if p == 0:
                one_pass(graphed, chunk, sq, sk, sv, lambda layer: s_qout[layer], s_out)     # the commit pass
            elif p == 1:
                torch.cuda.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph):
                    one_pass(graphed, chunk, sq, sk, sv, lambda layer: s_qout[layer], s_out)
                s_out.fill_(float("nan"))
                graph.replay()
            else:
                s_out.fill_(float("nan"))
                graph.replay()
            torch.cuda.synchronize()
            assert np.array_equal(bits(s_out), bits(e_out)), (chunk, p)
        eager.check_device()
        graphed.check_device()
        for layer in range(L):
            assert np.array_equal(bits(graphed.kv_view(layer, 0)), bits(eager.kv_view(layer, 0)))
            assert np.array_equal(bits(graphed.kv_view(layer, 1)), bits(eager.kv_view(layer, 1)))
        assert graphed.state(probe)["slot_frame"] == eager.state(probe)["slot_frame"]
        hq, hk, hv = host[probe]
        orc.append(0, F64(hk), F64(hv), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        qr = orc.rope_q(F64(hq), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        want, _ = orc.attn(0, qr, chunk * C)
        check_attn(f64(s_out[probe]), want)
    # calls made: per chunk one commit and one captured overwrite on the graphed handle
    assert graphed.state(0)["overwrites"] == wl.n_chunks and eager.state(0)["overwrites"] == wl.n_chunks * (passes - 1)
    eager.close()
    graphed.close()
