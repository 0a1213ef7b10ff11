"""GPU parity on seeded random small shapes: every combination the fixed cases do not name
(head sizes, head counts, ragged frame sizes down to one token, chunk / sink / window sizes,
no sink, bf16 and 8-bit caches), through append, overwrite passes, decode, recache, the
several-streams launch and the clip step with its backward, every row against the oracle."""
import numpy as np
import pytest
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

from gpu_util import check_attn, dev, f64

pytestmark = pytest.mark.gpu

F64 = synth.bf16_bits_to_f64


def random_workload(rng, i):
    D = int(rng.choice([64, 128]))
    H = int(rng.integers(1, 5))
    gh, gw = int(rng.integers(1, 12)), int(rng.integers(1, 24))
    C = int(rng.integers(1, 4))
    S = C * int(rng.integers(0, 3))
    W = C * int(rng.integers(1, 5))
    n_chunks = (S + W) // C + int(rng.integers(1, 4))
    return synth.Workload("random_%d" % i, 1, H, D, gh, gw, C, S, W, n_chunks=n_chunks, seed=1000 + i)


@pytest.mark.parametrize("i", range(16))
def test_random_stream(oracle_mod, i):
    rng = np.random.default_rng(4242 + i)
    wl = random_workload(rng, i)
    e4m3 = bool(rng.integers(0, 2))
    C, P, H, D = wl.chunk_frames, wl.tokens_per_frame, wl.heads, wl.head_dim
    cache = B.Cache(*wl.cache_args, kv_format=B.LL_KV_E4M3 if e4m3 else B.LL_KV_BF16)
    orc = oracle_mod.Oracle(*wl.cache_args)
    if e4m3:
        ks = (6.0 / 448.0 * (1.0 + 0.2 * rng.random(H))).astype(np.float32)
        vs = (5.0 / 448.0 * (1.0 + 0.2 * rng.random(H))).astype(np.float32)
        cache.set_kv_scales(0, ks, vs)
        orc.set_kv_e4m3(ks[None], vs[None])
    recache_at = int(rng.integers(0, wl.n_chunks))
    print("shape", wl.name, dict(H=H, D=D, grid=(wl.grid_h, wl.grid_w), C=C, S=wl.sink_frames, W=wl.window_frames,
                                 chunks=wl.n_chunks, e4m3=e4m3, recache_at=recache_at))
    for chunk in range(wl.n_chunks):
        for pass_id in range(int(rng.integers(1, 3))):               # sometimes an overwrite pass first
            q, k, v = synth.chunk_qkv(wl, chunk, pass_id=pass_id)
            dq = dev(q)
            q_out = torch.empty_like(dq)
            cache.rope_append_kv(0, dq, dev(k), dev(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
            orc.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        out = torch.full_like(dq, float("nan"))
        lse = torch.full((H, C * P), float("nan"), device="cuda")
        cache.sink_window_attn(0, q_out, chunk * C, out, lse)
        cache.check_device()
        want, want_lse = orc.attn(0, orc.rope_q(F64(q), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta), chunk * C)
        check_attn(f64(out), want)
        assert np.abs(lse.cpu().numpy().T - want_lse).max() <= 2e-2
        st, ost = cache.state(), orc.state()
        assert st["end"] == ost["end"] and st["slot_frame"] == list(ost["slot_frame"]) and st["evictions"] == ost["evictions"]
        if chunk == recache_at:
            end = (chunk + 1) * C
            n = max(0, end - max(wl.sink_frames, end - wl.window_frames))
            if n > 0:
                rq, rk, rv = synth.chunk_qkv(wl, chunk, pass_id=synth.RECACHE_PASS, n_frames=n)
                drq = dev(rq)
                rq_out, r_out = torch.empty_like(drq), torch.full_like(drq, float("nan"))
                cache.recache(0, drq, dev(rk), dev(rv), n, wl.grid_h, wl.grid_w, wl.rope_theta, rq_out, r_out)
                cache.check_device()
                _, want, _ = orc.recache(0, F64(rq), F64(rk), F64(rv), n, wl.grid_h, wl.grid_w, wl.rope_theta)
                check_attn(f64(r_out), want)
    cache.close()


@pytest.mark.parametrize("i", range(8))
def test_random_clip_and_backward(oracle_mod, i):
    rng = np.random.default_rng(777 + i)
    D = int(rng.choice([64, 128]))
    H = int(rng.integers(1, 4))
    gh, gw = int(rng.integers(1, 9)), int(rng.integers(1, 20))
    C = int(rng.integers(1, 4))
    S = C * int(rng.integers(0, 2))
    clip_chunks = int(rng.integers(1, 5))
    window = C * int(rng.integers(1, 4))
    ctx = int(rng.integers(0, 4)) if S == 0 else int(rng.integers(S // C, S // C + 3))
    W = window + clip_chunks * C - C + C * int(rng.integers(0, 2))
    wl = synth.Workload("random_clip_%d" % i, 1, H, D, gh, gw, C, S, W, n_chunks=0, seed=2000 + i)
    P, T, fs = wl.tokens_per_frame, clip_chunks * C, ctx * C
    print("clip", dict(H=H, D=D, grid=(gh, gw), C=C, S=S, W=W, ctx=ctx, clip_chunks=clip_chunks, window=window))
    cache = B.Cache(*wl.cache_args)
    orc = oracle_mod.Oracle(*wl.cache_args)
    for chunk in range(ctx):
        _, k, v = synth.chunk_qkv(wl, chunk)
        cache.rope_append_kv(0, None, dev(k), dev(v), chunk * C, gh, gw, wl.rope_theta)
        orc.append(0, F64(k), F64(v), chunk * C, gh, gw, wl.rope_theta)
    q, k, v = synth.chunk_qkv(wl, 50, n_frames=T)
    g = synth.normal_bf16(rng, q.shape)
    dq_in = dev(q)
    q_out, out = torch.empty_like(dq_in), torch.full_like(dq_in, float("nan"))
    lse = torch.empty(H, T * P, device="cuda")
    cache.clip_append_attn(0, dq_in, dev(k), dev(v), fs, T, window, gh, gw, wl.rope_theta, q_out, out, lse)
    cache.check_device()
    _, want, _ = orc.clip(0, F64(q), F64(k), F64(v), fs, T, window, gh, gw, wl.rope_theta)
    check_attn(f64(out), want)
    ws = torch.empty(B.ll_clip_backward_workspace_bytes(cache.h, T) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    grads = [torch.full_like(dq_in, float("nan")) for _ in range(3)]
    B.ll_clip_attn_backward(cache.h, 0, q_out, out, dev(g), lse, fs, T, window, gh, gw, wl.rope_theta, *grads, ws)
    cache.check_device()
    res = orc.clip_backward(0, F64(q), F64(g), fs, T, window, gh, gw, wl.rope_theta)
    for name, got, w, m in zip(("dq", "dk", "dv"), grads, res[:3], res[3:]):
        err = np.abs(f64(got) - w)
        assert np.isfinite(f64(got)).all(), name
        assert (err <= 2.0 ** -7 * m + 2e-4).all(), (name, (err / (2.0 ** -7 * m + 2e-4)).max())
    cache.close()
