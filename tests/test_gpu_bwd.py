"""GPU parity of the clip step's backward pass: dq, dk, dv through the C ABI against the
oracle's fp64 gradients (which are pinned by finite differences of the forward clip)."""
import numpy as np
import pytest
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

from gpu_util import bits, dev, f64, guarded

pytestmark = pytest.mark.gpu

F64 = synth.bf16_bits_to_f64

# (workload, context chunks before the clip, clip chunks, local window in frames)
CASES = [
    (synth.Workload("bwd_d128", 1, 2, 128, 6, 25, 3, 3, 12, n_chunks=0, seed=81), 2, 3, 6),      # sink + context + clip
    (synth.Workload("bwd_wrap", 1, 2, 128, 5, 13, 3, 3, 12, n_chunks=0, seed=82), 4, 3, 6),      # the clip's slots wrap round the ring
    (synth.Workload("bwd_d64", 1, 3, 64, 7, 19, 1, 1, 8, n_chunks=0, seed=83), 3, 4, 3),         # 133-token frames, one-frame chunks
    (synth.Workload("bwd_first", 1, 2, 128, 4, 30, 2, 2, 8, n_chunks=0, seed=84), 0, 3, 4),      # the clip opens the stream (holds the sink)
]

# Error bar: every gradient element is a sum of terms; P and dS are rounded to bf16 before the
# tensor-core products (2^-9 of each term), delta is formed from the bf16 output of the forward
# (2^-9 of the terms of d_out.out, which enters every dS of the row), the result is rounded to
# bf16 once (2^-9 of itself).  With M the sum of the absolute values of an element's terms (the
# oracle returns it) the arithmetic cannot be off by more than a small multiple of 2^-9 M; the
# bar is 2^-7 M plus a floor for elements whose terms are all tiny (measured worst: 0.24 of
# 2^-6 M).
REL_TO_TERMS = 2.0 ** -7
FLOOR = 2e-4


def check_grad(name, got, want, mag):
    err = np.abs(got - want)
    bound = REL_TO_TERMS * mag + FLOOR
    worst = (err / bound).max()
    print("backward %s: max |err| %.3e, max |grad| %.3e, worst err/bound %.3f, mean err/terms %.2e"
          % (name, err.max(), np.abs(want).max(), worst, (err / (mag + 1e-30)).mean()))
    assert np.isfinite(got).all()
    assert worst <= 1.0, name
    assert (err / (mag + FLOOR)).mean() <= 2.0 ** -9, name          # on average well inside one bf16 rounding of the terms


@pytest.mark.parametrize("wl,ctx,clip_chunks,window", CASES, ids=lambda x: getattr(x, "name", None))
def test_clip_backward_matches_oracle(oracle_mod, wl, ctx, clip_chunks, window):
    C, P, H, D = wl.chunk_frames, wl.tokens_per_frame, wl.heads, wl.head_dim
    cache = B.Cache(*wl.cache_args)
    orc = oracle_mod.Oracle(*wl.cache_args)
    for chunk in range(ctx):
        _, k, v = synth.chunk_qkv(wl, chunk)
        cache.rope_append_kv(0, None, dev(k), dev(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        orc.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
    T = clip_chunks * C
    fs = ctx * C
    q, k, v = synth.chunk_qkv(wl, 100, n_frames=T)
    g_bits = synth.normal_bf16(np.random.default_rng([wl.seed, 7]), q.shape)
    dq_in, dk_in, dv_in, dg = dev(q), dev(k), dev(v), dev(g_bits)
    n = T * P
    q_out = torch.empty_like(dq_in)
    out = torch.empty_like(dq_in)
    lse = torch.empty(H, n, device="cuda", dtype=torch.float32)
    cache.clip_append_attn(0, dq_in, dk_in, dv_in, fs, T, window, wl.grid_h, wl.grid_w, wl.rope_theta, q_out, out, lse)
    ws = torch.empty(B.ll_clip_backward_workspace_bytes(cache.h, T) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    grads = [guarded((n, H, D), fill=float("nan")) for _ in range(3)]
    state_before = cache.state()
    B.ll_clip_attn_backward(cache.h, 0, q_out, out, dg, lse, fs, T, window, wl.grid_h, wl.grid_w, wl.rope_theta,
                            grads[0][0], grads[1][0], grads[2][0], ws)
    cache.check_device()
    assert cache.state() == state_before
    for _, guard in grads:
        guard()
    orc.clip(0, F64(q), F64(k), F64(v), fs, T, window, wl.grid_h, wl.grid_w, wl.rope_theta)
    want = orc.clip_backward(0, F64(q), F64(g_bits), fs, T, window, wl.grid_h, wl.grid_w, wl.rope_theta)
    for name, (got, _), w, m in zip(("dq", "dk", "dv"), grads, want[:3], want[3:]):
        check_grad("%s %s" % (wl.name, name), f64(got), w, m)
    # the same call again gives the same bits
    first = [bits(g).copy() for g, _ in grads]
    B.ll_clip_attn_backward(cache.h, 0, q_out, out, dg, lse, fs, T, window, wl.grid_h, wl.grid_w, wl.rope_theta,
                            grads[0][0], grads[1][0], grads[2][0], ws)
    cache.check_device()
    for before, (g, _) in zip(first, grads):
        assert np.array_equal(before, bits(g))
    cache.close()


def test_clip_backward_argument_checks():
    wl = CASES[0][0]
    C = wl.chunk_frames
    cache = B.Cache(*wl.cache_args)
    q, k, v = (dev(t) for t in synth.chunk_qkv(wl, 0, n_frames=2 * C))
    q_out, out = torch.empty_like(q), torch.empty_like(q)
    lse = torch.empty(wl.heads, q.shape[0], device="cuda")
    cache.clip_append_attn(0, q, k, v, 0, 2 * C, 6, wl.grid_h, wl.grid_w, wl.rope_theta, q_out, out, lse)
    ws = torch.empty(B.ll_clip_backward_workspace_bytes(cache.h, 2 * C), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.LLError) as e:                     # not the newest frames of the stream
        B.ll_clip_attn_backward(cache.h, 0, q_out, out, out, lse, 0, C, 6, wl.grid_h, wl.grid_w, wl.rope_theta, q, k, v, ws)
    assert e.value.code == B.LL_ERR_BAD_POSITION
    with pytest.raises(B.LLError) as e:                     # workspace too small
        B.ll_clip_attn_backward(cache.h, 0, q_out, out, out, lse, 0, 2 * C, 6, wl.grid_h, wl.grid_w, wl.rope_theta, q, k, v,
                                ws[:256])
    assert e.value.code == B.LL_ERR_INVALID_ARG
    cache.check_device()
    cache.close()


def test_clip_backward_closed_forms_at_the_benchmark_shape(oracle_mod):
    """Config-1 layer shape, a 21-frame clip behind 12 frames of context, K = 0: every weight is
    1/n (n = 12 frames of keys), so the gradients have closed forms that need no oracle run:
    dq = 0; dv is the same for all tokens of a frame, (1/n) * sum over the chunks that see the
    frame of the chunk's summed d_out; dk_j = (1/(n sqrt(D))) sum_i (d_out_i.v_j - d_out_i.o_i) q_i
    over the rows i that see j (checked on sampled key rows, in the rotated frame)."""
    base = synth.CONFIGS[1]
    C, P, H, D, S, Wa = base.chunk_frames, base.tokens_per_frame, base.heads, base.head_dim, base.sink_frames, base.window_frames
    clip_chunks, ctx = 7, 4
    T = clip_chunks * C
    cache = B.Cache(1, H, D, P, C, S, Wa + T - C)
    rng = np.random.default_rng(91)
    zeros = torch.zeros(C * P, H, D, device="cuda", dtype=torch.bfloat16)
    v_ctx = []
    for chunk in range(ctx):
        v = synth.normal_bf16(rng, (C * P, H, D))
        v_ctx.append(F64(v))
        cache.rope_append_kv(0, None, zeros, dev(v), chunk * C, base.grid_h, base.grid_w, base.rope_theta)
    q = synth.normal_bf16(rng, (T * P, H, D))
    v = synth.normal_bf16(rng, (T * P, H, D))
    g = synth.normal_bf16(rng, (T * P, H, D))
    dq_in, dv_in, dg = dev(q), dev(v), dev(g)
    k0 = torch.zeros_like(dq_in)
    q_out, out = torch.empty_like(dq_in), torch.empty_like(dq_in)
    lse = torch.empty(H, T * P, device="cuda", dtype=torch.float32)
    fs = ctx * C
    cache.clip_append_attn(0, dq_in, k0, dv_in, fs, T, Wa, base.grid_h, base.grid_w, base.rope_theta, q_out, out, lse)
    ws = torch.empty(B.ll_clip_backward_workspace_bytes(cache.h, T) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    dq, dk, dv = (torch.full_like(dq_in, float("nan")) for _ in range(3))
    B.ll_clip_attn_backward(cache.h, 0, q_out, out, dg, lse, fs, T, Wa, base.grid_h, base.grid_w, base.rope_theta, dq, dk, dv, ws)
    cache.check_device()
    n = (S + Wa) * P
    assert np.abs(lse.cpu().numpy() - np.log(n)).max() < 1e-3
    assert float(dq.float().abs().max()) == 0.0
    # frames (absolute) each clip chunk sees, and the d_out sums per chunk
    gf, vf, qf = F64(g), F64(v), F64(q)
    all_v = np.concatenate(v_ctx + [vf]).reshape(ctx * C + T, P, H, D)             # by absolute frame
    chunk_sum = gf.reshape(clip_chunks, C * P, H, D).sum(axis=1)
    sees = lambda c_, f: f < fs + (c_ + 1) * C and (f < S or f >= fs + (c_ + 1) * C - Wa)
    got_dv = f64(dv).reshape(T, P, H, D)
    for i in range(T):
        want = sum(chunk_sum[c_] for c_ in range(clip_chunks) if sees(c_, fs + i)) / n
        err = np.abs(got_dv[i] - want[None])
        # one bf16 rounding of 1/n, one of the result, fp32 accumulation over up to 14040 rows
        assert err.max() <= 2.0 ** -7 * np.abs(want).max() + 1e-6, (i, err.max())
    # dk on sampled key rows, in the rotated frame: rotate the stored gradient forward again
    o_bar = np.stack([sum(all_v[f].sum(axis=0) for f in range(ctx * C + T) if sees(c_, f)) / n for c_ in range(clip_chunks)])
    q_rot = oracle_mod.rope(qf, fs, base.grid_h, base.grid_w, base.rope_theta)
    dk_rot = oracle_mod.rope(f64(dk), fs, base.grid_h, base.grid_w, base.rope_theta)
    for j in synth.sample_rows(T * P, 24, seed=3, edges=False):
        fj = fs + j // P
        want = np.zeros((H, D))
        mag = np.zeros((H, D))
        for c_ in range(clip_chunks):
            if not sees(c_, fj):
                continue
            rows = slice(c_ * C * P, (c_ + 1) * C * P)
            w = (np.einsum("ihd,hd->ih", gf[rows], vf[j]) - np.einsum("ihd,hd->ih", gf[rows], o_bar[c_])) / (n * np.sqrt(D))
            want += np.einsum("ih,ihd->hd", w, q_rot[rows])
            mag += np.einsum("ih,ihd->hd", np.abs(w), np.abs(q_rot[rows]))
        err = np.abs(dk_rot[j] - want)
        assert (err <= 2.0 ** -7 * mag + 2e-5).all(), (j, (err / (2.0 ** -7 * mag + 2e-5)).max())
    cache.close()
