"""GPU parity of the QKV projection with norm, rotation and append in its epilogue:
cache rows, rotated queries and the attention that follows, against the oracle's
fp64 projection + RMS norm + rotation + append + attention."""
import numpy as np
import pytest
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

from gpu_util import bits, check_attn, dev, f64, guarded

pytestmark = pytest.mark.gpu

F64 = synth.bf16_bits_to_f64

# (workload, d_model): heads * head_dim a multiple of 256 or of 192 (the two tile widths, at
# both head sizes); ragged last token tile; a d_model that is not a multiple of the GEMM's
# 64-wide K block
SHAPES = [
    (synth.Workload("qkv_d128", 1, 2, 128, 6, 25, 3, 3, 6, n_chunks=4, seed=71), 192),
    (synth.Workload("qkv_d64", 1, 4, 64, 9, 14, 2, 2, 4, n_chunks=4, seed=72), 136),
    (synth.Workload("qkv_wide", 1, 6, 128, 5, 13, 2, 2, 4, n_chunks=3, seed=73), 320),      # 768 = 4 x 192: the 192-wide tiles
    (synth.Workload("qkv_d64_192", 1, 3, 64, 7, 11, 2, 2, 4, n_chunks=3, seed=74), 200),     # 192 = 3 heads of 64 in one tile
]


def draw(wl, d_model, chunk):
    rng = np.random.default_rng([wl.seed, chunk, d_model])
    x = synth.normal_bf16(rng, (wl.chunk_tokens, d_model))
    return x


def weights(wl, d_model):
    rng = np.random.default_rng([wl.seed, 999])
    n = 3 * wl.heads * wl.head_dim
    w = synth.f32_to_bf16_bits((rng.standard_normal((n, d_model)) / np.sqrt(d_model)).astype(np.float32))
    bias = (0.1 * rng.standard_normal(n)).astype(np.float32)
    gq = (1.0 + 0.2 * rng.standard_normal(n // 3)).astype(np.float32)
    gk = (1.0 + 0.2 * rng.standard_normal(n // 3)).astype(np.float32)
    return w, bias, gq, gk


def close_to(got, want, mag, what):
    """One bf16 rounding of the exact value plus the fp32 accumulation error of a sum whose
    terms have total magnitude `mag` (the product of bf16 numbers is exact in fp32; the sum of
    d_model of them carries a few fp32 roundings)."""
    err = np.abs(got - want)
    bound = 2.0 ** -8 * np.abs(want) + 2e-5 * mag + 1e-30
    assert (err <= bound).all(), "%s: worst error/bound %.3f" % (what, (err / bound).max())
    half_ulp = 2.0 ** (np.floor(np.log2(np.abs(want) + 1e-300)) - 8)      # of bf16: 8 significant bits
    return float((err <= half_ulp + 2e-6 * mag).mean())


@pytest.mark.parametrize("with_norm", [False, True], ids=["plain", "norm"])
@pytest.mark.parametrize("wl,d_model", SHAPES, ids=lambda x: getattr(x, "name", str(x)))
def test_projection_epilogue_matches_oracle(oracle_mod, wl, d_model, with_norm):
    C, P, H, D = wl.chunk_frames, wl.tokens_per_frame, wl.heads, wl.head_dim
    HD, nq = H * D, C * P
    eps = 1e-6
    cache = B.Cache(*wl.cache_args)
    orc = oracle_mod.Oracle(*wl.cache_args)
    w, bias, gq, gk = weights(wl, d_model)
    dw = dev(w)
    dbias, dgq, dgk = (torch.from_numpy(a).cuda() for a in (bias, gq, gk))
    ws = torch.empty(B.ll_qkv_proj_workspace_bytes(cache.h) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    wf = F64(w)
    for chunk in range(wl.n_chunks):
        x = draw(wl, d_model, chunk)
        dx = dev(x)
        q_out, q_guard = guarded((nq, H, D))
        row_scale = torch.full((nq,), float("nan"), device="cuda")
        out, out_guard = guarded((nq, H, D), fill=float("nan"))
        for rep in range(2):                                  # commit, then overwrite in place
            B.ll_qkv_proj_append(cache.h, 0, dx, dw, dbias, dgq if with_norm else None, dgk if with_norm else None,
                                 eps, chunk * C, C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out,
                                 row_scale if with_norm else None, ws if with_norm else None)
        B.ll_sink_window_attn_scaled(cache.h, 0, q_out, row_scale if with_norm else None, chunk * C, C, out)
        cache.check_device()
        q_guard()
        out_guard()
        # oracle: fp64 projection, norm, rotation, append, attention
        xf = F64(x)
        q, k, v = oracle_mod.qkv_proj(xf, wf, bias)
        mag = np.abs(xf) @ np.abs(wf).T + np.abs(bias)[None, :]          # magnitude of what each output sums
        mq, mk, mv = mag[:, :HD], mag[:, HD:2 * HD], mag[:, 2 * HD:]
        if with_norm:
            rq = 1.0 / np.sqrt((q * q).mean(axis=1) + eps)
            rk = 1.0 / np.sqrt((k * k).mean(axis=1) + eps)
            q_hat = oracle_mod.rms_norm(q.reshape(nq, H, D), gq, eps)
            k_hat = oracle_mod.rms_norm(k.reshape(nq, H, D), gk, eps)
            mq, mk = mq * rq[:, None] * np.abs(gq)[None, :], mk * rk[:, None] * np.abs(gk)[None, :]
            got_scale = row_scale.cpu().numpy().astype(np.float64)
            assert np.abs(got_scale / rq - 1).max() <= 1e-5
        else:
            q_hat, k_hat = q.reshape(nq, H, D), k.reshape(nq, H, D)
            got_scale = np.ones(nq)
        orc.append(0, k_hat, v.reshape(nq, H, D), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        assert cache.state()["slot_frame"] == list(orc.state()["slot_frame"])
        # rotated queries (times their row factor) against the oracle's; a rotated element mixes
        # the two elements of its pair, so the magnitude is the pair's
        want_q = orc.rope_q(q_hat, chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        pair = lambda m: np.repeat(m.reshape(nq, H, D // 2, 2).sum(axis=3), 2, axis=2).reshape(nq, H, D)
        got_q = f64(q_out) * got_scale[:, None, None]
        close_to(got_q, want_q, pair(mq), "q")
        # cache rows of the chunk's frames
        K, V = orc.read_layer()
        kc, vc = cache.kv_view(0, 0), cache.kv_view(0, 1)
        exact = []
        for i in range(C):
            slot = orc.slot_of(chunk * C + i)
            rows = slice(slot * P, (slot + 1) * P)
            tok = slice(i * P, (i + 1) * P)
            got_k = f64(kc[:, rows, :]).transpose(1, 0, 2)
            got_v = f64(vc[:, rows, :]).transpose(1, 0, 2)
            exact.append(close_to(got_k, K[slot], pair(mk.reshape(nq, H, D))[tok], "k"))
            exact.append(close_to(got_v, V[slot], mv.reshape(nq, H, D)[tok], "v"))
        assert min(exact) >= 0.97, exact                      # nearly every element is the correctly rounded one
        want, _ = orc.attn(0, want_q, chunk * C)
        check_attn(f64(out), want)
    cache.close()


def test_projection_at_the_benchmark_shape(oracle_mod):
    """4680 tokens x 1536 -> 3 x 12 x 128 with norm and bias, first chunk of a stream: sampled
    token rows of q, k, v against the fp64 projection, then attention on sampled rows."""
    wl = synth.CONFIGS[1]
    d_model = 1536
    C, P, H, D = wl.chunk_frames, wl.tokens_per_frame, wl.heads, wl.head_dim
    HD, nq = H * D, C * P
    eps = 1e-6
    cache = B.Cache(*wl.cache_args)
    orc = oracle_mod.Oracle(*wl.cache_args)
    w, bias, gq, gk = weights(wl, d_model)
    x = draw(wl, d_model, 0)
    dbias, dgq, dgk = (torch.from_numpy(a).cuda() for a in (bias, gq, gk))
    ws = torch.empty(B.ll_qkv_proj_workspace_bytes(cache.h) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    q_out = torch.empty(nq, H, D, device="cuda", dtype=torch.bfloat16)
    row_scale = torch.empty(nq, device="cuda")
    out = torch.full_like(q_out, float("nan"))
    B.ll_qkv_proj_append(cache.h, 0, dev(x), dev(w), dbias, dgq, dgk, eps, 0, C, wl.grid_h, wl.grid_w, wl.rope_theta,
                         q_out, row_scale, ws)
    B.ll_sink_window_attn_scaled(cache.h, 0, q_out, row_scale, 0, C, out)
    cache.check_device()
    q, k, v = oracle_mod.qkv_proj(F64(x), F64(w), bias)
    q_hat = oracle_mod.rms_norm(q.reshape(nq, H, D), gq, eps)
    k_hat = oracle_mod.rms_norm(k.reshape(nq, H, D), gk, eps)
    orc.append(0, k_hat, v.reshape(nq, H, D), 0, wl.grid_h, wl.grid_w, wl.rope_theta)
    want_q = orc.rope_q(q_hat, 0, wl.grid_h, wl.grid_w, wl.rope_theta)
    rows = synth.sample_rows(nq, 256, seed=7)
    got_q = f64(q_out) * row_scale.cpu().numpy().astype(np.float64)[:, None, None]
    assert np.abs(got_q[rows] - want_q[rows]).max() <= 2.0 ** -8 * np.abs(want_q).max() + 1e-3
    K, V = orc.read_layer()
    vc, kc = cache.kv_view(0, 1), cache.kv_view(0, 0)
    for i in range(C):
        got_v = f64(vc[:, i * P:(i + 1) * P, :]).transpose(1, 0, 2)
        got_k = f64(kc[:, i * P:(i + 1) * P, :]).transpose(1, 0, 2)
        assert np.abs(got_v - V[i]).max() <= 2.0 ** -8 * np.abs(V[i]).max() + 1e-3
        assert np.abs(got_k - K[i]).max() <= 2.0 ** -8 * np.abs(K[i]).max() + 1e-3
    want, _ = orc.attn(0, want_q, 0, rows=rows)
    check_attn(f64(out)[rows], want)
    cache.close()


def test_projection_argument_checks():
    wl = synth.Workload("qkv_small", 1, 2, 64, 4, 4, 1, 1, 2, n_chunks=1, seed=0)      # heads*head_dim = 128: neither tile width divides it
    cache = B.Cache(*wl.cache_args)
    x = torch.zeros(16, 64, device="cuda", dtype=torch.bfloat16)
    w = torch.zeros(3 * 128, 64, device="cuda", dtype=torch.bfloat16)
    q_out = torch.zeros(16, 2, 64, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(B.LLError) as e:
        B.ll_qkv_proj_append(cache.h, 0, x, w, None, None, None, 0.0, 0, 1, 4, 4, 10000.0, q_out)
    assert e.value.code == B.LL_ERR_UNSUPPORTED_SHAPE and cache.state()["end"] == 0
    cache.close()
