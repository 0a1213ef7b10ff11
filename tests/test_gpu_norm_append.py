"""GPU parity of the append with the q/k RMS norm in front: the cache rows and the
rotated queries against the CPU oracle (norm, then rotation, one rounding to
bf16), V rows bit-exact, integer state as for the plain append; and attention
over a cache filled this way."""
import numpy as np
import pytest
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

from gpu_util import bits, check_attn, dev, f64, new_cache, ulp_distance

pytestmark = pytest.mark.gpu

F64 = synth.bf16_bits_to_f64

CASES = [
    synth.Workload("norm_d128", 1, 12, 128, 6, 10, 3, 3, 6, n_chunks=4, seed=51),      # the model's row: 1536 elements
    synth.Workload("norm_d64", 1, 3, 64, 9, 14, 2, 2, 4, n_chunks=5, seed=52),          # 24 vectors: ragged over the lanes
    synth.Workload("norm_one_head", 1, 1, 128, 7, 19, 1, 1, 3, n_chunks=5, seed=53),    # 16 vectors: half a warp idle
    synth.Workload("norm_wide", 1, 40, 128, 4, 4, 1, 1, 2, n_chunks=3, seed=54),        # 5120 elements per row
]
EPS = 1e-6


def close_bits(got_bits, want_f64):
    """The kernel scales and rotates in fp32 and rounds once to bf16.  Its result may differ
    from the rounded fp64 value by the rounding itself (half a bf16 ulp of the value) plus the
    fp32 error of the row factor, the gain product and the rotation, which is relative to the
    rotated pair's length, not to the element (an element can be a small difference of two
    large products): 8e-6 of sqrt(even^2 + odd^2).  At least 99% of the elements are bit-exact."""
    want_bits = synth.f32_to_bf16_bits(want_f64.astype(np.float32))
    assert (got_bits == want_bits).mean() >= 0.99, "only %.4f exact" % (got_bits == want_bits).mean()
    err = np.abs(F64(got_bits) - want_f64)
    half_ulp = 0.5 * 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want_f64), 2.0 ** -126))) - 7)
    pair = np.sqrt(want_f64[..., 0::2] ** 2 + want_f64[..., 1::2] ** 2)
    tol = 1.001 * half_ulp + 8e-6 * np.repeat(pair, 2, axis=-1)
    assert (err <= tol).all(), "worst excess %.3e" % (err - tol).max()


@pytest.mark.parametrize("wl", CASES, ids=lambda w: w.name)
def test_norm_rope_append_matches_oracle(oracle_mod, wl):
    cache = new_cache(wl)
    orc = oracle_mod.Oracle(1, wl.heads, wl.head_dim, wl.tokens_per_frame, wl.chunk_frames, wl.sink_frames,
                            wl.window_frames, faithful=True)
    P, C, H, D = wl.tokens_per_frame, wl.chunk_frames, wl.heads, wl.head_dim
    rng = np.random.default_rng(wl.seed)
    gq = (1.0 + 0.3 * rng.standard_normal((H, D))).astype(np.float32)
    gk = (1.0 + 0.3 * rng.standard_normal((H, D))).astype(np.float32)
    dgq, dgk = torch.from_numpy(gq).cuda(), torch.from_numpy(gk).cuda()
    for chunk in range(wl.n_chunks):
        q, k, v = synth.chunk_qkv(wl, chunk)
        scale = 0.05 if chunk == 1 else 3.0 if chunk == 2 else 1.0          # small rows feel eps, large ones do not
        q = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(q) * scale)
        k = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(k) * scale)
        dq, dk, dv = dev(q), dev(k), dev(v)
        q_out = torch.full_like(dq, float("nan"))
        fs = chunk * C
        cache.norm_rope_append_kv(0, dq, dk, dv, dgq, dgk, EPS, fs, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
        cache.check_device()
        kn = oracle_mod.rms_norm(F64(k), gk.astype(np.float64), EPS)
        qn = oracle_mod.rms_norm(F64(q), gq.astype(np.float64), EPS)
        orc.append(0, kn, F64(v), fs, wl.grid_h, wl.grid_w, wl.rope_theta)
        st, ost = cache.state(), orc.state()
        assert st["end"] == ost["end"] and st["slot_frame"] == list(ost["slot_frame"])
        K, V = orc.read_layer()                                 # K already rounded to bf16 (storage-faithful mode)
        kc, vc = cache.kv_view(0, 0), cache.kv_view(0, 1)
        for i in range(C):
            slot = orc.slot_of(fs + i)
            got_k = bits(kc[:, slot * P:(slot + 1) * P, :]).transpose(1, 0, 2)
            want_k = oracle_mod.rope(kn[i * P:(i + 1) * P], fs + i, wl.grid_h, wl.grid_w, wl.rope_theta)
            close_bits(got_k, want_k)
            got_v = bits(vc[:, slot * P:(slot + 1) * P, :]).transpose(1, 0, 2)
            assert np.array_equal(got_v, v[i * P:(i + 1) * P])
        close_bits(bits(q_out), oracle_mod.rope(qn, fs, wl.grid_h, wl.grid_w, wl.rope_theta))
        # attention over the cache built this way
        out = torch.empty_like(dq)
        cache.sink_window_attn(0, q_out, fs, out)
        cache.check_device()
        want, _ = orc.attn(0, orc.rope_q(qn, fs, wl.grid_h, wl.grid_w, wl.rope_theta), fs)
        check_attn(f64(out), want)
    cache.close()


def test_norm_append_equals_norm_then_plain_append_when_the_norm_is_trivial(oracle_mod):
    """Rows whose mean square is exactly 1 with gain 1 and eps 0: the norm changes nothing, so
    the fused call must write the very bits of the plain append."""
    wl = synth.Workload("norm_trivial", 1, 2, 64, 4, 4, 1, 1, 2, n_chunks=1, seed=55)
    a, b = new_cache(wl), new_cache(wl)
    n = wl.chunk_tokens
    signs = np.where(np.random.default_rng(5).random((n, 2, 64)) < 0.5, -1.0, 1.0).astype(np.float32)
    x = synth.f32_to_bf16_bits(signs)                                        # every element +-1
    dx, dv = dev(x), dev(synth.chunk_qkv(wl, 0)[2])
    ones = torch.ones(2 * 64, device="cuda")
    qa, qb = torch.empty_like(dx), torch.empty_like(dx)
    a.norm_rope_append_kv(0, dx, dx, dv, ones, ones, 0.0, 0, wl.grid_h, wl.grid_w, wl.rope_theta, qa)
    b.rope_append_kv(0, dx, dx, dv, 0, wl.grid_h, wl.grid_w, wl.rope_theta, qb)
    a.check_device()
    assert np.array_equal(bits(qa), bits(qb))
    assert np.array_equal(bits(a.kv_view(0, 0)), bits(b.kv_view(0, 0)))
    assert np.array_equal(bits(a.kv_view(0, 1)), bits(b.kv_view(0, 1)))
    a.close()
    b.close()
