"""GPU parity of the dense (cross-) attention entry point against the CPU oracle:
prompt-sized key sets, ragged query and key counts, both head sizes."""
import numpy as np
import pytest
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

from gpu_util import bits, check_attn, dev, f64

pytestmark = pytest.mark.gpu

F64 = synth.bf16_bits_to_f64


def draw(shape, seed):
    return synth.normal_bf16(np.random.default_rng(seed), shape)


@pytest.mark.parametrize("n_q,n_k,H,D", [(600, 512, 2, 128), (133, 77, 3, 64), (1, 1, 1, 128), (257, 129, 2, 128),
                                          (1000, 300, 4, 64), (256, 128, 1, 128), (40, 1000, 2, 128)])
def test_cross_attn_matches_oracle(oracle_mod, n_q, n_k, H, D):
    cache = B.Cache(1, H, D, 8, 1, 1, 1)                 # lends shape, scratch and status words only
    q, k, v = draw((n_q, H, D), 1), draw((n_k, H, D), 2), draw((n_k, H, D), 3)
    dq, dk, dv = dev(q), dev(k), dev(v)
    out = torch.full_like(dq, float("nan"))
    lse = torch.full((H, n_q), float("nan"), device="cuda")
    before = cache.state()
    cache.cross_attn(dq, dk, dv, out, lse)
    cache.check_device()
    want, want_lse = oracle_mod.dense_attn(F64(q), F64(k), F64(v))
    check_attn(f64(out), want)
    assert np.abs(lse.cpu().numpy().T - want_lse).max() <= 2e-2
    assert cache.state() == before
    again = torch.empty_like(out)
    cache.cross_attn(dq, dk, dv, again)                   # without lse; same bits
    assert np.array_equal(bits(again), bits(out))
    cache.close()


def test_cross_attn_at_the_model_shape(oracle_mod):
    """One chunk of video tokens (4680) over a 512-token prompt, 12 heads of 128."""
    n_q, n_k, H, D = 4680, 512, 12, 128
    cache = B.Cache(1, H, D, 1560, 3, 3, 9)
    q, k, v = draw((n_q, H, D), 4), draw((n_k, H, D), 5), draw((n_k, H, D), 6)
    dq, dk, dv = dev(q), dev(k), dev(v)
    out = torch.full_like(dq, float("nan"))
    cache.cross_attn(dq, dk, dv, out)
    cache.check_device()
    assert torch.isfinite(out.float()).all()
    rows = synth.sample_rows(n_q, 96, seed=3)
    want, _ = oracle_mod.dense_attn(F64(q), F64(k), F64(v), rows=rows)
    check_attn(f64(out)[rows], want)
    # the handle's self-attention path is untouched by it
    wl = synth.CONFIGS[1]
    qq, kk, vv = synth.chunk_qkv(wl, 0)
    q_out = torch.empty_like(dev(qq))
    cache.rope_append_kv(0, dev(qq), dev(kk), dev(vv), 0, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
    o2 = torch.empty_like(q_out)
    cache.sink_window_attn(0, q_out, 0, o2)
    cache.check_device()
    assert torch.isfinite(o2.float()).all()
    cache.close()
