"""GPU parity of the 8-bit (E4M3) cache: codes written by the append kernel against the
oracle's storage rule, and attention over such a cache against the oracle's attention
over the same quantised rows, under the same bar as the bf16 path."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

from gpu_util import bits, check_attn, check_attn_outliers, dev, f64, guarded

pytestmark = pytest.mark.gpu

F64 = synth.bf16_bits_to_f64
MEDIUM = synth.Workload("kv8_medium", 2, 2, 128, 10, 20, 3, 3, 9, n_chunks=6, seed=61)
MEDIUM64 = synth.Workload("kv8_d64", 1, 3, 64, 9, 14, 2, 2, 4, n_chunks=6, seed=62)
ODD = synth.Workload("kv8_odd", 1, 1, 128, 7, 19, 1, 1, 3, n_chunks=6, seed=63)


def decode_table():
    """Value of every E4M3 code (from the bit pattern), NaN codes as nan."""
    t = np.full(256, np.nan)
    for code in range(256):
        sgn, e, m = code >> 7, (code >> 3) & 15, code & 7
        if e == 15 and m == 7:
            continue
        mag = (m / 8.0) * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7)
        t[code] = -mag if sgn else mag
    return t


def scales_for(wl, amax):
    """One scale per layer and head, different for every head, mapping about `amax` onto 448."""
    k = np.array([[amax / 448.0 * (1.0 + 0.13 * h + 0.05 * l) for h in range(wl.heads)] for l in range(wl.layers)],
                 dtype=np.float32)
    return k, (k * np.float32(0.8)).astype(np.float32)


def new_pair(oracle_mod, wl, amax=6.0, faithful=False, layers=None):
    L = layers or wl.layers
    cache = B.Cache(L, wl.heads, wl.head_dim, wl.tokens_per_frame, wl.chunk_frames, wl.sink_frames,
                    wl.window_frames, kv_format=B.LL_KV_E4M3)
    orc = oracle_mod.Oracle(L, wl.heads, wl.head_dim, wl.tokens_per_frame, wl.chunk_frames, wl.sink_frames,
                            wl.window_frames, faithful=faithful)
    ks, vs = scales_for(dataclasses.replace(wl, layers=L), amax)
    orc.set_kv_e4m3(ks, vs)
    for l in range(L):
        cache.set_kv_scales(l, ks[l], vs[l])
    return cache, orc, ks, vs


def check_codes(cache, orc, layer, ks, vs, wl):
    """Stored codes x scale against the oracle's rows: V bit-exact; K within one code step and
    exact on all but a few elements in ten thousand (the kernel rotates in fp32, the oracle in
    fp64, so a quotient sitting on a rounding boundary can fall either way)."""
    table = decode_table()
    P = wl.tokens_per_frame
    K, V = orc.read_layer(layer)
    kc = cache.kv_view(layer, 0).cpu().numpy()
    vc = cache.kv_view(layer, 1).cpu().numpy()
    st = cache.state(layer)
    order = np.argsort(np.where(np.isnan(table), np.inf, table))       # codes sorted by value
    rank = np.empty(256, dtype=np.int64)
    rank[order] = np.arange(256)
    for slot, frame in enumerate(st["slot_frame"]):
        if frame < 0:
            continue
        got_v = table[vc[:, slot * P:(slot + 1) * P, :]].transpose(1, 0, 2) * vs[layer][None, :, None].astype(np.float64)
        assert np.array_equal(got_v, V[slot]), (layer, slot)
        codes = kc[:, slot * P:(slot + 1) * P, :].transpose(1, 0, 2)
        got_k = table[codes] * ks[layer][None, :, None].astype(np.float64)
        same = got_k == K[slot]
        assert same.mean() >= 0.9995, same.mean()
        if not same.all():
            # the oracle's value as a code: nearest table entry of value / scale
            want_val = K[slot] / ks[layer][None, :, None].astype(np.float64)
            finite = np.where(np.isnan(table), 1e9, table)
            want_code = np.abs(want_val[~same][:, None] - finite[None, :]).argmin(axis=1)
            step = np.abs(rank[codes[~same]] - rank[want_code])
            # -0 and +0 are two codes of one value: a step across zero counts two
            assert step.max() <= 2, step.max()


@pytest.mark.parametrize("wl", [synth.CONFIGS[0], MEDIUM, MEDIUM64, ODD], ids=lambda w: w.name)
def test_e4m3_append_and_attention_match_the_quantised_oracle(oracle_mod, wl):
    cache, orc, ks, vs = new_pair(oracle_mod, wl)
    C, P = wl.chunk_frames, wl.tokens_per_frame
    nq = C * P
    layer = wl.layers - 1
    worst = (0.0, 0.0)
    for chunk in range(wl.n_chunks):
        q, k, v = synth.chunk_qkv(wl, chunk)
        dq, dk, dv = dev(q), dev(k), dev(v)
        q_out, q_guard = guarded(dq.shape)
        out, out_guard = guarded(dq.shape, fill=float("nan"))
        lse = torch.full((wl.heads, nq), float("nan"), device="cuda", dtype=torch.float32)
        for rep in range(2):                     # the second call overwrites the chunk in place
            cache.rope_append_kv(layer, dq, dk, dv, chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
            orc.append(layer, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        cache.sink_window_attn(layer, q_out, chunk * C, out, lse)
        cache.check_device()
        q_guard()
        out_guard()
        st, ost = cache.state(layer), orc.state(layer)
        assert st["end"] == ost["end"] and st["slot_frame"] == list(ost["slot_frame"])
        check_codes(cache, orc, layer, ks, vs, wl)
        want, want_lse = orc.attn(layer, orc.rope_q(F64(q), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta), chunk * C)
        e = check_attn(f64(out), want)
        worst = (max(worst[0], e[0]), max(worst[1], e[1]))
        assert np.abs(lse.cpu().numpy().T - want_lse).max() <= 2e-2
    print("parity %s (E4M3 cache): worst max-abs %.3e mean-abs %.3e" % (wl.name, worst[0], worst[1]))
    # recache over the 8-bit cache: rows rewritten as codes, sink untouched, block-causal attention
    W = wl.window_frames
    end = wl.n_chunks * C
    n = end - max(wl.sink_frames, end - W)
    rq, rk, rv = synth.chunk_qkv(wl, wl.n_chunks, pass_id=synth.RECACHE_PASS, n_frames=n)
    drq = dev(rq)
    rq_out, r_out = torch.empty_like(drq), torch.full_like(drq, float("nan"))
    cache.recache(layer, drq, dev(rk), dev(rv), n, wl.grid_h, wl.grid_w, wl.rope_theta, rq_out, r_out)
    cache.check_device()
    _, want, _ = orc.recache(layer, F64(rq), F64(rk), F64(rv), n, wl.grid_h, wl.grid_w, wl.rope_theta)
    check_attn(f64(r_out), want)
    check_codes(cache, orc, layer, ks, vs, wl)
    cache.close()


def test_e4m3_and_bf16_caches_share_a_launch(oracle_mod):
    """One launch over an 8-bit stream and a bf16 stream: each item uses its own format."""
    wl = MEDIUM
    C = wl.chunk_frames
    c8, o8, ks, vs = new_pair(oracle_mod, wl, layers=1)
    c16 = B.Cache(1, wl.heads, wl.head_dim, wl.tokens_per_frame, C, wl.sink_frames, wl.window_frames)
    o16 = oracle_mod.Oracle(1, wl.heads, wl.head_dim, wl.tokens_per_frame, C, wl.sink_frames, wl.window_frames)
    items, wants = [], []
    for cache, orc, last, stream in ((c8, o8, 4, 0), (c16, o16, 2, 1)):
        for chunk in range(last + 1):
            q, k, v = synth.chunk_qkv(wl, chunk, stream=stream)
            dq = dev(q)
            q_out = torch.empty_like(dq)
            cache.rope_append_kv(0, dq, dev(k), dev(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
            orc.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        want, _ = orc.attn(0, orc.rope_q(F64(q), last * C, wl.grid_h, wl.grid_w, wl.rope_theta), last * C)
        out = torch.full_like(q_out, float("nan"))
        items.append((cache, 0, q_out, last * C, out, None))
        wants.append(want)
    B.Cache.sink_window_attn_batched(items)
    for item, want in zip(items, wants):
        item[0].check_device()
        check_attn(f64(item[4]), want)
        item[0].close()


def test_e4m3_config1_sampled_rows_and_outliers(oracle_mod):
    """The benchmark layer shape at steady state over an 8-bit cache, sampled rows; then the
    outlier workload (1 % of the entries x20, scales sized for it) with its three figures."""
    for wl, amax in ((synth.CONFIGS[1], 6.0), (dataclasses.replace(synth.CONFIGS[4], name="kv8_outliers"), 120.0)):
        C = wl.chunk_frames
        outl = wl.outlier_frac > 0
        cache, orc, ks, vs = new_pair(oracle_mod, wl, amax=amax, layers=1)
        orc_abs = orc_truth = None
        if outl:
            orc_abs = oracle_mod.Oracle(1, wl.heads, wl.head_dim, wl.tokens_per_frame, C, wl.sink_frames, wl.window_frames)
            orc_truth = oracle_mod.Oracle(1, wl.heads, wl.head_dim, wl.tokens_per_frame, C, wl.sink_frames, wl.window_frames)
            orc_abs.set_kv_e4m3(ks, vs)
            orc_truth.set_kv_e4m3(ks, vs)
        for chunk in range(5):
            q, k, v = synth.chunk_qkv(wl, chunk)
            dq = dev(q)
            q_out = torch.empty_like(dq)
            cache.rope_append_kv(0, dq, dev(k), dev(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_out)
            orc.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
            if outl:
                orc_abs.append(0, F64(k), np.abs(F64(v)), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
                orc_truth.append(0, F64(k), F64(v), chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        out = torch.full_like(q_out, float("nan"))
        cache.sink_window_attn(0, q_out, 4 * C, out)
        cache.check_device()
        rows = synth.sample_rows(wl.chunk_tokens, 256, seed=4)
        # the outlier workload's reference takes the queries as the path holds them (rotated, bf16)
        qr = oracle_mod.rope(F64(q), 4 * C, wl.grid_h, wl.grid_w, wl.rope_theta, round_bf16=outl)
        want, _ = orc.attn(0, qr, 4 * C, rows=rows)
        got = f64(out)[rows]
        if outl:
            scale = orc_abs.attn(0, qr, 4 * C, rows=rows)[0]
            truth = orc_truth.attn(0, orc_truth.rope_q(F64(q), 4 * C, wl.grid_h, wl.grid_w, wl.rope_theta), 4 * C, rows=rows)[0]
            check_attn_outliers(got, want, scale, truth, label="E4M3 cache, config-4 inputs")
        else:
            e = check_attn(got, want)
            print("parity config1 (E4M3 cache): max-abs %.3e mean-abs %.3e" % e)
        cache.close()


def test_e4m3_storage_is_half_and_the_format_is_fixed_at_bind():
    wl = synth.CONFIGS[2]
    h16 = B.ll_cache_create(*wl.cache_args)
    h8 = B.ll_cache_create(*wl.cache_args)
    B.ll_cache_set_kv_format(h8, B.LL_KV_E4M3)
    b16, b8 = B.ll_cache_storage_bytes(h16), B.ll_cache_storage_bytes(h8)
    kv = wl.heads * (wl.sink_frames + wl.window_frames) * wl.tokens_per_frame * wl.head_dim
    # 30 layers: codes take half of bf16; one bf16 staging pair is added once
    assert abs((b16 - b8) - (wl.layers * 2 * kv - 4 * kv)) < 64 * 1024
    assert b8 < 0.54 * b16
    B.ll_cache_destroy(h16)
    B.ll_cache_destroy(h8)
    small = synth.Workload("fmt", 1, 2, 64, 4, 4, 1, 1, 2, n_chunks=1, seed=0)
    cache = B.Cache(*small.cache_args, kv_format=B.LL_KV_E4M3)
    with pytest.raises(B.LLError) as e:
        B.ll_cache_set_kv_format(cache.h, B.LL_KV_BF16)
    assert e.value.code == B.LL_ERR_INVALID_ARG
    with pytest.raises(B.LLError) as e:
        cache.set_kv_scales(0, [1.0, -1.0], [1.0, 1.0])
    assert e.value.code == B.LL_ERR_INVALID_ARG
    q, k, v = (dev(t) for t in synth.chunk_qkv(small, 0))
    g = torch.ones(2 * 64, device="cuda")
    with pytest.raises(B.LLError) as e:
        cache.norm_rope_append_kv(0, q, k, v, g, g, 1e-6, 0, 4, 4)
    assert e.value.code == B.LL_ERR_UNSUPPORTED_SHAPE
    assert cache.state()["end"] == 0
    cache.close()
