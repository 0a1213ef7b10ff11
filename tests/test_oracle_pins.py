"""Pins for the CPU oracle: facts fixed by the paper and by mathematics.

None of these tests re-types the oracle's own formula.  Each one checks the
oracle against something independent: a literal list-based cache (Sec. 3.3
"Frame Sink"), a flat library-softmax attention over the full history, closed
forms, a complex-number textbook RoPE, and constants the paper prints.
"""
import os

import numpy as np
import pytest
from scipy.special import logsumexp, softmax

from paper_2509_22622_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def golden():
    out = {}
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.split("#")[0].split()
            if line:
                out[line[0]] = [int(t) for t in line[1:]]
    return out


def rand(shape, seed):
    return synth.bf16_bits_to_f64(synth.normal_bf16(np.random.default_rng(seed), shape))


# ---------------------------------------------------------------------------
# independent references used by the pins
# ---------------------------------------------------------------------------

def literal_cache_frames(end, S, W):
    """Sec. 3.3 read literally: the first chunk stays, the rest is the last W frames."""
    frames = list(range(end))
    sink = frames[:S]
    rest = frames[S:]
    window = [f for f in frames[-W:] if f in rest] if W > 0 else []
    return sink + window


def textbook_rope_1d(x, pos, theta):
    """RoFormer's rotary embedding on pairs (2i, 2i+1), as complex multiplication."""
    d = x.shape[-1]
    z = x[..., 0::2] + 1j * x[..., 1::2]
    freq = theta ** (-np.arange(0, d, 2) / d)
    z = z * np.exp(1j * pos * freq)
    out = np.empty_like(x)
    out[..., 0::2] = z.real
    out[..., 1::2] = z.imag
    return out


def flat_block_causal(q, keys, vals, q_chunk, key_chunk):
    """Full-history attention with library softmax.  q [nq,H,D]; keys/vals [nk,H,D];
    key j is visible iff its chunk id <= the query's chunk id."""
    D = q.shape[-1]
    s = np.einsum("qhd,khd->hqk", q, keys) / np.sqrt(D)
    mask = key_chunk[None, :] <= q_chunk[:, None]
    s = np.where(mask[None], s, -np.inf)
    p = softmax(s, axis=-1)
    return np.einsum("hqk,khd->qhd", p, vals), logsumexp(s, axis=-1).T


# ---------------------------------------------------------------------------
# slot rule, visible set, sink persistence
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("C,S,W", [(1, 1, 2), (3, 3, 9), (2, 2, 4), (1, 0, 3), (2, 4, 6), (3, 3, 3)])
def test_resident_frames_match_literal_cache(oracle_mod, C, S, W):
    """After every append the slot table holds exactly sink + last W frames."""
    o = oracle_mod.Oracle(1, 1, 2, 1, C, S, W)
    for chunk in range(12):
        x = np.zeros((C, 1, 2))
        o.append(0, x, x, chunk * C, 1, 1)
        st = o.state()
        end = (chunk + 1) * C
        assert st["end"] == end
        resident = sorted(int(f) for f in st["slot_frame"] if f >= 0)
        assert resident == sorted(set(literal_cache_frames(end, S, W)))
        # every resident frame sits where the slot rule says
        for f in resident:
            assert st["slot_frame"][o.slot_of(f)] == f


@pytest.mark.parametrize("C,S,W", [(1, 1, 2), (3, 3, 9), (2, 2, 4), (1, 0, 3), (3, 3, 3)])
def test_visible_set_bruteforce(oracle_mod, C, S, W):
    """visible(fq, fk) for the newest chunk == the literal cache content, for every fq, fk."""
    o = oracle_mod.Oracle(1, 1, 2, 1, C, S, W)
    for chunk in range(10):
        end = (chunk + 1) * C
        expect = set(literal_cache_frames(end, S, W))
        for fq in range(chunk * C, end):
            got = {fk for fk in range(-2, end + 4) if o.visible(fq, fk)}
            assert got == expect, (chunk, fq)


def test_visible_set_is_block_causal_for_old_queries(oracle_mod):
    """A query of an older chunk sees nothing from later chunks, all of its own chunk."""
    o = oracle_mod.Oracle(1, 1, 2, 1, 3, 3, 9)
    for fq in range(0, 30):
        hi = (fq // 3 + 1) * 3
        vis = {fk for fk in range(40) if o.visible(fq, fk)}
        assert max(vis) == hi - 1
        assert set(range(fq // 3 * 3, hi)) <= vis
        assert vis == set(literal_cache_frames(hi, 3, 9))


def test_steady_state_key_count_matches_paper(oracle_mod):
    g = golden()
    C, S, W = g["chunk_frames"][0], g["sink_frames"][0], g["window_frames"][0]
    o = oracle_mod.Oracle(1, 1, 2, 1, C, S, W)
    n_vis = sum(o.visible(20 * C, fk) for fk in range(100))
    assert n_vis == g["effective_frames"][0]
    assert n_vis * g["tokens_per_frame"][0] == g["max_keys"][0]
    # a 21-frame clip under sink 3 + window 18 is full block-causal attention
    o2 = oracle_mod.Oracle(1, 1, 2, 1, C, S, 18)
    for fq in range(g["clip_latent_frames"][0]):
        hi = (fq // C + 1) * C
        assert {fk for fk in range(30) if o2.visible(fq, fk)} == set(range(hi))


def test_sink_never_evicted_and_bytes_stable(oracle_mod):
    C, S, W, P, H, D = 2, 2, 4, 3, 2, 8
    o = oracle_mod.Oracle(1, H, D, P, C, S, W)
    sink_k = sink_v = None
    for chunk in range(9):
        k, v = rand((C * P, H, D), 10 + chunk), rand((C * P, H, D), 50 + chunk)
        o.append(0, k, v, chunk * C, 1, 3)
        K, V = o.read_layer()
        if chunk == 0:
            sink_k, sink_v = K[:S].copy(), V[:S].copy()
            assert np.array_equal(V[:S].reshape(C * P, H, D), v)
        if chunk == 4:   # a recache in the middle must not touch the sink
            n = min(W, (chunk + 1) * C - S)
            qn, kn, vn = (rand((n * P, H, D), 90 + i) for i in range(3))
            o.recache(0, qn, kn, vn, n, 1, 3)
            K, V = o.read_layer()
        assert list(o.state()["slot_frame"][:S]) == list(range(S))
        assert np.array_equal(K[:S], sink_k) and np.array_equal(V[:S], sink_v)
    assert o.state()["evictions"] == 9 * C - S - W


def test_append_position_rules(oracle_mod):
    o = oracle_mod.Oracle(1, 1, 2, 1, 2, 2, 4)
    x = np.zeros((2, 1, 2))
    with pytest.raises(oracle_mod.OracleError):
        o.append(0, x, x, 2, 1, 1)          # skips chunk 0
    o.append(0, x, x, 0, 1, 1)
    o.append(0, x, x, 0, 1, 1)              # overwrite newest: state unchanged
    assert o.state()["end"] == 2
    o.append(0, x, x, 2, 1, 1)
    with pytest.raises(oracle_mod.OracleError):
        o.append(0, x, x, 0, 1, 1)          # not the newest chunk any more
    o.reset()
    assert o.state()["end"] == 0 and all(o.state()["slot_frame"] == -1)


# ---------------------------------------------------------------------------
# RoPE
# ---------------------------------------------------------------------------

def test_rope_band_sizes_match_definition(oracle_mod):
    g = golden()
    assert list(oracle_mod.rope_split(128)) == g["rope_pairs_d128"]
    assert [2 * n for n in oracle_mod.rope_split(64)] == g["rope_dims_d64"]


@pytest.mark.parametrize("D", [64, 128])
def test_rope_reduces_to_textbook_1d(oracle_mod, D):
    """On a 1x1 grid only the t band turns, and it is RoFormer's rotation."""
    n_t, n_h, n_w = oracle_mod.rope_split(D)
    x = rand((5, 3, D), 3)
    got = oracle_mod.rope(x, frame_start=7, gh=1, gw=1, theta=10000.0)
    for i in range(5):
        want = x[i].copy()
        want[:, :2 * n_t] = textbook_rope_1d(x[i][:, :2 * n_t], 7 + i, 10000.0)
        np.testing.assert_allclose(got[i], want, rtol=0, atol=1e-12)


@pytest.mark.parametrize("D", [64, 128])
def test_rope_each_axis_is_textbook_on_its_band(oracle_mod, D):
    """Frame 0: t band idle; h and w bands turn by y and x (row-major tokens)."""
    n_t, n_h, n_w = oracle_mod.rope_split(D)
    gh, gw = 3, 4
    x = rand((gh * gw, 2, D), 4)
    got = oracle_mod.rope(x, 0, gh, gw, 100.0)
    a, b = 2 * n_t, 2 * (n_t + n_h)
    for n in range(gh * gw):
        yy, xx = divmod(n, gw)
        want = x[n].copy()
        want[:, a:b] = textbook_rope_1d(x[n][:, a:b], yy, 100.0)
        want[:, b:] = textbook_rope_1d(x[n][:, b:], xx, 100.0)
        np.testing.assert_allclose(got[n], want, rtol=0, atol=1e-12)


def test_rope_identity_norm_and_relative_property(oracle_mod):
    D, gh, gw = 128, 2, 3
    x = rand((gh * gw, 2, D), 5)
    r = oracle_mod.rope(x, 0, gh, gw)
    assert np.array_equal(r[0], x[0])                       # position (0,0,0)
    pair_norm = lambda a: a[..., 0::2] ** 2 + a[..., 1::2] ** 2
    np.testing.assert_allclose(pair_norm(r), pair_norm(x), rtol=1e-12)
    # scores depend on position differences only: shift t of both q and k
    q, k = rand((gh * gw, 2, D), 6), rand((gh * gw, 2, D), 7)
    s0 = np.einsum("qhd,khd->hqk", oracle_mod.rope(q, 3, gh, gw), oracle_mod.rope(k, 1, gh, gw))
    s1 = np.einsum("qhd,khd->hqk", oracle_mod.rope(q, 903, gh, gw), oracle_mod.rope(k, 901, gh, gw))
    np.testing.assert_allclose(s0, s1, rtol=0, atol=1e-9)
    # ...but do change when only one side moves
    s2 = np.einsum("qhd,khd->hqk", oracle_mod.rope(q, 4, gh, gw), oracle_mod.rope(k, 1, gh, gw))
    assert np.abs(s2 - s0).max() > 1e-3


def test_round_bf16_matches_bit_rounding(oracle_mod):
    x = np.random.default_rng(0).standard_normal(2000).astype(np.float32)
    want = synth.bf16_bits_to_f64(synth.f32_to_bf16_bits(x))
    np.testing.assert_array_equal(oracle_mod.round_bf16(x.astype(np.float64)), want)
    ties = np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, -(2 + 2.0 ** -7)])
    np.testing.assert_array_equal(oracle_mod.round_bf16(ties), [1.0, 1.015625, -2.0])


# ---------------------------------------------------------------------------
# attention
# ---------------------------------------------------------------------------

def stream(o, n_chunks, gh, gw, seed, theta=10000.0):
    """Append n_chunks chunks, attend each as it arrives.  Returns per-chunk
    (out, lse) plus the flat roped history for the flat reference."""
    P = gh * gw
    outs, hist_k, hist_v, hist_q = [], [], [], []
    for c in range(n_chunks):
        q, k, v = (rand((o.C * P, o.H, o.D), seed + 3 * c + i) for i in range(3))
        o.append(0, k, v, c * o.C, gh, gw, theta)
        qr = o.rope_q(q, c * o.C, gh, gw, theta)
        outs.append(o.attn(0, qr, c * o.C))
        hist_q.append(qr)
        hist_k.append(oracle_mod_rope(k, c * o.C, gh, gw, theta))
        hist_v.append(v)
    return outs, hist_q, hist_k, hist_v


def oracle_mod_rope(x, fs, gh, gw, theta):
    import oracle
    return oracle.rope(x, fs, gh, gw, theta)


@pytest.mark.parametrize("C,S,W,n_chunks", [(1, 1, 7, 8), (2, 2, 8, 5), (2, 0, 10, 5), (3, 3, 9, 4)])
def test_window_covering_history_is_full_causal(oracle_mod, C, S, W, n_chunks):
    """W >= total - S: sink+window equals flat block-causal attention."""
    gh, gw, H, D = 2, 3, 2, 16
    P = gh * gw
    o = oracle_mod.Oracle(1, H, D, P, C, S, W)
    outs, hq, hk, hv = stream(o, n_chunks, gh, gw, 100)
    keys, vals = np.concatenate(hk), np.concatenate(hv)
    key_chunk = np.repeat(np.arange(n_chunks), C * P)
    for c in range(n_chunks):
        want, want_lse = flat_block_causal(hq[c], keys, vals, np.full(C * P, c), key_chunk)
        np.testing.assert_allclose(outs[c][0], want, rtol=0, atol=1e-12)
        np.testing.assert_allclose(outs[c][1], want_lse, rtol=0, atol=1e-12)


def test_short_window_equals_flat_attention_over_literal_cache(oracle_mod):
    """With eviction: equals library-softmax attention over sink + last W frames."""
    C, S, W, gh, gw, H, D = 2, 2, 4, 2, 2, 2, 16
    P = gh * gw
    o = oracle_mod.Oracle(1, H, D, P, C, S, W)
    outs, hq, hk, hv = stream(o, 7, gh, gw, 200)
    keys, vals = np.concatenate(hk), np.concatenate(hv)
    differs = False
    for c in range(7):
        frames = literal_cache_frames((c + 1) * C, S, W)
        idx = np.concatenate([np.arange(f * P, (f + 1) * P) for f in frames])
        s = np.einsum("qhd,khd->hqk", hq[c], keys[idx]) / np.sqrt(D)
        want = np.einsum("hqk,khd->qhd", softmax(s, axis=-1), vals[idx])
        np.testing.assert_allclose(outs[c][0], want, rtol=0, atol=1e-12)
        full, _ = flat_block_causal(hq[c], keys, vals, np.full(C * P, c), np.repeat(np.arange(7), C * P))
        differs |= np.abs(full - want).max() > 1e-6
    assert differs      # once frames are evicted the result is not full attention


def test_single_visible_key_returns_its_value(oracle_mod):
    o = oracle_mod.Oracle(1, 2, 8, 1, 1, 1, 2)
    q, k, v = rand((1, 2, 8), 1), rand((1, 2, 8), 2), rand((1, 2, 8), 3)
    o.append(0, k, v, 0, 1, 1)
    out, lse = o.attn(0, o.rope_q(q, 0, 1, 1), 0)
    np.testing.assert_array_equal(out, v)
    np.testing.assert_allclose(lse[0], np.einsum("hd,hd->h", q[0], k[0]) / np.sqrt(8), atol=1e-13)


def test_softmax_rows_sum_to_one_and_keys_are_the_resident_rows(oracle_mod):
    C, S, W, gh, gw, H, D = 1, 1, 2, 4, 4, 2, 64
    P = gh * gw
    o = oracle_mod.Oracle(1, H, D, P, C, S, W)
    for c in range(6):
        q, k, v = (rand((P, H, D), 300 + 3 * c + i) for i in range(3))
        o.append(0, k, v, c, gh, gw)
        qr = o.rope_q(q, c, gh, gw)
        out, lse = o.attn(0, qr, c)
        K, V = o.read_layer()
        for row in (0, P - 1):
            for h in range(H):
                p, kr = o.attn_probs(0, qr, c, row, h)
                assert abs(p.sum() - 1.0) < 1e-12
                frames = literal_cache_frames(c + 1, S, W)
                want_rows = sorted(o.slot_of(f) * P + n for f in frames for n in range(P))
                assert sorted(kr) == want_rows
                vv = V.reshape(-1, H, D)[kr, h]
                np.testing.assert_allclose(p @ vv, out[row, h], atol=1e-12)
                kk = K.reshape(-1, H, D)[kr, h]
                s = kk @ qr[row, h] / np.sqrt(D)
                np.testing.assert_allclose(logsumexp(s), lse[row, h], atol=1e-12)


def test_zero_keys_give_visible_histogram(oracle_mod):
    """K == 0: uniform weights, so with V = one-hot(frame id) the output is the
    histogram of visible frames; with V constant the output is that constant."""
    C, S, W, gh, gw, H = 3, 3, 9, 2, 2, 1
    P = gh * gw
    D = 32
    o = oracle_mod.Oracle(1, H, D, P, C, S, W)
    for c in range(8):
        k = np.zeros((C * P, H, D))
        v = np.zeros((C * P, H, D))
        for i in range(C):
            v[i * P:(i + 1) * P, :, c * C + i] = 1.0
        o.append(0, k, v, c * C, gh, gw)
        out, lse = o.attn(0, rand((C * P, H, D), c), c * C)
        frames = literal_cache_frames((c + 1) * C, S, W)
        want = np.zeros(D)
        want[frames] = 1.0 / len(frames)
        np.testing.assert_allclose(out, np.broadcast_to(want, out.shape), atol=1e-15)
        np.testing.assert_allclose(lse, np.log(len(frames) * P), atol=1e-13)
    o2 = oracle_mod.Oracle(1, H, D, P, C, S, W)
    for c in range(5):
        o2.append(0, rand((C * P, H, D), 40 + c), np.full((C * P, H, D), 0.75), c * C, gh, gw)
        out, _ = o2.attn(0, rand((C * P, H, D), c), c * C)
        np.testing.assert_allclose(out, 0.75, atol=1e-14)


def test_recache_equals_streaming_when_nothing_was_evicted(oracle_mod):
    """Bulk block-causal recache over chunks 1..k == attending them one by one."""
    C, S, W, gh, gw, H, D = 2, 2, 6, 2, 2, 2, 16
    P = gh * gw
    o = oracle_mod.Oracle(1, H, D, P, C, S, W)
    qs, ks, vs, outs = [], [], [], []
    for c in range(4):                       # sink chunk + 3 ring chunks, no eviction
        q, k, v = (rand((C * P, H, D), 500 + 3 * c + i) for i in range(3))
        o.append(0, k, v, c * C, gh, gw)
        outs.append(o.attn(0, o.rope_q(q, c * C, gh, gw), c * C))
        qs.append(q); ks.append(k); vs.append(v)
    before = o.state()
    qr, out, lse = o.recache(0, np.concatenate(qs[1:]), np.concatenate(ks[1:]),
                             np.concatenate(vs[1:]), 3 * C, gh, gw)
    after = o.state()
    assert before["end"] == after["end"] and np.array_equal(before["slot_frame"], after["slot_frame"])
    np.testing.assert_allclose(out, np.concatenate([x[0] for x in outs[1:]]), atol=1e-13)
    np.testing.assert_allclose(lse, np.concatenate([x[1] for x in outs[1:]]), atol=1e-13)


def test_recache_after_wraparound_matches_flat_reference(oracle_mod):
    """Ring wrapped: recache rows see sink + window frames up to their own chunk."""
    C, S, W, gh, gw, H, D = 1, 1, 3, 2, 2, 2, 16
    P = gh * gw
    o = oracle_mod.Oracle(1, H, D, P, C, S, W)
    sink_k = sink_v = None
    for c in range(6):
        k, v = rand((P, H, D), 700 + c), rand((P, H, D), 800 + c)
        o.append(0, k, v, c, gh, gw)
        if c == 0:
            sink_k, sink_v = oracle_mod.rope(k, 0, gh, gw), v
    q, k, v = (rand((W * P, H, D), 900 + i) for i in range(3))
    qr, out, lse = o.recache(0, q, k, v, W, gh, gw)
    r0 = 6 - W
    kr = oracle_mod.rope(k, r0, gh, gw)
    np.testing.assert_allclose(qr, oracle_mod.rope(q, r0, gh, gw), atol=0)
    keys = np.concatenate([sink_k, kr]); vals = np.concatenate([sink_v, v])
    key_chunk = np.concatenate([np.full(P, -1), np.repeat(np.arange(W), P)])
    want, want_lse = flat_block_causal(qr, keys, vals, np.repeat(np.arange(W), P), key_chunk)
    np.testing.assert_allclose(out, want, atol=1e-12)
    np.testing.assert_allclose(lse, want_lse, atol=1e-12)
    # the next chunk then attends over the rebuilt ring
    q2, k2, v2 = (rand((P, H, D), 950 + i) for i in range(3))
    o.append(0, k2, v2, 6, gh, gw)
    out2, _ = o.attn(0, o.rope_q(q2, 6, gh, gw), 6)
    keys2 = np.concatenate([sink_k, kr[P:], oracle_mod.rope(k2, 6, gh, gw)])
    vals2 = np.concatenate([sink_v, v[P:], v2])
    s = np.einsum("qhd,khd->hqk", oracle_mod.rope(q2, 6, gh, gw), keys2) / np.sqrt(D)
    np.testing.assert_allclose(out2, np.einsum("hqk,khd->qhd", softmax(s, -1), vals2), atol=1e-12)


def test_recache_with_only_sink_is_a_noop(oracle_mod):
    o = oracle_mod.Oracle(1, 1, 4, 1, 2, 2, 4)
    x = np.zeros((2, 1, 4))
    o.append(0, x, x, 0, 1, 1)
    e = np.zeros((0, 1, 4))
    qr, out, lse = o.recache(0, e, e, e, 0, 1, 1)
    assert out.shape[0] == 0
    with pytest.raises(oracle_mod.OracleError):
        o.recache(0, x, x, x, 2, 1, 1)


def test_sampled_rows_equal_full_evaluation(oracle_mod):
    C, S, W, gh, gw, H, D = 2, 2, 4, 2, 3, 2, 16
    P = gh * gw
    o = oracle_mod.Oracle(1, H, D, P, C, S, W)
    for c in range(4):
        q, k, v = (rand((C * P, H, D), 600 + 3 * c + i) for i in range(3))
        o.append(0, k, v, c * C, gh, gw)
    qr = o.rope_q(q, 3 * C, gh, gw)
    full, lse = o.attn(0, qr, 3 * C)
    rows = np.array([0, 5, C * P - 1])
    part, lse_p = o.attn(0, qr, 3 * C, rows=rows)
    np.testing.assert_array_equal(part, full[rows])
    np.testing.assert_array_equal(lse_p, lse[rows])


def test_faithful_mode_rounds_stored_keys_only(oracle_mod):
    C, S, W, gh, gw, H, D = 1, 1, 2, 2, 2, 1, 64
    P = gh * gw
    a = oracle_mod.Oracle(1, H, D, P, C, S, W, faithful=False)
    b = oracle_mod.Oracle(1, H, D, P, C, S, W, faithful=True)
    k, v = rand((P, H, D), 1), rand((P, H, D), 2)
    a.append(0, k, v, 0, gh, gw); b.append(0, k, v, 0, gh, gw)
    Ka, Va = a.read_layer(); Kb, Vb = b.read_layer()
    np.testing.assert_array_equal(Va, Vb)
    np.testing.assert_array_equal(Kb[0], oracle_mod.round_bf16(Ka[0]))
    assert np.abs(Ka[0] - Kb[0]).max() <= 2.0 ** -8 * np.abs(Ka[0]).max()


def test_ring_fills_from_its_first_slot(oracle_mod):
    """The slot contract: while the ring is filling, resident frames are a
    contiguous prefix of the storage (frame f sits in slot f), and the first
    evicted frame is the oldest window frame."""
    C, S, W = 3, 3, 9
    o = oracle_mod.Oracle(1, 1, 2, 1, C, S, W)
    x = np.zeros((C, 1, 2))
    for chunk in range(4):
        o.append(0, x, x, chunk * C, 1, 1)
        sf = list(o.state()["slot_frame"])
        end = (chunk + 1) * C
        assert sf == list(range(end)) + [-1] * (S + W - end)
    o.append(0, x, x, 12, 1, 1)      # frames 12..14 replace frames 3..5 in place
    assert list(o.state()["slot_frame"]) == [0, 1, 2, 12, 13, 14, 6, 7, 8, 9, 10, 11]
    assert o.state()["evictions"] == 3


def test_seek_equals_full_replay(oracle_mod):
    """Skipping evicted history gives the same attention as replaying all of it."""
    C, S, W, gh, gw, H, D = 2, 2, 4, 2, 2, 2, 16
    P = gh * gw
    full = oracle_mod.Oracle(1, H, D, P, C, S, W)
    data = [tuple(rand((C * P, H, D), 1000 + 3 * c + i) for i in range(3)) for c in range(9)]
    for c, (q, k, v) in enumerate(data):
        full.append(0, k, v, c * C, gh, gw)
    want = full.attn(0, full.rope_q(data[8][0], 16, gh, gw), 16)
    short = oracle_mod.Oracle(1, H, D, P, C, S, W)
    short.append(0, data[0][1], data[0][2], 0, gh, gw)          # the sink chunk
    short.seek(0, 14)                                           # window = chunks 7, 8
    with pytest.raises(oracle_mod.OracleError):
        short.attn(0, short.rope_q(data[8][0], 16, gh, gw), 12)  # nothing resident yet
    for c in (7, 8):
        short.append(0, data[c][1], data[c][2], c * C, gh, gw)
    got = short.attn(0, short.rope_q(data[8][0], 16, gh, gw), 16)
    np.testing.assert_array_equal(got[0], want[0])
    np.testing.assert_array_equal(got[1], want[1])
    assert list(short.state()["slot_frame"]) == list(full.state()["slot_frame"])
    with pytest.raises(oracle_mod.OracleError):
        short.seek(0, 4)                                        # cannot go back


# ---------------------------------------------------------------------------
# a clip in one step (Sec. 3.3, "Consistency between Training and Inference")
# ---------------------------------------------------------------------------

def clip_flat_reference(oracle_mod, hist_q, hist_k, hist_v, first_clip_chunk, C, S, window, gh, gw):
    """Library-softmax attention of the clip's queries over the frames Sec. 3.3 keeps for them,
    written from the text: the sink frames, and of all other frames up to the query's own chunk
    the last `window` ones.  hist_* hold every chunk of the stream so far, raw."""
    P = gh * gw
    D = hist_q[0].shape[-1]
    keys = np.concatenate([oracle_mod.rope(k, c * C, gh, gw) for c, k in enumerate(hist_k)])
    vals = np.concatenate(hist_v)
    outs, lses = [], []
    for c in range(first_clip_chunk, len(hist_q)):
        upto = list(range((c + 1) * C))
        frames = [f for f in upto if f < S] + [f for f in upto[-window:] if f >= S]
        idx = np.concatenate([np.arange(f * P, (f + 1) * P) for f in frames])
        qr = oracle_mod.rope(hist_q[c], c * C, gh, gw)
        s = np.einsum("qhd,khd->hqk", qr, keys[idx]) / np.sqrt(D)
        outs.append(np.einsum("hqk,khd->qhd", softmax(s, axis=-1), vals[idx]))
        lses.append(logsumexp(s, axis=-1).T)
    return np.concatenate(outs), np.concatenate(lses)


@pytest.mark.parametrize("C,S,window,clip_chunks,before", [(1, 1, 2, 3, 4), (2, 2, 4, 2, 3), (1, 0, 1, 4, 2),
                                                            (2, 2, 2, 3, 0), (1, 2, 3, 2, 1)])
def test_clip_equals_flat_attention_over_sink_context_tail_and_clip(oracle_mod, C, S, window, clip_chunks, before):
    gh, gw, H, D = 2, 3, 2, 16
    P = gh * gw
    T = clip_chunks * C
    ring = window + T - C                      # resident set of S + (window - C) + T frames: O(W + T + S)
    o = oracle_mod.Oracle(1, H, D, P, C, S, ring)
    hq, hk, hv = [], [], []
    for c in range(before + clip_chunks):
        q, k, v = (rand((C * P, H, D), 1000 + 10 * c + i) for i in range(3))
        hq.append(q); hk.append(k); hv.append(v)
        if c < before:
            o.append(0, k, v, c * C, gh, gw)
    q, k, v = (np.concatenate(h[before:]) for h in (hq, hk, hv))
    qr, out, lse = o.clip(0, q, k, v, before * C, T, window, gh, gw)
    want, want_lse = clip_flat_reference(oracle_mod, hq, hk, hv, before, C, S, window, gh, gw)
    np.testing.assert_allclose(out, want, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, want_lse, rtol=0, atol=1e-12)
    np.testing.assert_array_equal(qr, oracle_mod.rope(q, before * C, gh, gw))
    assert o.state()["end"] == (before + clip_chunks) * C


def test_clip_equals_chunk_by_chunk_decoding_with_that_window(oracle_mod):
    """Train/inference consistency itself: the clip step gives every chunk exactly what
    streaming inference with a ring of `window` frames gives it."""
    C, S, window, gh, gw, H, D = 2, 2, 4, 2, 2, 2, 16
    P = gh * gw
    clip_chunks, before = 4, 5
    T = clip_chunks * C
    big = oracle_mod.Oracle(1, H, D, P, C, S, window + T - C)
    small = oracle_mod.Oracle(1, H, D, P, C, S, window)
    outs = []
    data = [[rand((C * P, H, D), 2000 + 10 * c + i) for i in range(3)] for c in range(before + clip_chunks)]
    for c, (q, k, v) in enumerate(data):
        small.append(0, k, v, c * C, gh, gw)
        if c < before:
            big.append(0, k, v, c * C, gh, gw)
        else:
            outs.append(small.attn(0, small.rope_q(q, c * C, gh, gw), c * C))
    q, k, v = (np.concatenate([d[i] for d in data[before:]]) for i in range(3))
    _, out, lse = big.clip(0, q, k, v, before * C, T, window, gh, gw)
    np.testing.assert_allclose(out, np.concatenate([x[0] for x in outs]), rtol=0, atol=1e-13)
    np.testing.assert_allclose(lse, np.concatenate([x[1] for x in outs]), rtol=0, atol=1e-13)
    # a longer window than the one asked for would see more: the result really depends on it
    big2 = oracle_mod.Oracle(1, H, D, P, C, S, window + T - C)
    for c in range(before):
        big2.append(0, data[c][1], data[c][2], c * C, gh, gw)
    _, out2, _ = big2.clip(0, q, k, v, before * C, T, window - C, gh, gw)
    assert np.abs(out2 - out).max() > 1e-6


def test_clip_rejects_a_ring_too_short_for_it(oracle_mod):
    C, S, window = 1, 1, 3
    o = oracle_mod.Oracle(1, 1, 8, 1, C, S, 4)
    x = rand((3, 1, 8), 5)
    with pytest.raises(oracle_mod.OracleError):
        o.clip(0, x, x, x, 0, 3, window, 1, 1)          # needs 3 + 3 - 1 = 5 ring frames
    o.clip(0, x[:2], x[:2], x[:2], 0, 2, window, 1, 1)  # 3 + 2 - 1 = 4 fits
    with pytest.raises(oracle_mod.OracleError):
        o.clip(0, x[:2], x[:2], x[:2], 0, 2, window, 1, 1)   # not at the stream's end any more


# ---------------------------------------------------------------------------
# dense attention (cross-attention to the prompt, Sec. 3.1)
# ---------------------------------------------------------------------------

def test_dense_attention_equals_library_softmax(oracle_mod):
    q, k, v = rand((37, 3, 16), 1), rand((29, 3, 16), 2), rand((29, 3, 16), 3)
    out, lse = oracle_mod.dense_attn(q, k, v)
    s = np.einsum("qhd,khd->hqk", q, k) / np.sqrt(16)
    np.testing.assert_allclose(out, np.einsum("hqk,khd->qhd", softmax(s, axis=-1), v), rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, logsumexp(s, axis=-1).T, rtol=0, atol=1e-12)
    rows = np.array([36, 0, 5])
    out_r, lse_r = oracle_mod.dense_attn(q, k, v, rows=rows)
    np.testing.assert_array_equal(out_r, out[rows])
    np.testing.assert_array_equal(lse_r, lse[rows])


def test_dense_attention_special_cases(oracle_mod):
    q, k, v = rand((5, 2, 8), 4), rand((1, 2, 8), 5), rand((1, 2, 8), 6)
    out, lse = oracle_mod.dense_attn(q, k, v)                       # one key: its value, lse = the score
    np.testing.assert_array_equal(out, np.broadcast_to(v, out.shape))
    np.testing.assert_allclose(lse, np.einsum("qhd,hd->qh", q, k[0]) / np.sqrt(8), atol=1e-13)
    k0 = np.zeros((7, 2, 8)); v7 = rand((7, 2, 8), 7)
    out, lse = oracle_mod.dense_attn(q, k0, v7)                     # equal scores: the mean of the values
    np.testing.assert_allclose(out, np.broadcast_to(v7.mean(axis=0), out.shape), atol=1e-14)
    np.testing.assert_allclose(lse, np.log(7.0), atol=1e-14)
    # permuting the keys (with their values) changes nothing; heads do not mix
    k9, v9 = rand((9, 2, 8), 8), rand((9, 2, 8), 9)
    perm = np.random.default_rng(0).permutation(9)
    a, _ = oracle_mod.dense_attn(q, k9, v9)
    b, _ = oracle_mod.dense_attn(q, k9[perm], v9[perm])
    np.testing.assert_allclose(a, b, atol=1e-13)
    k9b = k9.copy(); k9b[:, 1] *= 2.0
    c, _ = oracle_mod.dense_attn(q, k9b, v9)
    np.testing.assert_array_equal(a[:, 0], c[:, 0])
    assert np.abs(a[:, 1] - c[:, 1]).max() > 1e-6


# ---------------------------------------------------------------------------
# RMS norm of q/k rows (upstream of the rotation; not in the paper)
# ---------------------------------------------------------------------------

def test_rms_norm_closed_forms(oracle_mod):
    # the 3-4-5 row: mean square 12.5
    y = oracle_mod.rms_norm(np.array([[[3.0, 4.0]]]), np.ones(2), 0.0)
    np.testing.assert_allclose(y, np.array([[[3.0, 4.0]]]) / np.sqrt(12.5), rtol=1e-15)
    # a constant row c with eps: c / sqrt(c^2 + eps) * gain
    g = np.array([0.5, -2.0, 1.0, 3.0])
    y = oracle_mod.rms_norm(np.full((1, 2, 2), -1.5), g, 0.25)
    np.testing.assert_allclose(y.reshape(-1), -1.5 / np.sqrt(2.5) * g, rtol=1e-15)
    # a zero row stays zero (eps keeps the division finite)
    assert np.all(oracle_mod.rms_norm(np.zeros((2, 1, 4)), np.ones(4), 1e-6) == 0.0)


def test_rms_norm_invariants(oracle_mod):
    x = rand((9, 3, 8), 77)
    g = rand((3, 8), 78)
    y = oracle_mod.rms_norm(x, g, 0.0)
    # gain 1: every token's whole row has mean square 1, whatever its scale
    y1 = oracle_mod.rms_norm(x, np.ones(24), 0.0)
    np.testing.assert_allclose((y1.reshape(9, -1) ** 2).mean(axis=1), 1.0, rtol=1e-13)
    np.testing.assert_allclose(oracle_mod.rms_norm(7.0 * x, g, 0.0), y, rtol=1e-13)
    # the gain multiplies element-wise, the norm is over the row, not per head
    np.testing.assert_allclose(y, y1 * g[None], rtol=1e-14)
    per_head = x / np.sqrt((x ** 2).mean(axis=2, keepdims=True))
    assert np.abs(per_head - y1).max() > 1e-3
    # tokens are independent
    x2 = x.copy(); x2[4] *= 3.0
    y2 = oracle_mod.rms_norm(x2, g, 1e-6)
    ye = oracle_mod.rms_norm(x, g, 1e-6)
    np.testing.assert_array_equal(np.delete(y2, 4, axis=0), np.delete(ye, 4, axis=0))
    # eps matters for small rows: with eps the output shrinks
    small = 1e-3 * x
    assert np.abs(oracle_mod.rms_norm(small, g, 1e-6)).max() < np.abs(oracle_mod.rms_norm(small, g, 0.0)).max()


# ---------------------------------------------------------------------------
# 8-bit (E4M3) cache storage
# ---------------------------------------------------------------------------

def e4m3_table():
    """Every finite E4M3 value decoded from its bit pattern: sign(1) exponent(4, bias 7)
    mantissa(3); exponent field 0 is subnormal; S.1111.111 is NaN (no infinities)."""
    vals = {}
    for code in range(256):
        sgn, e, m = code >> 7, (code >> 3) & 15, code & 7
        if e == 15 and m == 7:
            continue
        mag = (m / 8.0) * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7)
        vals[code] = -mag if sgn else mag
    return vals


def brute_force_e4m3(x):
    """Nearest table value, ties to the code with an even mantissa, clamped to +-448."""
    table = e4m3_table()
    pos = sorted((v, c) for c, v in table.items() if c < 128)
    a = min(abs(float(x)), 448.0)
    best = min(pos, key=lambda vc: (abs(vc[0] - a), vc[1] & 1))
    return best[0] if x >= 0 else -best[0]


def test_e4m3_rounding_equals_brute_force_over_the_code_table(oracle_mod):
    table = e4m3_table()
    assert len(table) == 254 and max(table.values()) == 448.0 and table[1] == 2.0 ** -9
    # every representable value is a fixed point
    for v in table.values():
        assert oracle_mod.round_e4m3(v) == v
    # every midpoint between neighbours (the ties), points just off them, random values, the ends
    pos = sorted(v for c, v in table.items() if c < 128)
    xs = []
    for lo, hi in zip(pos[:-1], pos[1:]):
        mid = 0.5 * (lo + hi)
        xs += [mid, np.nextafter(mid, 0.0), np.nextafter(mid, 1e9), 0.75 * lo + 0.25 * hi]
    rng = np.random.default_rng(0)
    xs += list(rng.standard_normal(2000) * np.exp(rng.uniform(-8, 7, 2000)))
    xs += [448.0, 449.0, 464.0, 1e6, 2.0 ** -10, 2.0 ** -11, 1e-30]
    for x in xs:
        for s in (x, -x):
            assert oracle_mod.round_e4m3(s) == brute_force_e4m3(s), s
    assert np.isnan(oracle_mod.round_e4m3(float("nan")))


def test_e4m3_cache_rows_and_attention_equal_a_flat_reference(oracle_mod):
    """The rows an 8-bit cache holds are scale * E4M3(fl32(x) / scale) of the rotated keys and
    the raw values (brute force over the code table), old rows stay as they were, and attention
    over such a cache is library softmax over exactly those numbers."""
    L, H, D, gh, gw, C, S, W = 2, 3, 64, 2, 3, 1, 1, 3
    P = gh * gw
    orc = oracle_mod.Oracle(L, H, D, P, C, S, W)
    ks = np.array([[0.02, 0.5, 1.0], [0.013, 0.25, 3.0]], dtype=np.float32)
    vs = np.array([[0.01, 0.125, 2.0], [0.7, 0.031, 1.5]], dtype=np.float32)
    k0, v0 = rand((P, H, D), 1), rand((P, H, D), 2)
    orc.append(1, k0, v0, 0, gh, gw)                       # written before the switch: stays exact
    orc.set_kv_e4m3(ks, vs)
    quant = np.vectorize(brute_force_e4m3)

    def stored(x, scale):                                  # x [P, H, D], scale [H]
        t = (x.astype(np.float32) / scale[None, :, None].astype(np.float32)).astype(np.float64)
        return quant(t) * scale[None, :, None].astype(np.float64)

    hist_k, hist_v = [oracle_mod.rope(k0, 0, gh, gw)], [v0]
    for f in range(1, 6):
        k, v = rand((P, H, D), 10 + f) * (1 + f), rand((P, H, D), 20 + f)
        orc.append(1, k, v, f, gh, gw)
        hist_k.append(stored(oracle_mod.rope(k, f, gh, gw), ks[1]))
        hist_v.append(stored(v, vs[1]))
    K, V = orc.read_layer(1)
    for f in (0, 3, 4, 5):                                 # resident: sink 0 and window 3..5
        slot = orc.slot_of(f)
        assert np.array_equal(K[slot], hist_k[f]) and np.array_equal(V[slot], hist_v[f]), f
    assert not np.array_equal(K[orc.slot_of(5)], oracle_mod.rope(k, 5, gh, gw))      # it did quantise
    q = oracle_mod.rope(rand((P, H, D), 99), 5, gh, gw)
    got, lse = orc.attn(1, q, 5)
    keys = np.concatenate([hist_k[f] for f in (0, 3, 4, 5)])
    vals = np.concatenate([hist_v[f] for f in (0, 3, 4, 5)])
    s = np.einsum("qhd,khd->hqk", q, keys) / np.sqrt(D)
    want = np.einsum("hqk,khd->qhd", softmax(s, axis=-1), vals)
    assert np.abs(got - want).max() < 1e-12
    assert np.abs(lse - logsumexp(s, axis=-1).T).max() < 1e-12
    # a recache writes quantised rows too and leaves the sink alone
    rq, rk, rv = rand((3 * P, H, D), 31), rand((3 * P, H, D), 32), rand((3 * P, H, D), 33)
    orc.recache(1, rq, rk, rv, 3, gh, gw)
    K2, V2 = orc.read_layer(1)
    assert np.array_equal(K2[0], hist_k[0]) and np.array_equal(V2[0], hist_v[0])
    for i, f in enumerate((3, 4, 5)):
        slot = orc.slot_of(f)
        assert np.array_equal(V2[slot], stored(rv[i * P:(i + 1) * P], vs[1]))
        assert np.array_equal(K2[slot], stored(oracle_mod.rope(rk[i * P:(i + 1) * P], f, gh, gw), ks[1]))
    # layer 0 uses its own scales
    orc.append(0, k0, v0, 0, gh, gw)
    K0, V0 = orc.read_layer(0)
    assert np.array_equal(V0[0], stored(v0, vs[0]))


def test_e4m3_storage_scales_by_powers_of_two_and_saturates(oracle_mod):
    """Doubling the scale and the data doubles the stored value exactly; values beyond
    448 scales clamp; the relative error inside the normal range is at most 2^-4."""
    H, D = 1, 8
    x = rand((1, H, D), 5) * 3.0
    outs = []
    for mult in (1.0, 2.0, 0.25):
        orc = oracle_mod.Oracle(1, H, D, 1, 1, 1, 1)
        orc.set_kv_e4m3(np.array([0.05 * mult], dtype=np.float32), np.array([0.05 * mult], dtype=np.float32))
        orc.append(0, x * 0.0, x * mult, 0, 1, 1)
        outs.append(orc.read_layer(0)[1][0] / mult)
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])
    assert np.abs(outs[0] - x).max() <= 2.0 ** -4 * np.abs(x).max()
    orc = oracle_mod.Oracle(1, H, D, 1, 1, 1, 1)
    orc.set_kv_e4m3(np.array([0.001], dtype=np.float32), np.array([0.001], dtype=np.float32))
    big = np.full((1, H, D), 7.0)
    orc.append(0, big * 0.0, -big, 0, 1, 1)
    assert np.array_equal(orc.read_layer(0)[1][0], np.full((1, H, D), -448.0 * float(np.float32(0.001))))


# ---------------------------------------------------------------------------
# QKV projection (the step in front of the path)
# ---------------------------------------------------------------------------

def test_qkv_projection_equals_the_written_out_sum_and_splits_q_k_v(oracle_mod):
    rng = np.random.default_rng(3)
    T, dm, n = 5, 7, 4
    x, w, b = rng.standard_normal((T, dm)), rng.standard_normal((3 * n, dm)), rng.standard_normal(3 * n)
    q, k, v = oracle_mod.qkv_proj(x, w, b)
    for t in range(T):
        for j in range(3 * n):
            want = b[j] + sum(x[t, i] * w[j, i] for i in range(dm))
            got = (q, k, v)[j // n][t, j % n]
            assert abs(got - want) < 1e-12
    # identity blocks: q = x, k = 2x, v = -x (catches a transposed weight or a wrong split)
    eye = np.eye(dm)
    q, k, v = oracle_mod.qkv_proj(x, np.concatenate([eye, 2 * eye, -eye]))
    assert np.array_equal(q, x) and np.array_equal(k, 2 * x) and np.array_equal(v, -x)


# ---------------------------------------------------------------------------
# gradients of the clip step
# ---------------------------------------------------------------------------

def _clip_loss(oracle_mod, shape, ctx, q, k, v, G, window):
    """sum(out * G) of a clip run on a fresh cache holding the context frames."""
    H, D, gh, gw, C, S, W = shape
    orc = oracle_mod.Oracle(1, H, D, gh * gw, C, S, W)
    for f, (ck, cv) in enumerate(ctx):
        orc.append(0, ck, cv, f * C, gh, gw)
    n_frames = q.shape[0] // (gh * gw)
    _, out, _ = orc.clip(0, q, k, v, len(ctx) * C, n_frames, window, gh, gw)
    return float((out * G).sum()), orc


def test_clip_backward_equals_central_finite_differences(oracle_mod):
    """Every element of dq, dk, dv against (L(x + e) - L(x - e)) / 2e of the pinned forward clip,
    L = sum(out * G): sink + context tail + earlier clip chunks all in play, window shorter than
    the clip, gradients through the rotation."""
    H, D, gh, gw, C, S, W = 2, 8, 1, 2, 1, 1, 5
    shape = (H, D, gh, gw, C, S, W)
    P, T, window = gh * gw, 3, 2
    rng = np.random.default_rng(11)
    ctx = [(rng.standard_normal((C * P, H, D)), rng.standard_normal((C * P, H, D))) for _ in range(2)]
    q, k, v = (rng.standard_normal((T * P, H, D)) for _ in range(3))
    G = rng.standard_normal((T * P, H, D))
    _, orc = _clip_loss(oracle_mod, shape, ctx, q, k, v, G, window)
    dq, dk, dv, mq, mk, mv = orc.clip_backward(0, q, G, 2 * C, T, window, gh, gw)
    eps = 1e-5
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        fd = np.zeros_like(x)
        for idx in np.ndindex(x.shape):
            xp, xm = x.copy(), x.copy()
            xp[idx] += eps
            xm[idx] -= eps
            args_p = dict(q=q, k=k, v=v); args_p[name] = xp
            args_m = dict(q=q, k=k, v=v); args_m[name] = xm
            fd[idx] = (_clip_loss(oracle_mod, shape, ctx, args_p["q"], args_p["k"], args_p["v"], G, window)[0] -
                       _clip_loss(oracle_mod, shape, ctx, args_m["q"], args_m["k"], args_m["v"], G, window)[0]) / (2 * eps)
        assert np.abs(fd - g).max() < 1e-7, (name, np.abs(fd - g).max())
        assert np.abs(g).max() > 1e-3                         # not trivially zero
    # the magnitudes bound the gradients they belong to (rotation pairs share one bound)
    assert (np.abs(dv) <= mv + 1e-12).all()
    pair = lambda a: np.repeat(np.abs(a).reshape(T * P, H, D // 2, 2).sum(axis=3), 2, axis=2).reshape(a.shape)
    assert (pair(dq) <= 2 * mq + 1e-12).all() and (pair(dk) <= 2 * mk + 1e-12).all()


def test_clip_backward_closed_forms(oracle_mod):
    """One visible key per query (one-token frames, no sink, window of one frame): o_i = v_i, so
    dv = d_out and dq = dk = 0.  And d_out = 0 gives zero gradients."""
    H, D = 2, 8
    orc = oracle_mod.Oracle(1, H, D, 1, 1, 0, 4)
    rng = np.random.default_rng(12)
    q, k, v, G = (rng.standard_normal((3, H, D)) for _ in range(4))
    orc.clip(0, q, k, v, 0, 3, 1, 1, 1)
    dq, dk, dv, *_ = orc.clip_backward(0, q, G, 0, 3, 1, 1, 1)
    assert np.abs(dv - G).max() < 1e-14 and np.abs(dq).max() < 1e-14 and np.abs(dk).max() < 1e-14
    dq, dk, dv, *_ = orc.clip_backward(0, q, 0 * G, 0, 3, 1, 1, 1)
    assert not dq.any() and not dk.any() and not dv.any()
