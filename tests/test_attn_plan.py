"""CPU-only: the work division of the attention kernel.

The library reports, per query group, how many columns go out whole and how the
steps of the rest are cut into shares (``ll_debug_attn_plan``).  Here the rule a
CTA follows to find its work is written out again in Python and checked for what
must hold whatever the shape: every step of every column is done exactly once,
a column split over several CTAs is split into contiguous parts whose owners
can be found from the first step alone, and no CTA does more than one step more
than another."""
import pytest
from hypothesis import example, given, settings, strategies as st

from paper_2509_22622_b200 import binding as B


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2509_22622_b200 import build
    build.build()


def cta_work(plan, cta):
    """(group, column, first step, one past last step) in the order the CTA takes them."""
    out = []
    G = plan.n_ctas
    g = 0
    for wave in range(plan.n_waves):
        col = wave * G + cta                                  # launch-wide column number
        if col >= plan.all_cols:                              # a partial last wave
            continue
        while col >= plan.col_begin[g] + plan.heads * plan.tiles[g]:
            g += 1
        out.append((g, col - plan.col_begin[g], 0, plan.n_kt[g]))
    k = plan.share_of_cta[cta]
    u, end = (plan.share_begin[k], plan.share_begin[k + 1]) if k >= 0 else (0, 0)
    while u < end:
        # the group whose shared steps hold u
        g = 0
        while g + 1 < plan.n_groups and u >= plan.step_begin[g + 1]:
            g += 1
        off = u - plan.step_begin[g]
        col, kt0 = divmod(off, plan.n_kt[g])
        kt1 = min(plan.n_kt[g], kt0 + (end - u))
        out.append((g, plan.wave_cols[g] + col, kt0, kt1))
        u += kt1 - kt0
    return out


def shares_of_column(plan, own, first, n_kt):
    """What a CTA holding share `own` with a part of the column whose shared steps are
    [first, first + n_kt) takes for the column's first and last share."""
    i0 = i1 = own
    while plan.share_begin[i0] > first:
        i0 -= 1
    while plan.share_begin[i1 + 1] < first + n_kt:
        i1 += 1
    return i0, i1


def check_plan(plan):
    if plan.n_groups == 0:
        return
    G = plan.n_ctas
    assert 1 <= G <= 160
    # shares: rising, non-empty, handed to CTAs in rising order, covering the shared steps
    sb = list(plan.share_begin[:plan.n_shares + 1])
    assert sb[0] == 0 and sb[-1] == plan.shared_steps and all(a < b for a, b in zip(sb, sb[1:]))
    assert [k for k in plan.share_of_cta[:G] if k >= 0] == list(range(plan.n_shares))
    done = {}
    loads, whole = [], []
    for cta in range(G):
        work = cta_work(plan, cta)
        loads.append(sum(k1 - k0 for _, _, k0, k1 in work))
        whole.append(sum(k1 - k0 for g, col, k0, k1 in work if col < plan.wave_cols[g]))
        for g, col, k0, k1 in work:
            assert 0 <= col < plan.heads * plan.tiles[g] and 0 <= k0 < k1 <= plan.n_kt[g]
            for k in range(k0, k1):
                assert (g, col, k) not in done, "step done twice"
                done[(g, col, k)] = cta
    total = sum(plan.heads * plan.tiles[g] * plan.n_kt[g] for g in range(plan.n_groups))
    assert len(done) == total, "steps left undone"
    # the shares level the CTAs: those that take one end within a step of each other, and a CTA
    # that takes none was at that level already
    assert plan.all_cols == sum(plan.heads * plan.tiles[g] for g in range(plan.n_groups))
    if plan.n_shares == 0:
        # short columns: everything goes out whole, the last wave possibly partial.  Two CTAs can
        # differ by what the columns of one wave differ, summed over the waves.
        def kt_of(col):
            g = max(g for g in range(plan.n_groups) if plan.col_begin[g] <= col)
            return plan.n_kt[g]
        spread = 0
        for wave in range(plan.n_waves):
            kts = [kt_of(c) for c in range(wave * G, min((wave + 1) * G, plan.all_cols))]
            spread += max(kts) - (min(kts) if len(kts) == G else 0)
        assert plan.shared_steps == 0 and plan.n_waves * G >= plan.all_cols > (plan.n_waves - 1) * G
        assert max(loads) - min(loads) <= spread
        return
    level = max((loads[i] for i in range(G) if plan.share_of_cta[i] >= 0), default=min(loads))
    for i in range(G):
        if plan.share_of_cta[i] >= 0:
            assert level - 1 <= loads[i] <= level
        else:
            assert loads[i] == whole[i] >= level - 1
    # a split column: its parts sit in consecutive shares, which every part's CTA finds from the
    # column's first and last shared step
    share_of = {cta: plan.share_of_cta[cta] for cta in range(G)}
    for g in range(plan.n_groups):
        for col in range(plan.wave_cols[g], plan.heads * plan.tiles[g]):
            owners = [share_of[done[(g, col, k)]] for k in range(plan.n_kt[g])]
            assert owners == sorted(owners) and sorted(set(owners)) == list(range(owners[0], owners[-1] + 1))
            first = plan.step_begin[g] + (col - plan.wave_cols[g]) * plan.n_kt[g]
            for own in set(owners):
                assert shares_of_column(plan, own, first, plan.n_kt[g]) == (owners[0], owners[-1])


def make_cache(heads, P, C, S, W, n_chunks):
    h = B.ll_cache_create(1, heads, 128, P, C, S, W)
    B.ll_cache_set_dry_run(h, True)
    gh = 1
    for chunk in range(n_chunks):
        B.ll_rope_append_kv(h, 0, None, None, None, chunk * C, C, gh, P // gh)
    return h


def test_plan_of_the_benchmark_layer():
    h = make_cache(12, 1560, 3, 3, 9, 6)
    plan = B.ll_debug_attn_plan(h, sm_count=148)
    assert (plan.n_ctas, plan.n_groups, plan.tiles[0], plan.n_kt[0]) == (148, 1, 19, 147)
    assert plan.wave_cols[0] == 148 and plan.shared_steps == 80 * 147      # 228 columns: 148 whole, 80 shared
    assert plan.n_waves == 1 and plan.n_shares == 148
    check_plan(plan)
    plan = B.ll_debug_attn_plan(h, recache=True, sm_count=148)
    assert plan.n_groups == 3 and [plan.n_kt[g] for g in range(3)] == [74, 111, 147]     # the ring has wrapped: two runs, each with a ragged tile
    # 684 columns: four waves across the group boundaries, the last 92 columns (of group 2) shared
    assert plan.n_waves == 4 and [plan.wave_cols[g] for g in range(3)] == [228, 228, 136]
    assert plan.shared_steps == 92 * 147
    check_plan(plan)
    B.ll_cache_destroy(h)


@settings(max_examples=150, deadline=None, derandomize=True)
@given(heads=st.integers(1, 12), P=st.integers(1, 700), C=st.integers(1, 3), s_chunks=st.integers(0, 2),
       w_chunks=st.integers(1, 4), n_chunks=st.integers(1, 12), sms=st.sampled_from([1, 7, 148, 160]),
       recache=st.booleans())
# fewer shared steps (3) than CTAs (7): only some CTAs take a share
@example(heads=11, P=86, C=3, s_chunks=0, w_chunks=1, n_chunks=1, sms=7, recache=False)
def test_every_step_is_done_exactly_once(heads, P, C, s_chunks, w_chunks, n_chunks, sms, recache):
    h = make_cache(heads, P, C, s_chunks * C, w_chunks * C, n_chunks)
    plan = B.ll_debug_attn_plan(h, recache=recache, sm_count=sms)
    check_plan(plan)
    B.ll_cache_destroy(h)


@settings(max_examples=150, deadline=None, derandomize=True)
@given(heads=st.integers(1, 12), D=st.sampled_from([64, 128]), sms=st.sampled_from([7, 148, 160]),
       streams=st.lists(st.tuples(st.integers(1, 700), st.integers(1, 3), st.integers(0, 2), st.integers(1, 4),
                                  st.integers(1, 12)), min_size=1, max_size=8))
def test_every_step_of_a_launch_over_several_streams_is_done_exactly_once(heads, D, sms, streams):
    """Streams that differ in frame size, chunk length, sink, window and position share a launch."""
    handles = []
    for P, C, s_chunks, w_chunks, n_chunks in streams:
        h = B.ll_cache_create(1, heads, D, P, C, s_chunks * C, w_chunks * C)
        B.ll_cache_set_dry_run(h, True)
        for chunk in range(n_chunks):
            B.ll_rope_append_kv(h, 0, None, None, None, chunk * C, C, 1, P)
        handles.append(h)
    plan = B.ll_debug_attn_plan_batched([(h, 0) for h in handles], sm_count=sms)
    assert plan.n_groups == len(streams) and plan.heads == heads
    check_plan(plan)
    for h in handles:
        B.ll_cache_destroy(h)


def test_plan_of_eight_ragged_streams():
    """The benchmark layer's shape at stream positions 0, 1, 2, 3, 6, 13, 29, 50: 1824 columns go out as
    twelve whole waves and 48 shared columns; the waves that straddle two streams give CTAs
    different loads, which the shares level out."""
    handles = [make_cache(12, 1560, 3, 3, 9, pos + 1) for pos in (0, 1, 2, 3, 6, 13, 29, 50)]
    plan = B.ll_debug_attn_plan_batched([(h, 0) for h in handles], sm_count=148)
    assert [plan.n_kt[g] for g in range(8)] == [37, 74, 110, 147, 147, 147, 147, 147]
    assert plan.n_waves == 12 and plan.shared_steps == 48 * 147
    check_plan(plan)
    for h in handles:
        B.ll_cache_destroy(h)


def test_short_columns_are_not_split():
    """A prompt-sized key set (4 key tiles per column): 228 columns go out as one full and one
    partial wave and nothing passes through the merge scratch."""
    h = B.ll_cache_create(1, 12, 128, 1560, 3, 3, 3)
    B.ll_cache_set_dry_run(h, True)
    B.ll_rope_append_kv(h, 0, None, None, None, 0, 3, 1, 1560)
    plan = B.ll_debug_attn_plan(h, sm_count=148)           # chunk 0 sees itself: 37 tiles per column, split
    assert plan.n_waves == 1 and plan.n_shares == 148
    small = B.ll_cache_create(1, 12, 128, 130, 3, 3, 3)     # 390 rows: 2 tiles x 12 heads = 24 columns of 4 key tiles
    B.ll_cache_set_dry_run(small, True)
    B.ll_rope_append_kv(small, 0, None, None, None, 0, 3, 1, 130)
    plan = B.ll_debug_attn_plan(small, sm_count=148)
    assert (plan.n_ctas, plan.n_waves, plan.n_shares, plan.shared_steps) == (24, 1, 0, 0)
    check_plan(plan)
    plan = B.ll_debug_attn_plan(small, sm_count=7)          # 24 columns on 7 CTAs: 3 full waves + 3 columns
    assert (plan.n_ctas, plan.n_waves, plan.n_shares) == (7, 4, 0)
    check_plan(plan)
    B.ll_cache_destroy(h)
    B.ll_cache_destroy(small)
