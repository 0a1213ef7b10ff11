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
    for g in range(plan.n_groups):
        for wave in range(plan.wave_cols[g] // G):
            out.append((g, wave * G + cta, 0, plan.n_kt[g]))
    S = plan.share_ctas
    u = plan.shared_steps * min(cta, S) // S
    end = plan.shared_steps * min(cta + 1, S) // S
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


def owner_of_shared_step(plan, u):
    return ((u + 1) * plan.share_ctas - 1) // plan.shared_steps


def check_plan(plan):
    if plan.n_groups == 0:
        return
    G = plan.n_ctas
    assert 1 <= G <= 160
    done = {}
    loads = []
    for cta in range(G):
        work = cta_work(plan, cta)
        loads.append(sum(k1 - k0 for _, _, k0, k1 in work))
        for g, col, k0, k1 in work:
            assert 0 <= col < plan.heads * plan.tiles[g] and 0 <= k0 < k1 <= plan.n_kt[g]
            for k in range(k0, k1):
                assert (g, col, k) not in done, "step done twice"
                done[(g, col, k)] = cta
    total = sum(plan.heads * plan.tiles[g] * plan.n_kt[g] for g in range(plan.n_groups))
    assert len(done) == total, "steps left undone"
    assert max(loads) - min(loads) <= 1, "every CTA gets the same whole columns and shares differ by one step at most"
    # a split column: its parts belong to consecutive CTAs, which the kernel finds from the column's
    # first and last shared step
    for g in range(plan.n_groups):
        for col in range(plan.wave_cols[g], plan.heads * plan.tiles[g]):
            owners = [done[(g, col, k)] for k in range(plan.n_kt[g])]
            assert owners == sorted(owners)
            first = plan.step_begin[g] + (col - plan.wave_cols[g]) * plan.n_kt[g]
            i0, i1 = owner_of_shared_step(plan, first), owner_of_shared_step(plan, first + plan.n_kt[g] - 1)
            assert (i0, i1) == (owners[0], owners[-1])
            assert sorted(set(owners)) == list(range(i0, i1 + 1))


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
    check_plan(plan)
    plan = B.ll_debug_attn_plan(h, recache=True, sm_count=148)
    assert plan.n_groups == 3 and [plan.n_kt[g] for g in range(3)] == [74, 111, 147]     # the ring has wrapped: two runs, each with a ragged tile
    check_plan(plan)
    B.ll_cache_destroy(h)


@settings(max_examples=40, deadline=None)
@given(heads=st.integers(1, 12), P=st.integers(1, 700), C=st.integers(1, 3), s_chunks=st.integers(0, 2),
       w_chunks=st.integers(1, 4), n_chunks=st.integers(1, 12), sms=st.sampled_from([1, 7, 148, 160]),
       recache=st.booleans())
# fewer shared steps (3) than CTAs (7): the CTAs that take one must still be consecutive
@example(heads=11, P=86, C=3, s_chunks=0, w_chunks=1, n_chunks=1, sms=7, recache=False)
def test_every_step_is_done_exactly_once(heads, P, C, s_chunks, w_chunks, n_chunks, sms, recache):
    h = make_cache(heads, P, C, s_chunks * C, w_chunks * C, n_chunks)
    plan = B.ll_debug_attn_plan(h, recache=recache, sm_count=sms)
    check_plan(plan)
    B.ll_cache_destroy(h)
