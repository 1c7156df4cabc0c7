"""Pins for the oracle's cache logic: the invariants the paper fixes
(refresh == normal calculation, one-step delay, Appendix A's printed index
example, the active-row counts behind O(L^3) vs O(L^2)), plus brute force for
the selection."""
import itertools
import os

import numpy as np
import pytest

from oracle import dkv_oracle as O
from tests.test_oracle_blocks import rng, small_model, small_weights

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def read_golden(name):
    out = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split("=")
        out[k.strip()] = [int(a) for a in v.split()]
    return out


# ------------------------------------------------------------ index plumbing

def test_concat_reorder_maps_printed_example():
    g = read_golden("concat_reorder_example.txt")
    L = g["seq_len"][0]
    un_prev, un_next = g["unmasked_prev"], g["unmasked_next"]
    m_prev = [i for i in range(L) if i not in un_prev]
    m_next = [i for i in range(L) if i not in un_next]
    order_prev, order_next, full_map, entries = O.concat_reorder_maps(un_prev, m_prev, un_next, m_next)
    assert order_prev == g["order_prev"]
    assert order_next == g["order_next"]
    assert full_map == g["map"]
    assert entries == g["cache_entries"]


def test_literal_cache_physical_order_follows_printed_example():
    """Run two Decode steps whose mask sets are those of the printed example
    and look at the physical order the literal cache holds."""
    g = read_golden("concat_reorder_example.txt")
    m = small_model()
    W = small_weights(m)
    L = 8
    x = rng(0).integers(0, 40, size=L)
    c = O.LiteralCache(m, W, L)
    c.step(x, np.arange(L))                                   # full step fills everything
    M_prev = [i for i in range(L) if i not in g["unmasked_prev"]]
    M_next = [i for i in range(L) if i not in g["unmasked_next"]]
    c.step(x, np.array(M_prev))                               # active = M_{t-1}
    assert c.order == g["order_prev"]
    c.step(x, np.array(M_next))
    assert c.order == g["order_next"]


# ---------------------------------------------------------------- policies

def test_refresh_schedule():
    dec = O.Policy(O.POLICY_DECODE, refresh_interval=8)
    assert [t for t in range(1, 26) if O.is_refresh_step(t, dec)] == [1, 9, 17, 25]
    assert all(O.is_refresh_step(t, O.Policy(O.POLICY_DECODE, 1)) for t in range(1, 10))
    assert [t for t in range(1, 20) if O.is_refresh_step(t, O.Policy(O.POLICY_PREFILL, 4))] == [1]
    assert [t for t in range(1, 20) if O.is_refresh_step(t, O.Policy(O.POLICY_DECODE, 0))] == [1]
    assert all(O.is_refresh_step(t, O.Policy(O.POLICY_NONE)) for t in range(1, 5))


def test_greedy_window_formula():
    # [c - ceil(w/2), c + floor(w/2)]: w=4 -> +-2 (5 rows); w=3 -> [-2,+1]
    assert O.greedy_window([10], 4, 100) == [8, 9, 10, 11, 12]
    assert O.greedy_window([10], 3, 100) == [8, 9, 10, 11]
    assert O.greedy_window([0], 4, 100) == [0, 1, 2]
    assert O.greedy_window([99], 4, 100) == [97, 98, 99]
    assert O.greedy_window([5, 7], 2, 100) == [4, 5, 6, 7, 8]


def simulate_counts(G, P, k, pol, order):
    """Active-row counts over a whole generation, masks driven by `order`."""
    L = P + G
    M = np.zeros(L, np.uint8)
    M[P:] = 1
    M_prev, D_prev, counts = None, None, []
    for t in range(1, G // k + 1):
        D = list(order[t - 1])
        counts.append(len(O.active_set(t, pol, L, P, M_prev, M, D, D_prev)))
        M_prev = M.copy()
        M[D] = 0
        D_prev = D
    return counts


@pytest.mark.parametrize("G,tot_vanilla,tot_decode,tot_greedy", [(256, 65536, 33151, 1786), (1024, 1048576, 525823, 7162)])
def test_active_row_totals_cubic_vs_quadratic(G, tot_vanilla, tot_decode, tot_greedy):
    """P=0, k=1, no refresh after step 1.  With O(L) attention work per active
    row, G^2 rows is the O(L^3) of the plain sampler and ~6G rows is O(L^2)."""
    order = rng(G).permutation(G).reshape(G, 1)
    assert sum(simulate_counts(G, 0, 1, O.Policy(O.POLICY_NONE), order)) == G * G == tot_vanilla
    c = simulate_counts(G, 0, 1, O.Policy(O.POLICY_DECODE, 0), order)
    assert c[0] == G and all(c[s] == G - s + 1 for s in range(1, G))      # #M_t + k
    assert sum(c) == G + sum(G - s + 1 for s in range(1, G)) == tot_decode
    # Greedy, window 4 around D_{t-1}; interior (no clipping) upper bound is 6 rows
    cg = simulate_counts(G, 0, 1, O.Policy(O.POLICY_GREEDY, 0, window=4), order)
    assert cg[0] == G and max(cg[1:]) <= 6
    assert G + 6 * (G - 1) == tot_greedy and sum(cg) <= tot_greedy


def test_active_counts_per_policy():
    G, P, k = 16, 8, 2
    order = rng(3).permutation(G).reshape(G // k, k) + P
    L = P + G
    c = simulate_counts(G, P, k, O.Policy(O.POLICY_DECODE, 4), order)
    for s, n in enumerate(c):
        assert n == (L if s % 4 == 0 else (G - s * k) + k)
    c = simulate_counts(G, P, k, O.Policy(O.POLICY_PD, 4), order)
    for s, n in enumerate(c):
        assert n == (L if s == 0 else G if s % 4 == 0 else (G - s * k) + k)
    c = simulate_counts(G, P, k, O.Policy(O.POLICY_PREFILL, 4), order)
    assert c == [L] + [G] * (G // k - 1)
    c = simulate_counts(G, P, k, O.Policy(O.POLICY_DECODE, 0, delay=0), order)
    assert c == [L] + [G - s * k for s in range(1, G // k)]
    c = simulate_counts(G, P, k, O.Policy(O.POLICY_GREEDY, 0, window=4), order)
    assert c[0] == L and all(n <= k * (4 + 2) for n in c[1:])


# --------------------------------------------------------------- selection

def test_select_unmask_brute_force():
    r = rng(5)
    for trial in range(30):
        L = 12
        conf = r.choice([0.1, 0.2, 0.3, 0.5], size=L)          # many ties
        masked = r.integers(0, 2, size=L).astype(np.uint8)
        lo, hi = 2, 11
        cands = [i for i in range(lo, hi) if masked[i]]
        for k in (1, 2, 3):
            if len(cands) < k:
                with pytest.raises(ValueError):
                    O.select_unmask(conf, masked, lo, hi, k)
                continue
            got = O.select_unmask(conf, masked, lo, hi, k)
            # brute force: the best k-subset under (higher conf, then lower position)
            best = min(itertools.combinations(cands, k), key=lambda s: sorted((-conf[i], i) for i in s))
            assert sorted(got) == sorted(best)
            assert all(masked[i] and lo <= i < hi for i in got) and len(set(got)) == k


def test_select_nan_counts_as_minus_inf():
    conf = np.array([np.nan, 0.1, 0.2])
    assert O.select_unmask(conf, np.ones(3, np.uint8), 0, 3, 2) == [2, 1]


# ------------------------------------------------------ generation invariants

def run(pol, form="literal", G=8, P=5, k=1, block=None, order=None, seed=0, keep_logits=True, n_steps=None):
    m = small_model()
    W = small_weights(m, seed)
    prompt = rng(20 + seed).integers(0, 40, size=P)
    return m, W, O.generate_one(m, W, prompt, G, k, pol, block, order, form, keep_logits=keep_logits, n_steps=n_steps)


def vanilla_logits(m, W, st):
    return O.vanilla_forward(m, W, st.x_in)[st.head_rows]


def test_policy_none_and_interval_one_equal_vanilla_every_step():
    greedy_order = (rng(9).permutation(8) + 5).reshape(8, 1)
    for pol, order in ((O.Policy(O.POLICY_NONE), None), (O.Policy(O.POLICY_DECODE, 1), None),
                       (O.Policy(O.POLICY_GREEDY, 1, window=2), greedy_order)):
        m, W, tr = run(pol, order=order)
        for st in tr:
            assert len(st.active) == len(st.x_in)
            np.testing.assert_allclose(st.logits, vanilla_logits(m, W, st), atol=1e-11)
    # and the two generate identical tokens
    a = O.final_tokens(run(O.Policy(O.POLICY_NONE))[2])
    b = O.final_tokens(run(O.Policy(O.POLICY_DECODE, 1))[2])
    np.testing.assert_array_equal(a, b)


@pytest.mark.parametrize("kind", [O.POLICY_DECODE, O.POLICY_PREFILL, O.POLICY_PD, O.POLICY_GREEDY])
def test_step_one_equals_vanilla_for_every_policy(kind):
    order = (rng(1).permutation(8) + 5).reshape(8, 1)
    m, W, tr = run(O.Policy(kind, 4, window=4), order=order if kind == O.POLICY_GREEDY else None, n_steps=1)
    np.testing.assert_allclose(tr[0].logits, vanilla_logits(m, W, tr[0]), atol=1e-11)


def test_cached_steps_differ_from_vanilla_but_refresh_steps_match():
    m, W, tr = run(O.Policy(O.POLICY_DECODE, 4))
    for st in tr:
        diff = np.abs(st.logits - vanilla_logits(m, W, st)).max()
        if (st.t - 1) % 4 == 0:
            assert diff < 1e-11
        elif st.t > 2:
            # stale K/V of decoded rows: an approximation, not the vanilla result
            assert diff > 1e-9


def test_fresh_cache_exactness():
    """Fill all slots by a full step on x, then run a cached step on the same
    x with an arbitrary active subset: those rows equal the vanilla rows."""
    m = small_model()
    W = small_weights(m, 2)
    L = 12
    x = rng(30).integers(0, 40, size=L)
    ref = O.vanilla_forward(m, W, x)
    for cls in (O.LiteralCache, O.SlotCache):
        c = cls(m, W, L)
        c.step(x, np.arange(L))
        A = np.array([1, 4, 5, 9, 11])
        out = c.step(x, A).dense()
        np.testing.assert_allclose(out[A], ref[A], atol=1e-11)
        assert np.isnan(out[[0, 2, 3]]).all()
        only = c.step(x, A, logit_rows=[4, 11])             # the head is row-wise
        np.testing.assert_allclose(only[np.array([4, 11])], ref[[4, 11]], atol=1e-11)
        assert np.isnan(only[5]).all()


@pytest.mark.parametrize("pol,order_needed", [
    (O.Policy(O.POLICY_DECODE, 3), False), (O.Policy(O.POLICY_PD, 3), False), (O.Policy(O.POLICY_PREFILL), False),
    (O.Policy(O.POLICY_DECODE, 0, delay=0), False), (O.Policy(O.POLICY_GREEDY, 4, window=4), True),
    (O.Policy(O.POLICY_GREEDY, 0, window=2, window_center=O.CENTER_CUR), True)])
def test_literal_algorithm_equals_slot_form(pol, order_needed):
    order = (rng(2).permutation(8) + 5).reshape(4, 2) if order_needed else None
    _, _, a = run(pol, "literal", k=2, order=order)
    _, _, b = run(pol, "slots", k=2, order=order)
    for sa, sb in zip(a, b):
        np.testing.assert_array_equal(sa.active, sb.active)
        np.testing.assert_array_equal(sa.written_step, sb.written_step)
        assert sa.chosen == sb.chosen
        np.testing.assert_array_equal(sa.pred, sb.pred)
        np.testing.assert_allclose(sa.logits, sb.logits, atol=1e-11)


def unmask_step(trace, L):
    u = np.zeros(L, dtype=np.int64)      # 0 = prompt
    for st in trace:
        for p in st.chosen:
            u[p] = st.t
    return u


def test_decode_provenance_one_step_delay():
    """A token unmasked at step s is recomputed with its decoded input at step
    s+1; that K/V is what later steps reuse, until the next refresh."""
    N, P, G = 5, 5, 12
    _, _, tr = run(O.Policy(O.POLICY_DECODE, N), G=G, P=P, keep_logits=False)
    u = unmask_step(tr, P + G)
    for st in tr:
        last_refresh = ((st.t - 1) // N) * N + 1
        for p in range(P + G):
            if st.masked_in[p] or p in st.chosen:
                expect = st.t                                # still active
            elif u[p] > 0 and u[p] + 1 <= st.t and u[p] + 1 > last_refresh:
                expect = u[p] + 1
            else:
                expect = last_refresh
            if st.masked_in[p]:
                assert st.written_step[p] == st.t
            elif p in st.chosen:
                assert st.written_step[p] == st.t
            else:
                assert st.written_step[p] == max(expect, last_refresh), (st.t, p)


def test_delay_zero_caches_at_the_unmask_step():
    P, G = 5, 8
    _, _, tr = run(O.Policy(O.POLICY_DECODE, 0, delay=0), G=G, P=P, keep_logits=False)
    u = unmask_step(tr, P + G)
    last = tr[-1]
    for p in range(P, P + G):
        if u[p] < last.t:
            assert last.written_step[p] == max(u[p], 1)


def test_prompt_rows_written_once_under_prefill_and_pd():
    for pol in (O.Policy(O.POLICY_PREFILL), O.Policy(O.POLICY_PD, 3)):
        _, _, tr = run(pol, keep_logits=False)
        for st in tr:
            assert (st.written_step[:5] == 1).all()
        if pol.kind == O.POLICY_PD:
            assert len(tr[3].active) == 8 and tr[3].refresh       # step 4: generation rows only


def test_generation_terminates_with_all_unmasked_and_block_order():
    P, G, k, block = 5, 8, 2, 4
    _, _, tr = run(O.Policy(O.POLICY_DECODE, 3), G=G, P=P, k=k, block=block, keep_logits=False)
    assert len(tr) == G // k
    seen = []
    for st in tr:
        blk = (st.t - 1) // (block // k)
        assert st.cand == (P + blk * block, P + (blk + 1) * block)
        assert len(st.chosen) == k and all(st.masked_in[p] and st.cand[0] <= p < st.cand[1] for p in st.chosen)
        # rows of later blocks stay active although they are not candidates
        if (st.t - 1) % 3:
            assert set(np.nonzero(st.masked_in)[0]) <= set(st.active)
        seen += st.chosen
    assert sorted(seen) == list(range(P, P + G))
    x = O.final_tokens(tr)
    assert (x != 49).all() and (x[:P] == tr[0].x_in[:P]).all()


def test_cache_ratio():
    _, _, tr = run(O.Policy(O.POLICY_NONE), keep_logits=False)
    assert O.cache_ratio(tr) == 0.0
    P, G = 5, 8
    _, _, tr = run(O.Policy(O.POLICY_DECODE, 0), G=G, P=P, keep_logits=False)
    L = P + G
    expect = np.mean([0.0] + [(L - ((G - s) + 1)) / L for s in range(1, G)])
    assert abs(O.cache_ratio(tr) - expect) < 1e-15


def test_cache_ratio_counts_prefill_rows_as_computed():
    """PD with a prompt-only prefill pass, P = 5, G = 8 (L = 13), one token per step, a refresh every
    4 steps.  Rows COMPUTED per step, written out by hand: step 1 computes the 5 prompt rows in the
    prefill pass and the 8 generation rows in its own pass (13 of 13: nothing is served from the
    cache); steps 2-4 compute the masked rows of the step before (8, 7, 6); step 5 (s = 4) is a
    refresh of the generation rows (8); steps 6-8 compute 4, 3, 2.  The prompt rows are cache-served
    in every step but the first.  Cache ratio = mean over steps of (13 - computed) / 13."""
    _, _, tr = run(O.Policy(O.POLICY_PD, 4, isolated_prefill=True), G=8, P=5, keep_logits=False)
    computed = [13, 8, 7, 6, 8, 4, 3, 2]
    assert [len(s.active) + s.prefilled for s in tr] == computed
    assert abs(O.cache_ratio(tr) - (0 + 5 + 6 + 7 + 5 + 9 + 10 + 11) / (8 * 13)) < 1e-15
    # the same policy without the separate pass computes the same 13 rows at step 1 in one pass
    _, _, tr2 = run(O.Policy(O.POLICY_PD, 4), G=8, P=5, keep_logits=False)
    assert [len(s.active) for s in tr2] == computed and O.cache_ratio(tr2) == O.cache_ratio(tr)


def test_greedy_uses_given_order_and_bounded_rows():
    order = (rng(4).permutation(8) + 5).reshape(8, 1)
    _, _, tr = run(O.Policy(O.POLICY_GREEDY, 0, window=4), order=order, keep_logits=False)
    for st in tr:
        assert st.chosen == [int(order[st.t - 1, 0])]
        if st.t > 1:
            assert len(st.active) <= 6
            assert st.chosen[0] in st.active and int(order[st.t - 2, 0]) in st.active


def test_bf16_rounding_emulation_stays_close_to_exact():
    m = small_model()
    W = small_weights(m, 3)
    x = rng(31).integers(0, 40, size=10)
    a = O.vanilla_forward(m, W, x)
    b = O.vanilla_forward(m, W, x, rnd=O.round_bf16)
    err = np.abs(a - b).max() / a.std()
    assert 1e-5 < err < 5e-2


# ------------------------------------------------- shifted outputs (Appendix B, Un-Shift)

def test_shifted_head_reads_the_previous_row_and_keeps_the_cache_rule():
    """shift=1: confidence and token of position j come from the logits of row
    j-1; with no cache (every row computed) those are the vanilla logits of
    row j-1.  The K/V caching rule itself is unchanged."""
    m = small_model()
    W = small_weights(m, 4)
    prompt = rng(40).integers(0, 40, size=5)
    tr = O.generate_one(m, W, prompt, 8, 1, O.Policy(O.POLICY_NONE, shift=1), keep_logits=True)
    for st in tr:
        ref = O.vanilla_forward(m, W, st.x_in)
        np.testing.assert_allclose(st.logits, ref[st.head_rows - 1], atol=1e-11)
        for j in st.head_rows:
            c, p = O.confidence(ref[j - 1], m.mask_id)
            assert st.pred[j] == p and abs(st.conf[j] - c) < 1e-12
    # Decode with shift: the active set is M_{t-1} plus the rows left of the candidates
    pol = O.Policy(O.POLICY_DECODE, 4, shift=1)
    tr = O.generate_one(m, W, prompt, 8, 1, pol, keep_logits=True)
    prev_mask = None
    for st in tr:
        if (st.t - 1) % 4 and prev_mask is not None:
            expect = set(np.nonzero(prev_mask)[0]) | {int(j) - 1 for j in st.head_rows}
            assert set(st.active.tolist()) == expect
        prev_mask = st.masked_in
    # literal and slot forms agree with the shift as well
    tr2 = O.generate_one(m, W, prompt, 8, 1, pol, form="slots", keep_logits=True)
    for a, b in zip(tr, tr2):
        np.testing.assert_array_equal(a.active, b.active)
        assert a.chosen == b.chosen
        np.testing.assert_allclose(a.logits, b.logits, atol=1e-11)


def test_un_and_right_shift_caches_a_row_only_when_input_and_prediction_are_decoded():
    """shift=2 (Appendix B, third variant): a row is served from the cache at
    step t only if, in the mask set the policy looks at (M_{t-1}), both its own
    token and the token to its right are decoded; everything else is computed.
    Checked from the trace alone, not through the oracle's own set arithmetic."""
    m = small_model()
    W = small_weights(m, 5)
    prompt = rng(41).integers(0, 40, size=5)
    L = 5 + 8
    pol = O.Policy(O.POLICY_DECODE, 4, shift=2)
    tr = O.generate_one(m, W, prompt, 8, 1, pol, keep_logits=True)
    prev_mask = None
    for st in tr:
        if (st.t - 1) % 4 == 0:
            assert len(st.active) == L                      # refresh and first step: everything
        else:
            act = set(st.active.tolist())
            for j in range(L):
                own_decoded = not prev_mask[j]
                right_decoded = j + 1 >= L or not prev_mask[j + 1]
                assert (j not in act) == (own_decoded and right_decoded), (st.t, j)
        # the rows that serve the candidates are computed, and their logits are the vanilla ones on a full step
        assert set((st.head_rows - 1).tolist()) <= set(st.active.tolist())
        if len(st.active) == L:
            ref = O.vanilla_forward(m, W, st.x_in)
            np.testing.assert_allclose(st.logits, ref[st.head_rows - 1], atol=1e-11)
        prev_mask = st.masked_in
    # it recomputes a superset of Un-Shift's rows, and both forms of the cache agree
    tr1 = O.generate_one(m, W, prompt, 8, 1, O.Policy(O.POLICY_DECODE, 4, shift=1), order=np.array([s.chosen for s in tr]))
    tr2 = O.generate_one(m, W, prompt, 8, 1, pol, order=np.array([s.chosen for s in tr]), form="slots", keep_logits=True)
    for a, b, c in zip(tr, tr1, tr2):
        assert set(b.active.tolist()) <= set(a.active.tolist())
        np.testing.assert_array_equal(a.active, c.active)
        np.testing.assert_allclose(a.logits, c.logits, atol=1e-11)
    # Prefill scope: the last prompt row predicts the first generated token, so it joins the generation rows
    trp = O.generate_one(m, W, prompt, 8, 1, O.Policy(O.POLICY_PREFILL, shift=2))
    assert trp[3].active.tolist() == list(range(4, L))


# ------------------------------------------------- isolated prompt-only prefill (Sec. 3.3, Prefill / PD)

def _block_masked_forward(m, W, x, P):
    """One pass over all rows with an attention mask written out by hand:
    prompt queries see the prompt keys only, generation queries see every key."""
    fw = O._Forward(m, W)
    L = len(x)
    h = fw.embed(x)
    g = m.n_q_heads // m.n_kv_heads
    for l in range(m.n_layers):
        q, k, v = fw.qkv(l, h, np.arange(L))
        a = np.zeros((L, m.n_q_heads, m.head_dim))
        for i in range(L):
            n_keys = P if i < P else L
            for hq in range(m.n_q_heads):
                s = np.array([q[i, hq] @ k[j, hq // g] for j in range(n_keys)]) / np.sqrt(m.head_dim)
                w = np.exp(s - s.max())
                w /= w.sum()
                a[i, hq] = sum(w[j] * v[j, hq // g] for j in range(n_keys))
        h = fw.after_attention(l, h, a)
    return fw.logits(h)


@pytest.mark.parametrize("form", ["literal", "slots"])
def test_isolated_prefill_equals_a_block_masked_forward(form):
    m = small_model()
    W = small_weights(m, 6)
    P, G = 6, 7
    prompt = rng(50).integers(0, 40, size=P)
    pol = O.Policy(O.POLICY_PD, 3, isolated_prefill=True)
    tr = O.generate_one(m, W, prompt, G, 1, pol, form=form, keep_logits=True)
    st = tr[0]
    assert st.active.tolist() == list(range(P, P + G)) and (st.written_step == 1).all()
    ref = _block_masked_forward(m, W, st.x_in, P)
    np.testing.assert_allclose(st.logits, ref[st.head_rows], atol=1e-10)
    # and it differs from the joint first step, where the prompt rows see the masked tail
    joint = O.generate_one(m, W, prompt, G, 1, O.Policy(O.POLICY_PD, 3), form=form, keep_logits=True)[0]
    assert np.abs(joint.logits - st.logits).max() > 1e-6
    # later steps never touch the prompt rows
    for s in tr[1:]:
        assert s.active.min() >= P and (s.written_step[:P] == 1).all()


def test_isolated_prefill_kv_do_not_depend_on_the_generation_part():
    m = small_model()
    W = small_weights(m, 6)
    prompt = rng(51).integers(0, 40, size=5)
    pol = O.Policy(O.POLICY_PREFILL, isolated_prefill=True)
    a = O.Sampler(m, W, prompt, 4, 1, pol, form="slots")
    b = O.Sampler(m, W, prompt, 9, 3, pol, form="slots")
    a.step(), b.step()
    np.testing.assert_array_equal(a.cache.K[:, :5], b.cache.K[:, :5])
    np.testing.assert_array_equal(a.cache.V[:, :5], b.cache.V[:, :5])
