"""Pins of the oracle's growth step of the draft token graph: top-k children, probability
pruning and sibling pruning (Sec. 4.2), tau-redundant nodes and their merge edges (Sec. 5.2,
Sec. 5.3: after merging no n-gram longer than tau repeats)."""
import numpy as np

import oracle


def fresh(B, Ncap, root_token=5):
    tokens = np.full((B, Ncap), -1, np.int32); tokens[:, 0] = root_token
    parent = np.full((B, Ncap), -1, np.int32)
    merge = np.full((B, Ncap), -1, np.int32)
    leaf = np.zeros((B, Ncap), np.uint8)
    prob = np.zeros((B, Ncap), np.float32); prob[:, 0] = 1.0
    n = np.ones((B,), np.int32)
    return [tokens, parent, merge, leaf, prob, n]


def forcing_logits(rows, V):
    """one logits row per entry of `rows`: the listed tokens get descending logits above the rest"""
    lg = np.full((1, len(rows), V), -20.0, np.float32)
    for r, toks in enumerate(rows):
        for i, t in enumerate(toks):
            lg[0, r, t] = 5.0 - i
    return lg


def grow(state, lg, frontier, k, tau, tp=0.0, ts=0.0):
    B, F, V = lg.shape
    fr = np.full((B, F), -1, np.int32)
    fl = np.zeros((B,), np.int32)
    for b, f in enumerate(frontier):
        fr[b, :len(f)] = f; fl[b] = len(f)
    out = oracle.draft_expand(lg, fr, fl, *state, k=k, tau=tau, theta_prob=tp, theta_sib=ts)
    return list(out[:6]), out[6], out[7], out[8]


def test_top_k_probabilities_and_both_prunings():
    P = np.array([.04, .4, .15, .25, .06, .1])
    lg = np.log(P)[None, None, :].astype(np.float32)
    st, nf, nfl, full = grow(fresh(1, 16), lg, [[0]], k=3, tau=4, tp=0.2, ts=0.0)
    tok, par, mrg, leaf, prob, n = st
    assert n[0] == 4 and list(tok[0, 1:4]) == [1, 3, 2] and list(par[0, 1:4]) == [0, 0, 0]
    assert np.allclose(prob[0, 1:4], [.4, .25, .15], atol=1e-6)
    assert list(leaf[0, 1:4]) == [0, 0, 1]                 # .15 < .2
    assert list(nf[0, :nfl[0]]) == [1, 2] and not full
    # sibling pruning against the best sibling: .5 * .4 = .2 prunes .15 only; .7 * .4 = .28 prunes .25 too
    assert list(grow(fresh(1, 16), lg, [[0]], 3, 4, 0.0, 0.5)[0][3][0, 1:4]) == [0, 0, 1]
    assert list(grow(fresh(1, 16), lg, [[0]], 3, 4, 0.0, 0.7)[0][3][0, 1:4]) == [0, 1, 1]


def test_ties_go_to_the_lowest_token_and_comparisons_are_strict():
    lg = np.zeros((1, 1, 4), np.float32)                    # four tokens at exactly 1/4
    st, nf, nfl, _ = grow(fresh(1, 8), lg, [[0]], k=3, tau=4, tp=0.25, ts=1.0)
    assert list(st[0][0, 1:4]) == [0, 1, 2]
    assert list(st[3][0, 1:4]) == [0, 0, 0]                 # q < theta is false at equality, for both rules
    st, _, _, _ = grow(fresh(1, 8), lg, [[0]], k=3, tau=4, tp=np.nextafter(0.25, 1.0), ts=0.0)
    assert list(st[3][0, 1:4]) == [1, 1, 1]


def test_order_matches_a_stable_library_sort():
    rng = np.random.default_rng(4)
    V, k = 50, 7
    lg = np.round(rng.normal(size=(1, 3, V)), 1).astype(np.float32)      # rounded: plenty of exact ties
    st, _, _, _ = grow(fresh(1, 64), lg, [[0, 0, 0]], k=k, tau=50)
    for r in range(3):
        want = np.argsort(-lg[0, r].astype(np.float64), kind="stable")[:k]
        assert list(st[0][0, 1 + r * k: 1 + (r + 1) * k]) == list(want)
        p = np.exp(lg[0, r].astype(np.float64)); p /= p.sum()
        assert np.allclose(st[4][0, 1 + r * k: 1 + (r + 1) * k], p[want], rtol=1e-6)


def test_worked_redundancy_example():
    V = 12
    # level 1: root (token 5) -> tokens 1, 2;  level 2: node 1 -> 3, 4; node 2 -> 3, 7
    for tau, want_merge in ((1, {5: 3}), (2, {}), (3, {})):
        st = fresh(1, 32)
        st, nf, nfl, _ = grow(st, forcing_logits([[1, 2]], V), [[0]], k=2, tau=tau)
        assert list(nf[0, :nfl[0]]) == [1, 2]
        st, nf, nfl, _ = grow(st, forcing_logits([[3, 4], [3, 7]], V), [[1, 2]], k=2, tau=tau)
        tok, par, mrg, leaf, prob, n = st
        assert list(tok[0, :7]) == [5, 1, 2, 3, 4, 3, 7] and list(par[0, :7]) == [-1, 0, 0, 1, 1, 2, 2]
        got = {c: int(mrg[0, c]) for c in range(7) if mrg[0, c] >= 0}
        assert got == want_merge
        assert [c for c in range(7) if leaf[0, c]] == sorted(want_merge)
        assert list(nf[0, :nfl[0]]) == [c for c in (3, 4, 5, 6) if c not in want_merge]
    # level 3 with tau = 2: node 3 (token 3) -> 8, 9; node 5 (token 3) -> 8, 6: (3, 8) re-occurs
    for tau, want in ((2, {9: 7}), (3, {})):
        st = fresh(1, 32)
        st, _, _, _ = grow(st, forcing_logits([[1, 2]], V), [[0]], 2, tau)
        st, _, _, _ = grow(st, forcing_logits([[3, 4], [3, 7]], V), [[1, 2]], 2, tau)
        st, nf, nfl, _ = grow(st, forcing_logits([[8, 9], [8, 6]], V), [[3, 5]], 2, tau)
        mrg = st[2]
        assert {c: int(mrg[0, c]) for c in range(11) if mrg[0, c] >= 0} == want
        assert list(nf[0, :nfl[0]]) == [c for c in (7, 8, 9, 10) if c not in want]


def grams(tok, par, n, length):
    out = []
    for c in range(n):
        g, a = [], c
        for _ in range(length):
            if a < 0:
                break
            g.append(int(tok[a])); a = par[a]
        if len(g) == length:
            out.append((tuple(g), c))
    return out


def test_no_gram_longer_than_tau_repeats_after_merging():
    rng = np.random.default_rng(12)
    V, k = 5, 3                                              # a tiny vocabulary forces repeats
    for tau in (1, 2, 3):
        st = fresh(2, 400, root_token=0)
        frontier = [[0], [0]]
        for level in range(6):
            F = max(1, max(len(f) for f in frontier))
            lg = rng.normal(size=(2, F, V)).astype(np.float32)
            before = st[5].copy()
            st, nf, nfl, full = grow(st, lg, frontier, k, tau)
            assert not full
            tok, par, mrg, leaf, prob, n = st
            for b in range(2):
                assert n[b] == before[b] + k * len(frontier[b])
                new = list(range(before[b], n[b]))
                assert list(nf[b, :nfl[b]]) == [c for c in new if not leaf[b, c]]
                seen = {}
                for g, c in grams(tok[b], par[b], n[b], tau):
                    if g in seen:
                        assert mrg[b, c] == seen[g] and leaf[b, c]       # merged into the first occurrence
                        assert mrg[b, seen[g]] == -1
                    else:
                        seen[g] = c
                        assert mrg[b, c] == -1
                longer = [g for g, _ in grams(tok[b], par[b], n[b], tau + 1)]
                assert len(longer) == len(set(longer))                  # Sec. 5.3
            frontier = [list(nf[b, :nfl[b]]) for b in range(2)]
            if not any(frontier):
                break
        assert (st[2] >= 0).any()                                        # something was merged at all


def test_capacity():
    lg = np.zeros((1, 2, 8), np.float32)
    st = fresh(1, 6)
    st, nf, nfl, full = grow(st, lg, [[0, 0]], k=3, tau=9)
    assert full and st[5][0] == 6 and nfl[0] == 5
