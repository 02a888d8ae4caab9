"""Pins for the CPU oracle's acceptance step: numpy argmax, hand-built DAGs with hand-derived
answers, special cases (chain, tree), invariants, and an independent dynamic-programming
solution of the same problem."""
import numpy as np
import pytest

import gsd_inputs as gi
import oracle
from helpers import dp_longest_accepted, load_accept_cases, logits_with_argmax

CASES = load_accept_cases()


def run_case(tokens, parents, amax, V=128, rng=None, Tcap=0):
    logits = logits_with_argmax(amax, V, rng)[None]
    ptr, idx = gi.parents_to_csr([parents])
    toks, lens, nodes, _ = oracle.accept(logits, np.array([tokens], dtype=np.int32), ptr, idx,
                                         Tcap=Tcap)
    m = int(lens[0])
    return list(toks[0, :m]), list(nodes[0, :m]), toks[0], nodes[0], m


@pytest.mark.parametrize("case", CASES, ids=[c["name"] for c in CASES])
def test_hand_built_dags(case):
    toks, nodes, raw_t, raw_n, m = run_case(case["tokens"], case["parents"], case["argmax"])
    assert toks == case["expect_tokens"]
    assert nodes == case["expect_nodes"]
    assert m == len(case["expect_tokens"])
    assert (raw_t[m:] == -1).all() and (raw_n[m:] == -1).all()


def test_argmax_matches_numpy_first_occurrence():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((50, 777)).astype(np.float32)
    x[3, [5, 400, 776]] = 9.0         # exact ties: the lowest index wins
    x[4, :] = 1.25                    # a constant row
    x[5, 0] = x[5, 776] = 7.0
    x[6, 10] = np.inf; x[6, 20] = np.inf
    x[7, :] = -np.inf
    assert np.array_equal(oracle.argmax(x), np.argmax(x, axis=1))


def test_argmax_nan_never_wins():
    x = np.zeros((4, 6), dtype=np.float32)
    x[0] = [np.nan, 1, 3, np.nan, 3, 2]; x[1] = np.nan
    x[2] = [np.nan, -np.inf, -np.inf, np.nan, np.nan, np.nan]
    x[3] = [-0.0, 0.0, -0.0, 0.0, -1, -2]          # signed zeros compare equal
    assert list(oracle.argmax(x)) == [2, 0, 1, 0]


def test_chain_equals_longest_prefix_match():
    # sequence-structured drafting (Sec. 3): accept the longest prefix on which the greedy
    # continuation of each position equals the next drafted token
    rng = np.random.default_rng(1)
    for trial in range(200):
        n = int(rng.integers(1, 12))
        tok = rng.integers(0, 3, size=n).tolist()
        amax = rng.integers(0, 3, size=n).tolist()
        parents = [[]] + [[i - 1] for i in range(1, n)]
        m = 0
        while m + 1 < n and tok[m + 1] == amax[m]:
            m += 1
        toks, nodes, *_ = run_case(tok, parents, amax, V=8)
        assert nodes == list(range(m + 1))
        assert toks == tok[1:m + 1] + [amax[m]]


def test_tree_equals_best_leaf_prefix_match():
    rng = np.random.default_rng(2)
    for trial in range(60):
        n = int(rng.integers(2, 40))
        parents, _ = gi.make_dag(n, min(6, n - 1), 3, 1, rng)
        tok = rng.integers(0, 3, size=n).tolist()
        amax = rng.integers(0, 3, size=n).tolist()
        best = 0
        for leaf in range(n):                   # every node's unique root path
            path = [leaf]
            while parents[path[-1]]:
                path.append(parents[path[-1]][0])
            path = path[::-1]
            m = 0
            while m + 1 < len(path) and tok[path[m + 1]] == amax[path[m]]:
                m += 1
            best = max(best, m)
        *_, m_got = run_case(tok, parents, amax, V=8)
        assert m_got == best + 1


@pytest.mark.parametrize("name", ["tiny", "llama7b", "llama13b", "llama70b"])
def test_invariants_and_dp_cross_check_on_configs(name):
    cfg = gi.CONFIGS[name]
    for trial in range(2):
        inp = gi.make_inputs(cfg, gi.seed_for(cfg, trial), attn=False)
        toks, lens, nodes, visited = oracle.accept(inp["logits"], inp["draft_tokens"],
                                                   inp["parent_ptr"], inp["parent_idx"])
        amax_all = np.argmax(inp["logits"], axis=2)
        assert (visited >= cfg.N).all()          # every node has at least one root path
        for b in range(cfg.B):
            parents, tok, amax = inp["parents"][b], inp["draft_tokens"][b], amax_all[b]
            m = int(lens[b])
            path = list(nodes[b, :m])
            assert 1 <= m <= cfg.depth + 1 and path[0] == 0
            for i in range(1, m):
                assert path[i - 1] in parents[path[i]]
                assert tok[path[i]] == amax[path[i - 1]]
                assert toks[b, i - 1] == tok[path[i]]
            assert toks[b, m - 1] == amax[path[-1]]
            assert (toks[b, m:] == -1).all()
            assert path == dp_longest_accepted(tok, amax, parents)


def test_dense_duplicate_tokens_against_dp():
    # few distinct tokens: many accepted paths and many ties
    rng = np.random.default_rng(3)
    for trial in range(100):
        n = int(rng.integers(2, 48))
        parents, _ = gi.make_dag(n, min(7, n - 1), 4, 3, rng)
        tok = rng.integers(0, 2, size=n).tolist()
        amax = rng.integers(0, 2, size=n).tolist()
        toks, nodes, *_ = run_case(tok, parents, amax, V=4)
        want = dp_longest_accepted(tok, amax, parents)
        assert nodes == want
        assert toks == [tok[v] for v in want[1:]] + [amax[want[-1]]]


def test_visit_cap_prunes_without_changing_the_answer():
    cfg = gi.CONFIGS["llama13b"]
    inp = gi.make_inputs(cfg, attn=False)
    a = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"])
    b = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"],
                      visit_cap=50)
    assert (b[3] < 0).all() and (np.abs(b[3]) < a[3]).all()
    for x, y in zip(a[:3], b[:3]):
        assert np.array_equal(x, y)


def test_malformed_dag_and_small_tcap_are_rejected():
    logits = logits_with_argmax([1, 2], 4)[None]
    tok = np.array([[0, 1]], dtype=np.int32)
    ptr = np.array([[0, 0, 1]], dtype=np.int32)
    with pytest.raises(ValueError):
        oracle.accept(logits, tok, ptr, np.array([[1]], dtype=np.int32))     # parent == child
    with pytest.raises(ValueError):
        oracle.accept(logits, tok, ptr, np.array([[0]], dtype=np.int32), Tcap=1)
