"""Pins of the oracle's non-deterministic verification (Sec. 3: accept with probability
min(1, p/q), the first rejection ends the hypothesis, the target model regenerates that token;
Sec. 6.4: the same on the token graph).  The random numbers are inputs, so every case is exact."""
import numpy as np
import pytest

import gsd_inputs as gi
import oracle

LOG = np.log


def chain(n):
    """parent CSR of the path 0 -> 1 -> ... -> n-1"""
    ptr = np.array([[0] + list(range(0, n))], dtype=np.int32)
    idx = np.array([list(range(0, n - 1)) or [0]], dtype=np.int32)
    return ptr, idx


def run(logits, tok, ptr, idx, q, u, us):
    t, l, nd = oracle.accept_sampled(np.asarray(logits, np.float32)[None], np.asarray(tok, np.int32)[None], ptr, idx,
                                     np.asarray(q, np.float32)[None], np.asarray(u, np.float32)[None],
                                     np.asarray([us], np.float32))
    n = int(l[0])
    return list(t[0, :n]), list(nd[0, :n])


def test_worked_chain():
    # P rows: node 0 -> [.5,.25,.125,.125]; node 1 -> [.1,.2,.3,.4]; tokens of nodes 1..3: 0, 0, 2
    P = np.array([[.5, .25, .125, .125], [.1, .2, .3, .4], [.25, .25, .25, .25], [.7, .1, .1, .1]])
    ptr, idx = chain(4)
    tok = [3, 0, 0, 2]
    # step 0->1: u q = .5*.8 = .4 < .5 accepted; step 1->2: .3*.5 = .15 < .1 is false: rejected
    toks, nodes = run(LOG(P), tok, ptr, idx, q=[1, .8, .5, .5], u=[0, .5, .3, .0], us=0.25)
    assert nodes == [0, 1]
    # regenerated at node 1: cumulative .1, .3 -> the first one above .25 is index 1
    assert toks == [0, 1]
    # with a smaller u the second step passes too (.1*.5 = .05 < .1) and the third (0 < .25)
    toks, nodes = run(LOG(P), tok, ptr, idx, q=[1, .8, .5, .5], u=[0, .5, .1, .0], us=0.95)
    assert nodes == [0, 1, 2, 3]
    assert toks == [0, 0, 2, 3]          # .7+.1+.1 = .9 is not above .95: index 3


def test_strict_comparisons():
    # V = 2 with equal logits: both probabilities are exactly one half
    ptr, idx = chain(2)
    lg = np.zeros((2, 2))
    # u q == p is a rejection; just below is an acceptance
    assert run(lg, [0, 1], ptr, idx, q=[1, 1], u=[0, .5], us=.1)[1] == [0]
    assert run(lg, [0, 1], ptr, idx, q=[1, 1], u=[0, np.nextafter(np.float32(.5), np.float32(0))], us=.1)[1] == [0, 1]
    # inverse CDF: the cumulative value has to exceed u
    assert run(lg, [0, 1], ptr, idx, q=[1, 1], u=[0, .9], us=.5)[0] == [1]
    assert run(lg, [0, 1], ptr, idx, q=[1, 1], u=[0, .9], us=.49)[0] == [0]


def test_draft_probability_scales_the_test():
    # p = 1/4; with q = 1/8 the ratio is above one: always accepted; with q = 1 only below 1/4
    ptr, idx = chain(2)
    lg = np.zeros((2, 4))
    assert run(lg, [0, 2], ptr, idx, q=[1, .125], u=[0, .999], us=.1)[1] == [0, 1]
    assert run(lg, [0, 2], ptr, idx, q=[1, 1.0], u=[0, .26], us=.1)[1] == [0]
    assert run(lg, [0, 2], ptr, idx, q=[1, 1.0], u=[0, .24], us=.1)[1] == [0, 1]
    # q = 0 (the draft gave the token no mass): accepted whenever the target gives it any
    assert run(lg, [0, 2], ptr, idx, q=[1, 0.0], u=[0, .999], us=.1)[1] == [0, 1]


def test_probability_is_read_from_the_parent_on_the_path():
    # node 3 (token 1) has the parents 1 and 2; node 1 gives token 1 mass .9, node 2 gives .05
    P = np.array([[.5, .5, 0, 0], [.05, .9, .05, 0], [.9, .05, .05, 0], [.25, .25, .25, .25]])
    with np.errstate(divide="ignore"):
        lg = LOG(P)
    ptr = np.array([[0, 0, 1, 2, 4]], dtype=np.int32)
    idx = np.array([[0, 0, 1, 2]], dtype=np.int32)
    tok = [0, 0, 1, 1]
    # u q = .5 for node 3: passes under node 1 only; nodes 1 and 2 both pass under the root
    toks, nodes = run(lg, tok, ptr, idx, q=[1, 1, 1, 1], u=[0, .4, .4, .5], us=.1)
    assert nodes == [0, 1, 3] and toks[:2] == [0, 1]
    # make the step 0 -> 1 fail: the only way to node 3 is through node 2, where it is rejected
    toks, nodes = run(lg, tok, ptr, idx, q=[1, 1, 1, 1], u=[0, .6, .4, .5], us=.1)
    assert nodes == [0, 2]


def peaked(cfg, inp):
    """logits that put (numerically) all mass on the argmax of the generated logits"""
    am = oracle.argmax(inp["logits"])
    lg = np.full(inp["logits"].shape, -80.0, dtype=np.float32)
    np.put_along_axis(lg, am[..., None].astype(np.int64), 0.0, axis=-1)
    return lg


@pytest.mark.parametrize("name", ["tiny", "llama7b"])
def test_reduces_to_the_deterministic_rule_for_one_hot_targets(name):
    # with a one-hot target distribution, q = 1 and any u in (0, 1) the test "u < min(1, p/q)"
    # is "the token is the target's argmax", and the regenerated token is that argmax
    cfg = gi.CONFIGS[name]
    longest = 0
    for trial in range(4):
        inp = gi.make_inputs(cfg, gi.seed_for(cfg, trial), attn=False)
        lg = peaked(cfg, inp)
        rng = np.random.default_rng(5 + trial)
        u = rng.uniform(0.01, 0.99, size=(cfg.B, cfg.N)).astype(np.float32)
        us = rng.uniform(0.01, 0.99, size=(cfg.B,)).astype(np.float32)
        q = np.ones((cfg.B, cfg.N), dtype=np.float32)
        t0, l0, n0, _ = oracle.accept(lg, inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"])
        t1, l1, n1 = oracle.accept_sampled(lg, inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], q, u, us)
        assert (l0 == l1).all() and (t0 == t1).all() and (n0 == n1).all()
        longest = max(longest, int(l0.max()))
    assert longest > 1             # the generator plants agreement: some path is really accepted


def test_u_zero_accepts_every_step_with_mass_and_larger_u_never_helps():
    cfg = gi.CONFIGS["tiny"]
    inp = gi.make_inputs(cfg, attn=False)
    lg = inp["logits"]
    B, N = cfg.B, cfg.N
    q = np.full((B, N), 0.3, dtype=np.float32)
    us = np.full((B,), 0.5, dtype=np.float32)
    zero = np.zeros((B, N), dtype=np.float32)
    _, l_all, nodes_all = oracle.accept_sampled(lg, inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], q, zero, us)
    # every step accepted: the hypothesis is a longest root path of the graph = deepest level + 1
    for b in range(B):
        depth = max(inp["levels"][b])
        assert l_all[b] == depth + 1
    rng = np.random.default_rng(9)
    u = rng.uniform(0, 1, size=(B, N)).astype(np.float32)
    prev = l_all
    for scale in (0.25, 0.5, 1.0):
        _, l, _ = oracle.accept_sampled(lg, inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], q,
                                        (u * scale).astype(np.float32), us)
        assert (l <= prev).all()
        prev = l


def test_acceptance_frequency_matches_min_one_p_over_q():
    # one step, many independent u: the fraction accepted is min(1, p/q) (Sec. 3)
    ptr, idx = chain(2)
    P = np.array([[.2, .8], [.5, .5]])
    n = 4000
    rng = np.random.default_rng(1)
    for q, want in ((.4, .5), (.1, 1.0), (.8, .25)):
        acc = 0
        for u in rng.uniform(0, 1, size=n):
            acc += len(run(LOG(P), [0, 0], ptr, idx, q=[1, q], u=[0, u], us=.3)[1]) == 2
        assert abs(acc / n - want) < 0.03
