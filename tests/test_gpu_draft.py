"""gsd_draft_expand on the GPU against the CPU oracle, level by level.  The order of the children
compares logits (exact on both sides); the pruning flags compare fp32 probabilities with
thresholds, so the thresholds of these tests are placed at least 0.2 % (relative) away from every
probability (and probability ratio) they are compared with - taken from a numpy fp64 softmax."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


def fresh(B, Ncap, root_token=5):
    tokens = np.full((B, Ncap), -1, np.int32); tokens[:, 0] = root_token
    parent = np.full((B, Ncap), -1, np.int32)
    merge = np.full((B, Ncap), -1, np.int32)
    leaf = np.zeros((B, Ncap), np.uint8)
    prob = np.zeros((B, Ncap), np.float32); prob[:, 0] = 1.0
    n = np.ones((B,), np.int32)
    return [tokens, parent, merge, leaf, prob, n]


def decisive_thresholds(lg, fl, k, rng, tp_range=(0.02, 0.4), ts_range=(0.05, 0.6)):
    x = lg.astype(np.float64)
    x = x - x.max(axis=-1, keepdims=True)
    P = np.exp(x); P /= P.sum(axis=-1, keepdims=True)
    top = -np.sort(-P, axis=-1)[..., :k]
    rows = [top[b, f] for b in range(lg.shape[0]) for f in range(fl[b])]
    q = np.concatenate(rows) if rows else np.zeros(0)
    ratio = np.concatenate([r / r[0] for r in rows]) if rows else np.zeros(0)
    def pick(values, lo_hi):
        for _ in range(4000):
            t = rng.uniform(*lo_hi)
            if (np.abs(values - t) > 0.002 * t).all():
                return float(np.float32(t))
        raise AssertionError("no decisive threshold found")
    return pick(q, tp_range), pick(ratio, ts_range)


def gpu_step(state, lg, fr, fl, k, tau, tp, ts, status=None):
    import paper_2407_16207_b200 as gsd
    dev = "cuda"
    t = [torch.from_numpy(a.copy()).to(dev) for a in state]
    nf, nfl = gsd.gsd_draft_expand(torch.from_numpy(lg).to(dev), torch.from_numpy(fr).to(dev), torch.from_numpy(fl).to(dev),
                                   *t, k=k, tau=tau, theta_prob=tp, theta_sib=ts, status=status)
    torch.cuda.synchronize()
    return [a.cpu().numpy() for a in t], nf.cpu().numpy(), nfl.cpu().numpy()


def compare(got, want, nf_g, nfl_g, nf_w, nfl_w):
    n = want[5]
    assert np.array_equal(got[5], n)
    for b in range(len(n)):
        for a in (0, 1, 2, 3):
            assert np.array_equal(got[a][b, :n[b]], want[a][b, :n[b]]), a
        assert np.allclose(got[4][b, :n[b]], want[4][b, :n[b]], rtol=2e-5, atol=1e-9)
        assert nfl_g[b] == nfl_w[b] and np.array_equal(nf_g[b, :nfl_g[b]], nf_w[b, :nfl_w[b]])


def grow_levels(B, V, k, tau, levels, Ncap, seed, logit_scale=3.0, round_to=None, drop=0.0, tp_range=(0.02, 0.4), ts_range=(0.05, 0.6)):
    rng = np.random.default_rng(seed)
    state = fresh(B, Ncap)
    frontier = [[0] for _ in range(B)]
    merged = 0
    for level in range(levels):
        F = max(1, max(len(f) for f in frontier))
        lg = (rng.normal(size=(B, F, V)) * logit_scale).astype(np.float32)
        if V > 4 * k:
            # a peaked draft distribution: a handful of tokens well above the rest
            hot = rng.integers(0, V, size=(B, F, 2 * k))
            np.put_along_axis(lg, hot, (rng.uniform(4, 7, size=hot.shape) * logit_scale + 4).astype(np.float32), axis=-1)
        if round_to:
            lg = np.round(lg / round_to).astype(np.float32) * np.float32(round_to)     # exact ties between logits
        if drop > 0:
            keep_top = np.argsort(-lg, axis=-1)[..., :k]
            mask = rng.uniform(size=lg.shape) < drop
            np.put_along_axis(mask, keep_top, False, axis=-1)
            lg[mask] = -np.inf
        fr = np.full((B, F), -1, np.int32); fl = np.zeros((B,), np.int32)
        for b, f in enumerate(frontier):
            fr[b, :len(f)] = f; fl[b] = len(f)
        tp, ts = decisive_thresholds(lg, fl, k, rng, tp_range, ts_range)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        got, nf_g, nfl_g = gpu_step(state, lg, fr, fl, k, tau, tp, ts, status=status)
        out = oracle.draft_expand(lg, fr, fl, *state, k=k, tau=tau, theta_prob=tp, theta_sib=ts)
        want, nf_w, nfl_w, full = list(out[:6]), out[6], out[7], out[8]
        compare(got, want, nf_g, nfl_g, nf_w, nfl_w)
        assert bool(int(status.item()) & 0x80) == full
        assert int(status.item()) & ~0x80 == 0
        state = want
        frontier = [list(nf_w[b, :nfl_w[b]]) for b in range(B)]
        merged += int((want[2] >= 0).sum())
        if full or not any(frontier):
            break
    return state, merged


def test_llama_vocabulary_four_levels():
    state, _ = grow_levels(B=3, V=32000, k=4, tau=2, levels=5, Ncap=512, seed=1, tp_range=(0.005, 0.05), ts_range=(0.02, 0.2))
    assert state[5].min() > 40


@pytest.mark.parametrize("tau", [1, 2, 3])
def test_tiny_vocabulary_many_repeats(tau):
    # 6 tokens, 3 children per node: grams re-occur all the time; rounded logits tie exactly
    state, merged = grow_levels(B=4, V=6, k=3, tau=tau, levels=6, Ncap=400, seed=10 + tau, logit_scale=1.0, round_to=0.5)
    assert merged > 0


def test_scalar_loads_filtered_entries_and_k8():
    grow_levels(B=2, V=1003, k=8, tau=2, levels=3, Ncap=512, seed=3, drop=0.6)


def test_long_runs_of_equal_logits():
    # thousands of entries tie with the k-th best: the order is decided by the token id alone
    # (on the GPU this is the path that keeps per-thread lists instead of a candidate buffer)
    rng = np.random.default_rng(8)
    B, F, V, k = 2, 3, 5000, 6
    lg = rng.integers(0, 2, size=(B, F, V)).astype(np.float32)       # values 0 and 1 only
    lg[0, 0, :] = 0.0                                                 # one row entirely flat
    fr = np.zeros((B, F), np.int32); fl = np.full((B,), F, np.int32)
    state = fresh(B, 64)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got, nf_g, nfl_g = gpu_step(state, lg, fr, fl, k, 9, 0.0, 0.0, status=status)
    out = oracle.draft_expand(lg, fr, fl, *state, k=k, tau=9, theta_prob=0.0, theta_sib=0.0)
    compare(got, list(out[:6]), nf_g, nfl_g, out[6], out[7])
    assert int(status.item()) == 0
    assert list(got[0][0, 1:1 + k]) == list(range(k))


def test_best_entries_in_one_threads_share():
    # The row kernel offers one candidate per thread; a thread's share is every 256th group of
    # four entries.  Here the k best entries of a row sit in one group, in groups 1024 entries
    # apart, or tie with entries elsewhere - all cases in which an entry that no thread offered
    # belongs to the k best and the row has to be read a second time.
    rng = np.random.default_rng(21)
    B, F, V, k = 2, 6, 32000, 4
    lg = (rng.normal(size=(B, F, V)) * 2).astype(np.float32)
    big = np.float32(30.0)
    lg[0, 0, 4000:4004] = [big + 3, big + 2, big + 1, big]              # one group of four
    lg[0, 1, [17, 17 + 1024, 17 + 2048, 17 + 3072]] = [big, big + 1, big + 2, big + 3]   # one thread, four groups
    lg[0, 2, [5, 6]] = big                                              # two equal maxima side by side
    lg[0, 2, [9000, 20000]] = big                                       # ... and two more elsewhere: ties by token id
    lg[0, 3, 31996:32000] = [big, big, big, big]                        # the last group of the row
    lg[0, 4, [100, 101]] = [big + 1, big - 1]                           # the second of a pair ranks third
    lg[0, 4, [7000, 15000]] = [big, big - 2]
    lg[0, 5, 0] = big                                                   # nothing special: one clear winner
    lg[1] = lg[0][::-1]
    fr = np.zeros((B, F), np.int32); fl = np.full((B,), F, np.int32)
    state = fresh(B, 64)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got, nf_g, nfl_g = gpu_step(state, lg, fr, fl, k, 9, 0.0, 0.0, status=status)
    out = oracle.draft_expand(lg, fr, fl, *state, k=k, tau=9, theta_prob=0.0, theta_sib=0.0)
    compare(got, list(out[:6]), nf_g, nfl_g, out[6], out[7])
    assert int(status.item()) == 0
    assert list(got[0][0, 1:5]) == [4000, 4001, 4002, 4003]
    assert list(got[0][0, 5:9]) == [17 + 3072, 17 + 2048, 17 + 1024, 17]
    assert list(got[0][0, 9:13]) == [5, 6, 9000, 20000]


def test_capacity_is_reported_and_respected():
    state, _ = grow_levels(B=2, V=64, k=4, tau=4, levels=8, Ncap=50, seed=5)
    assert (state[5] == 50).any()


def test_bad_frontier_is_flagged():
    lg = np.zeros((1, 2, 16), np.float32)
    fr = np.array([[0, 7]], np.int32)          # node 7 does not exist yet
    fl = np.array([2], np.int32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    gpu_step(fresh(1, 32), lg, fr, fl, 2, 2, 0.0, 0.0, status=status)
    assert int(status.item()) & 0x100
