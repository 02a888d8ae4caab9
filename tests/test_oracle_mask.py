"""Pins for the oracle's ancestor-mask builder: closed forms (chain, star, tree paths), a
boolean matrix closure computed with numpy, and hand-built DAGs."""
import numpy as np
import pytest

import gsd_inputs as gi
import oracle


def bits_of(mask_row, N):
    return {j for j in range(N) if (int(mask_row[j // 32]) >> (j % 32)) & 1}


def csr(parents):
    return gi.parents_to_csr([parents])


def test_chain_is_lower_triangular_and_star_sees_root_only():
    N = 70                                                   # three mask words
    ptr, idx = csr([[]] + [[i - 1] for i in range(1, N)])
    m = oracle.build_mask(ptr, idx)[0]
    for n in range(N):
        assert bits_of(m[n], N) == set(range(n + 1))
    ptr, idx = csr([[]] + [[0] for _ in range(1, N)])
    m = oracle.build_mask(ptr, idx)[0]
    for n in range(1, N):
        assert bits_of(m[n], N) == {0, n}
    assert (m[:, 2] >> np.uint32(N - 64)).max() == 0        # no bits at positions >= N


def test_hand_built_diamond_with_level_skip():
    # 0 -> 1, 0 -> 2, {1,2} -> 3, 3 -> 4, 0 -> 4 (skip edge), 5 has no parent
    ptr, idx = csr([[], [0], [0], [1, 2], [0, 3], []])
    m = oracle.build_mask(ptr, idx)[0]
    want = [{0}, {0, 1}, {0, 2}, {0, 1, 2, 3}, {0, 1, 2, 3, 4}, {5}]
    assert [bits_of(m[n], 6) for n in range(6)] == want


@pytest.mark.parametrize("name", ["tiny", "llama7b", "llama13b", "llama70b"])
def test_matches_boolean_matrix_closure(name):
    cfg = gi.CONFIGS[name]
    inp = gi.make_inputs(cfg, attn=False, accept=False)
    got = oracle.build_mask(inp["parent_ptr"], inp["parent_idx"])
    N = cfg.N
    for b in range(cfg.B):
        A = np.eye(N, dtype=bool)
        for v, ps in enumerate(inp["parents"][b]):
            A[v, ps] = True
        R = A.copy()
        for _ in range(int(np.ceil(np.log2(max(N, 2)))) + 1):      # repeated squaring
            R = (R.astype(np.int64) @ R.astype(np.int64)) > 0
        for n in range(N):
            assert bits_of(got[b, n], N) == set(np.nonzero(R[n])[0].tolist())


def test_tree_rows_are_root_paths():
    rng = np.random.default_rng(5)
    parents, _ = gi.make_dag(60, 6, 3, 1, rng)
    ptr, idx = csr(parents)
    m = oracle.build_mask(ptr, idx)[0]
    for n in range(60):
        path, v = {n}, n
        while parents[v]:
            v = parents[v][0]
            path.add(v)
        assert bits_of(m[n], 60) == path


def test_bad_parent_indices_are_ignored():
    ptr = np.array([[0, 0, 2, 3]], dtype=np.int32)
    idx = np.array([[0, 5, 2]], dtype=np.int32)             # node 1: {0, 5(bad)}, node 2: {2(self, bad)}
    m = oracle.build_mask(ptr, idx)[0]
    assert [bits_of(m[n], 3) for n in range(3)] == [{0}, {0, 1}, {2}]
