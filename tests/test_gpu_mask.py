"""gsd_build_mask on the GPU against the oracle's upward search: bit-exact."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
import oracle
from gpu_util import i32_tensor

pytestmark = pytest.mark.gpu


def gpu_mask(ptr, idx, status=None):
    import paper_2407_16207_b200 as gsd
    out = gsd.gsd_build_mask(i32_tensor(ptr, "cuda"), i32_tensor(idx, "cuda"), status=status)
    torch.cuda.synchronize()
    return out.cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("name", ["tiny", "llama7b", "llama13b", "llama70b", "sweep512"])
def test_configs_bit_exact_and_equal_to_the_generated_mask(name):
    cfg = gi.sweep_config(4, 512, 512) if name == "sweep512" else gi.CONFIGS[name]
    inp = gi.make_inputs(cfg, attn=False, accept=False)
    got = gpu_mask(inp["parent_ptr"], inp["parent_idx"])
    assert np.array_equal(got, oracle.build_mask(inp["parent_ptr"], inp["parent_idx"]))
    assert np.array_equal(got, inp["ancestor_mask"])


def test_chain_of_maximum_length_and_odd_sizes():
    for N in (1, 31, 33, 100, 512):
        ptr, idx = gi.parents_to_csr([[[]] + [[i - 1] for i in range(1, N)]])
        got = gpu_mask(ptr, idx)
        assert np.array_equal(got, oracle.build_mask(ptr, idx))


def test_bad_edges_are_ignored_and_flagged():
    ptr = np.array([[0, 0, 2, 3]], dtype=np.int32)
    idx = np.array([[0, 5, 2]], dtype=np.int32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = gpu_mask(ptr, idx, status)
    assert np.array_equal(got, oracle.build_mask(ptr, idx))
    assert int(status.item()) == 0x1
