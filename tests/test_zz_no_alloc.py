"""gsd_accept_static: acceptance for callers that cannot provide scratch memory.

A plug-in inside a serving process whose host has already taken the GPU's memory, or code
on a path where cudaMalloc is not allowed, calls this variant; the scratch sits in a fixed
array inside the library.  Its results must equal those of gsd_accept, call after call
(the shared array keeps the previous call's contents, so the second call checks the
clearing).  This file sorts last on purpose: it runs after every other test."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
import oracle
from gpu_util import accept_tensors

pytestmark = pytest.mark.gpu


def both(inp):
    import paper_2407_16207_b200 as gsd
    t = accept_tensors(inp)
    args = (t["logits"], t["draft_tokens"], t["parent_ptr"], t["parent_idx"])
    want = gsd.gsd_accept(*args)
    got = gsd.gsd_accept_static(*args)
    torch.cuda.synchronize()
    return [x.cpu().numpy() for x in want], [x.cpu().numpy() for x in got]


def test_two_calls_in_a_row_match_gsd_accept():
    # integer results: the comparison is exact, as in the other acceptance tests
    first = gi.make_inputs(gi.CONFIGS["llama13b"], attn=False)
    second = gi.make_inputs(gi.CONFIGS["llama7b"], attn=False)     # fewer rows: stale keys remain beyond them
    for inp in (first, second, first):
        want, got = both(inp)
        for w, g in zip(want, got):
            assert np.array_equal(w, g)
        # and against the CPU oracle directly, so that this file stands on its own
        ref = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"])
        for r, g in zip(ref[:3], got):
            assert np.array_equal(r, g)


def test_free_device_memory_does_not_move():
    # the call's promise is that it allocates nothing: with the outputs allocated up front, the
    # driver's free-byte count (cudaMemGetInfo) is the same after twenty more calls
    import ctypes
    import paper_2407_16207_b200 as gsd
    inp = gi.make_inputs(gi.CONFIGS["llama7b"], attn=False)
    t = accept_tensors(inp)
    B, N, V = t["logits"].shape
    toks = torch.empty((B, N), dtype=torch.int32, device="cuda")
    lens = torch.empty((B,), dtype=torch.int32, device="cuda")
    nodes = torch.empty((B, N), dtype=torch.int32, device="cuda")
    p = gsd.binding.AcceptParams(B, N, V, t["parent_idx"].shape[1], N)
    L = gsd.lib()
    stream = torch.cuda.current_stream().cuda_stream

    def call():
        rc = L.gsd_accept_static(t["logits"].data_ptr(), t["draft_tokens"].data_ptr(), t["parent_ptr"].data_ptr(),
                                 t["parent_idx"].data_ptr(), toks.data_ptr(), lens.data_ptr(), nodes.data_ptr(),
                                 ctypes.byref(p), None, stream)
        assert rc == 0

    call()                                   # the first call on a device looks the array up
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for _ in range(20):
        call()
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    ref = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"])
    assert np.array_equal(toks.cpu().numpy(), ref[0]) and np.array_equal(lens.cpu().numpy(), ref[1])


def test_size_limit_is_refused_cleanly():
    import paper_2407_16207_b200 as gsd
    B, N, V = 33, 512, 8                                             # 16896 rows > 16384
    assert B * N > gsd.binding.GSD_STATIC_MAX_ROWS
    logits = torch.zeros((B, N, V), dtype=torch.float32, device="cuda")
    tok = torch.zeros((B, N), dtype=torch.int32, device="cuda")
    ptr = torch.zeros((B, N + 1), dtype=torch.int32, device="cuda")
    idx = torch.zeros((B, 1), dtype=torch.int32, device="cuda")
    with pytest.raises(gsd.GsdError) as e:
        gsd.gsd_accept_static(logits, tok, ptr, idx)
    assert e.value.code == -4 and "GSD_STATIC_MAX_ROWS" in str(e.value)
    # the largest allowed size goes through and agrees with gsd_accept
    B = 32
    logits = torch.randn((B, N, V), dtype=torch.float32, device="cuda")
    tok, ptr = tok[:B].contiguous(), ptr[:B].contiguous()
    idx = idx[:B].contiguous()
    want = gsd.gsd_accept(logits, tok, ptr, idx)
    got = gsd.gsd_accept_static(logits, tok, ptr, idx)
    for w, g in zip(want, got):
        assert torch.equal(w, g)
