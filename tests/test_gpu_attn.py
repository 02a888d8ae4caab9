"""gsd_verify_attn on the GPU against the fp64 CPU oracle.

Tolerance (bf16 output against fp64): max-abs <= 1e-2 and mean-abs <= 1e-3."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
import oracle
from gpu_util import attn_tensors, out_to_f64

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 1e-2, 1e-3
KERNELS = [1, 2]        # GSD_ATTN_MMA, GSD_ATTN_TCGEN05


def gpu_attn(inp, **kw):
    import paper_2407_16207_b200 as gsd
    t = attn_tensors(inp)
    try:
        out = gsd.gsd_verify_attn(t["q"], t["k_cache"], t["v_cache"], t["draft_k"], t["draft_v"],
                                  t["ancestor_mask"], t["seq_lens"], **kw)
    except gsd.GsdError as e:
        if e.code == -6:
            pytest.skip("kernel variant does not cover this shape")
        raise
    torch.cuda.synchronize()
    return out


def cpu_attn(inp, **kw):
    return oracle.attn(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"], inp["draft_v"],
                       inp["ancestor_mask"], inp["seq_lens"], **kw)


def assert_close(got64, want):
    assert np.isfinite(got64).all()
    err = np.abs(got64 - want)
    assert err.max() <= MAX_ABS, f"max-abs {err.max():.3e}"
    assert err.mean() <= MEAN_ABS, f"mean-abs {err.mean():.3e}"


def assert_close_scaled(got64, want):
    # for batches with almost no prefix: rows that see a handful of keys keep values of a few
    # units, whose bf16 rounding step is larger, so the error is taken relative to max(1, |value|)
    assert np.isfinite(got64).all()
    err = np.abs(got64 - want) / np.maximum(1.0, np.abs(want))
    assert err.max() <= MAX_ABS, f"max-abs {err.max():.3e}"
    assert err.mean() <= MEAN_ABS, f"mean-abs {err.mean():.3e}"


def variant(cfg, **kw):
    return gi.VerifyConfig(**{**cfg.__dict__, **kw})


@pytest.mark.parametrize("kernel", [0] + KERNELS)
@pytest.mark.parametrize("name", ["tiny", "llama7b", "llama13b"])
def test_configs_full_compare(name, kernel):
    cfg = gi.CONFIGS[name]
    for trial in range(2 if name != "llama13b" else 1):
        inp = gi.make_inputs(cfg, gi.seed_for(cfg, trial), accept=False)
        assert_close(out_to_f64(gpu_attn(inp, kernel=kernel)), cpu_attn(inp))


@pytest.fixture(scope="module")
def llama70b_all_rows():
    """The full-size configuration with the oracle's answer for ALL 131072 rows, computed once
    (some tens of seconds on the host cores) and shared by the three kernel selections."""
    cfg = gi.CONFIGS["llama70b"]
    inp = gi.make_inputs(cfg, accept=False)
    return inp, cpu_attn(inp)


@pytest.mark.parametrize("kernel", [0] + KERNELS)
def test_llama70b_every_row(kernel, llama70b_all_rows):
    inp, want = llama70b_all_rows
    got = out_to_f64(gpu_attn(inp, kernel=kernel))
    assert got.shape == want.shape
    assert_close(got, want)
    # no single (sequence, kv head) unit hides behind the global mean
    cfg = inp["cfg"]
    err = np.abs(got - want).reshape(cfg.B, cfg.N, cfg.Hkv, cfg.G, cfg.D)
    assert err.mean(axis=(1, 3, 4)).max() <= MEAN_ABS


@pytest.mark.parametrize("num_splits", [-1, -2])
def test_llama70b_every_row_with_plans_made_on_the_device(num_splits, llama70b_all_rows):
    # GSD_ATTN_SPLIT_BALANCED / GSD_ATTN_SPLIT_PER_SEQUENCE at full size, every row against the oracle
    inp, want = llama70b_all_rows
    got = out_to_f64(gpu_attn(inp, kernel=2, num_splits=num_splits))
    assert_close(got, want)
    cfg = inp["cfg"]
    err = np.abs(got - want).reshape(cfg.B, cfg.N, cfg.Hkv, cfg.G, cfg.D)
    assert err.mean(axis=(1, 3, 4)).max() <= MEAN_ABS


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("shape", [
    dict(B=2, Hq=8, Hkv=2, D=64, L=(1, 300), N=37, depth=8),          # GQA, D=64, ragged, odd N
    dict(B=3, Hq=6, Hkv=2, D=128, L=(100, 700), N=130, depth=12, kmax=4, pmax=3),
    dict(B=2, Hq=8, Hkv=1, D=128, L=(0, 65), N=200, depth=14, kmax=4, pmax=3),   # MQA, short prefixes
    dict(B=1, Hq=16, Hkv=2, D=128, L=129, N=512, depth=18, kmax=4, pmax=3),      # maximum N
    dict(B=1, Hq=2, Hkv=2, D=64, L=5, N=1, depth=0),                   # a single node
])
def test_ragged_shapes_nan_padding(shape, kernel):
    base = dict(name="t", config_id=7, kmax=3, pmax=2, V=8, vtok=8, p_agree=0.5)
    cfg = gi.VerifyConfig(**{**base, **shape})
    inp = gi.make_inputs(cfg, 77, accept=False, pad_fill="nan")
    assert_close(out_to_f64(gpu_attn(inp, kernel=kernel)), cpu_attn(inp))


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("Hq,Hkv,N", [(8, 2, 40), (2, 2, 128)])
def test_prefix_lengths_around_the_tile_edges(kernel, Hq, Hkv, N):
    # the last tile of a prefix holds 1, 127, 128 (none ragged), 1, 127, ... keys; NaN behind every
    # sequence end (a tile loaded past the end, or a key of the overlap counted twice, would show)
    lens = np.array([0, 1, 127, 128, 129, 255, 256, 257, 300, 383, 384, 385], dtype=np.int32)
    cfg = gi.VerifyConfig("t", 7, len(lens), Hq, Hkv, 128, 385, N, 8, 3, 2, 8, 8, 0.5)
    inp = gi.make_inputs(cfg, 19, accept=False)
    inp["seq_lens"][:] = lens
    for b, n in enumerate(lens):
        inp["k_cache"][b, int(n):] = 0x7FC0
        inp["v_cache"][b, int(n):] = 0x7FC0
    want = cpu_attn(inp)
    for splits in (0, 2):
        assert_close_scaled(out_to_f64(gpu_attn(inp, kernel=kernel, num_splits=splits)), want)


@pytest.mark.parametrize("kernel", KERNELS)
def test_arbitrary_mask_bits_and_empty_rows(kernel):
    # random bit patterns (not triangular, padding bits set), some rows with no key at all
    cfg = gi.VerifyConfig("t", 7, 2, 8, 4, 128, (0, 40), 70, 8, 3, 2, 8, 8, 0.5)
    inp = gi.make_inputs(cfg, 5, accept=False, pad_fill="nan")
    rng = np.random.default_rng(9)
    inp["ancestor_mask"] = rng.integers(0, 2 ** 32, size=inp["ancestor_mask"].shape, dtype=np.uint32)
    inp["ancestor_mask"][0, 3] = 0
    inp["ancestor_mask"][1, :, :] &= np.uint32(0x00010001)
    inp["seq_lens"][0] = 0
    got = out_to_f64(gpu_attn(inp, kernel=kernel))
    want = cpu_attn(inp)
    assert_close(got, want)
    assert np.all(got[0, 3] == 0)


@pytest.mark.parametrize("kernel", KERNELS)
def test_split_count_invariance_and_determinism(kernel):
    cfg = gi.CONFIGS["llama7b"]
    inp = gi.make_inputs(cfg, accept=False)
    want = cpu_attn(inp)
    outs = {}
    for s in (1, 2, 3, 7):
        outs[s] = gpu_attn(inp, kernel=kernel, num_splits=s)
        assert_close(out_to_f64(outs[s]), want)
        again = gpu_attn(inp, kernel=kernel, num_splits=s)
        assert torch.equal(outs[s], again)                     # bit-identical run to run
    for s in (2, 3, 7):
        assert (outs[s].float() - outs[1].float()).abs().max().item() <= 4e-3


@pytest.mark.parametrize("kernel", KERNELS)
def test_softmax_scale_override(kernel):
    cfg = gi.CONFIGS["tiny"] if kernel == 1 else variant(gi.CONFIGS["tiny"], D=128)
    inp = gi.make_inputs(cfg, accept=False)
    assert_close(out_to_f64(gpu_attn(inp, kernel=kernel, softmax_scale=0.3)), cpu_attn(inp, scale=0.3))


def test_canary_padding_is_untouched():
    import paper_2407_16207_b200 as gsd
    cfg = gi.CONFIGS["tiny"]
    inp = gi.make_inputs(cfg, accept=False)
    t = attn_tensors(inp)
    n = t["q"].numel()
    buf = torch.full((n + 512,), 7.0, dtype=torch.bfloat16, device="cuda")
    out = buf[256:256 + n].view_as(t["q"])
    gsd.gsd_verify_attn(t["q"], t["k_cache"], t["v_cache"], t["draft_k"], t["draft_v"],
                        t["ancestor_mask"], t["seq_lens"], out=out)
    torch.cuda.synchronize()
    assert (buf[:256] == 7.0).all() and (buf[256 + n:] == 7.0).all()


def test_bad_seq_len_is_clamped_and_flagged():
    cfg = gi.CONFIGS["tiny"]
    inp = gi.make_inputs(cfg, accept=False)
    want = cpu_attn(inp)
    inp2 = dict(inp)
    inp2["seq_lens"] = np.array([10_000], dtype=np.int32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = out_to_f64(gpu_attn(inp2, status=status))
    assert int(status.item()) == 0x10
    assert_close(got, want)          # clamped to Lmax == the true length here


def sampled_rows_check(inp, out, rng, n_random=256, node_step=0, units=None):
    """Rows the oracle recomputes one by one: every `node_step`-th node (all GQA heads) of the
    listed (sequence, kv head) units plus `n_random` random rows."""
    cfg = inp["cfg"]
    if units is None:
        units = [(int(rng.integers(cfg.B)), int(rng.integers(cfg.Hkv)))]
    node_step = node_step or max(1, cfg.N // 64)
    rows = [(b0, n, c0 * cfg.G + g) for b0, c0 in units for n in range(0, cfg.N, node_step) for g in range(cfg.G)]
    rows += [(int(rng.integers(cfg.B)), int(rng.integers(cfg.N)), int(rng.integers(cfg.Hq)))
             for _ in range(n_random)]
    want = oracle.attn_rows(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"],
                            inp["draft_v"], inp["ancestor_mask"], inp["seq_lens"], rows)
    idx = torch.tensor(rows, device=out.device, dtype=torch.long)
    assert_close(out_to_f64(out[idx[:, 0], idx[:, 1], idx[:, 2]]), want)


SWEEP_B, SWEEP_L, SWEEP_N = (1, 8, 32), (512, 2048, 8192, 32768), (32, 128, 512)


@pytest.mark.parametrize("L", SWEEP_L)
@pytest.mark.parametrize("B", SWEEP_B)
def test_sweep_points_sampled_rows(B, L):
    # every point of the 70B-shaped sweep (64 q heads over 8 kv heads, D 128; 3 x 4 x 3 = 36
    # points, up to 4.3 GB of KV cache): one whole (sequence, kv head) unit of stacked rows
    # (every node for N = 32, every N/64-th node otherwise, all 8 heads of each) plus 256 random
    # rows, recomputed one by one by the oracle.  The three graph sizes of a (B, L) pair share
    # one KV cache (it is drawn from (seed, B, L) alone).
    first = None
    for N in SWEEP_N:
        cfg = gi.sweep_config(B, L, N)
        inp = gi.make_inputs(cfg, accept=False, kv_from=first)
        first = first or inp
        out = gpu_attn(inp)
        sampled_rows_check(inp, out, np.random.default_rng(B * 1000 + N + L))
        del out
        torch.cuda.empty_cache()


RANDOM_SHAPES = []
_rng = np.random.default_rng(20240716)
for _i in range(24):
    _G = int(_rng.choice([1, 2, 4, 8, 16]))
    _Hkv = int(_rng.choice([1, 2, 3]))
    _N = int(_rng.integers(1, 330))
    _lo = int(_rng.integers(0, 500))
    RANDOM_SHAPES.append((int(_rng.integers(1, 4)), _G * _Hkv, _Hkv, (_lo, _lo + int(_rng.integers(0, 400))), _N,
                          int(_rng.choice([0, 0, 1, 2, 3, 5]))))


@pytest.mark.parametrize("shape", RANDOM_SHAPES, ids=[f"B{b}_Hq{hq}_Hkv{hk}_L{l[0]}-{l[1]}_N{n}_s{sp}" for b, hq, hk, l, n, sp in RANDOM_SHAPES])
def test_random_shapes_full_compare(shape):
    # odd sizes: rows that do not fill a tile, one- and two-row-tile units in one call, empty and
    # ragged prefixes that differ per sequence, one to three draft tiles, forced split counts
    B, Hq, Hkv, L, N, splits = shape
    depth = max(1, min(N - 1, 12)) if N > 1 else 0
    cfg = gi.VerifyConfig("r", 9, B, Hq, Hkv, 128, L, N, depth, 4, 3, 8, 8, 0.5)
    inp = gi.make_inputs(cfg, 1000 + N, accept=False, pad_fill="nan")
    want = cpu_attn(inp)
    for kernel in (0, 2):
        assert_close(out_to_f64(gpu_attn(inp, kernel=kernel, num_splits=splits)), want)


def test_many_units_per_cta_sampled_rows():
    # 4096 units of work for 148 persistent CTAs (about 28 each, more than the kernel decodes up
    # front), short ragged prefix (one partial cache tile) and four draft tiles per unit
    cfg = gi.sweep_config(32, 100, 512)
    inp = gi.make_inputs(cfg, accept=False)
    out = gpu_attn(inp)
    # first, last and a middle (sequence, kv head)
    sampled_rows_check(inp, out, np.random.default_rng(77), n_random=1024, node_step=16,
                       units=[(0, 0), (31, 7), (17, 3)])


def test_dominant_key_and_large_score_jumps():
    # one cache key scores 2^k times above the rest from some tile on: the running maximum has
    # to be raised (accumulator rescale path) and nothing may overflow
    cfg = gi.VerifyConfig("t", 7, 1, 8, 1, 128, 700, 130, 10, 4, 3, 8, 8, 0.5)
    inp = gi.make_inputs(cfg, 3, accept=False)
    k = gi.bf16_bits_to_f32(inp["k_cache"])
    q = gi.bf16_bits_to_f32(inp["q"])
    q[0, :, :, 5] = 24.0
    k[0, :, 0, 5] = 0.0
    k[0, 300, 0, 5] = 6.0          # +144/sqrt(128) = +12.7 in score units at key 300
    k[0, 650, 0, 5] = 24.0         # +50.9 at key 650 (a later tile)
    inp["q"], inp["k_cache"] = gi.f32_to_bf16_bits(q), gi.f32_to_bf16_bits(k)
    dk = gi.bf16_bits_to_f32(inp["draft_k"]); dk[0, :, 0, 5] = 0.0
    inp["draft_k"] = gi.f32_to_bf16_bits(dk)
    want = cpu_attn(inp)
    for kernel in KERNELS:
        assert_close(out_to_f64(gpu_attn(inp, kernel=kernel)), want)
