"""Seeded synthetic inputs for the GSD verification step (shared by the tests, the
benchmark and the CPU checker).

This module only *draws inputs*: draft DAGs with bounded in/out degree, node tokens,
bf16 Q/K/V tensors, prefix lengths and fp32 logits with a planted agreement rate.
It contains none of the method's arithmetic (no attention, no argmax, no path search).
The ancestor bitmask it emits is part of the input format: row n has bit j set iff
draft node j is node n itself or one of its ancestors in the DAG (the "each token only
attends to its ancestors" rule of tree attention, Sec. 4.1, extended to the merged
graph of Sec. 5.3).

The shapes follow LLaMA-2 7B / 13B / 70B attention layers (the models of Sec. 6.1);
they stand in for the paper's GSM8K / XSum / Alpaca / WMT-14 workloads, which are not
used here.

Everything is numpy; bf16 tensors are carried as uint16 bit patterns.
Random numbers come from numpy's Philox counter-based generator keyed by the seed; the
large tensors are drawn slice by slice from jumped copies of their stream, so several host
threads can fill them and the values do not depend on the thread count.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace
from typing import Dict, List, Optional, Sequence, Tuple, Union

import numpy as np

__all__ = [
    "VerifyConfig", "CONFIGS", "sweep_config", "level_sizes", "make_dag", "closure_mask",
    "parents_to_csr", "children_of", "f32_to_bf16_bits", "bf16_bits_to_f32",
    "make_inputs", "seed_for",
]


@dataclass(frozen=True)
class VerifyConfig:
    """One synthetic workload. `L` is a fixed prefix length or an inclusive (lo, hi) range."""
    name: str
    config_id: int
    B: int
    Hq: int
    Hkv: int
    D: int
    L: Union[int, Tuple[int, int]]
    N: int
    depth: int
    kmax: int
    pmax: int
    V: int
    vtok: int          # node tokens are uniform in [0, vtok)
    p_agree: float

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def W(self) -> int:
        return (self.N + 31) // 32


CONFIGS: Dict[str, VerifyConfig] = {
    # tiny case: the CPU checker finishes in well under a second
    "tiny": VerifyConfig("tiny", 1, 1, 4, 4, 64, 128, 16, 5, 3, 2, 1000, 1000, 0.7),
    # LLaMA-2-7B attention layer shape
    "llama7b": VerifyConfig("llama7b", 2, 1, 32, 32, 128, 2048, 64, 8, 3, 2, 32000, 32000, 0.7),
    # LLaMA-2-13B attention layer shape, ragged prefixes
    "llama13b": VerifyConfig("llama13b", 3, 4, 40, 40, 128, (1024, 4096), 128, 12, 4, 3,
                             32000, 32000, 0.6),
    # LLaMA-2-70B GQA attention layer shape
    "llama70b": VerifyConfig("llama70b", 4, 8, 64, 8, 128, 4096, 256, 16, 4, 3, 32000, 32000, 0.7),
}


def sweep_config(B: int, L: int, N: int) -> VerifyConfig:
    """A point of the 70B-shaped sweep: depth = 2*log2(N), degree bounds as in llama70b."""
    depth = 2 * int(round(np.log2(N)))
    return VerifyConfig(f"sweep_B{B}_L{L}_N{N}", 5, B, 64, 8, 128, L, N, depth, 4, 3,
                        32000, 32000, 0.7)


def seed_for(cfg: VerifyConfig, trial: int = 0) -> int:
    return 1000 * cfg.config_id + trial


def _rng(seed: int, stream: int) -> np.random.Generator:
    # one independent Philox stream per tensor so tensors can be regenerated separately
    return np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, stream]))


# ----------------------------------------------------------------------------- bf16
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even. Finite inputs only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------- DAG
def level_sizes(N: int, depth: int, kmax: int) -> List[int]:
    """Sizes of levels 0..depth: one root, the other N-1 nodes spread as evenly as the
    growth bound size(l) <= kmax * size(l-1) allows."""
    if N < 1 or depth < 0:
        raise ValueError("need N >= 1 and depth >= 0")
    sizes = [1]
    remaining = N - 1
    for lvl in range(1, depth + 1):
        left = depth - lvl + 1
        want = -(-remaining // left)
        take = min(want, kmax * sizes[-1])
        sizes.append(take)
        remaining -= take
    if remaining != 0:
        raise ValueError(f"{N} nodes do not fit depth {depth} with out-degree <= {kmax}")
    return sizes


def make_dag(N: int, depth: int, kmax: int, pmax: int, rng: np.random.Generator
             ) -> Tuple[List[List[int]], List[int]]:
    """Level-structured DAG in level (BFS) order, hence topologically numbered.

    Every non-root node first gets one parent drawn uniformly among the previous-level
    nodes that still have fewer than kmax children; then a parent count is drawn
    uniformly in 1..pmax and further distinct previous-level parents are added while
    nodes with spare child capacity remain.  Returns (parents per node sorted ascending,
    level of each node)."""
    sizes = level_sizes(N, depth, kmax)
    parents: List[List[int]] = [[] for _ in range(N)]
    level = [0] * N
    nchild = [0] * N
    start = 1
    prev = [0]
    for lvl in range(1, depth + 1):
        cur = list(range(start, start + sizes[lvl]))
        start += sizes[lvl]
        for v in cur:
            level[v] = lvl
            free = [p for p in prev if nchild[p] < kmax]
            p = free[int(rng.integers(len(free)))]
            parents[v].append(p)
            nchild[p] += 1
        for v in cur:
            want = int(rng.integers(1, pmax + 1))
            while len(parents[v]) < want:
                free = [p for p in prev if nchild[p] < kmax and p not in parents[v]]
                if not free:
                    break
                p = free[int(rng.integers(len(free)))]
                parents[v].append(p)
                nchild[p] += 1
        for v in cur:
            parents[v].sort()
        if cur:
            prev = cur
    return parents, level


def children_of(parents: Sequence[Sequence[int]]) -> List[List[int]]:
    ch: List[List[int]] = [[] for _ in parents]
    for v, ps in enumerate(parents):
        for p in ps:
            ch[p].append(v)
    return ch


def closure_mask(parents: Sequence[Sequence[int]], W: int = 0) -> np.ndarray:
    """[N, W] uint32: bit j of row n (word j // 32, bit j % 32) set iff j == n or j is an
    ancestor of n along any path.  Requires every parent index < child index."""
    N = len(parents)
    W = W or (N + 31) // 32
    anc = [0] * N
    for v in range(N):
        bits = 1 << v
        for p in parents[v]:
            if not 0 <= p < v:
                raise ValueError("parents must precede children")
            bits |= anc[p]
        anc[v] = bits
    out = np.zeros((N, W), dtype=np.uint32)
    for v in range(N):
        for w in range(W):
            out[v, w] = (anc[v] >> (32 * w)) & 0xFFFFFFFF
    return out


def parents_to_csr(parents_per_seq: Sequence[Sequence[Sequence[int]]], Ecap: int = 0
                   ) -> Tuple[np.ndarray, np.ndarray]:
    """Per-sequence parent lists -> (ptr [B, N+1], idx [B, Ecap]) int32; unused idx slots are -1."""
    B = len(parents_per_seq)
    N = len(parents_per_seq[0])
    emax = max(sum(len(p) for p in ps) for ps in parents_per_seq)
    Ecap = max(Ecap, emax, 1)
    ptr = np.zeros((B, N + 1), dtype=np.int32)
    idx = np.full((B, Ecap), -1, dtype=np.int32)
    for b, ps in enumerate(parents_per_seq):
        e = 0
        for v, pv in enumerate(ps):
            ptr[b, v] = e
            for p in pv:
                idx[b, e] = p
                e += 1
        ptr[b, N] = e
    return ptr, idx


# ----------------------------------------------------------------------------- tensors
def _normal_bf16(seed: int, stream: int, shape: Tuple[int, ...]) -> np.ndarray:
    """N(0,1) values rounded to bf16.  Slice i along the first axis is drawn from the Philox
    stream (seed, stream) jumped i times, so the slices can be filled by several host threads
    and the result does not depend on how many there are."""
    out = np.empty(shape, dtype=np.uint16)
    flat = out.reshape(shape[0], -1) if len(shape) > 1 else out.reshape(1, -1)
    base = np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, stream])
    step = 1 << 22                          # the fp32 temporary of a piece stays at 16 MB

    def fill(i: int) -> None:
        g = np.random.Generator(base.jumped(i))
        for a in range(0, flat.shape[1], step):
            b = min(a + step, flat.shape[1])
            flat[i, a:b] = f32_to_bf16_bits(g.standard_normal(b - a, dtype=np.float32))

    workers = min(flat.shape[0], os.cpu_count() or 1)
    if workers <= 1 or flat.size < (1 << 22):
        for i in range(flat.shape[0]):
            fill(i)
    else:
        with ThreadPoolExecutor(max_workers=workers) as ex:
            list(ex.map(fill, range(flat.shape[0])))
    return out


def make_inputs(cfg: VerifyConfig, seed: int | None = None, *, attn: bool = True,
                accept: bool = True, pad_fill: str = "junk",
                kv_from: Optional[Dict[str, object]] = None) -> Dict[str, object]:
    """Draw one batch for `cfg`.

    Keys: cfg, seed, parents (list per sequence), levels, draft_tokens [B,N] i32,
    parent_ptr [B,N+1] i32, parent_idx [B,Ecap] i32, ancestor_mask [B,N,W] u32,
    seq_lens [B] i32, Lmax; with attn: q [B,N,Hq,D], k_cache/v_cache [B,Lmax,Hkv,D],
    draft_k/draft_v [B,N,Hkv,D] (uint16 bf16 bits); with accept: logits [B,N,V] f32.

    pad_fill: what cache rows at positions >= seq_lens[b] hold: "junk" (large finite
    values of random sign), "nan" (quiet-NaN patterns) or "zero".
    kv_from: an earlier batch drawn with the same seed, B, Hkv, D, prefix lengths and pad_fill;
    its k_cache / v_cache arrays are used as they are instead of being drawn a second time
    (the draw depends on nothing else, so they would come out identical).
    """
    if seed is None:
        seed = seed_for(cfg)
    B, N, Hq, Hkv, D, V = cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D, cfg.V
    g_dag = _rng(seed, 1)
    parents_all, levels_all = [], []
    for _ in range(B):
        ps, lv = make_dag(N, cfg.depth, cfg.kmax, cfg.pmax, g_dag)
        parents_all.append(ps)
        levels_all.append(lv)
    tokens = _rng(seed, 2).integers(0, cfg.vtok, size=(B, N), dtype=np.int32)
    ptr, idx = parents_to_csr(parents_all)
    mask = np.stack([closure_mask(ps, cfg.W) for ps in parents_all])
    if isinstance(cfg.L, tuple):
        seq_lens = _rng(seed, 3).integers(cfg.L[0], cfg.L[1] + 1, size=B, dtype=np.int32)
    else:
        seq_lens = np.full(B, cfg.L, dtype=np.int32)
    Lmax = int(seq_lens.max()) if B else 0
    out: Dict[str, object] = dict(cfg=cfg, seed=seed, parents=parents_all, levels=levels_all,
                                  draft_tokens=tokens, parent_ptr=ptr, parent_idx=idx,
                                  ancestor_mask=mask, seq_lens=seq_lens, Lmax=Lmax)
    if attn:
        out["q"] = _normal_bf16(seed, 4, (B, N, Hq, D))
        if kv_from is not None:
            kc, vc = kv_from["k_cache"], kv_from["v_cache"]
            if (kv_from["seed"] != seed or kc.shape != (B, max(Lmax, 1), Hkv, D)
                    or not np.array_equal(kv_from["seq_lens"], seq_lens)):
                raise ValueError("kv_from was drawn for another cache shape or seed")
        else:
            kc = _normal_bf16(seed, 5, (B, max(Lmax, 1), Hkv, D))
            vc = _normal_bf16(seed, 6, (B, max(Lmax, 1), Hkv, D))
        g_pad = _rng(seed, 9)
        for b in range(B):
            n_pad = kc.shape[1] - int(seq_lens[b])
            if n_pad <= 0 or kv_from is not None:
                continue
            shp = (n_pad, Hkv, D)
            if pad_fill == "junk":
                sign = g_pad.integers(0, 2, size=shp).astype(np.float32) * 2 - 1
                fill = f32_to_bf16_bits(sign * np.float32(3.0e37))
            elif pad_fill == "nan":
                fill = np.full(shp, 0x7FC0, dtype=np.uint16)
            elif pad_fill == "zero":
                fill = np.zeros(shp, dtype=np.uint16)
            else:
                raise ValueError(pad_fill)
            kc[b, int(seq_lens[b]):] = fill
            vc[b, int(seq_lens[b]):] = fill
        out["k_cache"], out["v_cache"] = kc, vc
        out["draft_k"] = _normal_bf16(seed, 7, (B, N, Hkv, D))
        out["draft_v"] = _normal_bf16(seed, 8, (B, N, Hkv, D))
    if accept:
        logits = np.empty((B, N, V), dtype=np.float32)
        base = np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, 10])

        def fill_logits(b: int) -> None:      # sequence b: the stream (seed, 10) jumped b times
            np.random.Generator(base.jumped(b)).standard_normal((N, V), dtype=np.float32, out=logits[b])

        if B > 1 and logits.size >= (1 << 22):
            with ThreadPoolExecutor(max_workers=min(B, os.cpu_count() or 1)) as ex:
                list(ex.map(fill_logits, range(B)))
        else:
            for b in range(B):
                fill_logits(b)
        g_pl = _rng(seed, 11)
        for b in range(B):
            ch = children_of(parents_all[b])
            for v in range(N):
                if ch[v] and g_pl.random() < cfg.p_agree:
                    c = ch[v][int(g_pl.integers(len(ch[v])))]
                    logits[b, v, tokens[b, c]] = 12.0
        out["logits"] = logits
    return out
