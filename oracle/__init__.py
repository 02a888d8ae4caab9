"""ctypes front end of the CPU oracle (`gsd_oracle.c`).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline
leg may import this; the product package never does.  It shares nothing with the CUDA
path.  See the header of `gsd_oracle.c` for what is computed and which passages of the
paper it follows (Sec. 3 deterministic verification, Sec. 4.1 tree attention and
longest-path selection, Sec. 5.3 merged token graph).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# GSD_ORACLE_SRC / GSD_ORACLE_LIB let the mutation tests point this loader at a deliberately
# broken copy of the source (to show that the pins notice); nothing else uses them.
_SRC = os.environ.get("GSD_ORACLE_SRC", os.path.join(_HERE, "gsd_oracle.c"))
_LIB = os.environ.get("GSD_ORACLE_LIB", os.path.join(_HERE, "_gsd_oracle.so"))
_lib: Optional[ctypes.CDLL] = None


class _Dims(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("N", ctypes.c_int32), ("Hq", ctypes.c_int32),
                ("Hkv", ctypes.c_int32), ("D", ctypes.c_int32), ("Lmax", ctypes.c_int32),
                ("scale", ctypes.c_double)]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over independent output rows) if it is stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
           "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.gsd_oracle_threads.restype = ctypes.c_int
        _lib.gsd_oracle_argmax_row.restype = ctypes.c_int32
        for name in ("gsd_oracle_attn", "gsd_oracle_attn_rows", "gsd_oracle_accept", "gsd_oracle_accept_sampled", "gsd_oracle_draft_expand",
                     "gsd_oracle_commit_kv", "gsd_oracle_build_mask", "gsd_oracle_unmerge_tree"):
            getattr(_lib, name).restype = ctypes.c_int
        _lib.gsd_oracle_argmax.restype = None
    return _lib


def threads() -> int:
    return int(_load().gsd_oracle_threads())


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _attn_args(q, k_cache, v_cache, draft_k, draft_v, ancestor_mask, seq_lens, scale):
    q = _c(q, np.uint16); k_cache = _c(k_cache, np.uint16); v_cache = _c(v_cache, np.uint16)
    draft_k = _c(draft_k, np.uint16); draft_v = _c(draft_v, np.uint16)
    ancestor_mask = _c(ancestor_mask, np.uint32); seq_lens = _c(seq_lens, np.int32)
    B, N, Hq, D = q.shape
    _, Lmax, Hkv, _ = k_cache.shape
    assert v_cache.shape == k_cache.shape
    assert draft_k.shape == (B, N, Hkv, D) and draft_v.shape == (B, N, Hkv, D)
    assert ancestor_mask.shape == (B, N, (N + 31) // 32)
    assert seq_lens.shape == (B,) and (seq_lens >= 0).all() and (seq_lens <= Lmax).all()
    assert Hq % Hkv == 0
    dims = _Dims(B, N, Hq, Hkv, D, Lmax, float(scale) if scale else 0.0)
    keep = (q, k_cache, v_cache, draft_k, draft_v, ancestor_mask, seq_lens)
    return dims, keep


def attn(q, k_cache, v_cache, draft_k, draft_v, ancestor_mask, seq_lens, scale: float = 0.0
         ) -> np.ndarray:
    """fp64 DAG-masked attention; bf16 inputs as uint16 bit patterns. Returns [B,N,Hq,D] f64."""
    dims, keep = _attn_args(q, k_cache, v_cache, draft_k, draft_v, ancestor_mask, seq_lens, scale)
    out = np.zeros(keep[0].shape, dtype=np.float64)
    rc = _load().gsd_oracle_attn(ctypes.byref(dims), *[_p(a) for a in keep], _p(out))
    if rc != 0:
        raise RuntimeError("oracle attention failed")
    return out


def attn_rows(q, k_cache, v_cache, draft_k, draft_v, ancestor_mask, seq_lens,
              rows: Sequence[Sequence[int]], scale: float = 0.0) -> np.ndarray:
    """Same as `attn` for the listed (b, n, h) rows only. Returns [len(rows), D] f64."""
    dims, keep = _attn_args(q, k_cache, v_cache, draft_k, draft_v, ancestor_mask, seq_lens, scale)
    rows = _c(rows, np.int32).reshape(-1, 3)
    out = np.zeros((rows.shape[0], dims.D), dtype=np.float64)
    rc = _load().gsd_oracle_attn_rows(ctypes.byref(dims), *[_p(a) for a in keep], _p(rows),
                                      ctypes.c_long(rows.shape[0]), _p(out))
    if rc != 0:
        raise RuntimeError("oracle attention failed")
    return out


def argmax(logits) -> np.ndarray:
    """Row-wise argmax over the last axis, ties to the lowest index, NaN never wins."""
    logits = _c(logits, np.float32)
    V = logits.shape[-1]
    rows = logits.size // V if V else 0
    out = np.zeros(logits.shape[:-1], dtype=np.int32)
    _load().gsd_oracle_argmax(_p(logits), ctypes.c_long(rows), ctypes.c_int32(V), _p(out))
    return out


def accept(logits, draft_tokens, parent_ptr, parent_idx, Tcap: int = 0, visit_cap: int = 0):
    """Brute-force longest accepted path.

    Returns (accepted_tokens [B,Tcap] padded with -1, accepted_len [B],
    accepted_nodes [B,Tcap] padded with -1, paths_visited [B]; a negative count means the
    walk stopped extending rejected paths after `visit_cap` paths)."""
    logits = _c(logits, np.float32); draft_tokens = _c(draft_tokens, np.int32)
    parent_ptr = _c(parent_ptr, np.int32); parent_idx = _c(parent_idx, np.int32)
    B, N, V = logits.shape
    assert draft_tokens.shape == (B, N) and parent_ptr.shape == (B, N + 1)
    Ecap = parent_idx.shape[1]
    Tcap = Tcap or N
    toks = np.zeros((B, Tcap), dtype=np.int32)
    lens = np.zeros((B,), dtype=np.int32)
    nodes = np.zeros((B, Tcap), dtype=np.int32)
    visited = np.zeros((B,), dtype=np.int64)
    rc = _load().gsd_oracle_accept(_p(logits), _p(draft_tokens), _p(parent_ptr), _p(parent_idx),
                                   ctypes.c_int32(B), ctypes.c_int32(N), ctypes.c_int32(V),
                                   ctypes.c_int32(Ecap), ctypes.c_int32(Tcap), _p(toks), _p(lens),
                                   _p(nodes), _p(visited), ctypes.c_int64(visit_cap))
    if rc != 0:
        raise ValueError("oracle accept: malformed DAG or Tcap too small")
    return toks, lens, nodes, visited


def accept_sampled(logits, draft_tokens, parent_ptr, parent_idx, draft_q, u_accept, u_sample, Tcap: int = 0,
                   draft_logits=None):
    """Non-deterministic verification with the random numbers passed in (see gsd_oracle_accept_sampled).
    With `draft_logits` [B,N,V] the regenerated token after a rejection comes from the residual
    max(0, P - Q) of the end node; without it, from the target distribution P.

    Returns (accepted_tokens [B,Tcap] padded with -1, accepted_len [B], accepted_nodes [B,Tcap])."""
    logits = _c(logits, np.float32); draft_tokens = _c(draft_tokens, np.int32)
    parent_ptr = _c(parent_ptr, np.int32); parent_idx = _c(parent_idx, np.int32)
    draft_q = _c(draft_q, np.float32); u_accept = _c(u_accept, np.float32); u_sample = _c(u_sample, np.float32)
    B, N, V = logits.shape
    assert draft_tokens.shape == (B, N) and parent_ptr.shape == (B, N + 1)
    assert draft_q.shape == (B, N) and u_accept.shape == (B, N) and u_sample.shape == (B,)
    if draft_logits is not None:
        draft_logits = _c(draft_logits, np.float32)
        assert draft_logits.shape == (B, N, V)
    Ecap = parent_idx.shape[1]
    Tcap = Tcap or N
    toks = np.zeros((B, Tcap), dtype=np.int32)
    lens = np.zeros((B,), dtype=np.int32)
    nodes = np.zeros((B, Tcap), dtype=np.int32)
    rc = _load().gsd_oracle_accept_sampled(_p(logits), _p(draft_tokens), _p(parent_ptr), _p(parent_idx),
                                           _p(draft_logits) if draft_logits is not None else None,
                                           _p(draft_q), _p(u_accept), _p(u_sample),
                                           ctypes.c_int32(B), ctypes.c_int32(N), ctypes.c_int32(V),
                                           ctypes.c_int32(Ecap), ctypes.c_int32(Tcap), _p(toks), _p(lens), _p(nodes))
    if rc != 0:
        raise ValueError("oracle accept_sampled: malformed DAG or Tcap too small")
    return toks, lens, nodes


def draft_expand(logits, frontier, frontier_len, tokens, tree_parent, merge_to, leaf, prob, num_nodes,
                 k: int, tau: int, theta_prob: float, theta_sib: float):
    """One growth step of the draft token graph (see gsd_oracle_draft_expand).  The graph arrays
    are copied; returns (tokens, tree_parent, merge_to, leaf, prob, num_nodes, new_frontier
    [B,F*k] padded with -1, new_frontier_len [B], out_of_capacity flag)."""
    logits = _c(logits, np.float32); frontier = _c(frontier, np.int32); frontier_len = _c(frontier_len, np.int32)
    tokens = _c(tokens, np.int32).copy(); tree_parent = _c(tree_parent, np.int32).copy()
    merge_to = _c(merge_to, np.int32).copy(); leaf = _c(leaf, np.uint8).copy()
    prob = _c(prob, np.float32).copy(); num_nodes = _c(num_nodes, np.int32).copy()
    B, F, V = logits.shape
    Ncap = tokens.shape[1]
    assert frontier.shape == (B, F) and frontier_len.shape == (B,)
    for a in (tree_parent, merge_to, leaf, prob):
        assert a.shape == (B, Ncap)
    nf = np.full((B, F * k), -1, dtype=np.int32)
    nfl = np.zeros((B,), dtype=np.int32)
    rc = _load().gsd_oracle_draft_expand(_p(logits), _p(frontier), _p(frontier_len), _p(tokens), _p(tree_parent),
                                         _p(merge_to), _p(leaf), _p(prob), _p(num_nodes), _p(nf), _p(nfl),
                                         ctypes.c_int32(B), ctypes.c_int32(F), ctypes.c_int32(V), ctypes.c_int32(Ncap),
                                         ctypes.c_int32(k), ctypes.c_int32(tau), ctypes.c_double(theta_prob),
                                         ctypes.c_double(theta_sib))
    if rc < 0:
        raise ValueError("oracle draft_expand: malformed input")
    return tokens, tree_parent, merge_to, leaf, prob, num_nodes, nf, nfl, bool(rc & 1)


def commit_kv(k_cache, v_cache, draft_k, draft_v, accepted_nodes, accepted_len, seq_lens):
    """Append the draft K/V rows of the accepted path to the cache (copies of the inputs are
    modified and returned).  Returns (k_cache, v_cache, seq_lens, number of sequences that hit Lmax)."""
    k_cache = _c(k_cache, np.uint16).copy(); v_cache = _c(v_cache, np.uint16).copy()
    draft_k = _c(draft_k, np.uint16); draft_v = _c(draft_v, np.uint16)
    accepted_nodes = _c(accepted_nodes, np.int32); accepted_len = _c(accepted_len, np.int32)
    seq_lens = _c(seq_lens, np.int32).copy()
    B, Lmax, Hkv, D = k_cache.shape
    N = draft_k.shape[1]
    Tcap = accepted_nodes.shape[1]
    assert draft_k.shape == (B, N, Hkv, D) and v_cache.shape == k_cache.shape
    rc = _load().gsd_oracle_commit_kv(_p(k_cache), _p(v_cache), _p(draft_k), _p(draft_v),
                                      _p(accepted_nodes), _p(accepted_len), _p(seq_lens),
                                      ctypes.c_int32(B), ctypes.c_int32(N), ctypes.c_int32(Hkv),
                                      ctypes.c_int32(D), ctypes.c_int32(Lmax), ctypes.c_int32(Tcap))
    return k_cache, v_cache, seq_lens, int(rc)


def build_mask(parent_ptr, parent_idx) -> np.ndarray:
    """Ancestor bitmask [B,N,ceil(N/32)] uint32 (self bit included) from the parent CSR."""
    parent_ptr = _c(parent_ptr, np.int32); parent_idx = _c(parent_idx, np.int32)
    B, N1 = parent_ptr.shape
    N = N1 - 1
    mask = np.zeros((B, N, (N + 31) // 32), dtype=np.uint32)
    rc = _load().gsd_oracle_build_mask(_p(parent_ptr), _p(parent_idx), ctypes.c_int32(B),
                                       ctypes.c_int32(N), ctypes.c_int32(parent_idx.shape[1]), _p(mask))
    if rc != 0:
        raise RuntimeError("oracle build_mask failed")
    return mask


def unmerge_tree(draft_tokens, parent_ptr, parent_idx, Ucap: int, max_depth: int):
    """The token graph unfolded into a tree, one node per root path (see gsd_oracle_unmerge_tree).
    Returns (tree_tokens, tree_parent, tree_source [B,Ucap] padded with -1, tree_count [B],
    out_of_capacity flag)."""
    draft_tokens = _c(draft_tokens, np.int32); parent_ptr = _c(parent_ptr, np.int32)
    parent_idx = _c(parent_idx, np.int32)
    B, N = draft_tokens.shape
    assert parent_ptr.shape == (B, N + 1)
    tt = np.zeros((B, Ucap), dtype=np.int32); tp = np.zeros((B, Ucap), dtype=np.int32)
    ts = np.zeros((B, Ucap), dtype=np.int32); cnt = np.zeros((B,), dtype=np.int32)
    rc = _load().gsd_oracle_unmerge_tree(_p(draft_tokens), _p(parent_ptr), _p(parent_idx), ctypes.c_int32(B),
                                         ctypes.c_int32(N), ctypes.c_int32(parent_idx.shape[1]),
                                         ctypes.c_int32(Ucap), ctypes.c_int32(max_depth), _p(tt), _p(tp), _p(ts),
                                         _p(cnt))
    if rc < 0:
        raise ValueError("oracle unmerge_tree: malformed input")
    return tt, tp, ts, cnt, bool(rc)
