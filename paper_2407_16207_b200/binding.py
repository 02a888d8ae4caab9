"""ctypes binding of libgsd.so with the same names as the C ABI (include/gsd.h).

The functions take torch tensors (CUDA tensors for the device calls, CPU tensors for the
host-buffer step), check dtype / shape / contiguity, and pass raw pointers, sizes and the
current CUDA stream.  PyTorch is used for memory and streams only.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

GSD_ATTN_AUTO, GSD_ATTN_MMA, GSD_ATTN_TCGEN05 = 0, 1, 2
GSD_ATTN_SPLIT_BALANCED = -1      # num_splits: equal shares of key tiles per CTA, dealt out on the device
GSD_ATTN_SPLIT_PER_SEQUENCE = -2  # num_splits: a split count per sequence, chosen on the device

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libgsd.so")
_lib: Optional[ctypes.CDLL] = None


class GsdError(RuntimeError):
    """A negative gsd_status returned by the library."""

    def __init__(self, code: int, what: str):
        super().__init__(what)
        self.code = code


class AttnParams(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("N", ctypes.c_int32), ("Hq", ctypes.c_int32),
                ("Hkv", ctypes.c_int32), ("D", ctypes.c_int32), ("Lmax", ctypes.c_int32),
                ("softmax_scale", ctypes.c_float), ("num_splits", ctypes.c_int32),
                ("kernel", ctypes.c_int32)]


class CommitParams(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("N", ctypes.c_int32), ("Hkv", ctypes.c_int32),
                ("D", ctypes.c_int32), ("Lmax", ctypes.c_int32), ("Tcap", ctypes.c_int32)]


class AcceptParams(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("N", ctypes.c_int32), ("V", ctypes.c_int32),
                ("Ecap", ctypes.c_int32), ("Tcap", ctypes.c_int32)]


class DraftParams(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("F", ctypes.c_int32), ("V", ctypes.c_int32),
                ("Ncap", ctypes.c_int32), ("k", ctypes.c_int32), ("tau", ctypes.c_int32),
                ("theta_prob", ctypes.c_float), ("theta_sib", ctypes.c_float)]


EXPORTS = ["gsd_version", "gsd_status_string", "gsd_last_cuda_error", "gsd_debug_attn_wait", "gsd_verify_attn",
           "gsd_verify_attn_workspace_bytes", "gsd_verify_attn_num_splits", "gsd_accept",
           "gsd_accept_workspace_bytes", "gsd_accept_static", "gsd_accept_sampled",
           "gsd_accept_sampled_workspace_bytes", "gsd_draft_expand", "gsd_draft_expand_workspace_bytes",
           "gsd_commit_kv", "gsd_build_mask", "gsd_unmerge_tree", "gsd_verify_step_host",
           "gsd_verify_step_host_arena_bytes"]


def library_path() -> str:
    return _LIB_PATH


def lib() -> ctypes.CDLL:
    """Load libgsd.so (built in-tree by paper_2407_16207_b200/build.py). No fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise GsdError(-100, f"{_LIB_PATH} is missing: run `python -m paper_2407_16207_b200.build` "
                                 "(there is no CPU fallback)")
        L = ctypes.CDLL(_LIB_PATH)
        vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        L.gsd_version.restype = i32
        L.gsd_status_string.restype = ctypes.c_char_p
        L.gsd_status_string.argtypes = [i32]
        L.gsd_last_cuda_error.restype = ctypes.c_char_p
        L.gsd_debug_attn_wait.restype = None
        L.gsd_debug_attn_wait.argtypes = [ctypes.c_uint64, ctypes.c_int32]
        L.gsd_verify_attn.restype = i32
        L.gsd_verify_attn.argtypes = [vp] * 8 + [ctypes.POINTER(AttnParams), vp, sz, vp, vp]
        L.gsd_verify_attn_workspace_bytes.restype = sz
        L.gsd_verify_attn_workspace_bytes.argtypes = [ctypes.POINTER(AttnParams)]
        L.gsd_verify_attn_num_splits.restype = i32
        L.gsd_verify_attn_num_splits.argtypes = [ctypes.POINTER(AttnParams)]
        L.gsd_accept.restype = i32
        L.gsd_accept.argtypes = [vp] * 7 + [ctypes.POINTER(AcceptParams), vp, sz, vp, vp]
        L.gsd_accept_sampled.restype = i32
        L.gsd_accept_sampled.argtypes = [vp] * 11 + [ctypes.POINTER(AcceptParams), vp, sz, vp, vp]
        L.gsd_accept_sampled_workspace_bytes.restype = sz
        L.gsd_accept_sampled_workspace_bytes.argtypes = [ctypes.POINTER(AcceptParams)]
        L.gsd_draft_expand.restype = i32
        L.gsd_draft_expand.argtypes = [vp] * 11 + [ctypes.POINTER(DraftParams), vp, sz, vp, vp]
        L.gsd_draft_expand_workspace_bytes.restype = sz
        L.gsd_draft_expand_workspace_bytes.argtypes = [ctypes.POINTER(DraftParams)]
        L.gsd_accept_static.restype = i32
        L.gsd_accept_static.argtypes = [vp] * 7 + [ctypes.POINTER(AcceptParams), vp, vp]
        L.gsd_build_mask.restype = i32
        L.gsd_build_mask.argtypes = [vp, vp, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp]
        L.gsd_unmerge_tree.restype = i32
        L.gsd_unmerge_tree.argtypes = [vp] * 7 + [ctypes.c_int32] * 5 + [vp, vp]
        L.gsd_commit_kv.restype = i32
        L.gsd_commit_kv.argtypes = [vp] * 7 + [ctypes.POINTER(CommitParams), vp, vp]
        L.gsd_accept_workspace_bytes.restype = sz
        L.gsd_accept_workspace_bytes.argtypes = [ctypes.POINTER(AcceptParams)]
        L.gsd_verify_step_host.restype = i32
        L.gsd_verify_step_host.argtypes = ([vp] * 8 + [ctypes.POINTER(AttnParams)] + [vp] * 7
                                           + [ctypes.POINTER(AcceptParams), vp, sz, vp, vp])
        L.gsd_verify_step_host_arena_bytes.restype = sz
        L.gsd_verify_step_host_arena_bytes.argtypes = [ctypes.POINTER(AttnParams),
                                                       ctypes.POINTER(AcceptParams)]
        _lib = L
    return _lib


def _check(rc: int) -> None:
    if rc != 0:
        L = lib()
        msg = L.gsd_status_string(rc).decode()
        detail = L.gsd_last_cuda_error().decode()
        if rc == -5 or (rc == -4 and detail.startswith("gsd_accept_static")):
            msg += ": " + detail
        raise GsdError(rc, f"gsd error {rc}: {msg}")


def gsd_version() -> int:
    return int(lib().gsd_version())


def gsd_debug_attn_wait(limit_ns: int = 0, withhold_first_k: bool = False) -> None:
    """Test hook for the bounded in-kernel waits of the tcgen05 attention kernel; see
    gsd_debug_attn_wait in include/gsd.h.  (0, False) restores the defaults."""
    lib().gsd_debug_attn_wait(int(limit_ns), 1 if withhold_first_k else 0)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _want(t: torch.Tensor, dtype, shape, name: str, cuda: bool) -> None:
    if t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
        raise ValueError(f"{name}: expected contiguous {dtype} {tuple(shape)}, got {t.dtype} "
                         f"{tuple(t.shape)}")
    if t.is_cuda != cuda:
        raise ValueError(f"{name}: expected a {'CUDA' if cuda else 'CPU'} tensor")


def _stream(t: torch.Tensor) -> int:
    return torch.cuda.current_stream(t.device).cuda_stream


def _attn_params(q, k_cache, draft_k, softmax_scale, num_splits, kernel) -> AttnParams:
    B, N, Hq, D = q.shape
    Lmax, Hkv = k_cache.shape[1], k_cache.shape[2]
    return AttnParams(B, N, Hq, Hkv, D, Lmax, float(softmax_scale), int(num_splits), int(kernel))


def _check_attn_tensors(q, k_cache, v_cache, draft_k, draft_v, ancestor_mask, seq_lens, cuda):
    bf = torch.bfloat16
    if q.dim() != 4 or k_cache.dim() != 4:
        raise ValueError("q must be [B,N,Hq,D] and k_cache [B,Lmax,Hkv,D]")
    B, N, Hq, D = q.shape
    Lmax, Hkv = k_cache.shape[1], k_cache.shape[2]
    _want(q, bf, (B, N, Hq, D), "q", cuda)
    _want(k_cache, bf, (B, Lmax, Hkv, D), "k_cache", cuda)
    _want(v_cache, bf, (B, Lmax, Hkv, D), "v_cache", cuda)
    _want(draft_k, bf, (B, N, Hkv, D), "draft_k", cuda)
    _want(draft_v, bf, (B, N, Hkv, D), "draft_v", cuda)
    if ancestor_mask.dtype not in (torch.int32, torch.uint32):
        raise ValueError("ancestor_mask must hold 32-bit words (int32 or uint32)")
    _want(ancestor_mask, ancestor_mask.dtype, (B, N, (N + 31) // 32), "ancestor_mask", cuda)
    _want(seq_lens, torch.int32, (B,), "seq_lens", cuda)


def gsd_verify_attn_num_splits(B, N, Hq, Hkv, D, Lmax, num_splits=0, kernel=GSD_ATTN_AUTO) -> int:
    p = AttnParams(B, N, Hq, Hkv, D, Lmax, 0.0, num_splits, kernel)
    return int(lib().gsd_verify_attn_num_splits(ctypes.byref(p)))


def gsd_verify_attn_workspace_bytes(B, N, Hq, Hkv, D, Lmax, num_splits=0,
                                    kernel=GSD_ATTN_AUTO) -> int:
    p = AttnParams(B, N, Hq, Hkv, D, Lmax, 0.0, num_splits, kernel)
    return int(lib().gsd_verify_attn_workspace_bytes(ctypes.byref(p)))


def gsd_verify_attn(q, k_cache, v_cache, draft_k, draft_v, ancestor_mask, seq_lens,
                    out: Optional[torch.Tensor] = None, *, softmax_scale: float = 0.0,
                    num_splits: int = 0, kernel: int = GSD_ATTN_AUTO,
                    workspace: Optional[torch.Tensor] = None,
                    status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """DAG-masked attention of the draft nodes; see gsd_verify_attn in include/gsd.h.
    Enqueued on the current stream; returns `out` [B,N,Hq,D] bf16."""
    _check_attn_tensors(q, k_cache, v_cache, draft_k, draft_v, ancestor_mask, seq_lens, True)
    if out is None:
        out = torch.empty_like(q)
    _want(out, torch.bfloat16, q.shape, "out", True)
    p = _attn_params(q, k_cache, draft_k, softmax_scale, num_splits, kernel)
    L = lib()
    with torch.cuda.device(q.device):
        need = int(L.gsd_verify_attn_workspace_bytes(ctypes.byref(p)))
        if workspace is None and need:
            workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        _check(L.gsd_verify_attn(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(),
                                 draft_k.data_ptr(), draft_v.data_ptr(), ancestor_mask.data_ptr(),
                                 seq_lens.data_ptr(), out.data_ptr(), ctypes.byref(p),
                                 _ptr(workspace), ws_bytes, _ptr(status), _stream(q)))
    return out


def gsd_accept_workspace_bytes(B, N, V=1, Ecap=1, Tcap=1) -> int:
    p = AcceptParams(B, N, V, Ecap, Tcap)
    return int(lib().gsd_accept_workspace_bytes(ctypes.byref(p)))


def gsd_accept(logits, draft_tokens, parent_ptr, parent_idx, *, Tcap: int = 0,
               want_nodes: bool = True, workspace: Optional[torch.Tensor] = None,
               status: Optional[torch.Tensor] = None,
               out: Optional[Tuple[torch.Tensor, torch.Tensor, Optional[torch.Tensor]]] = None
               ) -> Tuple[torch.Tensor, torch.Tensor, Optional[torch.Tensor]]:
    """Greedy verification + longest accepted path; see gsd_accept in include/gsd.h.
    Returns (accepted_tokens [B,Tcap], accepted_len [B], accepted_nodes [B,Tcap] or None)."""
    if logits.dim() != 3:
        raise ValueError("logits must be [B,N,V]")
    B, N, V = logits.shape
    _want(logits, torch.float32, (B, N, V), "logits", True)
    _want(draft_tokens, torch.int32, (B, N), "draft_tokens", True)
    _want(parent_ptr, torch.int32, (B, N + 1), "parent_ptr", True)
    if parent_idx.dim() != 2:
        raise ValueError("parent_idx must be [B,Ecap]")
    Ecap = parent_idx.shape[1]
    _want(parent_idx, torch.int32, (B, Ecap), "parent_idx", True)
    Tcap = Tcap or N
    if out is None:
        toks = torch.empty((B, Tcap), dtype=torch.int32, device=logits.device)
        lens = torch.empty((B,), dtype=torch.int32, device=logits.device)
        nodes = torch.empty((B, Tcap), dtype=torch.int32, device=logits.device) if want_nodes else None
    else:
        toks, lens, nodes = out
    p = AcceptParams(B, N, V, Ecap, Tcap)
    L = lib()
    with torch.cuda.device(logits.device):
        need = int(L.gsd_accept_workspace_bytes(ctypes.byref(p)))
        if workspace is None:
            workspace = torch.empty(max(need, 8), dtype=torch.uint8, device=logits.device)
        _check(L.gsd_accept(logits.data_ptr(), draft_tokens.data_ptr(), parent_ptr.data_ptr(),
                            parent_idx.data_ptr(), toks.data_ptr(), lens.data_ptr(), _ptr(nodes),
                            ctypes.byref(p), workspace.data_ptr(),
                            workspace.numel() * workspace.element_size(), _ptr(status),
                            _stream(logits)))
    return toks, lens, nodes


def gsd_accept_sampled_workspace_bytes(B, N) -> int:
    p = AcceptParams(B, N, 1, 1, 1)
    return int(lib().gsd_accept_sampled_workspace_bytes(ctypes.byref(p)))


def gsd_accept_sampled(logits, draft_tokens, parent_ptr, parent_idx, draft_q, u_accept, u_sample, *,
                       draft_logits: Optional[torch.Tensor] = None,
                       Tcap: int = 0, want_nodes: bool = True, workspace: Optional[torch.Tensor] = None,
                       status: Optional[torch.Tensor] = None,
                       out: Optional[Tuple[torch.Tensor, torch.Tensor, Optional[torch.Tensor]]] = None
                       ) -> Tuple[torch.Tensor, torch.Tensor, Optional[torch.Tensor]]:
    """Non-deterministic verification with the random numbers passed in; see gsd_accept_sampled in
    include/gsd.h.  `draft_logits` [B,N,V] (optional) makes the regenerated token come from the
    residual max(0, P - Q).  Returns (accepted_tokens [B,Tcap], accepted_len [B], accepted_nodes
    or None)."""
    if logits.dim() != 3:
        raise ValueError("logits must be [B,N,V]")
    B, N, V = logits.shape
    _want(logits, torch.float32, (B, N, V), "logits", True)
    _want(draft_tokens, torch.int32, (B, N), "draft_tokens", True)
    _want(parent_ptr, torch.int32, (B, N + 1), "parent_ptr", True)
    if parent_idx.dim() != 2:
        raise ValueError("parent_idx must be [B,Ecap]")
    Ecap = parent_idx.shape[1]
    _want(parent_idx, torch.int32, (B, Ecap), "parent_idx", True)
    _want(draft_q, torch.float32, (B, N), "draft_q", True)
    _want(u_accept, torch.float32, (B, N), "u_accept", True)
    _want(u_sample, torch.float32, (B,), "u_sample", True)
    if draft_logits is not None:
        _want(draft_logits, torch.float32, (B, N, V), "draft_logits", True)
    Tcap = Tcap or N
    if out is None:
        toks = torch.empty((B, Tcap), dtype=torch.int32, device=logits.device)
        lens = torch.empty((B,), dtype=torch.int32, device=logits.device)
        nodes = torch.empty((B, Tcap), dtype=torch.int32, device=logits.device) if want_nodes else None
    else:
        toks, lens, nodes = out
        _want(toks, torch.int32, (B, Tcap), "accepted_tokens", True)
        _want(lens, torch.int32, (B,), "accepted_len", True)
    p = AcceptParams(B, N, V, Ecap, Tcap)
    L = lib()
    with torch.cuda.device(logits.device):
        need = int(L.gsd_accept_sampled_workspace_bytes(ctypes.byref(p)))
        if workspace is None:
            workspace = torch.empty(max(need, 8), dtype=torch.uint8, device=logits.device)
        _check(L.gsd_accept_sampled(logits.data_ptr(), draft_tokens.data_ptr(), parent_ptr.data_ptr(),
                                    parent_idx.data_ptr(), _ptr(draft_logits), draft_q.data_ptr(),
                                    u_accept.data_ptr(),
                                    u_sample.data_ptr(), toks.data_ptr(), lens.data_ptr(), _ptr(nodes),
                                    ctypes.byref(p), workspace.data_ptr(),
                                    workspace.numel() * workspace.element_size(), _ptr(status),
                                    _stream(logits)))
    return toks, lens, nodes


def gsd_draft_expand(logits, frontier, frontier_len, tokens, tree_parent, merge_to, leaf, prob, num_nodes, *,
                     k: int, tau: int, theta_prob: float, theta_sib: float,
                     workspace: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None,
                     out: Optional[Tuple[torch.Tensor, torch.Tensor]] = None
                     ) -> Tuple[torch.Tensor, torch.Tensor]:
    """One growth step of the draft token graph, in place; see gsd_draft_expand in include/gsd.h.
    Returns (new_frontier [B,F*k], new_frontier_len [B])."""
    if logits.dim() != 3:
        raise ValueError("logits must be [B,F,V]")
    B, F, V = logits.shape
    Ncap = tokens.shape[1]
    _want(logits, torch.float32, (B, F, V), "logits", True)
    _want(frontier, torch.int32, (B, F), "frontier", True)
    _want(frontier_len, torch.int32, (B,), "frontier_len", True)
    for name, t, dt in (("tokens", tokens, torch.int32), ("tree_parent", tree_parent, torch.int32),
                        ("merge_to", merge_to, torch.int32), ("leaf", leaf, torch.uint8), ("prob", prob, torch.float32)):
        _want(t, dt, (B, Ncap), name, True)
    _want(num_nodes, torch.int32, (B,), "num_nodes", True)
    if out is None:
        nf = torch.full((B, F * k), -1, dtype=torch.int32, device=logits.device)
        nfl = torch.zeros((B,), dtype=torch.int32, device=logits.device)
    else:
        nf, nfl = out
        _want(nf, torch.int32, (B, F * k), "new_frontier", True)
        _want(nfl, torch.int32, (B,), "new_frontier_len", True)
    p = DraftParams(B, F, V, Ncap, int(k), int(tau), float(theta_prob), float(theta_sib))
    L = lib()
    with torch.cuda.device(logits.device):
        need = int(L.gsd_draft_expand_workspace_bytes(ctypes.byref(p)))
        if workspace is None:
            workspace = torch.empty(max(need, 8), dtype=torch.uint8, device=logits.device)
        _check(L.gsd_draft_expand(logits.data_ptr(), frontier.data_ptr(), frontier_len.data_ptr(),
                                  tokens.data_ptr(), tree_parent.data_ptr(), merge_to.data_ptr(), leaf.data_ptr(),
                                  prob.data_ptr(), num_nodes.data_ptr(), nf.data_ptr(), nfl.data_ptr(),
                                  ctypes.byref(p), workspace.data_ptr(),
                                  workspace.numel() * workspace.element_size(), _ptr(status), _stream(logits)))
    return nf, nfl


def gsd_build_mask(parent_ptr, parent_idx, out: Optional[torch.Tensor] = None, *,
                   status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Ancestor bitmask [B,N,ceil(N/32)] (int32 words) from the parent CSR; see gsd_build_mask in
    include/gsd.h.  Enqueued on the current stream."""
    B, N1 = parent_ptr.shape
    N = N1 - 1
    Ecap = parent_idx.shape[1]
    _want(parent_ptr, torch.int32, (B, N + 1), "parent_ptr", True)
    _want(parent_idx, torch.int32, (B, Ecap), "parent_idx", True)
    if out is None:
        out = torch.empty((B, N, (N + 31) // 32), dtype=torch.int32, device=parent_ptr.device)
    _want(out, out.dtype, (B, N, (N + 31) // 32), "ancestor_mask", True)
    with torch.cuda.device(parent_ptr.device):
        _check(lib().gsd_build_mask(parent_ptr.data_ptr(), parent_idx.data_ptr(), out.data_ptr(),
                                    B, N, Ecap, _ptr(status), _stream(parent_ptr)))
    return out


def gsd_unmerge_tree(draft_tokens, parent_ptr, parent_idx, *, Ucap: int, max_depth: int,
                     status: Optional[torch.Tensor] = None,
                     out: Optional[Tuple[torch.Tensor, torch.Tensor, torch.Tensor, torch.Tensor]] = None
                     ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor, torch.Tensor]:
    """The token graph unfolded into a tree (one node per root path); see gsd_unmerge_tree in
    include/gsd.h.  Returns (tree_tokens, tree_parent, tree_source [B,Ucap], tree_count [B])."""
    B, N = draft_tokens.shape
    Ecap = parent_idx.shape[1]
    _want(draft_tokens, torch.int32, (B, N), "draft_tokens", True)
    _want(parent_ptr, torch.int32, (B, N + 1), "parent_ptr", True)
    _want(parent_idx, torch.int32, (B, Ecap), "parent_idx", True)
    dev = draft_tokens.device
    if out is None:
        tt = torch.empty((B, Ucap), dtype=torch.int32, device=dev)
        tp = torch.empty((B, Ucap), dtype=torch.int32, device=dev)
        ts = torch.empty((B, Ucap), dtype=torch.int32, device=dev)
        cnt = torch.empty((B,), dtype=torch.int32, device=dev)
    else:
        tt, tp, ts, cnt = out
        for name, t in (("tree_tokens", tt), ("tree_parent", tp), ("tree_source", ts)):
            _want(t, torch.int32, (B, Ucap), name, True)
        _want(cnt, torch.int32, (B,), "tree_count", True)
    with torch.cuda.device(dev):
        _check(lib().gsd_unmerge_tree(draft_tokens.data_ptr(), parent_ptr.data_ptr(), parent_idx.data_ptr(),
                                      tt.data_ptr(), tp.data_ptr(), ts.data_ptr(), cnt.data_ptr(), B, N, Ecap,
                                      int(Ucap), int(max_depth), _ptr(status), _stream(draft_tokens)))
    return tt, tp, ts, cnt


def gsd_commit_kv(k_cache, v_cache, draft_k, draft_v, accepted_nodes, accepted_len, seq_lens, *,
                  status: Optional[torch.Tensor] = None) -> None:
    """Append the draft K/V rows of the accepted path to the cache in place and advance
    seq_lens; see gsd_commit_kv in include/gsd.h.  Enqueued on the current stream."""
    B, Lmax, Hkv, D = k_cache.shape
    N = draft_k.shape[1]
    Tcap = accepted_nodes.shape[1]
    bf = torch.bfloat16
    _want(k_cache, bf, (B, Lmax, Hkv, D), "k_cache", True)
    _want(v_cache, bf, (B, Lmax, Hkv, D), "v_cache", True)
    _want(draft_k, bf, (B, N, Hkv, D), "draft_k", True)
    _want(draft_v, bf, (B, N, Hkv, D), "draft_v", True)
    _want(accepted_nodes, torch.int32, (B, Tcap), "accepted_nodes", True)
    _want(accepted_len, torch.int32, (B,), "accepted_len", True)
    _want(seq_lens, torch.int32, (B,), "seq_lens", True)
    p = CommitParams(B, N, Hkv, D, Lmax, Tcap)
    with torch.cuda.device(k_cache.device):
        _check(lib().gsd_commit_kv(k_cache.data_ptr(), v_cache.data_ptr(), draft_k.data_ptr(),
                                   draft_v.data_ptr(), accepted_nodes.data_ptr(),
                                   accepted_len.data_ptr(), seq_lens.data_ptr(), ctypes.byref(p),
                                   _ptr(status), _stream(k_cache)))


GSD_STATIC_MAX_ROWS = 16384


def gsd_accept_static(logits, draft_tokens, parent_ptr, parent_idx, *, Tcap: int = 0,
                      want_nodes: bool = True, status: Optional[torch.Tensor] = None
                      ) -> Tuple[torch.Tensor, torch.Tensor, Optional[torch.Tensor]]:
    """gsd_accept for callers that cannot provide scratch memory: the library's own fixed
    array is used instead (B * N <= GSD_STATIC_MAX_ROWS; calls on one device must not overlap).
    The C call allocates nothing; this wrapper only allocates the result tensors it returns.
    See gsd_accept_static in include/gsd.h."""
    B, N, V = logits.shape
    _want(logits, torch.float32, (B, N, V), "logits", True)
    _want(draft_tokens, torch.int32, (B, N), "draft_tokens", True)
    _want(parent_ptr, torch.int32, (B, N + 1), "parent_ptr", True)
    Ecap = parent_idx.shape[1]
    _want(parent_idx, torch.int32, (B, Ecap), "parent_idx", True)
    Tcap = Tcap or N
    toks = torch.empty((B, Tcap), dtype=torch.int32, device=logits.device)
    lens = torch.empty((B,), dtype=torch.int32, device=logits.device)
    nodes = torch.empty((B, Tcap), dtype=torch.int32, device=logits.device) if want_nodes else None
    p = AcceptParams(B, N, V, Ecap, Tcap)
    with torch.cuda.device(logits.device):
        _check(lib().gsd_accept_static(logits.data_ptr(), draft_tokens.data_ptr(),
                                       parent_ptr.data_ptr(), parent_idx.data_ptr(),
                                       toks.data_ptr(), lens.data_ptr(), _ptr(nodes),
                                       ctypes.byref(p), _ptr(status), _stream(logits)))
    return toks, lens, nodes


def gsd_verify_step_host_arena_bytes(B, N, Hq, Hkv, D, Lmax, V, Ecap, Tcap, num_splits=0,
                                     kernel=GSD_ATTN_AUTO) -> int:
    ap = AttnParams(B, N, Hq, Hkv, D, Lmax, 0.0, num_splits, kernel)
    cp = AcceptParams(B, N, V, Ecap, Tcap)
    return int(lib().gsd_verify_step_host_arena_bytes(ctypes.byref(ap), ctypes.byref(cp)))


def gsd_verify_step_host(q, k_cache, v_cache, draft_k, draft_v, ancestor_mask, seq_lens, logits,
                         draft_tokens, parent_ptr, parent_idx, arena: torch.Tensor, *,
                         out=None, accepted=None, Tcap: int = 0, softmax_scale: float = 0.0,
                         num_splits: int = 0, kernel: int = GSD_ATTN_AUTO):
    """One whole verification step from HOST tensors through a caller-owned device arena;
    see gsd_verify_step_host in include/gsd.h.  Synchronises the current stream.
    Returns (out [B,N,Hq,D] bf16 CPU, accepted_tokens, accepted_len, accepted_nodes, status)."""
    _check_attn_tensors(q, k_cache, v_cache, draft_k, draft_v, ancestor_mask, seq_lens, False)
    B, N, V = logits.shape
    Ecap = parent_idx.shape[1]
    _want(logits, torch.float32, (B, N, V), "logits", False)
    _want(draft_tokens, torch.int32, (B, N), "draft_tokens", False)
    _want(parent_ptr, torch.int32, (B, N + 1), "parent_ptr", False)
    _want(parent_idx, torch.int32, (B, Ecap), "parent_idx", False)
    Tcap = Tcap or N
    if out is None:
        out = torch.empty_like(q)
    if accepted is None:
        accepted = (torch.empty((B, Tcap), dtype=torch.int32), torch.empty((B,), dtype=torch.int32),
                    torch.empty((B, Tcap), dtype=torch.int32))
    toks, lens, nodes = accepted
    ap = _attn_params(q, k_cache, draft_k, softmax_scale, num_splits, kernel)
    cp = AcceptParams(B, N, V, Ecap, Tcap)
    dev_status = ctypes.c_int32(0)
    if not arena.is_cuda:
        raise ValueError("arena must be a CUDA tensor")
    with torch.cuda.device(arena.device):
        _check(lib().gsd_verify_step_host(
            q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), draft_k.data_ptr(),
            draft_v.data_ptr(), ancestor_mask.data_ptr(), seq_lens.data_ptr(), out.data_ptr(),
            ctypes.byref(ap), logits.data_ptr(), draft_tokens.data_ptr(), parent_ptr.data_ptr(),
            parent_idx.data_ptr(), toks.data_ptr(), lens.data_ptr(), _ptr(nodes), ctypes.byref(cp),
            arena.data_ptr(), arena.numel() * arena.element_size(),
            ctypes.addressof(dev_status), _stream(arena)))
    return out, toks, lens, nodes, int(dev_status.value)
