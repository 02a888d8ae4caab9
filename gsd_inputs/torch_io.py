"""Marshalling of generated inputs (numpy, bf16 as uint16 bit patterns) into torch tensors on a
device or in host memory, and back.  No arithmetic of the method; used by the tests, the smoke
check and the benchmark."""
import numpy as np
import torch


def bf16_tensor(bits: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def i32_tensor(a: np.ndarray, device) -> torch.Tensor:
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint32:
        a = a.view(np.int32)
    return torch.from_numpy(a.astype(np.int32, copy=False)).to(device)


def attn_tensors(inp, device="cuda"):
    return dict(q=bf16_tensor(inp["q"], device), k_cache=bf16_tensor(inp["k_cache"], device),
                v_cache=bf16_tensor(inp["v_cache"], device), draft_k=bf16_tensor(inp["draft_k"], device),
                draft_v=bf16_tensor(inp["draft_v"], device),
                ancestor_mask=i32_tensor(inp["ancestor_mask"], device),
                seq_lens=i32_tensor(inp["seq_lens"], device))


def accept_tensors(inp, device="cuda"):
    return dict(logits=torch.from_numpy(inp["logits"]).to(device),
                draft_tokens=i32_tensor(inp["draft_tokens"], device),
                parent_ptr=i32_tensor(inp["parent_ptr"], device),
                parent_idx=i32_tensor(inp["parent_idx"], device))


def out_to_f64(out: torch.Tensor) -> np.ndarray:
    return out.detach().float().cpu().numpy().astype(np.float64)
