"""The tests' names for the marshalling helpers (generated numpy inputs -> torch tensors)."""
from gsd_inputs.torch_io import (accept_tensors, attn_tensors, bf16_bits, bf16_tensor,  # noqa: F401
                                 i32_tensor, out_to_f64)
