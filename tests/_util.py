"""Helpers shared by the GPU parity tests: storage arrays <-> device tensors."""
import numpy as np
import torch

import ec_synth as syn


def to_dev(a: np.ndarray | None, dtype: int | None = None, device="cuda"):
    """numpy storage array -> device tensor (uint16 bf16 bit patterns become torch.bfloat16)."""
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a))
    if a.dtype == np.uint16:
        t = t.view(torch.bfloat16)
    return t.to(device)


def to_storage(t: torch.Tensor) -> np.ndarray:
    """device tensor -> numpy storage array (bf16 comes back as uint16 bit patterns)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.uint16).numpy().copy()
    return t.numpy().copy()


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()
