"""Shared test plumbing: tensor <-> numpy bit views and batch slicing.  No method arithmetic."""
import numpy as np
import torch


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns (same shape)."""
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def from_bits(u: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(u.view(np.int16).copy()).view(torch.bfloat16)


def sample_np(batch, b):
    """numpy views of one sample of a workloads.Batch, as the oracle wants them."""
    rows = batch.sample_rows(b)
    return dict(q_bits=bits(batch.q[rows]), k_bits=bits(batch.k[rows]),
                hidden_bits=bits(batch.hidden[rows]), pos_ids=batch.pos_ids[rows].numpy(),
                v0=int(batch.vis_start[b]), nv=int(batch.vis_len[b]))
