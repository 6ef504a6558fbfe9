"""Stand-in language model that produces the logits the hot path consumes.

logits(prev) = E[prev] @ W (+ b): an embedding look-up followed by one dense
projection.  It replaces the paper's language models (Section 4.1), which are
not available here.  It is an input producer: it lives outside the library and
outside the timed hot path, and uses torch's stock matmul.
"""
from __future__ import annotations

import numpy as np
import torch


class StandInLM:
    def __init__(self, E, W, b, logits: str, device):
        self.device = torch.device(device)
        self.out_dtype = torch.float32 if logits == "f32" else torch.bfloat16
        op = torch.float32 if logits == "f32" else torch.bfloat16
        self.E = torch.as_tensor(E).to(self.device, op)
        self.W = torch.as_tensor(W).to(self.device, op)
        self.b = None if b is None else torch.as_tensor(b).to(self.device, torch.float32)
        self.V = self.W.shape[1]
        self.d = self.W.shape[0]

    @torch.no_grad()
    def logits(self, prev: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
        """prev: integer tensor [R] of previous tokens -> logits [R, V]."""
        h = self.E.index_select(0, prev.to(self.device, torch.int64))
        if self.b is None:
            if out is not None:
                return torch.matmul(h, self.W, out=out)
            return torch.matmul(h, self.W)
        z = (torch.matmul(h, self.W).float() + self.b).to(self.out_dtype)
        if out is not None:
            out.copy_(z)
            return out
        return z

    @torch.no_grad()
    def hidden(self, prev: torch.Tensor) -> torch.Tensor:
        """The final hidden vectors [R, d] of which logits(prev) is the projection."""
        return self.E.index_select(0, prev.to(self.device, torch.int64))

    @torch.no_grad()
    def projection_rows(self) -> torch.Tensor:
        """The projection with one vocabulary entry per row, [V, d] contiguous (the layout a fused
        projection kernel takes; the same numbers as W)."""
        if getattr(self, "_wt", None) is None:
            self._wt = self.W.t().contiguous()
        return self._wt

    def flops_per_row(self) -> int:
        return 2 * self.d * self.V


def markov_table(E: np.ndarray, W: np.ndarray, b: np.ndarray | None) -> np.ndarray:
    """All V rows of next-token logits, float32 [V, V] (small vocabularies only)."""
    Z = E.astype(np.float32) @ W.astype(np.float32)
    if b is not None:
        Z = Z + b.astype(np.float32)[None, :]
    return np.ascontiguousarray(Z, dtype=np.float32)
