"""Projections that consume the same X (q/k/v, gate/up) as ONE LoRA linear.

For projections g = 1..G with weights W_g [d_g, d_in] and adapters A_g [r, d_in], B_g [d_g, r]

    Y_g = X W_g^T + s (X A_g^T) B_g^T

is one layer with W = rows of all W_g, A = rows of all A_g (rank G r) and a block-diagonal B [sum d_g, G r]:
the kernels read X once per pass instead of G times, the narrow projections (k, v: 1024 columns) stop paying
for badly filled grids, and G launch chains become one.  The zero blocks of B cost only a few rank-r MMA columns.
Gradients: dX is the sum over the group by construction, dA_g are row blocks of dA, dB_g the diagonal blocks of dB
(the off-diagonal blocks are gradients with respect to entries that are zero by construction and are dropped).

All arithmetic runs in the CUDA kernels behind the C ABI; this module only lays out the operands.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch

from .binding import LoraLinearPlan


class GroupedLoraPlan:
    """Plan for G projections sharing X.  G * r must be a multiple of 8 and at most 64."""

    def __init__(self, T: int, d_in: int, d_outs: Sequence[int], r: int, device: int = 0):
        self.d_outs = [int(d) for d in d_outs]
        self.G, self.r = len(self.d_outs), int(r)
        if self.G * self.r > 64:
            raise ValueError("grouped projections: G * r must not exceed 64")
        self.offsets = [0]
        for d in self.d_outs:
            self.offsets.append(self.offsets[-1] + d)
        self.plan = LoraLinearPlan(T, d_in, self.offsets[-1], self.G * self.r, device)
        self.T, self.d_in = int(T), int(d_in)

    def close(self):
        self.plan.close()

    # -- operand layout --------------------------------------------------------------------------
    def pack(self, Ws, As, Bs) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """(W_cat, A_cat, B_cat) for the group; B_cat is block-diagonal.  One-time set-up for the frozen W; A_cat and
        B_cat can serve as the adapters' own storage (see ``views``)."""
        W = torch.cat(list(Ws), dim=0).contiguous()
        A = torch.cat(list(As), dim=0).contiguous()
        B = torch.zeros((self.offsets[-1], self.G * self.r), dtype=Bs[0].dtype, device=Bs[0].device)
        for g, Bg in enumerate(Bs):
            B[self.offsets[g]:self.offsets[g + 1], g * self.r:(g + 1) * self.r] = Bg
        return W, A, B

    def views(self, A_cat: torch.Tensor, B_cat: torch.Tensor):
        """Per-projection views (no copies) of the stacked adapters."""
        As = [A_cat[g * self.r:(g + 1) * self.r] for g in range(self.G)]
        Bs = [B_cat[self.offsets[g]:self.offsets[g + 1], g * self.r:(g + 1) * self.r] for g in range(self.G)]
        return As, Bs

    def split_outputs(self, Y_cat: torch.Tensor) -> List[torch.Tensor]:
        return [Y_cat[:, self.offsets[g]:self.offsets[g + 1]] for g in range(self.G)]

    # -- the two calls ---------------------------------------------------------------------------
    def fwd(self, X, W_cat, A_cat, B_cat, scale: float, Y_cat=None, stream=None) -> torch.Tensor:
        """Y_cat [T, sum d_g]; ``split_outputs`` gives the per-projection column blocks."""
        return self.plan.fwd(X, W_cat, A_cat, B_cat, scale, Y_cat, stream)

    def bwd(self, dY_cat, X, W_cat, A_cat, B_cat, scale: float, dX=None, dA_cat=None, dB_cat=None, stream=None,
            saved_p: bool = False):
        """(dX, [dA_g], [dB_g]); dA_g / dB_g are views into dA_cat [G r, d_in] / dB_cat [sum d_g, G r]."""
        dX, dA_cat, dB_cat = self.plan.bwd(dY_cat, X, W_cat, A_cat, B_cat, scale, dX, dA_cat, dB_cat, stream, saved_p)
        dAs, dBs = self.views(dA_cat, dB_cat)
        return dX, dAs, dBs
