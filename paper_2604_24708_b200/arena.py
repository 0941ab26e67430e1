"""Device memory layout helper: N replicas of a ragged tensor list packed into stacked arenas.

Layout in HBM (one allocation per quantity, no per-tensor allocations):

    param      fp32  [N][P_pad]     replica r of tensor k at  r * P_pad + offset_k
    exp_avg    fp32  [N][P_pad]     (AdamW only; [P_pad] when the moments are shared by all replicas)
    exp_avg_sq fp32  [N][P_pad]     (AdamW only; likewise)
    grad       fp32 or bf16 [N][P_pad]   (or [P_pad] when one gradient is shared)
    param_bf16 bf16  [P_pad]        (optional: the averaged parameters of the last converge, one copy)

Every offset_k is a multiple of ``align_elems`` (8 by default: 32 bytes of fp32, 16 bytes of
bf16), so every tensor takes the library's 128-bit path.  Only memory and descriptors are
handled here; all arithmetic is in the CUDA library.
"""
from __future__ import annotations

from typing import List, Sequence

import torch

from . import binding as B


class StackedArena:
    def __init__(self, numels: Sequence[int], groups: Sequence[int], n_replicas: int, optimizer: int,
                 grad_dtype: int, device: str = "cuda:0", align_elems: int = 8, shared_grad: bool = False,
                 shared_state: bool = False, sgd_momentum: bool = False, bf16_copy: bool = False):
        if not torch.cuda.is_available():
            raise RuntimeError("StackedArena needs a CUDA device (there is no CPU path)")
        self.numels = [int(x) for x in numels]
        self.groups = [int(g) for g in groups]
        self.n = int(n_replicas)
        self.optimizer = optimizer
        self.grad_dtype = grad_dtype
        self.device = torch.device(device)
        a = int(align_elems)
        self.offsets: List[int] = []
        cur = 0
        for ne in self.numels:
            self.offsets.append(cur)
            cur += (ne + a - 1) // a * a
        self.p_pad = cur
        gd = torch.bfloat16 if grad_dtype == B.HDET_DTYPE_BF16 else torch.float32
        self.param = torch.zeros((self.n, self.p_pad), dtype=torch.float32, device=self.device)
        adam = optimizer == B.HDET_OPT_ADAMW
        self.shared_state = bool(shared_state) and adam
        sshape = (self.p_pad,) if self.shared_state else (self.n, self.p_pad)
        self.exp_avg = (torch.zeros(sshape, dtype=torch.float32, device=self.device)
                        if (adam or sgd_momentum) else None)     # Adam first moment, or the SGD momentum buffer
        self.exp_avg_sq = torch.zeros(sshape, dtype=torch.float32, device=self.device) if adam else None
        self.shared_grad = bool(shared_grad)
        gshape = (self.p_pad,) if shared_grad else (self.n, self.p_pad)
        self.grad = torch.zeros(gshape, dtype=gd, device=self.device)
        # optional: one bf16 copy of the averaged parameters, written by every converge
        self.param_bf16 = torch.zeros((self.p_pad,), dtype=torch.bfloat16, device=self.device) if bf16_copy else None

    def descriptors(self) -> List[B.hdet_tensor]:
        out = []
        gsz = self.grad.element_size()
        for off, ne, grp in zip(self.offsets, self.numels, self.groups):
            t = B.hdet_tensor()
            t.param = self.param.data_ptr() + 4 * off
            t.grad = self.grad.data_ptr() + gsz * off
            if self.exp_avg is not None:
                t.exp_avg = self.exp_avg.data_ptr() + 4 * off
            if self.exp_avg_sq is not None:
                t.exp_avg_sq = self.exp_avg_sq.data_ptr() + 4 * off
            t.numel = ne
            t.param_stride = self.p_pad
            t.grad_stride = 0 if self.shared_grad else self.p_pad
            t.state_stride = 0 if self.shared_state else self.p_pad
            t.group = grp
            if self.param_bf16 is not None:
                t.param_bf16 = self.param_bf16.data_ptr() + 2 * off
            out.append(t)
        return out

    def resident_bytes(self) -> int:
        ts = [t for t in (self.param, self.grad, self.exp_avg, self.exp_avg_sq, self.param_bf16) if t is not None]
        return sum(t.numel() * t.element_size() for t in ts)
