"""Device-buffer plumbing for one layer of the hot path: uploads a workload's tensors,
allocates the outputs and the workspace, and issues the C-ABI calls.  No arithmetic."""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np
import torch

from . import binding as B
from .workloads import Workload


def to_device_bf16(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch bf16 tensor on the device (bit-exact)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)


def bf16_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class Layer:
    """All device buffers of one layer step for a workload."""

    def __init__(self, w: Workload, data: Dict[str, "np.ndarray | torch.Tensor"], device="cuda",
                 want_lse=True, want_slc=True):
        self.w = w
        self.dev = torch.device(device)
        N, D = w.n_heads, w.d_head
        self.shape = B.Shape(N, D, w.cu("T"), w.cu("Lq"))
        self.policy = B.make_policy(w.n_sink, w.n_recent, list(w.budget), w.n_streams)
        self.cu_B = B.pafu_kept_counts(self.shape, self.policy)
        # numpy bf16 bit patterns are uploaded; tensors already on the device are used as they are
        up = lambda k: data[k] if isinstance(data[k], torch.Tensor) else to_device_bf16(data[k], self.dev)
        self.K, self.V, self.Q, self.Kq, self.Vq = up("K"), up("V"), up("Q"), up("Kq"), up("Vq")
        self.w1, self.b1, self.w2, self.b2 = up("w1"), up("b1"), up("w2"), up("b2")
        self.head = B.Head(self.w1, self.b1, self.w2, self.b2, w.act, w.final)
        nT, nB, nQ = int(self.shape.cu_T[-1]), int(self.cu_B[-1]), int(self.shape.cu_Lq[-1])
        f32 = dict(dtype=torch.float32, device=self.dev)
        bf = dict(dtype=torch.bfloat16, device=self.dev)
        self.scores = torch.empty(max(nT, 1), **f32)
        self.idx = torch.empty(max(nB, 1), dtype=torch.int32, device=self.dev)
        self.Kc = torch.empty((max(nB, 1), N, D), **bf)
        self.Vc = torch.empty((max(nB, 1), N, D), **bf)
        self.SLc = torch.empty(max(nB, 1), **f32) if want_slc else None
        self.O = torch.empty((max(nQ, 1), N, D), **bf)
        self.LSE = torch.empty((N, max(nQ, 1)), **f32) if want_lse else None
        ws_bytes = B.pafu_workspace_bytes(self.shape, self.policy, self.head)
        assert ws_bytes > 0
        self.ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=self.dev)
        self.nT, self.nB, self.nQ = nT, nB, nQ
        self.args = B.step_args(self.shape, self.head, self.policy, self.K, self.V, self.Q, self.Kq,
                                self.Vq, 0.0, self.scores, self.idx, self.Kc, self.Vc, self.SLc,
                                self.O, self.LSE, self.ws)

    # individual steps -----------------------------------------------------------------
    def score(self):
        B.pafu_score(self.head, self.K, self.scores, self.ws, n_tokens=self.nT,
                     ldx=self.w.d_model)

    def select(self, scores: Optional[torch.Tensor] = None):
        B.pafu_select(self.scores if scores is None else scores, self.shape, self.policy, self.idx,
                      self.ws)

    def compact(self):
        B.pafu_compact(self.K, self.V, self.scores if self.SLc is not None else None, self.idx,
                       self.shape, self.policy, self.Kc, self.Vc, self.SLc)

    def attn(self):
        B.pafu_chunk_attn(self.Q, self.Kc, self.Vc, self.cu_B, self.Kq, self.Vq, self.shape, 0.0,
                          self.O, self.LSE, self.ws)

    def attn_indexed(self):
        B.pafu_chunk_attn_indexed(self.Q, self.K, self.V, self.idx, self.cu_B, self.Kq, self.Vq,
                                  self.shape, 0.0, self.O, self.LSE, self.ws)

    def step(self):
        B.pafu_step(self.args)

    def step_indexed(self):
        B.pafu_step_indexed(self.args)

    def check_status(self):
        st = B.pafu_workspace_status(self.ws)
        if st != 0:
            raise B.PafuError(st, "pafu_workspace_status")
