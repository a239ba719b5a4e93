"""Moves a synthetic workload onto the GPU and drives the two C-ABI calls of a verify step.
Used by the tests, the smoke check and the benchmark; holds no arithmetic of its own."""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np
import torch

from .binding import OwlContext, OwlDims, make_dims
from .workloads import Workload


def dims_of(wl: Workload, path_stride: int = 64) -> OwlDims:
    sp = wl.spec
    return make_dims(batch=sp.batch, total_nodes=wl.total_nodes, max_nodes=wl.max_nodes,
                     num_q_heads=sp.num_q_heads, num_kv_heads=sp.num_kv_heads, head_dim=sp.head_dim,
                     page_size=sp.page_size, max_pages_per_seq=wl.max_pages_per_seq, num_pages=wl.num_pages,
                     vocab=sp.vocab if wl.logits is not None else 0, path_stride=path_stride, sm_scale=wl.sm_scale)


def _bf16(a: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)


@dataclasses.dataclass
class DeviceWorkload:
    """Device-resident tensors of one workload plus preallocated outputs."""
    dims: OwlDims
    q: torch.Tensor
    k_cache: torch.Tensor
    v_cache: torch.Tensor
    block_table: torch.Tensor
    ctx_lens: torch.Tensor
    node_offsets: torch.Tensor
    tree_parent: torch.Tensor
    draft_tokens: torch.Tensor
    logits: Optional[torch.Tensor]
    out: torch.Tensor
    lse: torch.Tensor
    accept_len: torch.Tensor
    accept_path: torch.Tensor
    bonus_token: torch.Tensor
    node_argmax: torch.Tensor

    @classmethod
    def upload(cls, wl: Workload, device="cuda", path_stride: int = 64) -> "DeviceWorkload":
        dev = torch.device(device)
        d = dims_of(wl, path_stride)
        N, Hq, D = wl.q.shape
        B = wl.spec.batch
        i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
        return cls(
            dims=d, q=_bf16(wl.q, dev), k_cache=_bf16(wl.k_cache, dev), v_cache=_bf16(wl.v_cache, dev),
            block_table=i32(wl.block_table), ctx_lens=i32(wl.ctx_lens), node_offsets=i32(wl.node_offsets),
            tree_parent=i32(wl.tree_parent), draft_tokens=i32(wl.draft_tokens),
            logits=None if wl.logits is None else torch.from_numpy(wl.logits).to(dev),
            out=torch.zeros((N, Hq, D), dtype=torch.bfloat16, device=dev),
            lse=torch.zeros((N, Hq), dtype=torch.float32, device=dev),
            accept_len=torch.zeros(B, dtype=torch.int32, device=dev),
            accept_path=torch.zeros((B, path_stride), dtype=torch.int32, device=dev),
            bonus_token=torch.zeros(B, dtype=torch.int32, device=dev),
            node_argmax=torch.zeros(N, dtype=torch.int32, device=dev))

    def attn(self, ctx: OwlContext, check: bool = True) -> int:
        return ctx.owl_verify_attn(self.dims, self.q, self.k_cache, self.v_cache, self.block_table, self.ctx_lens,
                                   self.node_offsets, self.tree_parent, self.out, self.lse, check=check)

    def accept(self, ctx: OwlContext, check: bool = True) -> int:
        return ctx.owl_tree_accept(self.dims, self.logits, self.draft_tokens, self.node_offsets, self.tree_parent,
                                   self.accept_len, self.accept_path, self.bonus_token, self.node_argmax, check=check)

    def step(self, ctx: OwlContext) -> None:
        """One verify step: attention of the drafted nodes, then acceptance from the logits."""
        if self.logits is None:
            self.attn(ctx)
        else:
            ctx.owl_verify_step(self.dims, self.q, self.k_cache, self.v_cache, self.block_table, self.ctx_lens,
                                self.node_offsets, self.tree_parent, self.out, self.lse, self.logits, self.draft_tokens,
                                self.accept_len, self.accept_path, self.bonus_token, self.node_argmax)

    def out_f32(self) -> np.ndarray:
        return self.out.float().cpu().numpy()
