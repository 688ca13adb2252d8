"""One node's LM head sharded by vocabulary over the ranks of a process group.

The paper's nodes each hold a whole model (Section 4: one GPU per agent), so this is not part of
its method; it is how the same policy-loss step runs when the head (or the batch) outgrows one
GPU.  Rank r keeps rows [lo_r, hi_r) of W_head and all tokens' hidden states.  Per step:

  1. projection of the own shard        -> (max, sum, target logit) per token        [3, T]
  2. all-gather of the triples          -> every rank holds [P, 3, T] in its own memory
  3. loss tail over the gathered triples (identical on every rank: log-sum-exp merge, ratio,
     clipped surrogate, gradient factor, loss)
  4. backward of the own shard          -> dW rows [lo_r, hi_r) (final), partial dhidden
  5. all-reduce (sum) of dhidden        [T, H]

Two collectives per step (12 T bytes gathered per rank, 4 T H bytes reduced), both through
torch.distributed (NCCL on GPUs): kernels only ever read local memory.  The compute steps are
behind a small backend object, so the orchestration (sharding, id offsets, buffer layout,
collectives) can be exercised on CPU ranks with a stand-in backend.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional, Tuple

import torch
import torch.distributed as dist


def shard_bounds(V: int, world: int, rank: int, align: int = 128) -> Tuple[int, int]:
    """Rows [lo, hi) of the vocabulary that `rank` holds: equal shares in whole blocks of `align`
    rows (the vocab tile of the kernels), the last rank takes the ragged rest."""
    blocks = -(-V // align)
    per = -(-blocks // world)
    lo = min(V, rank * per * align)
    hi = min(V, (rank + 1) * per * align)
    return lo, hi


class CudaBackend:
    """The three compute steps on the CUDA library."""

    def __init__(self):
        from . import binding as B
        self.B = B
        self._ws: Optional[torch.Tensor] = None

    def _workspace(self, nbytes: int, device) -> torch.Tensor:
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
        return self._ws

    def lse_partial(self, hidden, W_shard, ids, vocab_offset, triple, status):
        B = self.B
        T, H, V = hidden.shape[0], hidden.shape[1], W_shard.shape[0]
        ws = self._workspace(B.sapo_workspace_bytes(B.WS_FWD, T, H, V, B._dtype_code(hidden)), hidden.device)
        B.sapo_lmhead_lse_partial(hidden, W_shard, ids, vocab_offset, triple, ws, status)

    def loss_from_partials(self, triples, V, ids, old_logp, adv, cu, eps_low, eps_high, grad_scale, out, status):
        self.B.sapo_policy_loss_from_partials(triples, V, ids, old_logp, adv, cu, eps_low, eps_high, grad_scale,
                                              out, status)

    def bwd_shard(self, hidden, W_shard, ids, vocab_offset, lse, gscale, dhidden, dW_shard, status):
        B = self.B
        T, H, V = hidden.shape[0], hidden.shape[1], W_shard.shape[0]
        kind = B.WS_BWD | (B.WS_OUT_BF16 if dhidden.dtype == torch.bfloat16 else 0)
        ws = self._workspace(B.sapo_workspace_bytes(kind, T, H, V, B._dtype_code(hidden)), hidden.device)
        B.sapo_policy_loss_bwd_shard(hidden, W_shard, ids, vocab_offset, lse, gscale, dhidden, dW_shard, False,
                                     ws, status)


@dataclass
class ShardedStep:
    out: Dict[str, torch.Tensor]       # logp, lse, ratio, surr, gscale, seq_surr, loss: the same on every rank
    dhidden: torch.Tensor              # [T, H], summed over the ranks
    dW_shard: torch.Tensor             # rows [lo, hi) of dW_head


class VocabShardedLoss:
    """Policy loss and gradients with W_head sharded by vocabulary over `group`."""

    def __init__(self, W_shard: torch.Tensor, V: int, vocab_offset: int, backend=None,
                 group: Optional[dist.ProcessGroup] = None, eps_low: float = 0.2, eps_high: float = 0.28,
                 grad_scale: float = 1.0):
        self.W, self.V, self.lo = W_shard, int(V), int(vocab_offset)
        self.backend = backend if backend is not None else CudaBackend()
        self.group = group
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.eps_low, self.eps_high, self.grad_scale = eps_low, eps_high, grad_scale

    def step(self, hidden: torch.Tensor, ids: torch.Tensor, old_logp: torch.Tensor, adv: torch.Tensor,
             cu_seqlens: torch.Tensor) -> ShardedStep:
        dev, T, H = hidden.device, hidden.shape[0], hidden.shape[1]
        S = cu_seqlens.numel() - 1
        f32 = lambda *shape: torch.empty(*shape, dtype=torch.float32, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        # 1. own shard -> one triple per token (a rank left without rows adds the neutral triple)
        mine = f32(3, T)
        empty = self.W.shape[0] == 0
        if empty:
            mine[0].fill_(float("-inf")); mine[1].zero_(); mine[2].zero_()
        else:
            self.backend.lse_partial(hidden, self.W, ids, self.lo, mine, status)
        # 2. everybody's triples into local memory: [P, 3, T], rank order
        triples = f32(self.world, 3, T)
        if self.world > 1:
            dist.all_gather_into_tensor(triples.view(-1), mine.view(-1), group=self.group)
        else:
            triples[0].copy_(mine)
        # 3. the loss tail, identical on every rank
        out = {k: f32(T) for k in ("logp", "lse", "ratio", "surr", "gscale")}
        out["seq_surr"], out["loss"] = f32(S), f32(1)
        self.backend.loss_from_partials(triples, self.V, ids, old_logp, adv, cu_seqlens, self.eps_low,
                                        self.eps_high, self.grad_scale, out, status)
        # 4. own shard's gradients
        dhidden = f32(T, H)
        dW = f32(self.W.shape[0], H)
        if empty:
            dhidden.zero_()
        else:
            self.backend.bwd_shard(hidden, self.W, ids, self.lo, out["lse"], out["gscale"], dhidden, dW, status)
        # 5. dhidden is a sum over the vocabulary: add the shards' shares
        if self.world > 1:
            dist.all_reduce(dhidden, op=dist.ReduceOp.SUM, group=self.group)
        self.status = status
        return ShardedStep(out, dhidden, dW)
