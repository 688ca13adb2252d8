"""One policy-scoring step = pack -> group advantages -> loss forward -> loss backward,
each a call into the CUDA library.  This module only owns buffers and sequences the calls
(it is the API a training loop would use); it performs no arithmetic of its own.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np
import torch

from . import binding as B
from . import inputs as gen


def _to_dev(a: np.ndarray, device) -> torch.Tensor:
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def _pinned(a: np.ndarray) -> torch.Tensor:
    t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else np.ascontiguousarray(a))
    return t.pin_memory()


@dataclass
class StepResult:
    loss: torch.Tensor
    fwd: Dict[str, torch.Tensor]
    dhidden: torch.Tensor
    dW: torch.Tensor
    packed: Dict[str, torch.Tensor]
    adv: torch.Tensor


class PolicyScorer:
    """Device-side state for scoring batches of one shape class.

    max_tokens / max_seqs bound the packed batch; W_head stays resident on the device.
    """

    def __init__(self, W_head: torch.Tensor, max_tokens: int, max_seqs: int, max_questions: int,
                 eps_low: float = 0.2, eps_high: float = 0.28, adv_eps: float = 1e-6,
                 ddof: int = 0, grad_scale: float = 1.0, device="cuda", active_backward: bool = False,
                 backward: Optional[str] = None, want_entropy: bool = False):
        if not torch.cuda.is_available():
            raise B.SapoError("PolicyScorer needs a CUDA device; there is no CPU path")
        B.load()
        self.device = device
        self.W = W_head
        self.V, self.H = int(W_head.shape[0]), int(W_head.shape[1])
        self.dtype = W_head.dtype
        self.dcode = B.DTYPE_F32 if self.dtype == torch.float32 else B.DTYPE_BF16
        self.max_tokens, self.max_seqs, self.max_q = int(max_tokens), int(max_seqs), int(max_questions)
        self.eps_low, self.eps_high = float(eps_low), float(eps_high)
        self.adv_eps, self.ddof, self.grad_scale = float(adv_eps), int(ddof), float(grad_scale)
        # "gather": the single-pass call with the hidden rows read in place from the rollout stores
        # (the pack copies no hidden rows)
        self.backward = backward if backward is not None else ("active" if active_backward else "dense")
        self.packed = B.alloc_packed(self.max_tokens, self.max_seqs, self.max_q, self.H, self.dtype, device,
                                     copy_hidden=self.backward != "gather")
        self.adv = torch.empty(self.max_seqs, dtype=torch.float32, device=device)
        self.fwd = B.alloc_fwd_outputs(self.max_tokens, self.max_seqs, device)
        # per-token entropy of the policy's distribution, if asked for (a by-product of the forward)
        self.entropy = (torch.empty(self.max_tokens, dtype=torch.float32, device=device)
                        if want_entropy else None)
        self.dhidden = torch.empty(self.max_tokens, self.H, dtype=torch.float32, device=device)
        self.dW = torch.empty(self.V, self.H, dtype=torch.float32, device=device)
        nf = B.sapo_workspace_bytes(B.WS_FWD, self.max_tokens, self.H, self.V, self.dcode)
        # how the gradients are formed: "dense" = forward call, then the backward call that
        # recomputes the logits; "active" = the same over tokens with a non-zero gradient factor
        # only; "fused" = one call that passes over the logits once (bf16 operands)
        if self.backward not in ("dense", "active", "fused", "gather"):
            raise ValueError(f"unknown backward mode {self.backward!r}")
        self.active_backward = self.backward == "active"
        which = {"dense": B.WS_BWD, "active": B.WS_BWD_ACTIVE, "fused": B.WS_FUSED,
                 "gather": B.WS_FUSED | B.WS_GATHER}[self.backward]
        nb = B.sapo_workspace_bytes(which, self.max_tokens, self.H, self.V, self.dcode)
        if nb == 0:
            raise B.SapoError(f"backward mode {self.backward!r} does not support these operands")
        self.n_active = torch.zeros(1, dtype=torch.int32, device=device)
        # forward and backward never overlap on the stream, so they share one scratch buffer
        self.workspace = torch.empty(max(nf + 4 * self.max_seqs + 256, nb), dtype=torch.uint8, device=device)
        self.status = B.new_status(device)

    # -- one step on device-resident buffers ------------------------------------------------
    def step(self, local: B.DeviceRollouts, ext: B.DeviceRollouts, sel: B.DeviceSelection,
             T: int, S: int) -> StepResult:
        """T and S are the packed token / sequence counts (known on the host from the
        selection; the pack kernel also writes them to packed['n_tokens'] / ['n_seqs'])."""
        p = self.packed
        B.sapo_pack_rollouts(local, ext, sel, p, self.status)
        Q = int(sel.q_offsets_local.numel() - 1)
        go = p["group_offsets"][:Q + 1]
        B.sapo_group_advantages(p["rewards"], go, self.adv_eps, self.ddof, self.adv, None, None,
                                self.status)
        cu = p["cu_seqlens"][:S + 1]
        if self.backward == "gather":
            B.sapo_policy_loss_fwd_bwd_gather(local.hidden, ext.hidden, p["tok_src"], self.W, p["ids"],
                                              p["old_logp"], self.adv, cu, self.eps_low, self.eps_high,
                                              self.grad_scale, self.fwd, self.dhidden, self.dW, False,
                                              self.workspace, self.status, T=T, entropy=self.entropy)
            return StepResult(self.fwd["loss"], self.fwd, self.dhidden, self.dW, p, self.adv)
        if self.backward == "fused":
            B.sapo_policy_loss_fwd_bwd(p["hidden"], self.W, p["ids"], p["old_logp"], self.adv, cu,
                                       self.eps_low, self.eps_high, self.grad_scale, self.fwd,
                                       self.dhidden, self.dW, False, self.workspace, self.status, T=T,
                                       entropy=self.entropy)
            return StepResult(self.fwd["loss"], self.fwd, self.dhidden, self.dW, p, self.adv)
        B.sapo_policy_loss_fwd(p["hidden"], self.W, p["ids"], p["old_logp"], self.adv, cu,
                               self.eps_low, self.eps_high, self.grad_scale, self.fwd,
                               self.workspace, self.status, T=T, entropy=self.entropy)
        if self.active_backward:
            B.sapo_policy_loss_bwd_active(p["hidden"], self.W, p["ids"], self.fwd["lse"], self.fwd["gscale"],
                                          self.dhidden, self.dW, False, self.workspace, self.status,
                                          self.n_active, T=T)
        else:
            B.sapo_policy_loss_bwd(p["hidden"], self.W, p["ids"], self.fwd["lse"], self.fwd["gscale"],
                                   self.dhidden, self.dW, False, self.workspace, self.status, T=T)
        return StepResult(self.fwd["loss"], self.fwd, self.dhidden, self.dW, p, self.adv)

    # -- one step from pinned host buffers -----------------------------------------------------
    def make_host_batch(self, batch: gen.Batch) -> Dict[str, torch.Tensor]:
        """Pinned host copies of everything a step consumes, plus matching device buffers."""
        if getattr(self, "_copy_stream", None) is not None:
            self._copy_stream.synchronize()          # no copy into the buffers this call replaces
        host, dev = {}, {}
        for side, buf in (("local", batch.local), ("ext", batch.ext)):
            for k in ("hidden", "ids", "old_logp", "offsets", "rewards"):
                a = getattr(buf, k)
                host[f"{side}.{k}"] = _pinned(a)
        for k in ("q_offsets_local", "local_idx", "q_offsets_ext", "ext_idx"):
            host[f"sel.{k}"] = _pinned(getattr(batch.sel, k))
        # two sets of device buffers: while a step computes on one, the next step's inputs are
        # copied into the other on a stream of their own
        other = {}
        for k, t in host.items():
            dev[k] = torch.empty(t.shape, dtype=t.dtype, device=self.device)
            other[k] = torch.empty(t.shape, dtype=t.dtype, device=self.device)
        self._host, self._dev = host, dev
        self._dev_sets = [dev, other]
        self._copy_stream = torch.cuda.Stream(device=self.device)
        self._copied = [torch.cuda.Event(), torch.cuda.Event()]
        self._consumed = [None, None]
        self._in_flight = [False, False]
        self._next_set = 0
        self._loss_host = torch.empty(1, dtype=torch.float32).pin_memory()
        self._logp_host = torch.empty(batch.T, dtype=torch.float32).pin_memory()
        self.h2d_bytes = sum(t.numel() * t.element_size() for t in host.values())
        self.d2h_bytes = 4 + 4 * batch.T
        return host

    def _start_copy(self, i: int) -> None:
        """Host -> device copy of the pinned inputs into buffer set i, on the copy stream, once
        the step that last read that set has finished."""
        with torch.cuda.stream(self._copy_stream):
            if self._consumed[i] is not None:
                self._copy_stream.wait_event(self._consumed[i])
            for k, t in self._host.items():
                self._dev_sets[i][k].copy_(t, non_blocking=True)
            self._copied[i].record(self._copy_stream)
        self._in_flight[i] = True

    def step_from_host(self, T: int, S: int, prefetch_next: bool = True) -> StepResult:
        """One step whose inputs start in pinned host memory: copy them to the device, run the
        step, read loss and log-probs back.  Every call makes exactly one copy of the inputs; with
        prefetch_next the copy it starts is the one the *next* call consumes (into the other buffer
        set, overlapping this call's kernels), and its own inputs are those the previous call
        fetched (or are copied now, on the first call)."""
        i = self._next_set
        if not self._in_flight[i]:
            self._start_copy(i)
        stream = torch.cuda.current_stream()
        stream.wait_event(self._copied[i])
        self._in_flight[i] = False
        d = self._dev_sets[i]
        view = lambda t: t.view(torch.bfloat16) if (t.dtype == torch.int16) else t
        local = B.DeviceRollouts(view(d["local.hidden"]), d["local.ids"], d["local.old_logp"],
                                 d["local.offsets"], d["local.rewards"])
        ext = B.DeviceRollouts(view(d["ext.hidden"]), d["ext.ids"], d["ext.old_logp"],
                               d["ext.offsets"], d["ext.rewards"])
        sel = B.DeviceSelection(d["sel.q_offsets_local"], d["sel.local_idx"], d["sel.q_offsets_ext"],
                                d["sel.ext_idx"])
        res = self.step(local, ext, sel, T, S)
        if self._consumed[i] is None:
            self._consumed[i] = torch.cuda.Event()
        self._consumed[i].record(stream)
        self._loss_host.copy_(res.loss, non_blocking=True)
        self._logp_host.copy_(res.fwd["logp"][:T], non_blocking=True)
        if prefetch_next:
            self._start_copy(1 - i)
            self._next_set = 1 - i
        return res

    def check_status(self) -> None:
        word = int(self.status.item())
        if word:
            raise B.SapoError("device status: " + ",".join(B.decode_status(word)))
