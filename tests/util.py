"""Test harness glue: move generated batches to the device, run the library through its
binding, and compare with the oracle under the stated tolerances."""
from __future__ import annotations

import math
from typing import Dict, Optional

import numpy as np
import torch

from oracle import sapo_oracle as orc
from paper_2509_08721_b200 import binding as B
from paper_2509_08721_b200 import inputs as gen

# tolerances of the parity bar
TOL_LOGP_ABS = 2e-3
TOL_LOSS_REL = 1e-3
TOL_GRAD_FRO = 2e-2
# advantages: compensated fp32 on the device, 6 fp32 ulp worst case for groups of up to 16
# (1 ulp deviation + 2.5 std + 1.5 scalar steps + 1 reciprocal and product), plus the rounding
# of the comparison itself
TOL_ADV_REL = 4e-7


def to_torch(a: np.ndarray, device="cuda") -> torch.Tensor:
    if a.dtype == np.uint16:                       # bf16 bit patterns
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def to_numpy(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def buf_dict(b: gen.RolloutBuffer) -> Dict[str, np.ndarray]:
    return {"hidden": b.hidden, "ids": b.ids, "old_logp": b.old_logp, "offsets": b.offsets,
            "rewards": b.rewards}


def sel_dict(s: gen.Selection) -> Dict[str, np.ndarray]:
    return {"q_offsets_local": s.q_offsets_local, "local_idx": s.local_idx,
            "q_offsets_ext": s.q_offsets_ext, "ext_idx": s.ext_idx}


def dev_rollouts(b: gen.RolloutBuffer) -> B.DeviceRollouts:
    return B.DeviceRollouts(to_torch(b.hidden), to_torch(b.ids), to_torch(b.old_logp),
                            to_torch(b.offsets), to_torch(b.rewards))


def dev_selection(s: gen.Selection) -> B.DeviceSelection:
    return B.DeviceSelection(to_torch(s.q_offsets_local), to_torch(s.local_idx),
                             to_torch(s.q_offsets_ext), to_torch(s.ext_idx))


def oracle_current_logp(batch: gen.Batch, rows_per_block: int = 1024) -> np.ndarray:
    """Log-probs of the packed tokens under the batch's head, from the oracle (float32)."""
    h = gen.as_f32(batch.built.hidden)
    W = gen.as_f32(batch.W).astype(np.float64)
    out = np.zeros(batch.T, dtype=np.float32)
    for a in range(0, batch.T, rows_per_block):
        b = min(batch.T, a + rows_per_block)
        out[a:b] = orc.token_logprobs(h[a:b], W, batch.built.ids[a:b])["logp"]
    return out


def torch_current_logp(hidden: torch.Tensor, W: torch.Tensor, ids: torch.Tensor,
                       rows: int = 2048) -> torch.Tensor:
    """A cheap stand-in for 'the current log-probs' used only to place old_logp near them
    when the oracle cannot score every token (it is an input recipe, not a reference)."""
    out = torch.empty(hidden.shape[0], dtype=torch.float32, device=hidden.device)
    for a in range(0, hidden.shape[0], rows):
        z = (hidden[a:a + rows] @ W.T).float()
        out[a:a + rows] = z.gather(1, ids[a:a + rows].long()[:, None])[:, 0] - torch.logsumexp(z, 1)
    return out


def gpu_pack(batch: gen.Batch, max_tokens: Optional[int] = None, max_seqs: Optional[int] = None):
    local, ext, sel = dev_rollouts(batch.local), dev_rollouts(batch.ext), dev_selection(batch.sel)
    T, S, Q = batch.T, batch.S, batch.sel.Q
    mt = T if max_tokens is None else max_tokens
    ms = S if max_seqs is None else max_seqs
    dt = torch.float32 if batch.dtype == gen.DTYPE_F32 else torch.bfloat16
    out = B.alloc_packed(mt, ms, Q, batch.H, dt)
    status = B.new_status()
    B.sapo_pack_rollouts(local, ext, sel, out, status)
    torch.cuda.synchronize()
    return out, int(status.item())


def gpu_scores(hidden, W, ids, old_logp, adv, cu, eps_low, eps_high, grad_scale=1.0,
               bwd_workspace_bytes: Optional[int] = None, want_bwd: bool = True,
               out_dtype: torch.dtype = torch.float32, accumulate_into=None):
    """fwd (+ bwd) through the binding on device tensors; returns device tensors."""
    T, H, V, S = hidden.shape[0], hidden.shape[1], W.shape[0], cu.numel() - 1
    dcode = B.DTYPE_F32 if hidden.dtype == torch.float32 else B.DTYPE_BF16
    status = B.new_status()
    out = B.alloc_fwd_outputs(T, S)
    ws_f = poisoned_workspace(B.sapo_workspace_bytes(B.WS_FWD, T, H, V, dcode))
    B.sapo_policy_loss_fwd(hidden, W, ids, old_logp, adv, cu, eps_low, eps_high, grad_scale, out,
                           ws_f, status)
    if want_bwd:
        kind = B.WS_BWD | (B.WS_OUT_BF16 if out_dtype == torch.bfloat16 else 0)
        nbytes = (B.sapo_workspace_bytes(kind, T, H, V, dcode)
                  if bwd_workspace_bytes is None else bwd_workspace_bytes)
        ws_b = poisoned_workspace(nbytes)
        out["dhidden"] = torch.empty(T, H, dtype=out_dtype, device="cuda")
        out["dW"] = torch.empty(V, H, dtype=out_dtype, device="cuda") if accumulate_into is None else accumulate_into
        B.sapo_policy_loss_bwd(hidden, W, ids, out["lse"], out["gscale"], out["dhidden"], out["dW"],
                               accumulate_into is not None, ws_b, status)
    torch.cuda.synchronize()
    out["status"] = int(status.item())
    return out


def poisoned_workspace(nbytes: int) -> torch.Tensor:
    """Scratch for a library call with every byte 0xFF: any bf16 or fp32 read from a place the call
    has not written first is a NaN, and shows in the outputs."""
    return torch.full((nbytes,), 0xFF, dtype=torch.uint8, device="cuda")


def gpu_scores_fused(hidden, W, ids, old_logp, adv, cu, eps_low, eps_high, grad_scale=1.0,
                     workspace_bytes: Optional[int] = None, out_dtype: torch.dtype = torch.float32,
                     accumulate_into=None, **variant):
    """Loss and gradients through the single-pass call; returns device tensors."""
    T, H, V, S = hidden.shape[0], hidden.shape[1], W.shape[0], cu.numel() - 1
    status = B.new_status()
    out = B.alloc_fwd_outputs(T, S)
    kind = B.WS_FUSED | (B.WS_OUT_BF16 if out_dtype == torch.bfloat16 else 0)
    nbytes = (B.sapo_workspace_bytes(kind, T, H, V, B.DTYPE_BF16)
              if workspace_bytes is None else workspace_bytes)
    ws = poisoned_workspace(nbytes)
    out["dhidden"] = torch.empty(T, H, dtype=out_dtype, device="cuda")
    out["dW"] = torch.empty(V, H, dtype=out_dtype, device="cuda") if accumulate_into is None else accumulate_into
    B.sapo_policy_loss_fwd_bwd(hidden, W, ids, old_logp, adv, cu, eps_low, eps_high, grad_scale, out,
                               out["dhidden"], out["dW"], accumulate_into is not None, ws, status, **variant)
    torch.cuda.synchronize()
    out["status"] = int(status.item())
    return out


def rel_fro(x: np.ndarray, ref: np.ndarray) -> float:
    d = np.linalg.norm(np.asarray(x, dtype=np.float64) - ref)
    n = np.linalg.norm(ref)
    return float(d / n) if n > 0 else float(d)


def check_loss(loss_gpu: float, loss_ref: float, adv_ref: np.ndarray) -> None:
    """Relative 1e-3 where the loss is well-conditioned; it is a cancelling sum
    -(1/S) sum_s A_s mean_t(rho) with sum_s A_s = 0 per group, so when |L| is tiny compared
    with the size of its terms (mean |A|) an absolute bound of 1e-5 * mean|A| applies."""
    scale = float(np.mean(np.abs(adv_ref))) if len(adv_ref) else 0.0
    err = abs(loss_gpu - loss_ref)
    if abs(loss_ref) >= 1e-2 * scale and loss_ref != 0.0:
        assert err <= TOL_LOSS_REL * abs(loss_ref), (loss_gpu, loss_ref)
    else:
        assert err <= 1e-5 * max(scale, 1e-30) + 1e-12, (loss_gpu, loss_ref, scale)


def check_forward(out: Dict[str, torch.Tensor], ref: Dict[str, np.ndarray], adv_ref: np.ndarray,
                  cu: np.ndarray, eps_low: float, eps_high: float, rows=None) -> None:
    """Per-token forward outputs against the oracle (optionally on a subset of rows)."""
    sl = slice(None) if rows is None else rows
    g = {k: to_numpy(out[k]).astype(np.float64)[sl] for k in ("logp", "lse", "ratio", "surr", "gscale")}
    assert np.max(np.abs(g["logp"] - ref["logp"])) <= TOL_LOGP_ABS
    assert np.max(np.abs(g["lse"] - ref["lse"])) <= TOL_LOGP_ABS
    assert np.allclose(g["ratio"], ref["ratio"], rtol=3e-3, atol=0)
    # the min/clip decision is taken in fp32 on the device and fp64 in the oracle: tokens
    # whose ratio sits within the log-prob tolerance of a clip edge may legitimately differ
    rho = ref["ratio"]
    near = np.minimum(np.abs(rho - (1 - eps_low)), np.abs(rho - (1 + eps_high))) < 4e-3
    A_tok = np.repeat(adv_ref, np.diff(cu))[sl] if rows is None else None
    scale_u = np.abs(ref["surr"]).max() + 1e-30
    assert np.max(np.abs(g["surr"] - ref["surr"])[~near]) <= 4e-3 * scale_u
    gs = np.abs(ref["gscale"]).max() + 1e-30
    assert np.max(np.abs(g["gscale"] - ref["gscale"])[~near]) <= 4e-3 * gs
