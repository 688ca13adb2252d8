"""ctypes binding of the SAPO B200 library: same names as the C ABI, argument marshalling
only.  torch supplies device memory and the current stream; every step of the path runs in
the library's CUDA kernels.  There is no fallback: if the shared library is missing or no
CUDA device is present, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Dict, Optional

import torch

from . import build as _build

DTYPE_BF16 = 0
DTYPE_F32 = 1
WS_FWD = 0
WS_BWD = 1
WS_BWD_ACTIVE = 2
WS_FUSED = 3
WS_OUT_BF16 = 0x100      # OR into the workspace kind: gradients in bf16
WS_GATHER = 0x200        # OR into the workspace kind: hidden rows read in place (..._gather)

ST_BITS = {
    0x01: "TOKEN_OVERFLOW", 0x02: "SEQ_OVERFLOW", 0x04: "BAD_INDEX", 0x08: "EMPTY_SEQUENCE",
    0x10: "BAD_TOKEN_ID", 0x20: "WAIT_TIMEOUT", 0x40: "NONFINITE_REWARD", 0x80: "EXP_RANGE",
    0x100: "NONFINITE_INPUT",
}

EXPORTS = ("sapo_pack_rollouts", "sapo_group_advantages", "sapo_policy_loss_fwd",
           "sapo_policy_loss_bwd", "sapo_workspace_bytes", "sapo_workspace_bytes_min",
           "sapo_status_string", "sapo_timing_enable", "sapo_timing_read", "sapo_launch_count",
           "sapo_policy_loss_fwd_static", "sapo_policy_loss_bwd_active", "sapo_policy_loss_fwd_bwd",
           "sapo_select_external", "sapo_group_advantages_warp", "sapo_debug_wait_timeout", "sapo_debug_bounds_violations",
           "sapo_policy_loss_fwd_bwd_gather", "sapo_lmhead_lse_partial", "sapo_policy_loss_from_partials", "sapo_policy_loss_bwd_shard",
           "sapo_select_workspace_bytes", "sapo_adam_step")
STATIC_SCRATCH_BYTES = 4 * 1024 * 1024
KERNEL_NAMES = ("pack_scan", "pack_copy", "group_adv", "split_bf16", "fwd_gemm", "loss_tail",
                "loss_final", "bwd_dz", "bwd_dh", "bwd_dw", "streamk_fixup", "compact", "select", "adam",
                "target_logit", "fwd_exp", "fused_tail")


class RolloutBufC(C.Structure):
    _fields_ = [("hidden", C.c_void_p), ("ids", C.c_void_p), ("old_logp", C.c_void_p),
                ("offsets", C.c_void_p), ("rewards", C.c_void_p), ("n_rollouts", C.c_int32)]


class SelectionC(C.Structure):
    _fields_ = [("q_offsets_local", C.c_void_p), ("local_idx", C.c_void_p),
                ("q_offsets_ext", C.c_void_p), ("ext_idx", C.c_void_p), ("Q", C.c_int32)]


class PackedC(C.Structure):
    _fields_ = [("hidden", C.c_void_p), ("ids", C.c_void_p), ("old_logp", C.c_void_p),
                ("rewards", C.c_void_p), ("cu_seqlens", C.c_void_p), ("seq_group", C.c_void_p),
                ("seq_is_ext", C.c_void_p), ("seq_src", C.c_void_p), ("tok_seq", C.c_void_p),
                ("tok_mask", C.c_void_p), ("group_offsets", C.c_void_p), ("n_tokens", C.c_void_p),
                ("n_seqs", C.c_void_p), ("max_tokens", C.c_int64), ("max_seqs", C.c_int32),
                ("tok_src", C.c_void_p)]


class LossCfgC(C.Structure):
    _fields_ = [("eps_low", C.c_float), ("eps_high", C.c_float), ("grad_scale", C.c_float),
                ("loss_agg", C.c_int32), ("kl_beta", C.c_float), ("ref_logp", C.c_void_p),
                ("entropy", C.c_void_p)]


_lib: Optional[C.CDLL] = None


def lib_path() -> str:
    return _build.LIB


def load() -> C.CDLL:
    """Load (building first if the sources are newer) and type the C ABI."""
    global _lib
    if _lib is not None:
        return _lib
    path = os.environ.get("SAPO_B200_LIB") or _build.LIB      # override: a differently built copy
    if not os.path.exists(path):
        path = _build.build()
    lib = C.CDLL(path)
    vp, i32, i64, f32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
    lib.sapo_pack_rollouts.restype = C.c_int
    lib.sapo_pack_rollouts.argtypes = [C.POINTER(RolloutBufC), C.POINTER(RolloutBufC),
                                       C.POINTER(SelectionC), i32, i32, C.POINTER(PackedC), vp, vp]
    lib.sapo_group_advantages.restype = C.c_int
    lib.sapo_group_advantages.argtypes = [vp, vp, i32, f32, i32, vp, vp, vp, vp, vp]
    lib.sapo_group_advantages_warp.restype = C.c_int
    lib.sapo_group_advantages_warp.argtypes = [vp, vp, i32, f32, i32, vp, vp, vp, vp, vp]
    lib.sapo_policy_loss_fwd.restype = C.c_int
    lib.sapo_policy_loss_fwd.argtypes = [vp, vp, i32, i64, i32, i32, i64, i64, vp, vp, vp, vp, i32,
                                         C.POINTER(LossCfgC), vp, vp, vp, vp, vp, vp, vp, vp, sz,
                                         vp, vp]
    lib.sapo_policy_loss_fwd_static.restype = C.c_int
    lib.sapo_policy_loss_fwd_static.argtypes = [vp, vp, i32, i64, i32, i32, i64, i64, vp, vp, vp, vp, i32,
                                                C.POINTER(LossCfgC), vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sapo_policy_loss_bwd.restype = C.c_int
    lib.sapo_policy_loss_bwd.argtypes = [vp, vp, i32, i64, i32, i32, i64, i64, vp, vp, vp, vp, vp,
                                         i32, i32, vp, sz, vp, vp]
    lib.sapo_policy_loss_bwd_active.restype = C.c_int
    lib.sapo_policy_loss_bwd_active.argtypes = [vp, vp, i32, i64, i32, i32, i64, i64, vp, vp, vp, vp, vp,
                                                i32, i32, vp, vp, sz, vp, vp]
    lib.sapo_policy_loss_fwd_bwd.restype = C.c_int
    lib.sapo_policy_loss_fwd_bwd.argtypes = [vp, vp, i32, i64, i32, i32, i64, i64, vp, vp, vp, vp, i32,
                                             C.POINTER(LossCfgC), vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32,
                                             vp, sz, vp, vp]
    lib.sapo_policy_loss_fwd_bwd_gather.restype = C.c_int
    lib.sapo_policy_loss_fwd_bwd_gather.argtypes = [vp, i64, vp, i64, vp, vp, i32, i64, i32, i32, i64, i64, vp, vp, vp,
                                                    vp, i32, C.POINTER(LossCfgC), vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                                    i32, i32, vp, sz, vp, vp]
    lib.sapo_select_external.restype = C.c_int
    lib.sapo_select_external.argtypes = [vp, vp, i32, i32, C.c_uint64, vp, vp, vp, vp, sz, vp]
    lib.sapo_select_workspace_bytes.restype = sz
    lib.sapo_select_workspace_bytes.argtypes = [i32]
    lib.sapo_adam_step.restype = C.c_int
    lib.sapo_adam_step.argtypes = [vp, vp, vp, vp, vp, i64, i32, i64, i32, f32, f32, f32, f32, vp]
    lib.sapo_workspace_bytes.restype = sz
    lib.sapo_workspace_bytes.argtypes = [i32, i64, i32, i32, i32]
    lib.sapo_workspace_bytes_min.restype = sz
    lib.sapo_workspace_bytes_min.argtypes = [i32, i64, i32, i32, i32]
    lib.sapo_timing_enable.restype = C.c_int
    lib.sapo_timing_enable.argtypes = [i32]
    lib.sapo_timing_read.restype = C.c_int
    lib.sapo_timing_read.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_int32)]
    lib.sapo_lmhead_lse_partial.restype = C.c_int
    lib.sapo_lmhead_lse_partial.argtypes = [vp, vp, i32, i64, i32, i32, i64, i64, vp, i32, vp, vp, sz, vp, vp]
    lib.sapo_policy_loss_from_partials.restype = C.c_int
    lib.sapo_policy_loss_from_partials.argtypes = [vp, i32, i64, i32, vp, vp, vp, vp, i32, C.POINTER(LossCfgC),
                                                   vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sapo_policy_loss_bwd_shard.restype = C.c_int
    lib.sapo_policy_loss_bwd_shard.argtypes = [vp, vp, i32, i64, i32, i32, i64, i64, vp, i32, vp, vp, vp, vp,
                                               i32, i32, vp, sz, vp, vp]
    lib.sapo_debug_wait_timeout.restype = C.c_int
    lib.sapo_debug_wait_timeout.argtypes = [i64, vp, vp]
    lib.sapo_debug_bounds_violations.restype = C.c_int64
    lib.sapo_debug_bounds_violations.argtypes = []
    lib.sapo_launch_count.restype = C.c_int64
    lib.sapo_launch_count.argtypes = []
    lib.sapo_status_string.restype = C.c_char_p
    lib.sapo_status_string.argtypes = [i32]
    _lib = lib
    return lib


class SapoError(RuntimeError):
    pass


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise SapoError(f"{what}: {load().sapo_status_string(rc).decode()} ({rc})")


def _require_cuda() -> None:
    if not torch.cuda.is_available():
        raise SapoError("the SAPO B200 library needs a CUDA device; there is no CPU path")


def _p(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _out_dtype_code(dhidden: torch.Tensor, dW_head: torch.Tensor) -> int:
    if dhidden.dtype != dW_head.dtype:
        raise SapoError("dhidden and dW_head must have the same element type")
    return _dtype_code(dhidden)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return DTYPE_BF16
    if t.dtype == torch.float32:
        return DTYPE_F32
    raise SapoError(f"unsupported element type {t.dtype}")


def sapo_timing_enable(on: bool) -> None:
    _check(load().sapo_timing_enable(1 if on else 0), "sapo_timing_enable")


def sapo_timing_read() -> Dict[str, Dict[str, float]]:
    """Summed milliseconds and launch count per kernel since the last read."""
    n = len(KERNEL_NAMES)
    ms = (C.c_float * n)()
    cnt = (C.c_int32 * n)()
    _check(load().sapo_timing_read(ms, cnt), "sapo_timing_read")
    return {KERNEL_NAMES[i]: {"ms": float(ms[i]), "launches": int(cnt[i])} for i in range(n)}


def sapo_launch_count() -> int:
    return int(load().sapo_launch_count())


def sapo_debug_wait_timeout(limit_clocks: int, status: torch.Tensor) -> None:
    """Make a bounded in-kernel wait run out (sets WAIT_TIMEOUT in `status`); see sapo.h."""
    _require_cuda()
    _check(load().sapo_debug_wait_timeout(int(limit_clocks), _p(status), _stream()), "sapo_debug_wait_timeout")


def decode_status(word: int):
    return [name for bit, name in ST_BITS.items() if word & bit]


def new_status(device="cuda") -> torch.Tensor:
    return torch.zeros(1, dtype=torch.int32, device=device)


# ------------------------------------------------------------------------------------------
@dataclass
class DeviceRollouts:
    """Device-resident rollout buffer (tensors named as in the C struct)."""
    hidden: torch.Tensor
    ids: torch.Tensor
    old_logp: torch.Tensor
    offsets: torch.Tensor
    rewards: torch.Tensor

    def c(self) -> RolloutBufC:
        return RolloutBufC(_p(self.hidden), _p(self.ids), _p(self.old_logp), _p(self.offsets),
                           _p(self.rewards), int(self.offsets.numel() - 1))


@dataclass
class DeviceSelection:
    q_offsets_local: torch.Tensor
    local_idx: torch.Tensor
    q_offsets_ext: torch.Tensor
    ext_idx: torch.Tensor

    def c(self) -> SelectionC:
        return SelectionC(_p(self.q_offsets_local), _p(self.local_idx), _p(self.q_offsets_ext),
                          _p(self.ext_idx), int(self.q_offsets_local.numel() - 1))


def alloc_packed(max_tokens: int, max_seqs: int, Q: int, H: int, dtype: torch.dtype,
                 device="cuda", copy_hidden: bool = True, tok_src: bool = False) -> Dict[str, torch.Tensor]:
    """Output buffers of sapo_pack_rollouts.  copy_hidden=False leaves out the packed copy of the
    hidden rows (then tok_src is needed: the loss reads the rows in place)."""
    i32, f32, u8 = torch.int32, torch.float32, torch.uint8
    e = lambda *s, dt: torch.empty(*s, dtype=dt, device=device)
    extra = {"tok_src": e(max_tokens, dt=torch.int64)} if (tok_src or not copy_hidden) else {}
    return {
        **extra, "H": H, "dtype": dtype,
        "hidden": e(max_tokens, H, dt=dtype) if copy_hidden else None, "ids": e(max_tokens, dt=i32),
        "old_logp": e(max_tokens, dt=f32), "rewards": e(max_seqs, dt=f32),
        "cu_seqlens": e(max_seqs + 1, dt=i32), "seq_group": e(max_seqs, dt=i32),
        "seq_is_ext": e(max_seqs, dt=u8), "seq_src": e(max_seqs, dt=i32),
        "tok_seq": e(max_tokens, dt=i32), "tok_mask": e(max_tokens, dt=u8),
        "group_offsets": e(Q + 1, dt=i32), "n_tokens": e(1, dt=i32), "n_seqs": e(1, dt=i32),
    }


def sapo_pack_rollouts(local: DeviceRollouts, ext: DeviceRollouts, sel: DeviceSelection,
                       out: Dict[str, torch.Tensor], status: torch.Tensor) -> None:
    """Enqueue the pack on the current stream; `out` comes from alloc_packed."""
    _require_cuda()
    H = int(out["H"])
    pc = PackedC(*[_p(out[k]) for k in ("hidden", "ids", "old_logp", "rewards", "cu_seqlens",
                                        "seq_group", "seq_is_ext", "seq_src", "tok_seq", "tok_mask",
                                        "group_offsets", "n_tokens", "n_seqs")],
                 int(out["ids"].numel()), int(out["seq_group"].numel()), _p(out.get("tok_src")))
    lc, ec, sc = local.c(), ext.c(), sel.c()
    rc = load().sapo_pack_rollouts(C.byref(lc), C.byref(ec), C.byref(sc), H,
                                   _dtype_code(local.hidden), C.byref(pc), _p(status), _stream())
    _check(rc, "sapo_pack_rollouts")


def sapo_group_advantages(rewards: torch.Tensor, group_offsets: torch.Tensor, adv_eps: float,
                          ddof: int, adv: torch.Tensor, mean: Optional[torch.Tensor],
                          std: Optional[torch.Tensor], status: torch.Tensor, warp_level: bool = False) -> None:
    """warp_level=True always takes the warp-level kernel (sapo_group_advantages_warp)."""
    _require_cuda()
    fn = load().sapo_group_advantages_warp if warp_level else load().sapo_group_advantages
    rc = fn(_p(rewards), _p(group_offsets), int(group_offsets.numel() - 1),
                                      float(adv_eps), int(ddof), _p(adv), _p(mean), _p(std),
                                      _p(status), _stream())
    _check(rc, "sapo_group_advantages")


def sapo_workspace_bytes(which: int, T: int, H: int, V: int, dtype: int) -> int:
    return int(load().sapo_workspace_bytes(which, T, H, V, dtype))


def sapo_workspace_bytes_min(which: int, T: int, H: int, V: int, dtype: int) -> int:
    return int(load().sapo_workspace_bytes_min(which, T, H, V, dtype))


def alloc_fwd_outputs(T: int, S: int, device="cuda") -> Dict[str, torch.Tensor]:
    f = lambda n: torch.empty(n, dtype=torch.float32, device=device)
    return {"logp": f(T), "lse": f(T), "ratio": f(T), "surr": f(T), "gscale": f(T),
            "seq_surr": f(S), "loss": f(1)}


def sapo_policy_loss_fwd(hidden: torch.Tensor, W_head: torch.Tensor, ids: torch.Tensor,
                         old_logp: torch.Tensor, adv: torch.Tensor, cu_seqlens: torch.Tensor,
                         eps_low: float, eps_high: float, grad_scale: float,
                         out: Dict[str, torch.Tensor], workspace: torch.Tensor,
                         status: torch.Tensor, T: Optional[int] = None, loss_agg: int = 0,
                         kl_beta: float = 0.0, ref_logp: Optional[torch.Tensor] = None,
                         entropy: Optional[torch.Tensor] = None) -> None:
    """entropy: optional float32 [T] output, the per-token entropy of the policy's distribution."""
    _require_cuda()
    T = int(hidden.shape[0]) if T is None else int(T)
    H, V = int(hidden.shape[1]), int(W_head.shape[0])
    S = int(cu_seqlens.numel() - 1)
    cfg = LossCfgC(eps_low, eps_high, grad_scale, int(loss_agg), float(kl_beta), _p(ref_logp), _p(entropy))
    rc = load().sapo_policy_loss_fwd(
        _p(hidden), _p(W_head), _dtype_code(hidden), T, H, V, hidden.stride(0), W_head.stride(0),
        _p(ids), _p(old_logp), _p(adv), _p(cu_seqlens), S, C.byref(cfg),
        _p(out["logp"]), _p(out["lse"]), _p(out["ratio"]), _p(out["surr"]), _p(out["gscale"]),
        _p(out.get("seq_surr")), _p(out["loss"]), _p(workspace), workspace.numel() * workspace.element_size(),
        _p(status), _stream())
    _check(rc, "sapo_policy_loss_fwd")


def sapo_policy_loss_fwd_static(hidden: torch.Tensor, W_head: torch.Tensor, ids: torch.Tensor,
                                old_logp: torch.Tensor, adv: torch.Tensor, cu_seqlens: torch.Tensor,
                                eps_low: float, eps_high: float, grad_scale: float,
                                out: Dict[str, torch.Tensor], status: torch.Tensor,
                                T: Optional[int] = None) -> None:
    """sapo_policy_loss_fwd for callers that may not allocate device memory: the scratch is the
    array built into the library (STATIC_SCRATCH_BYTES), so no workspace tensor is passed.
    Raises SapoError when the sizes need more scratch than that, or for fp32 operands."""
    _require_cuda()
    T = int(hidden.shape[0]) if T is None else int(T)
    H, V = int(hidden.shape[1]), int(W_head.shape[0])
    S = int(cu_seqlens.numel() - 1)
    cfg = LossCfgC(eps_low, eps_high, grad_scale, 0, 0.0, None, None)
    rc = load().sapo_policy_loss_fwd_static(
        _p(hidden), _p(W_head), _dtype_code(hidden), T, H, V, hidden.stride(0), W_head.stride(0),
        _p(ids), _p(old_logp), _p(adv), _p(cu_seqlens), S, C.byref(cfg),
        _p(out["logp"]), _p(out["lse"]), _p(out["ratio"]), _p(out["surr"]), _p(out["gscale"]),
        _p(out.get("seq_surr")), _p(out["loss"]), _p(status), _stream())
    _check(rc, "sapo_policy_loss_fwd_static")


def sapo_policy_loss_bwd(hidden: torch.Tensor, W_head: torch.Tensor, ids: torch.Tensor,
                         lse: torch.Tensor, gscale: torch.Tensor, dhidden: torch.Tensor,
                         dW_head: torch.Tensor, accumulate_dW: bool, workspace: torch.Tensor,
                         status: torch.Tensor, T: Optional[int] = None) -> None:
    _require_cuda()
    T = int(hidden.shape[0]) if T is None else int(T)
    H, V = int(hidden.shape[1]), int(W_head.shape[0])
    rc = load().sapo_policy_loss_bwd(
        _p(hidden), _p(W_head), _dtype_code(hidden), T, H, V, hidden.stride(0), W_head.stride(0),
        _p(ids), _p(lse), _p(gscale), _p(dhidden), _p(dW_head), _out_dtype_code(dhidden, dW_head),
        1 if accumulate_dW else 0,
        _p(workspace), workspace.numel() * workspace.element_size(), _p(status), _stream())
    _check(rc, "sapo_policy_loss_bwd")


def sapo_policy_loss_bwd_active(hidden: torch.Tensor, W_head: torch.Tensor, ids: torch.Tensor,
                                lse: torch.Tensor, gscale: torch.Tensor, dhidden: torch.Tensor,
                                dW_head: torch.Tensor, accumulate_dW: bool, workspace: torch.Tensor,
                                status: torch.Tensor, n_active: Optional[torch.Tensor] = None,
                                T: Optional[int] = None) -> None:
    """Backward over the tokens with a non-zero gradient factor only (same results)."""
    _require_cuda()
    T = int(hidden.shape[0]) if T is None else int(T)
    H, V = int(hidden.shape[1]), int(W_head.shape[0])
    rc = load().sapo_policy_loss_bwd_active(
        _p(hidden), _p(W_head), _dtype_code(hidden), T, H, V, hidden.stride(0), W_head.stride(0),
        _p(ids), _p(lse), _p(gscale), _p(dhidden), _p(dW_head), _out_dtype_code(dhidden, dW_head),
        1 if accumulate_dW else 0, _p(n_active),
        _p(workspace), workspace.numel() * workspace.element_size(), _p(status), _stream())
    _check(rc, "sapo_policy_loss_bwd_active")


def sapo_policy_loss_fwd_bwd(hidden: torch.Tensor, W_head: torch.Tensor, ids: torch.Tensor,
                             old_logp: torch.Tensor, adv: torch.Tensor, cu_seqlens: torch.Tensor,
                             eps_low: float, eps_high: float, grad_scale: float,
                             out: Dict[str, torch.Tensor], dhidden: torch.Tensor, dW_head: torch.Tensor,
                             accumulate_dW: bool, workspace: torch.Tensor, status: torch.Tensor,
                             T: Optional[int] = None, loss_agg: int = 0, kl_beta: float = 0.0,
                             ref_logp: Optional[torch.Tensor] = None,
                             entropy: Optional[torch.Tensor] = None) -> None:
    """Loss and both gradients in one call with a single pass over the logits (bf16 only)."""
    _require_cuda()
    T = int(hidden.shape[0]) if T is None else int(T)
    H, V = int(hidden.shape[1]), int(W_head.shape[0])
    S = int(cu_seqlens.numel() - 1)
    cfg = LossCfgC(eps_low, eps_high, grad_scale, int(loss_agg), float(kl_beta), _p(ref_logp), _p(entropy))
    rc = load().sapo_policy_loss_fwd_bwd(
        _p(hidden), _p(W_head), _dtype_code(hidden), T, H, V, hidden.stride(0), W_head.stride(0),
        _p(ids), _p(old_logp), _p(adv), _p(cu_seqlens), S, C.byref(cfg),
        _p(out["logp"]), _p(out["lse"]), _p(out["ratio"]), _p(out["surr"]), _p(out["gscale"]),
        _p(out.get("seq_surr")), _p(out["loss"]), _p(dhidden), _p(dW_head), _out_dtype_code(dhidden, dW_head),
        1 if accumulate_dW else 0,
        _p(workspace), workspace.numel() * workspace.element_size(), _p(status), _stream())
    _check(rc, "sapo_policy_loss_fwd_bwd")


def sapo_policy_loss_fwd_bwd_gather(local_hidden: torch.Tensor, ext_hidden: torch.Tensor, tok_src: torch.Tensor,
                                    W_head: torch.Tensor, ids: torch.Tensor, old_logp: torch.Tensor,
                                    adv: torch.Tensor, cu_seqlens: torch.Tensor, eps_low: float, eps_high: float,
                                    grad_scale: float, out: Dict[str, torch.Tensor], dhidden: torch.Tensor,
                                    dW_head: torch.Tensor, accumulate_dW: bool, workspace: torch.Tensor,
                                    status: torch.Tensor, T: Optional[int] = None, loss_agg: int = 0,
                                    kl_beta: float = 0.0, ref_logp: Optional[torch.Tensor] = None,
                                    entropy: Optional[torch.Tensor] = None) -> None:
    """sapo_policy_loss_fwd_bwd with the hidden rows read in place from the two rollout stores
    through tok_src (int64 [T], from sapo_pack_rollouts): no packed copy of the hidden states."""
    _require_cuda()
    T = int(tok_src.shape[0]) if T is None else int(T)
    H, V = int(W_head.shape[1]), int(W_head.shape[0])
    S = int(cu_seqlens.numel() - 1)
    ld = int(local_hidden.stride(0)) if local_hidden.shape[0] > 0 else int(ext_hidden.stride(0))
    if local_hidden.shape[0] > 0 and ext_hidden.shape[0] > 0 and local_hidden.stride(0) != ext_hidden.stride(0):
        raise SapoError("the two rollout stores must have the same row pitch")
    cfg = LossCfgC(eps_low, eps_high, grad_scale, int(loss_agg), float(kl_beta), _p(ref_logp), _p(entropy))
    rc = load().sapo_policy_loss_fwd_bwd_gather(
        _p(local_hidden), int(local_hidden.shape[0]), _p(ext_hidden), int(ext_hidden.shape[0]), _p(tok_src),
        _p(W_head), _dtype_code(W_head), T, H, V, ld, W_head.stride(0),
        _p(ids), _p(old_logp), _p(adv), _p(cu_seqlens), S, C.byref(cfg),
        _p(out["logp"]), _p(out["lse"]), _p(out["ratio"]), _p(out["surr"]), _p(out["gscale"]),
        _p(out.get("seq_surr")), _p(out["loss"]), _p(dhidden), _p(dW_head), _out_dtype_code(dhidden, dW_head),
        1 if accumulate_dW else 0,
        _p(workspace), workspace.numel() * workspace.element_size(), _p(status), _stream())
    _check(rc, "sapo_policy_loss_fwd_bwd_gather")


def sapo_lmhead_lse_partial(hidden: torch.Tensor, W_shard: torch.Tensor, ids: torch.Tensor, vocab_offset: int,
                            triple: torch.Tensor, workspace: torch.Tensor, status: torch.Tensor) -> None:
    """(max, sum, target logit) per token over one vocabulary shard; triple is float32 [3, T]."""
    _require_cuda()
    T, H, V = int(hidden.shape[0]), int(hidden.shape[1]), int(W_shard.shape[0])
    rc = load().sapo_lmhead_lse_partial(
        _p(hidden), _p(W_shard), _dtype_code(hidden), T, H, V, hidden.stride(0), W_shard.stride(0), _p(ids),
        int(vocab_offset), _p(triple), _p(workspace), workspace.numel() * workspace.element_size(), _p(status),
        _stream())
    _check(rc, "sapo_lmhead_lse_partial")


def sapo_policy_loss_from_partials(triples: torch.Tensor, V: int, ids: torch.Tensor, old_logp: torch.Tensor,
                                   adv: torch.Tensor, cu_seqlens: torch.Tensor, eps_low: float, eps_high: float,
                                   grad_scale: float, out: Dict[str, torch.Tensor], status: torch.Tensor,
                                   loss_agg: int = 0, kl_beta: float = 0.0,
                                   ref_logp: Optional[torch.Tensor] = None) -> None:
    """The loss tail over the gathered triples of all shards, float32 [n_parts, 3, T]."""
    _require_cuda()
    n_parts, T = int(triples.shape[0]), int(triples.shape[2])
    cfg = LossCfgC(eps_low, eps_high, grad_scale, int(loss_agg), float(kl_beta), _p(ref_logp), None)
    rc = load().sapo_policy_loss_from_partials(
        _p(triples), n_parts, T, int(V), _p(ids), _p(old_logp), _p(adv), _p(cu_seqlens),
        int(cu_seqlens.numel() - 1), C.byref(cfg), _p(out["logp"]), _p(out["lse"]), _p(out["ratio"]),
        _p(out["surr"]), _p(out["gscale"]), _p(out["seq_surr"]), _p(out["loss"]), _p(status), _stream())
    _check(rc, "sapo_policy_loss_from_partials")


def sapo_policy_loss_bwd_shard(hidden: torch.Tensor, W_shard: torch.Tensor, ids: torch.Tensor, vocab_offset: int,
                               lse: torch.Tensor, gscale: torch.Tensor, dhidden: torch.Tensor,
                               dW_shard: torch.Tensor, accumulate_dW: bool, workspace: torch.Tensor,
                               status: torch.Tensor) -> None:
    """Backward of one vocabulary shard: dW_shard is final, dhidden is to be summed over the shards."""
    _require_cuda()
    T, H, V = int(hidden.shape[0]), int(hidden.shape[1]), int(W_shard.shape[0])
    rc = load().sapo_policy_loss_bwd_shard(
        _p(hidden), _p(W_shard), _dtype_code(hidden), T, H, V, hidden.stride(0), W_shard.stride(0), _p(ids),
        int(vocab_offset), _p(lse), _p(gscale), _p(dhidden), _p(dW_shard), _out_dtype_code(dhidden, dW_shard),
        1 if accumulate_dW else 0, _p(workspace), workspace.numel() * workspace.element_size(), _p(status),
        _stream())
    _check(rc, "sapo_policy_loss_bwd_shard")


def sapo_select_external(rewards: torch.Tensor, group_offsets: torch.Tensor, J: int, seed: int):
    """Filter the pool (drop entries with all-equal rewards) and draw J of the rest uniformly.
    Returns (selected [J] int32, n_selected [1], n_candidates [1]) device tensors."""
    _require_cuda()
    n = int(group_offsets.numel() - 1)
    dev = group_offsets.device
    selected = torch.empty(max(J, 1), dtype=torch.int32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    n_cand = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = torch.empty(int(load().sapo_select_workspace_bytes(n)) // 8 + 1, dtype=torch.int64, device=dev)
    rc = load().sapo_select_external(_p(rewards), _p(group_offsets), n, int(J), int(seed) & (2**64 - 1),
                                     _p(selected), _p(n_sel), _p(n_cand), _p(ws), ws.numel() * 8, _stream())
    _check(rc, "sapo_select_external")
    return selected, n_sel, n_cand


def sapo_adam_step(master: torch.Tensor, m: torch.Tensor, v: torch.Tensor, grad: torch.Tensor,
                   w_bf16: Optional[torch.Tensor], step: int, lr: float = 1e-3, beta1: float = 0.9,
                   beta2: float = 0.999, eps: float = 1e-8) -> None:
    """One Adam step on a 2-D fp32 master weight; rewrites its bf16 copy if given."""
    _require_cuda()
    rows, cols = int(master.shape[0]), int(master.shape[1])
    ld = int(w_bf16.stride(0)) if w_bf16 is not None else cols
    rc = load().sapo_adam_step(_p(master), _p(m), _p(v), _p(grad), _p(w_bf16), rows, cols, ld, int(step),
                               lr, beta1, beta2, eps, _stream())
    _check(rc, "sapo_adam_step")
