"""The compacting backward (only tokens with a non-zero gradient factor are contracted) against
the oracle and against the regular backward."""
import numpy as np
import pytest
import torch

from oracle import sapo_oracle as orc
from paper_2509_08721_b200 import binding as B
from paper_2509_08721_b200 import inputs as gen
from tests import util as U

pytestmark = pytest.mark.gpu


def forward(batch, adv_np, eps=(0.2, 0.28)):
    b = batch.built
    hidden, W, ids = U.to_torch(b.hidden), U.to_torch(batch.W), U.to_torch(b.ids)
    T, H, V, S = hidden.shape[0], hidden.shape[1], W.shape[0], batch.S
    out, status = B.alloc_fwd_outputs(T, S), B.new_status()
    ws = torch.empty(B.sapo_workspace_bytes(B.WS_FWD, T, H, V, B.DTYPE_BF16), dtype=torch.uint8, device="cuda")
    B.sapo_policy_loss_fwd(hidden, W, ids, U.to_torch(b.old_logp), U.to_torch(adv_np.astype(np.float32)),
                           U.to_torch(b.cu_seqlens), eps[0], eps[1], 1.0, out, ws, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    return hidden, W, ids, out


def backward(kind, hidden, W, ids, out, ws_bytes=None):
    T, H, V = hidden.shape[0], hidden.shape[1], W.shape[0]
    which = B.WS_BWD_ACTIVE if kind == "active" else B.WS_BWD
    n = B.sapo_workspace_bytes(which, T, H, V, B.DTYPE_BF16) if ws_bytes is None else ws_bytes
    ws = torch.empty(n, dtype=torch.uint8, device="cuda")
    dH = torch.full((T, H), float("nan"), device="cuda")
    dW = torch.full((V, H), float("nan"), device="cuda")
    status = B.new_status()
    n_active = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    if kind == "active":
        B.sapo_policy_loss_bwd_active(hidden, W, ids, out["lse"], out["gscale"], dH, dW, False, ws, status, n_active)
    else:
        B.sapo_policy_loss_bwd(hidden, W, ids, out["lse"], out["gscale"], dH, dW, False, ws, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    return dH, dW, int(n_active.item())


def make(seed, Q=8, H=128, V=3000, lengths=("uniform", 30, 120), noise=0.15):
    recipe = gen.Recipe("act", gen.DTYPE_BF16, H, V, Q, 2, 2, lengths, ("bernoulli", 0.5),
                        equal_reward_fraction=0.25, noise_sigma=noise)
    batch = gen.make_batch(recipe, seed)
    gen.install_old_logp(batch, U.oracle_current_logp(batch))
    adv = orc.group_advantages(batch.built.rewards, batch.built.group_offsets, adv_eps=1e-6)["adv"]
    return batch, adv


@pytest.mark.parametrize("seed,min_panel", [(51, False), (52, True)])
def test_active_backward_matches_oracle_and_regular_backward(seed, min_panel):
    batch, adv = make(seed)
    b = batch.built
    hidden, W, ids, out = forward(batch, adv)
    g = out["gscale"].cpu().numpy()
    n_ref = int((g != 0).sum())
    assert 0 < n_ref < batch.T                       # zero-advantage groups and clipped tokens exist
    ws_bytes = None
    if min_panel:                                    # one 128-token panel: several chunks of active rows
        ws_bytes = (B.sapo_workspace_bytes(B.WS_BWD_ACTIVE, batch.T, 128, 3000, B.DTYPE_BF16)
                    - B.sapo_workspace_bytes(B.WS_BWD, batch.T, 128, 3000, B.DTYPE_BF16)
                    + B.sapo_workspace_bytes_min(B.WS_BWD, batch.T, 128, 3000, B.DTYPE_BF16))
        assert n_ref > 256
    dH, dW, n_active = backward("active", hidden, W, ids, out, ws_bytes)
    assert n_active == n_ref
    ref = orc.policy_loss_bwd(gen.as_f32(b.hidden), gen.as_f32(batch.W), b.ids,
                              out["lse"].cpu().numpy(), g)
    assert U.rel_fro(dH.cpu().numpy(), ref["dhidden"]) <= U.TOL_GRAD_FRO
    assert U.rel_fro(dW.cpu().numpy(), ref["dW"]) <= U.TOL_GRAD_FRO
    assert torch.all(dH[torch.from_numpy(g == 0).cuda()] == 0)
    dH2, dW2, _ = backward("regular", hidden, W, ids, out)
    assert U.rel_fro(dH.cpu().numpy(), dH2.double().cpu().numpy()) <= 1e-4
    assert U.rel_fro(dW.cpu().numpy(), dW2.double().cpu().numpy()) <= 1e-4


def test_active_backward_with_no_and_with_all_tokens_active():
    batch, adv = make(53, Q=4, lengths=("uniform", 5, 40), noise=0.01)
    hidden, W, ids, out = forward(batch, np.zeros_like(adv))          # every advantage zero
    dH, dW, n_active = backward("active", hidden, W, ids, out)
    assert n_active == 0 and torch.all(dH == 0) and torch.all(dW == 0)
    hidden, W, ids, out = forward(batch, np.ones_like(adv), eps=(0.9, 0.9))   # nothing clipped
    dH, dW, n_active = backward("active", hidden, W, ids, out)
    assert n_active == batch.T
    dH2, dW2, _ = backward("regular", hidden, W, ids, out)
    assert U.rel_fro(dH.cpu().numpy(), dH2.double().cpu().numpy()) <= 1e-4
    assert U.rel_fro(dW.cpu().numpy(), dW2.double().cpu().numpy()) <= 1e-4
