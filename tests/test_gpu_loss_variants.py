"""Loss variants on the device against the oracle: token-level aggregation and the optional
KL penalty towards a reference policy (the paper runs with the penalty weight at zero)."""
import numpy as np
import pytest
import torch

from oracle import sapo_oracle as orc
from paper_2509_08721_b200 import binding as B
from paper_2509_08721_b200 import inputs as gen
from tests import util as U

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("loss_agg,kl_beta", [(1, 0.0), (0, 0.25), (1, 0.25)])
def test_loss_variants_match_the_oracle(loss_agg, kl_beta):
    recipe = gen.Recipe("var", gen.DTYPE_BF16, 128, 2000, 4, 2, 2, ("uniform", 10, 90), ("bernoulli", 0.5))
    batch = gen.make_batch(recipe, 61)
    b = batch.built
    cur = U.oracle_current_logp(batch)
    gen.install_old_logp(batch, cur)
    rng = np.random.default_rng(3)
    ref_lp = (cur + rng.normal(size=batch.T).astype(np.float32) * np.float32(0.2)).astype(np.float32)
    adv = orc.group_advantages(b.rewards, b.group_offsets, adv_eps=1e-6)["adv"]
    h, W = gen.as_f32(b.hidden), gen.as_f32(batch.W)
    ref = orc.policy_loss_fwd(h, W, b.ids, b.old_logp, adv, b.cu_seqlens, 0.2, 0.28, grad_scale=1.5,
                              loss_agg=loss_agg, kl_beta=kl_beta, ref_logp=ref_lp)
    grads = orc.policy_loss_bwd(h, W, b.ids, ref["lse"], ref["gscale"])

    hidden, Wd, ids = U.to_torch(b.hidden), U.to_torch(batch.W), U.to_torch(b.ids)
    T, S, H, V = batch.T, batch.S, 128, 2000
    out, status = B.alloc_fwd_outputs(T, S), B.new_status()
    ws = torch.empty(B.sapo_workspace_bytes(B.WS_FWD, T, H, V, B.DTYPE_BF16), dtype=torch.uint8, device="cuda")
    B.sapo_policy_loss_fwd(hidden, Wd, ids, U.to_torch(b.old_logp), U.to_torch(adv.astype(np.float32)),
                           U.to_torch(b.cu_seqlens), 0.2, 0.28, 1.5, out, ws, status,
                           loss_agg=loss_agg, kl_beta=kl_beta,
                           ref_logp=U.to_torch(ref_lp) if kl_beta else None)
    wsb = torch.empty(B.sapo_workspace_bytes(B.WS_BWD, T, H, V, B.DTYPE_BF16), dtype=torch.uint8, device="cuda")
    dH = torch.empty(T, H, device="cuda")
    dW = torch.empty(V, H, device="cuda")
    B.sapo_policy_loss_bwd(hidden, Wd, ids, out["lse"], out["gscale"], dH, dW, False, wsb, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    U.check_forward(out, ref, adv, b.cu_seqlens, 0.2, 0.28)
    seq = out["seq_surr"].cpu().numpy().astype(np.float64)
    scale = np.abs(adv).max() + kl_beta
    assert np.max(np.abs(seq - ref["seq_surr"])) <= 1e-3 * scale
    assert abs(out["loss"].item() - ref["loss"]) <= 1e-3 * abs(ref["loss"]) + 1e-5 * scale
    assert U.rel_fro(dH.cpu().numpy(), grads["dhidden"]) <= U.TOL_GRAD_FRO
    assert U.rel_fro(dW.cpu().numpy(), grads["dW"]) <= U.TOL_GRAD_FRO


def test_kl_without_reference_is_rejected():
    x = torch.zeros(8, 16, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(16, 16, dtype=torch.bfloat16, device="cuda")
    i = torch.zeros(8, dtype=torch.int32, device="cuda")
    f = torch.zeros(8, device="cuda")
    cu = torch.tensor([0, 8], dtype=torch.int32, device="cuda")
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SapoError):
        B.sapo_policy_loss_fwd(x, W, i, f, f[:1], cu, 0.2, 0.2, 1.0, B.alloc_fwd_outputs(8, 1), ws,
                               B.new_status(), kl_beta=0.1)
