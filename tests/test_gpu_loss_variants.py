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


ENTROPY_SHAPES = [
    # hidden, vocab, lengths: a ragged vocabulary tail, several vocab tiles and splits, a peaked head
    (64, 1000, ("uniform", 1, 40), 0.02),
    (328, 2500, ("uniform", 30, 120), 0.02),
    (128, 20000, ("uniform", 50, 90), 0.2),
]


@pytest.mark.parametrize("H,V,lengths,w_std", ENTROPY_SHAPES, ids=["vocab_tail", "many_tiles", "peaked"])
@pytest.mark.parametrize("fused", [False, True], ids=["separate_calls", "single_pass"])
def test_per_token_entropy_matches_the_oracle(H, V, lengths, w_std, fused):
    """The entropy of the policy's distribution at every position, a by-product of the forward
    epilogue, against the oracle's -sum p log p at the log-prob tolerance; asking for it must not
    change any other output."""
    recipe = gen.Recipe("ent", gen.DTYPE_BF16, H, V, 4, 2, 2, lengths, ("bernoulli", 0.5))
    batch = gen.make_batch(recipe, 71)
    b = batch.built
    if w_std != 0.02:                      # a head with a wide logit spread: low-entropy rows
        batch.W = gen.f32_to_bf16_bits(gen.as_f32(batch.W) * np.float32(w_std / 0.02))
    gen.install_old_logp(batch, U.oracle_current_logp(batch))
    adv = np.linspace(-1.0, 1.0, batch.S).astype(np.float32)
    ref_ent = orc.token_entropy(gen.as_f32(b.hidden), gen.as_f32(batch.W))
    args = (U.to_torch(b.hidden), U.to_torch(batch.W), U.to_torch(b.ids), U.to_torch(b.old_logp),
            U.to_torch(adv), U.to_torch(b.cu_seqlens), 0.2, 0.28)
    T, S = batch.T, batch.S
    ent = torch.full((T,), -1.0, device="cuda")
    if fused:
        plain = U.gpu_scores_fused(*args)
        out = U.gpu_scores_fused(*args, entropy=ent)
    else:
        plain = U.gpu_scores(*args, want_bwd=False)
        status = B.new_status()
        out = B.alloc_fwd_outputs(T, S)
        ws = torch.empty(B.sapo_workspace_bytes(B.WS_FWD, T, H, V, B.DTYPE_BF16), dtype=torch.uint8, device="cuda")
        B.sapo_policy_loss_fwd(*args, 1.0, out, ws, status, entropy=ent)
        torch.cuda.synchronize()
        assert status.item() == 0
    got = ent.cpu().numpy().astype(np.float64)
    assert np.max(np.abs(got - ref_ent)) <= U.TOL_LOGP_ABS, np.max(np.abs(got - ref_ent))
    assert got.min() >= -1e-4 and got.max() <= np.log(V) + 1e-4
    for k in ("logp", "lse", "ratio", "surr", "gscale", "loss"):
        assert torch.equal(out[k], plain[k]), k


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
