"""What the loss calls promise about their per-token arguments: every token of [0, T) gets
defined outputs even when T is the capacity of the packed buffers rather than the token count
(the pack leaves the count on the device), a cu_seqlens that leaves [0, T] is clamped and
reported, and non-finite old log-probs or advantages mask their tokens and are reported."""
import numpy as np
import pytest
import torch

from oracle import sapo_oracle as orc
from paper_2509_08721_b200 import binding as B
from paper_2509_08721_b200 import inputs as gen
from tests import util as U

pytestmark = pytest.mark.gpu


def _recipe(**kw):
    base = dict(name="contract", dtype=gen.DTYPE_BF16, H=320, V=2500, Q=5, I=2, J=2,
                length_law=("uniform", 30, 110), reward_law=("bernoulli", 0.5))
    base.update(kw)
    return gen.Recipe(**base)


def _oracle(batch, adv):
    b = batch.built
    return orc.policy_loss_fwd_bwd_rows(gen.as_f32(b.hidden), gen.as_f32(batch.W), b.ids, b.old_logp, adv,
                                        b.cu_seqlens, 0.2, 0.28)


@pytest.mark.parametrize("fused", [False, True], ids=["separate_calls", "single_pass"])
@pytest.mark.parametrize("extra", [37, 300])
def test_scoring_the_whole_capacity_without_reading_the_token_count(fused, extra):
    batch = gen.make_batch(_recipe(), 77)
    gen.install_old_logp(batch, U.oracle_current_logp(batch))
    T, S, cap = batch.T, batch.S, batch.T + extra
    packed, st = U.gpu_pack(batch, max_tokens=cap, max_seqs=S)
    assert st == 0
    assert not packed["hidden"][T:].view(torch.int16).any()      # the pack zero-fills the unused slots
    adv_ref = orc.group_advantages(batch.built.rewards, batch.built.group_offsets,
                                   adv_eps=float(np.float32(1e-6)))["adv"]
    adv = U.to_torch(adv_ref.astype(np.float32))
    W = U.to_torch(batch.W)
    args = (packed["hidden"], W, packed["ids"], packed["old_logp"], adv, packed["cu_seqlens"], 0.2, 0.28)
    # T is taken from hidden.shape[0] = capacity: more tokens than the sequences cover
    out = U.gpu_scores_fused(*args) if fused else U.gpu_scores(*args)
    assert out["status"] == 0
    ref = _oracle(batch, adv_ref)
    head = {k: out[k][:T] for k in ("logp", "lse", "ratio", "surr", "gscale")}
    U.check_forward(head, ref, adv_ref, batch.built.cu_seqlens, 0.2, 0.28)
    for k in ("logp", "lse", "ratio", "surr", "gscale"):
        assert not out[k][T:].any(), k                            # masked: defined, and zero
    assert not out["dhidden"][T:].any()
    U.check_loss(float(out["loss"].item()), ref["loss"], adv_ref)
    assert U.rel_fro(out["dhidden"][:T].cpu().numpy(), ref["dhidden"]) <= U.TOL_GRAD_FRO
    assert U.rel_fro(out["dW"].cpu().numpy(), ref["dW"]) <= U.TOL_GRAD_FRO


@pytest.mark.parametrize("fused", [False, True], ids=["separate_calls", "single_pass"])
def test_cu_seqlens_outside_the_token_range_is_clamped_and_reported(fused):
    batch = gen.make_batch(_recipe(Q=3), 78)
    gen.install_old_logp(batch, U.oracle_current_logp(batch))
    b = batch.built
    T, S = batch.T, batch.S
    cu = b.cu_seqlens.copy()
    cu[-1] = T + 1000                                             # the last sequence claims tokens that do not exist
    adv = np.linspace(-1, 1, S).astype(np.float32)
    args = (U.to_torch(b.hidden), U.to_torch(batch.W), U.to_torch(b.ids), U.to_torch(b.old_logp),
            U.to_torch(adv), U.to_torch(cu), 0.2, 0.28)
    out = U.gpu_scores_fused(*args) if fused else U.gpu_scores(*args)
    assert out["status"] == 0x04
    # clamped to [0, T] the table is the true one: same results as the oracle's on it
    ref = orc.policy_loss_fwd(gen.as_f32(b.hidden), gen.as_f32(batch.W), b.ids, b.old_logp, adv, b.cu_seqlens,
                              0.2, 0.28)
    U.check_forward(out, ref, adv.astype(np.float64), b.cu_seqlens, 0.2, 0.28)
    U.check_loss(float(out["loss"].item()), ref["loss"], adv.astype(np.float64))
    assert torch.isfinite(out["dW"]).all() and torch.isfinite(out["dhidden"]).all()


@pytest.mark.parametrize("fused", [False, True], ids=["separate_calls", "single_pass"])
def test_nonfinite_old_logp_or_advantage_masks_the_tokens_and_is_reported(fused):
    batch = gen.make_batch(_recipe(Q=3), 79)
    gen.install_old_logp(batch, U.oracle_current_logp(batch))
    b = batch.built
    T, S = batch.T, batch.S
    adv = np.linspace(-1, 1, S).astype(np.float32)
    old = b.old_logp.copy()
    t_bad = int(b.cu_seqlens[1]) + 3                              # a token of the second sequence
    old[t_bad] = np.nan
    adv_bad = adv.copy()
    s_bad = S - 1
    adv_bad[s_bad] = np.inf                                       # and a whole sequence
    args = (U.to_torch(b.hidden), U.to_torch(batch.W), U.to_torch(b.ids), U.to_torch(old),
            U.to_torch(adv_bad), U.to_torch(b.cu_seqlens), 0.2, 0.28)
    out = U.gpu_scores_fused(*args) if fused else U.gpu_scores(*args)
    assert out["status"] == 0x100
    # the oracle on finite stand-ins: every other token is unaffected
    adv_fin = adv.copy()
    adv_fin[s_bad] = 0.0
    ref = orc.policy_loss_fwd(gen.as_f32(b.hidden), gen.as_f32(batch.W), b.ids, b.old_logp, adv_fin, b.cu_seqlens,
                              0.2, 0.28)
    masked = np.zeros(T, dtype=bool)
    masked[t_bad] = True
    masked[b.cu_seqlens[s_bad]:b.cu_seqlens[s_bad + 1]] = True
    for k in ("ratio", "surr", "gscale"):
        got = out[k].cpu().numpy()
        assert np.all(got[masked] == 0.0), k
    keep = ~masked
    assert np.max(np.abs(out["logp"].cpu().numpy() - ref["logp"])) <= U.TOL_LOGP_ABS    # log-probs stay defined
    assert np.allclose(out["ratio"].cpu().numpy()[keep], ref["ratio"][keep], rtol=3e-3)
    # the masked token counts in its sequence's length but adds nothing
    seq1 = slice(int(b.cu_seqlens[1]), int(b.cu_seqlens[2]))
    u = ref["surr"][seq1].copy()
    u[t_bad - seq1.start] = 0.0
    assert abs(out["seq_surr"][1].item() - u.mean()) <= 1e-3 * np.abs(adv).max()
    assert out["seq_surr"][s_bad].item() == 0.0
    assert torch.isfinite(out["loss"]).all()
    assert torch.isfinite(out["dW"]).all() and torch.isfinite(out["dhidden"]).all()
    assert not out["dhidden"][t_bad].any()


def test_a_bounded_wait_that_runs_out_sets_the_status_bit_and_leaves_the_context_usable():
    """Every in-kernel wait of the library has a limit.  The probe waits 100,000 clocks on a
    barrier nobody arrives at: it must come back with WAIT_TIMEOUT set, and a regular call right
    after it must run clean."""
    status = B.new_status()
    B.sapo_debug_wait_timeout(100_000, status)
    torch.cuda.synchronize()
    assert status.item() == 0x20 and B.decode_status(status.item()) == ["WAIT_TIMEOUT"]
    # nothing is left behind: a scoring step on the same stream is clean and correct
    batch = gen.make_batch(_recipe(Q=2), 80)
    gen.install_old_logp(batch, U.oracle_current_logp(batch))
    b = batch.built
    adv = np.linspace(-1, 1, batch.S).astype(np.float32)
    out = U.gpu_scores_fused(U.to_torch(b.hidden), U.to_torch(batch.W), U.to_torch(b.ids), U.to_torch(b.old_logp),
                             U.to_torch(adv), U.to_torch(b.cu_seqlens), 0.2, 0.28)
    assert out["status"] == 0
    ref = orc.policy_loss_fwd(gen.as_f32(b.hidden), gen.as_f32(batch.W), b.ids, b.old_logp, adv, b.cu_seqlens,
                              0.2, 0.28)
    U.check_forward(out, ref, adv.astype(np.float64), b.cu_seqlens, 0.2, 0.28)
    # a limit outside the allowed range is refused on the host
    with pytest.raises(B.SapoError):
        B.sapo_debug_wait_timeout(10**9, status)


@pytest.mark.parametrize("V,parts", [(2500, 2), (1000, 3)])
def test_vocabulary_shards_on_one_device_add_up_to_the_unsharded_call(V, parts):
    """The three shard entry points, run for every shard in turn on one GPU (no rank waits for
    another): the gathered triples give the same forward outputs as the unsharded call, the
    shards' dW rows and the sum of their dhidden shares match the oracle."""
    from paper_2509_08721_b200.vocab_parallel import CudaBackend, shard_bounds
    batch = gen.make_batch(_recipe(V=V, Q=3), 81)
    gen.install_old_logp(batch, U.oracle_current_logp(batch))
    b = batch.built
    T, S, H = batch.T, batch.S, batch.H
    adv = np.linspace(-1, 1, S).astype(np.float32)
    hidden, W, ids = U.to_torch(b.hidden), U.to_torch(batch.W), U.to_torch(b.ids)
    old, adv_d, cu = U.to_torch(b.old_logp), U.to_torch(adv), U.to_torch(b.cu_seqlens)
    be, status = CudaBackend(), B.new_status()
    triples = torch.empty(parts, 3, T, device="cuda")
    spans = [shard_bounds(V, parts, r) for r in range(parts)]
    for r, (lo, hi) in enumerate(spans):
        be.lse_partial(hidden, W[lo:hi], ids, lo, triples[r], status)
    out = B.alloc_fwd_outputs(T, S)
    be.loss_from_partials(triples, V, ids, old, adv_d, cu, 0.2, 0.28, 1.0, out, status)
    dH = torch.zeros(T, H, device="cuda")
    dW = torch.empty(V, H, device="cuda")
    for lo, hi in spans:
        share = torch.empty(T, H, device="cuda")
        be.bwd_shard(hidden, W[lo:hi], ids, lo, out["lse"], out["gscale"], share, dW[lo:hi], status)
        dH += share
    torch.cuda.synchronize()
    assert status.item() == 0
    ref = orc.policy_loss_fwd(gen.as_f32(b.hidden), gen.as_f32(batch.W), b.ids, b.old_logp, adv, b.cu_seqlens,
                              0.2, 0.28)
    grads = orc.policy_loss_bwd(gen.as_f32(b.hidden), gen.as_f32(batch.W), b.ids, ref["lse"], ref["gscale"])
    U.check_forward(out, ref, adv.astype(np.float64), b.cu_seqlens, 0.2, 0.28)
    U.check_loss(float(out["loss"].item()), ref["loss"], adv.astype(np.float64))
    assert U.rel_fro(dH.cpu().numpy(), grads["dhidden"]) <= U.TOL_GRAD_FRO
    assert U.rel_fro(dW.cpu().numpy(), grads["dW"]) <= U.TOL_GRAD_FRO
    whole = U.gpu_scores(hidden, W, ids, old, adv_d, cu, 0.2, 0.28, want_bwd=False)
    assert (out["logp"] - whole["logp"]).abs().max().item() <= 1e-5
