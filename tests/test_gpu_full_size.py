"""Parity at the full workload sizes, in the launch configurations bench.py times
(PolicyScorer: pack -> advantages -> forward -> backward with the default workspace, and
pack -> advantages -> the single-pass call).

Workload 2 is small enough for the oracle to score every token's forward pass; gradients are
checked on sampled rows.  Workloads 3-5 are checked on sampled whole sequences, on properties
of the gradients that hold at any size, and end to end on "lite" variants (same H, V, group
structure and distributions, shorter completions) that the oracle can finish."""
import numpy as np
import pytest
import torch

from oracle import sapo_oracle as orc
from paper_2509_08721_b200 import binding as B
from paper_2509_08721_b200 import inputs as gen
from paper_2509_08721_b200.pipeline import PolicyScorer, _to_dev
from tests import util as U

pytestmark = pytest.mark.gpu


MODES = ["dense", "fused"]     # separate forward / backward calls; the single-pass call


def run_scorer(batch, recipe, backward="dense"):
    scorer = PolicyScorer(_to_dev(batch.W, "cuda"), batch.T, batch.S, recipe.Q,
                          eps_low=batch.eps_low, eps_high=batch.eps_high, backward=backward)
    scorer.make_host_batch(batch)
    res = scorer.step_from_host(batch.T, batch.S)
    torch.cuda.synchronize()
    scorer.check_status()
    return scorer, res


def check_gradient_invariants(res, hidden_dev, W_dev, T):
    """sum_v dW[v,:] = 0 (because sum_v dz[t,v] = 0) and <dW, W> = <dH, hidden> (both equal
    sum_t dz_t . z_t); scaled by the size of the terms."""
    dW, dH = res.dW.double(), res.dhidden[:T].double()
    col = dW.sum(0)
    scale = dW.abs().sum(0) + 1e-30
    assert (col.abs() / scale).max().item() < 2e-2          # bf16 rounding of dz, summed over V
    a = (dW * W_dev.double()).sum().item()
    b = (dH * hidden_dev[:T].double()).sum().item()
    size = (dW.abs() * W_dev.double().abs()).sum().item() + 1e-30
    assert abs(a - b) <= 2e-3 * size, (a, b, size)


_W2 = {}


def workload2_reference():
    """The batch and the oracle's forward pass over all of its tokens (computed once per run)."""
    if not _W2:
        recipe = gen.config(2)
        batch = gen.make_batch(recipe, 2000)
        T, b = batch.T, batch.built
        h = gen.as_f32(b.hidden)
        W64 = gen.as_f32(batch.W).astype(np.float64)
        lse, logp = np.zeros(T), np.zeros(T)
        for a in range(0, T, 1024):
            e = min(T, a + 1024)
            lp = orc.token_logprobs(h[a:e], W64, b.ids[a:e])
            lse[a:e], logp[a:e] = lp["lse"], lp["logp"]
        gen.install_old_logp(batch, logp.astype(np.float32))
        adv = orc.group_advantages(b.rewards, b.group_offsets, adv_eps=float(np.float32(1e-6)))["adv"]
        ref = orc.surrogate_from_logp(logp, b.old_logp, adv, b.cu_seqlens, batch.eps_low, batch.eps_high)
        ref["logp"], ref["lse"] = logp, lse
        _W2.update(recipe=recipe, batch=batch, h=h, W64=W64, adv=adv, ref=ref)
    return _W2


@pytest.mark.parametrize("backward", MODES)
def test_workload2_full_size(backward):
    w2 = workload2_reference()
    recipe, batch, h, W64, adv, ref = (w2[k] for k in ("recipe", "batch", "h", "W64", "adv", "ref"))
    T, S, b = batch.T, batch.S, batch.built
    lse = ref["lse"]

    scorer, res = run_scorer(batch, recipe, backward)
    # pack, bit for bit
    assert np.array_equal(U.to_numpy(res.packed["hidden"])[:T], b.hidden)
    assert np.array_equal(U.to_numpy(res.packed["ids"])[:T], b.ids)
    assert np.array_equal(U.to_numpy(res.packed["cu_seqlens"])[:S + 1], b.cu_seqlens)
    assert np.allclose(res.adv[:S].cpu().numpy(), adv, rtol=U.TOL_ADV_REL, atol=1e-9)
    out = {k: v[:T] for k, v in res.fwd.items() if k not in ("seq_surr", "loss")}
    U.check_forward(out, ref, adv, b.cu_seqlens, batch.eps_low, batch.eps_high)
    seq = res.fwd["seq_surr"][:S].cpu().numpy().astype(np.float64)
    assert np.max(np.abs(seq - ref["seq_surr"])) <= 1e-3 * np.abs(adv).max()
    U.check_loss(float(res.loss.item()), ref["loss"], adv)
    # gradients on sampled rows
    rng = np.random.default_rng(7)
    rows = np.sort(rng.choice(T, size=192, replace=False))
    dz = orc.dlogits(h[rows], W64, b.ids[rows], lse[rows], ref["gscale"][rows])
    e_h = U.rel_fro(res.dhidden[rows].cpu().numpy(), dz @ W64)
    vrows = np.unique(np.concatenate([rng.choice(batch.V, size=120, replace=False), b.ids[:8]]))
    dW_ref = orc.dW_rows(h, W64, b.ids, lse, ref["gscale"], vrows)
    e_w = U.rel_fro(res.dW[torch.from_numpy(vrows).cuda()].cpu().numpy(), dW_ref)
    assert e_h <= U.TOL_GRAD_FRO and e_w <= U.TOL_GRAD_FRO, (e_h, e_w)
    check_gradient_invariants(res, res.packed["hidden"], scorer.W, T)


FULL = [(3, None, 1200), (4, None, 500), (5, 0.75, 1500), (5, 0.0, 1500)]


@pytest.mark.parametrize("backward", MODES)
@pytest.mark.parametrize("number,ext_fraction,sample_tokens", FULL,
                         ids=["cfg3", "cfg4", "cfg5_J6", "cfg5_J0"])
def test_workloads_3_to_5_full_size_sampled(number, ext_fraction, sample_tokens, backward):
    recipe = gen.config(number, ext_fraction=ext_fraction)
    batch = gen.make_batch(recipe, 1000 * number)
    T, S = batch.T, batch.S
    b = batch.built
    W_dev = _to_dev(batch.W, "cuda")
    # old log-probs: noise around a chunked torch estimate of the current ones (an input recipe)
    cur = U.torch_current_logp(_to_dev(b.hidden, "cuda"), W_dev, U.to_torch(b.ids)).cpu().numpy()
    gen.install_old_logp(batch, cur)
    adv = orc.group_advantages(b.rewards, b.group_offsets, adv_eps=float(np.float32(1e-6)))["adv"]

    scorer, res = run_scorer(batch, recipe, backward)
    assert np.array_equal(U.to_numpy(res.packed["ids"])[:T], b.ids)
    assert np.array_equal(U.to_numpy(res.packed["cu_seqlens"])[:S + 1], b.cu_seqlens)
    assert np.allclose(res.adv[:S].cpu().numpy(), adv, rtol=U.TOL_ADV_REL, atol=1e-9)

    # sampled whole sequences (prefer ones with a non-zero advantage), scored one by one
    rng = np.random.default_rng(number)
    order = rng.permutation(S)
    order = np.concatenate([order[adv[order] != 0], order[adv[order] == 0][:1]])
    W64 = gen.as_f32(batch.W).astype(np.float64)
    used = 0
    for s in order:
        a, e = int(b.cu_seqlens[s]), int(b.cu_seqlens[s + 1])
        if used + (e - a) > sample_tokens and used > 0:
            continue
        used += e - a
        hs = gen.as_f32(b.hidden[a:e])
        lp = orc.token_logprobs(hs, W64, b.ids[a:e])
        ref = orc.surrogate_from_logp(lp["logp"], b.old_logp[a:e], adv[s:s + 1], [0, e - a],
                                      batch.eps_low, batch.eps_high, n_seqs_total=S)
        ref["logp"], ref["lse"] = lp["logp"], lp["lse"]
        out = {k: res.fwd[k][a:e] for k in ("logp", "lse", "ratio", "surr", "gscale")}
        U.check_forward(out, ref, adv[s:s + 1], np.array([0, e - a]), batch.eps_low, batch.eps_high)
        assert abs(res.fwd["seq_surr"][s].item() - ref["seq_surr"][0]) <= 1e-3 * (abs(adv[s]) + 1e-12)
        dz = orc.dlogits(hs, W64, b.ids[a:e], lp["lse"], ref["gscale"])
        dH_ref = dz @ W64
        got = res.dhidden[a:e].cpu().numpy()
        if adv[s] == 0:
            assert np.all(got == 0.0)
        else:
            assert U.rel_fro(got, dH_ref) <= U.TOL_GRAD_FRO
        if used >= sample_tokens:
            break
    # the loss is the mean of the per-sequence surrogates the device reported
    seq = res.fwd["seq_surr"][:S].double().cpu().numpy()
    assert abs(res.loss.item() - (-seq.mean())) <= 1e-6 * np.abs(seq).mean() + 1e-9
    check_gradient_invariants(res, res.packed["hidden"], scorer.W, T)
    if number == 3:      # a quarter of the questions have equal rewards: no gradient from them
        go = b.group_offsets
        rows = slice(int(b.cu_seqlens[go[0]]), int(b.cu_seqlens[go[4]]))
        assert torch.all(res.dhidden[rows] == 0)


LITE = [(3, None, 128), (4, None, 128), (5, 0.5, 64)]


@pytest.mark.parametrize("number,ext_fraction,length_div", LITE, ids=["cfg3", "cfg4", "cfg5"])
def test_workloads_3_to_5_lite_end_to_end(number, ext_fraction, length_div):
    """Full H and V, group structure and reward law of the workload, completions shortened so
    that the oracle finishes: every output, dW included, against the oracle."""
    from tests.test_gpu_parity import run_case
    recipe = gen.config(number, ext_fraction=ext_fraction, length_div=length_div)
    if number != 3:
        recipe = gen.Recipe(**{**recipe.__dict__, "Q": 8})
    batch = gen.make_batch(recipe, 1000 * number + 1)
    run_case(batch)
