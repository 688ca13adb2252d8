"""Pins for the fp64 oracle: each check fixes it to something other than itself — a closed
form, a library routine, an invariant, brute force on tiny inputs or finite differences —
so that a dropped term, a wrong sign or index, or a transposed operand fails at least one.
CPU only."""
import math
import os

import numpy as np
import pytest
from scipy.special import log_softmax, logsumexp

from oracle import sapo_oracle as orc
from paper_2509_08721_b200 import inputs as gen


def buf_dict(b):
    return {"hidden": b.hidden, "ids": b.ids, "old_logp": b.old_logp, "offsets": b.offsets,
            "rewards": b.rewards}


def sel_dict(s):
    return {"q_offsets_local": s.q_offsets_local, "local_idx": s.local_idx,
            "q_offsets_ext": s.q_offsets_ext, "ext_idx": s.ext_idx}


def tiny_recipe(**kw):
    base = dict(name="tiny", dtype=gen.DTYPE_F32, H=5, V=17, Q=3, I=2, J=2,
                length_law=("uniform", 1, 4), reward_law=("bernoulli", 0.5))
    base.update(kw)
    return gen.Recipe(**base)


# ------------------------------------------------------------------------------- pack
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_pack_reproduces_the_generators_construction(seed):
    """The generator builds the packed batch first and then scatters it into buffers;
    packing those buffers must give the construction back bit for bit."""
    b = gen.make_batch(tiny_recipe(Q=5, length_law=("uniform", 1, 9)), seed,
                       selections=[(2, 2), (0, 3), (4, 0), (1, 1), (3, 5)])
    p = orc.pack_rollouts(buf_dict(b.local), buf_dict(b.ext), sel_dict(b.sel))
    c = b.built
    assert np.array_equal(p["hidden"].view(np.uint32), c.hidden.view(np.uint32))
    assert np.array_equal(p["ids"], c.ids)
    assert np.array_equal(p["old_logp"].view(np.uint32), c.logp_noise.view(np.uint32))
    assert np.array_equal(p["rewards"], c.rewards)
    for k in ("cu_seqlens", "seq_group", "seq_is_ext", "seq_src", "group_offsets"):
        assert np.array_equal(p[k], getattr(c, k)), k
    assert p["n_tokens"] == c.cu_seqlens[-1] == len(p["tok_seq"])
    # tok_seq by brute force
    for t in range(p["n_tokens"]):
        s = p["tok_seq"][t]
        assert c.cu_seqlens[s] <= t < c.cu_seqlens[s + 1]


def test_pack_without_external_picks_is_the_selected_local_rollouts():
    """J = 0 is plain RL fine-tuning (Section 3.2, last sentence): selecting every local
    rollout in order must return the local buffer unchanged."""
    b = gen.make_batch(tiny_recipe(Q=2, I=3, J=0, distractor_fraction=0.0), 5)
    n = b.local.n_rollouts
    sel = {"q_offsets_local": np.array([0, 2, n], np.int32),
           "local_idx": np.arange(n, dtype=np.int32),
           "q_offsets_ext": np.zeros(3, np.int32), "ext_idx": np.zeros(0, np.int32)}
    p = orc.pack_rollouts(buf_dict(b.local), buf_dict(b.ext), sel)
    assert np.array_equal(p["hidden"], b.local.hidden)
    assert np.array_equal(p["ids"], b.local.ids)
    assert np.array_equal(p["cu_seqlens"], b.local.offsets.astype(np.int32))
    assert not p["seq_is_ext"].any()
    assert np.array_equal(p["seq_group"], np.array([0, 0] + [1] * (n - 2)))


def test_pack_order_local_then_external_and_empty():
    b = gen.make_batch(tiny_recipe(Q=2), 9, selections=[(1, 2), (2, 1)])
    p = orc.pack_rollouts(buf_dict(b.local), buf_dict(b.ext), sel_dict(b.sel))
    assert p["seq_is_ext"].tolist() == [0, 1, 1, 0, 0, 1]
    assert p["group_offsets"].tolist() == [0, 3, 6]
    empty = {"q_offsets_local": np.zeros(1, np.int32), "local_idx": np.zeros(0, np.int32),
             "q_offsets_ext": np.zeros(1, np.int32), "ext_idx": np.zeros(0, np.int32)}
    p0 = orc.pack_rollouts(buf_dict(b.local), buf_dict(b.ext), empty)
    assert p0["n_tokens"] == 0 and p0["cu_seqlens"].tolist() == [0]


# ------------------------------------------------------------------------- advantages
def test_advantages_sum_to_zero_and_equal_rewards_give_zero():
    rng = np.random.default_rng(0)
    r = rng.random(40).astype(np.float32)
    go = np.array([0, 8, 9, 25, 40], np.int32)
    r[25:40] = 0.75                      # an all-equal group
    out = orc.group_advantages(r, go)
    for g in range(4):
        assert abs(out["adv"][go[g]:go[g + 1]].sum()) < 1e-9
    assert np.all(out["adv"][25:40] == 0.0)
    assert out["adv"][8] == 0.0          # a group of one


@pytest.mark.parametrize("G,k", [(8, 1), (8, 3), (16, 8), (8, 7)])
def test_advantages_closed_form_for_binary_rewards(G, k):
    """k ones among G with the population std: A1 = (1-p)/(sqrt(p(1-p))+eps),
    A0 = -p/(sqrt(p(1-p))+eps), p = k/G."""
    eps = 1e-6
    r = np.zeros(G, np.float32)
    r[:k] = 1.0
    out = orc.group_advantages(r, np.array([0, G], np.int32), adv_eps=eps, ddof=0)
    p = k / G
    sd = math.sqrt(p * (1 - p))
    assert np.allclose(out["adv"][:k], (1 - p) / (sd + eps), rtol=1e-13)
    assert np.allclose(out["adv"][k:], -p / (sd + eps), rtol=1e-13)
    assert math.isclose(out["mean"][0], p) and math.isclose(out["std"][0], sd)


def test_advantages_match_numpy_statistics_and_ddof():
    rng = np.random.default_rng(3)
    r = rng.normal(size=12)
    for ddof in (0, 1):
        out = orc.group_advantages(r, np.array([0, 12], np.int32), adv_eps=1e-6, ddof=ddof)
        assert np.allclose(out["adv"], (r - r.mean()) / (r.std(ddof=ddof) + 1e-6), rtol=1e-12)
    # scale invariance up to eps: rewards c*r give the same advantages when eps -> 0
    a1 = orc.group_advantages(r, np.array([0, 12], np.int32), adv_eps=0.0)["adv"]
    a2 = orc.group_advantages(7.5 * r, np.array([0, 12], np.int32), adv_eps=0.0)["adv"]
    assert np.allclose(a1, a2, rtol=1e-12)


# ---------------------------------------------------------------------------- log-prob
def test_logprob_matches_library_log_softmax():
    rng = np.random.default_rng(1)
    h = rng.normal(size=(7, 6))
    W = rng.normal(size=(13, 6))
    ids = rng.integers(0, 13, size=7)
    out = orc.token_logprobs(h, W, ids)
    z = np.einsum("tk,vk->tv", h, W)          # independent contraction path
    assert np.allclose(out["lse"], logsumexp(z, axis=1), rtol=1e-13)
    assert np.allclose(out["logp"], log_softmax(z, axis=1)[np.arange(7), ids], rtol=1e-12)
    # a transposed W would not even have this shape; a transposed contraction fails here:
    assert np.allclose(out["z"][2, 5], sum(h[2, k] * W[5, k] for k in range(6)))


def test_logprob_special_cases():
    rng = np.random.default_rng(2)
    h = rng.normal(size=(4, 3))
    ids = np.array([0, 1, 1, 0])
    # zero head: uniform distribution, logp = -ln V exactly
    out = orc.token_logprobs(h, np.zeros((9, 3)), ids % 9)
    assert np.allclose(out["logp"], -math.log(9.0), rtol=1e-15)
    # two-word vocabulary with W = [w, 0]: logp_0 = log sigmoid(h.w)
    w = rng.normal(size=3)
    out = orc.token_logprobs(h, np.stack([w, np.zeros(3)]), ids)
    a = h @ w
    ref = np.where(ids == 0, -np.log1p(np.exp(-a)), -np.log1p(np.exp(a)))
    assert np.allclose(out["logp"], ref, rtol=1e-12)
    # adding one vector to every row of W shifts all logits of a token equally
    W = rng.normal(size=(11, 3))
    u = rng.normal(size=3)
    ids = rng.integers(0, 11, size=4)
    assert np.allclose(orc.token_logprobs(h, W, ids)["logp"],
                       orc.token_logprobs(h, W + u, ids)["logp"], rtol=1e-11)
    # probabilities sum to one
    o = orc.token_logprobs(h, W, ids)
    assert np.allclose(np.exp(o["z"] - o["lse"][:, None]).sum(1), 1.0, rtol=1e-13)
    # large logits do not overflow
    big = orc.token_logprobs(1e3 * h, W, ids)
    assert np.all(np.isfinite(big["logp"]))


# ----------------------------------------------------------------------------- surrogate
def _toy(seed=0, T_s=(3, 5, 2, 4), V=17, H=5):
    rng = np.random.default_rng(seed)
    cu = np.concatenate([[0], np.cumsum(T_s)]).astype(np.int32)
    T = int(cu[-1])
    h = rng.normal(size=(T, H))
    W = rng.normal(size=(V, H)) * 0.5
    ids = rng.integers(0, V, size=T)
    adv = np.array([1.3, -0.7, 0.0, 0.4])[:len(T_s)]
    return rng, cu, h, W, ids, adv


def test_loss_with_old_equal_current_is_minus_mean_advantage():
    rng, cu, h, W, ids, adv = _toy()
    cur = orc.token_logprobs(h, W, ids)["logp"]
    out = orc.policy_loss_fwd(h, W, ids, cur, adv, cu)
    assert np.allclose(out["ratio"], 1.0)
    assert np.allclose(out["seq_surr"], adv, rtol=1e-13)
    assert math.isclose(out["loss"], -adv.mean(), rel_tol=1e-13)
    # gradient = plain policy gradient: g_t = -A_s / (S T_s)
    S = len(adv)
    T_s = np.diff(cu)
    expect = np.concatenate([np.full(T_s[s], -adv[s] / (S * T_s[s])) for s in range(S)])
    assert np.allclose(out["gscale"], expect, rtol=1e-13)


def test_loss_inside_the_clip_band_and_fully_clipped():
    rng, cu, h, W, ids, adv = _toy(1)
    cur = orc.token_logprobs(h, W, ids)["logp"]
    S, T_s = len(adv), np.diff(cu)
    # inside the band: L = -(1/S) sum_s A_s mean_t rho_t
    d = rng.uniform(-0.1, 0.1, size=len(cur))
    out = orc.policy_loss_fwd(h, W, ids, cur - d, adv, cu, 0.2, 0.28)
    rho = np.exp(d)
    expect = -sum(adv[s] * rho[cu[s]:cu[s + 1]].mean() for s in range(S)) / S
    assert math.isclose(out["loss"], expect, rel_tol=1e-12)
    assert np.all(out["active"] == 1.0)
    # asymmetric thresholds: rho = 1.25 is inside (1+0.28) but outside (1+0.2)
    one = orc.surrogate_from_logp(np.log([1.25]), [0.0], [1.0], [0, 1], 0.2, 0.28)
    assert math.isclose(one["surr"][0], 1.25) and one["gscale"][0] != 0.0
    one = orc.surrogate_from_logp(np.log([1.25]), [0.0], [1.0], [0, 1], 0.2, 0.2)
    assert math.isclose(one["surr"][0], 1.2) and one["gscale"][0] == 0.0
    # lower side, negative advantage: rho = 0.7 < 0.8 -> clipped value 0.8*A is the min
    one = orc.surrogate_from_logp(np.log([0.7]), [0.0], [-2.0], [0, 1], 0.2, 0.28)
    assert math.isclose(one["surr"][0], -1.6) and one["gscale"][0] == 0.0
    # lower side, positive advantage: unclipped 0.7*A is the min, gradient flows
    one = orc.surrogate_from_logp(np.log([0.7]), [0.0], [2.0], [0, 1], 0.2, 0.28)
    assert math.isclose(one["surr"][0], 1.4)
    assert math.isclose(one["gscale"][0], -2.0 * 0.7)
    # every token clipped on the binding side: loss is a constant, gradient exactly zero
    sign = np.concatenate([np.full(T_s[s], 1.0 if adv[s] >= 0 else -1.0) for s in range(S)])
    out = orc.policy_loss_fwd(h, W, ids, cur - 0.5 * sign, adv, cu, 0.2, 0.28)
    assert np.all(out["gscale"] == 0.0)
    expect = -sum(adv[s] * (1.28 if adv[s] >= 0 else 0.8) for s in range(S)) / S
    assert math.isclose(out["loss"], expect, rel_tol=1e-12)


def test_token_level_aggregation_and_kl_term():
    """loss_agg = 1 weighs every token 1/T; the KL penalty is the non-negative estimator
    exp(d) - d - 1 of d = ref - logp, zero (with zero slope) when the policies agree."""
    rng, cu, h, W, ids, adv = _toy(3)
    T_s, S = np.diff(cu), len(adv)
    T = int(cu[-1])
    cur = orc.token_logprobs(h, W, ids)["logp"]
    # rho = 1: token-level loss is -(1/T) sum_s T_s A_s
    out = orc.policy_loss_fwd(h, W, ids, cur, adv, cu, loss_agg=1)
    assert math.isclose(out["loss"], -(T_s * adv).sum() / T, rel_tol=1e-13)
    assert np.allclose(out["gscale"], -np.repeat(adv, T_s) / T, rtol=1e-13)
    # equal lengths: both aggregations coincide
    cu_eq = np.array([0, 3, 6, 9, 12], np.int32)
    d = rng.uniform(-0.1, 0.1, size=12)
    a0 = orc.surrogate_from_logp(cur[:12], cur[:12] - d, adv, cu_eq, 0.2, 0.28, loss_agg=0)
    a1 = orc.surrogate_from_logp(cur[:12], cur[:12] - d, adv, cu_eq, 0.2, 0.28, loss_agg=1)
    assert math.isclose(a0["loss"], a1["loss"], rel_tol=1e-13)
    # KL: ref = logp gives no penalty and no gradient; otherwise positive, equal to the
    # importance-weighted form E_q[...] term by term, and added with weight beta
    k0 = orc.surrogate_from_logp(cur, cur, adv, cu, 0.2, 0.28, kl_beta=0.3, ref_logp=cur)
    b0 = orc.surrogate_from_logp(cur, cur, adv, cu, 0.2, 0.28)
    assert np.all(k0["kl"] == 0.0) and math.isclose(k0["loss"], b0["loss"], rel_tol=1e-15)
    assert np.allclose(k0["gscale"], b0["gscale"], rtol=1e-15)
    ref = cur + rng.normal(size=T) * 0.3
    k = orc.surrogate_from_logp(cur, cur, adv, cu, 0.2, 0.28, kl_beta=0.3, ref_logp=ref)
    ratio = np.exp(ref - cur)
    assert np.all(k["kl"] > 0) and np.allclose(k["kl"], ratio - np.log(ratio) - 1, rtol=1e-13)
    pen = sum(k["kl"][cu[s]:cu[s + 1]].mean() for s in range(S)) / S
    assert math.isclose(k["loss"], b0["loss"] + 0.3 * pen, rel_tol=1e-12)


def test_variant_gradients_match_finite_differences():
    rng, cu, h, W, ids, adv = _toy(5, T_s=(2, 3, 1, 2), V=11, H=4)
    cur = orc.token_logprobs(h, W, ids)["logp"]
    old = cur + rng.normal(size=len(cur)) * 0.3
    ref = cur + rng.normal(size=len(cur)) * 0.2
    kw = dict(eps_low=0.2, eps_high=0.28, loss_agg=1, kl_beta=0.4, ref_logp=ref)
    f = orc.policy_loss_fwd(h, W, ids, old, adv, cu, **kw)
    g = orc.policy_loss_bwd(h, W, ids, f["lse"], f["gscale"])
    d = 1e-6
    for (arr, grad) in ((h, g["dhidden"]), (W, g["dW"])):
        num = np.zeros_like(arr)
        for idx in np.ndindex(*arr.shape):
            keep = arr[idx]
            arr[idx] = keep + d
            fp = orc.policy_loss_fwd(h, W, ids, old, adv, cu, **kw)["loss"]
            arr[idx] = keep - d
            fm = orc.policy_loss_fwd(h, W, ids, old, adv, cu, **kw)["loss"]
            arr[idx] = keep
            num[idx] = (fp - fm) / (2 * d)
        assert np.allclose(grad, num, rtol=1e-6, atol=1e-9)


# ------------------------------------------------------------------------------ gradient
def _loss_only(h, W, ids, old, adv, cu, lo, hi):
    return orc.policy_loss_fwd(h, W, ids, old, adv, cu, lo, hi)["loss"]


@pytest.mark.parametrize("seed", [2, 4, 5])
def test_gradient_matches_central_finite_differences(seed):
    rng, cu, h, W, ids, adv = _toy(seed, T_s=(2, 3, 1, 2), V=11, H=4)
    cur = orc.token_logprobs(h, W, ids)["logp"]
    old = cur + rng.normal(size=len(cur)) * 0.3      # some tokens beyond the clip edges
    lo, hi = 0.2, 0.28
    f = orc.policy_loss_fwd(h, W, ids, old, adv, cu, lo, hi)
    # stay away from the kink of min/clip, where the derivative is one-sided
    edge = np.minimum(np.abs(f["ratio"] - (1 - lo)), np.abs(f["ratio"] - (1 + hi)))
    assert edge.min() > 1e-4
    nz = adv[np.repeat(np.arange(len(adv)), np.diff(cu))] != 0
    assert 0 < f["active"][nz].sum() < nz.sum()        # both branches of the min occur
    g = orc.policy_loss_bwd(h, W, ids, f["lse"], f["gscale"])
    d = 1e-6
    for (arr, grad) in ((h, g["dhidden"]), (W, g["dW"])):
        num = np.zeros_like(arr)
        for idx in np.ndindex(*arr.shape):
            keep = arr[idx]
            arr[idx] = keep + d
            fp = _loss_only(h, W, ids, old, adv, cu, lo, hi)
            arr[idx] = keep - d
            fm = _loss_only(h, W, ids, old, adv, cu, lo, hi)
            arr[idx] = keep
            num[idx] = (fp - fm) / (2 * d)
        assert np.allclose(grad, num, rtol=1e-6, atol=1e-9)


def test_gradient_closed_forms_and_invariants():
    rng, cu, h, W, ids, adv = _toy(4)
    T, V = h.shape[0], W.shape[0]
    # zero head: dH = 0 and dW_v = sum_t g_t ([y_t = v] - 1/V) h_t
    f0 = orc.policy_loss_fwd(h, 0 * W, ids, np.full(T, -math.log(V)), adv, cu)
    g0 = orc.policy_loss_bwd(h, 0 * W, ids, f0["lse"], f0["gscale"])
    assert np.allclose(g0["dhidden"], 0.0, atol=1e-15)
    ref = np.zeros_like(W)
    for t in range(T):
        for v in range(V):
            ref[v] += f0["gscale"][t] * ((1.0 if ids[t] == v else 0.0) - 1.0 / V) * h[t]
    assert np.allclose(g0["dW"], ref, rtol=1e-12, atol=1e-15)
    # general head
    cur = orc.token_logprobs(h, W, ids)["logp"]
    f = orc.policy_loss_fwd(h, W, ids, cur + rng.normal(size=T) * 0.05, adv, cu)
    g = orc.policy_loss_bwd(h, W, ids, f["lse"], f["gscale"])
    assert np.allclose(g["dW"].sum(axis=0), 0.0, atol=1e-13)               # sum_v dz = 0
    assert math.isclose((g["dW"] * W).sum(), (g["dhidden"] * h).sum(), rel_tol=1e-10)
    s0 = 2                                                               # the A = 0 sequence
    assert np.all(g["dhidden"][cu[s0]:cu[s0 + 1]] == 0.0)
    # brute-force dH and dW from the element-wise definition
    dz = orc.dlogits(h, W, ids, f["lse"], f["gscale"])
    p = np.exp(orc.logits(h, W) - f["lse"][:, None])
    t, v = 4, int(ids[4])
    assert math.isclose(dz[t, v], f["gscale"][t] * (1 - p[t, v]), rel_tol=1e-12)
    assert math.isclose(dz[t, (v + 1) % V], -f["gscale"][t] * p[t, (v + 1) % V], rel_tol=1e-12)
    assert np.allclose(g["dhidden"][t], sum(dz[t, vv] * W[vv] for vv in range(V)), rtol=1e-12)
    assert np.allclose(g["dW"][3], sum(dz[tt, 3] * h[tt] for tt in range(T)), rtol=1e-12)


def test_row_blocked_evaluation_equals_the_whole_matrix_form():
    rng, cu, h, W, ids, adv = _toy(6, T_s=(5, 7, 3, 6))
    cur = orc.token_logprobs(h, W, ids)["logp"]
    old = cur + rng.normal(size=len(cur)) * 0.1
    f = orc.policy_loss_fwd(h, W, ids, old, adv, cu, 0.2, 0.28, grad_scale=2.0)
    g = orc.policy_loss_bwd(h, W, ids, f["lse"], f["gscale"])
    r = orc.policy_loss_fwd_bwd_rows(h, W, ids, old, adv, cu, 0.2, 0.28, grad_scale=2.0,
                                     rows_per_block=4)
    for k in ("logp", "lse", "ratio", "surr", "gscale", "seq_surr"):
        assert np.allclose(r[k], f[k], rtol=1e-13)
    assert math.isclose(r["loss"], f["loss"], rel_tol=1e-13)
    assert np.allclose(r["dhidden"], g["dhidden"], rtol=1e-12, atol=1e-16)
    assert np.allclose(r["dW"], g["dW"], rtol=1e-12, atol=1e-16)


def test_dW_rows_equals_the_rows_of_the_full_gradient():
    rng, cu, h, W, ids, adv = _toy(8, T_s=(4, 6, 2, 5))
    cur = orc.token_logprobs(h, W, ids)["logp"]
    f = orc.policy_loss_fwd(h, W, ids, cur + rng.normal(size=len(cur)) * 0.1, adv, cu)
    g = orc.policy_loss_bwd(h, W, ids, f["lse"], f["gscale"])
    rows = [0, 3, int(ids[0]), 16]
    assert np.allclose(orc.dW_rows(h, W, ids, f["lse"], f["gscale"], rows), g["dW"][rows],
                       rtol=1e-12, atol=1e-16)


# ------------------------------------------------------------- pool filter and sampling
def test_philox_matches_the_published_known_answers():
    path = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_known_answers.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        assert list(orc.philox4x32(v[0:4], v[4:6])) == v[6:10]


def test_select_external_filters_zero_advantage_and_samples_uniformly():
    rng = np.random.default_rng(0)
    sizes = rng.integers(1, 9, size=60)
    go = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    r = rng.integers(0, 2, size=go[-1]).astype(np.float32)
    const = np.array([len(set(r[go[g]:go[g + 1]])) == 1 for g in range(60)])
    out = orc.select_external(r, go, 10, seed=123)
    assert np.array_equal(out["candidates"], ~const)            # brute-force filter
    sel = out["selected"]
    assert len(sel) == 10 == len(set(sel.tolist())) and np.all(np.diff(sel) > 0)
    assert not const[sel].any()                                 # only informative rollouts
    # fewer candidates than asked for: all of them; J = 0: none
    assert np.array_equal(orc.select_external(r, go, 1000, seed=5)["selected"], np.nonzero(~const)[0])
    assert orc.select_external(r, go, 0, seed=5)["n_selected"] == 0
    # same seed, same draw; the draw is uniform over the candidates (frequency test over seeds)
    assert np.array_equal(orc.select_external(r, go, 10, seed=123)["selected"], sel)
    cand = np.nonzero(~const)[0]
    hits = np.zeros(60)
    n_seeds = 600
    for seed in range(n_seeds):
        hits[orc.select_external(r, go, 10, seed=seed)["selected"]] += 1
    p = 10 / len(cand)
    sd = math.sqrt(n_seeds * p * (1 - p))
    assert np.all(np.abs(hits[cand] - n_seeds * p) < 5 * sd) and hits[const].sum() == 0


def test_adam_step_matches_the_library_optimizer():
    import torch
    rng = np.random.default_rng(2)
    theta0 = rng.normal(size=(7, 5))
    p = torch.nn.Parameter(torch.tensor(theta0, dtype=torch.float64))
    opt = torch.optim.Adam([p], lr=1e-3)                     # library defaults: 0.9, 0.999, 1e-8
    theta, m, v = theta0.copy(), np.zeros_like(theta0), np.zeros_like(theta0)
    for t in range(1, 4):
        g = rng.normal(size=theta0.shape) * (10.0 ** -t)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        theta, m, v = orc.adam_step(theta, g, m, v, t)
        assert np.allclose(theta, p.detach().numpy(), rtol=1e-12, atol=1e-15)
    # first step of Adam moves every weight by lr against the sign of its gradient
    th1, _, _ = orc.adam_step(np.zeros(4), np.array([3.0, -2.0, 1e-3, -5e2]), np.zeros(4), np.zeros(4), 1)
    assert np.allclose(th1, [-1e-3, 1e-3, -1e-3, 1e-3], rtol=1e-4)


# ------------------------------------------------------------------ the input generator
def test_generator_recipes_have_the_stated_shapes():
    r = gen.config(1)
    b = gen.make_batch(r, 1001)
    assert (b.H, b.V, b.S, b.T) == (64, 1000, 32, 1024) and b.W.dtype == np.float32
    assert set(np.unique(b.built.rewards)) <= {0.0, 1.0}
    r3 = gen.config(3, length_div=64)
    b3 = gen.make_batch(gen.Recipe(**{**r3.__dict__, "H": 16, "V": 50}), 3001)
    for q in range(4):                      # a quarter of 16 questions: all-equal rewards
        a, e = b3.built.group_offsets[q], b3.built.group_offsets[q + 1]
        assert np.unique(b3.built.rewards[a:e]).size == 1
    r4 = gen.config(4, length_div=16)
    b4 = gen.make_batch(gen.Recipe(**{**r4.__dict__, "H": 8, "V": 40}), 4001)
    L = np.diff(b4.built.cu_seqlens)
    assert L.min() >= 8 and L.max() <= 128 and b4.S == 256
    assert set(np.unique(b4.built.rewards)) <= {0.0, 0.5, 1.0}
    for f, J in ((0.0, 0), (0.25, 2), (0.5, 4), (0.75, 6)):
        assert gen.config(5, ext_fraction=f).J == J
    x = np.array([1.0, 1.0078125, -3.140625], np.float32)          # exactly representable
    assert np.array_equal(gen.bf16_bits_to_f32(gen.f32_to_bf16_bits(x)), x)
    ties = np.array([1.00390625, 1.01171875], np.float32)          # halfway: round to even
    assert gen.bf16_bits_to_f32(gen.f32_to_bf16_bits(ties)).tolist() == [1.0, 1.015625]


# ------------------------------------------------------------------------------ entropy
def test_entropy_pins():
    """token_entropy against what fixes it: a uniform head gives ln V; scipy's entropy of the
    row distributions; the two-outcome closed form -(p ln p + q ln q); the identity
    H = lse - sum_v p z; and the bound 0 <= H <= ln V."""
    from scipy.special import softmax
    from scipy.stats import entropy as scipy_entropy
    rng = np.random.default_rng(17)
    T, H, V = 9, 6, 23
    h = rng.normal(size=(T, H))
    W = rng.normal(size=(V, H))
    ent = orc.token_entropy(h, W)
    # uniform head
    assert np.allclose(orc.token_entropy(h, np.zeros((V, H))), np.log(V), rtol=0, atol=1e-13)
    # library routine on the row distributions
    z = h @ W.T
    assert np.allclose(ent, scipy_entropy(softmax(z, axis=1), axis=1), rtol=1e-12, atol=1e-13)
    # identity with the log-sum-exp the oracle also reports
    lp = orc.token_logprobs(h, W, np.zeros(T, dtype=np.int64))
    assert np.allclose(ent, lp["lse"] - (softmax(z, axis=1) * z).sum(axis=1), rtol=1e-12, atol=1e-12)
    assert np.all(ent >= 0) and np.all(ent <= np.log(V) + 1e-12)
    # two outcomes: logits (a, 0) -> p = sigmoid(a)
    a = np.array([[-3.0], [0.0], [0.7], [5.0]])
    W2 = np.array([[1.0], [0.0]])
    p = 1.0 / (1.0 + np.exp(-a[:, 0]))
    closed = -(p * np.log(p) + (1 - p) * np.log(1 - p))
    assert np.allclose(orc.token_entropy(a, W2), closed, rtol=1e-13, atol=1e-15)
    # a peaked row has (almost) no entropy; shifting every logit of a row changes nothing
    assert orc.token_entropy(np.array([[50.0]]), W2)[0] < 1e-19
    u = rng.normal(size=H)
    assert np.allclose(orc.token_entropy(h, W + u[None, :]), ent, rtol=1e-11, atol=1e-12)
