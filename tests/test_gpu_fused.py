"""The single-pass call sapo_policy_loss_fwd_bwd against the fp64 oracle, element by element,
under the same tolerances as the separate forward and backward calls, and against those
calls themselves."""
import numpy as np
import pytest
import torch

from oracle import sapo_oracle as orc
from paper_2509_08721_b200 import binding as B
from paper_2509_08721_b200 import inputs as gen
from tests import util as U
from tests.test_gpu_parity import small_recipe

pytestmark = pytest.mark.gpu


def oracle_case(batch, eps_low, eps_high, grad_scale=1.0, noise_scale=1.0, **variant):
    batch.built.logp_noise *= np.float32(noise_scale)
    gen.install_old_logp(batch, U.oracle_current_logp(batch))
    b = batch.built
    adv = orc.group_advantages(b.rewards, b.group_offsets, adv_eps=float(np.float32(batch.adv_eps)))["adv"]
    h, W = gen.as_f32(b.hidden), gen.as_f32(batch.W)
    ref = orc.policy_loss_fwd(h, W, b.ids, b.old_logp, adv, b.cu_seqlens, eps_low, eps_high,
                              grad_scale=grad_scale, **variant)
    ref.update(orc.policy_loss_bwd(h, W, b.ids, ref["lse"], ref["gscale"]))
    return adv, ref


def device_inputs(batch, adv):
    b = batch.built
    return (U.to_torch(b.hidden), U.to_torch(batch.W), U.to_torch(b.ids), U.to_torch(b.old_logp),
            U.to_torch(adv.astype(np.float32)), U.to_torch(b.cu_seqlens))


def check_all(out, ref, adv, batch, eps_low, eps_high, extra_scale=0.0):
    assert out["status"] == 0
    U.check_forward(out, ref, adv, batch.built.cu_seqlens, eps_low, eps_high)
    seq = out["seq_surr"].cpu().numpy().astype(np.float64)
    scale = np.abs(adv).max() + extra_scale + 1e-30
    assert np.max(np.abs(seq - ref["seq_surr"])) <= 1e-3 * scale
    if extra_scale == 0.0:
        U.check_loss(float(out["loss"].item()), ref["loss"], adv)
    else:
        assert abs(out["loss"].item() - ref["loss"]) <= 1e-3 * abs(ref["loss"]) + 1e-5 * scale
    e_h = U.rel_fro(out["dhidden"].cpu().numpy(), ref["dhidden"])
    e_w = U.rel_fro(out["dW"].cpu().numpy(), ref["dW"])
    assert e_h <= U.TOL_GRAD_FRO and e_w <= U.TOL_GRAD_FRO, (e_h, e_w)


SHAPES = [
    ("one_tile", small_recipe(H=64, V=200, Q=2, length_law=("uniform", 3, 20))),
    ("vocab_tail", small_recipe(H=64, V=1000)),
    ("k_tail", small_recipe(H=72, V=777, Q=4, length_law=("uniform", 20, 90))),
    ("many_tiles", small_recipe(H=328, V=2500, Q=6, I=3, J=3, length_law=("uniform", 30, 120))),
    ("single_tokens", small_recipe(H=128, V=300, Q=4, length_law=("fixed", 1))),
    ("one_group", small_recipe(H=64, V=520, Q=1, I=3, J=0)),
    ("k_split", small_recipe(H=128, V=20000, Q=2, length_law=("uniform", 50, 90))),
    ("k_split_rounds", small_recipe(H=512, V=8192, Q=8, length_law=("uniform", 150, 230))),
]


@pytest.mark.parametrize("name,recipe", SHAPES, ids=[c[0] for c in SHAPES])
def test_fused_matches_oracle_small_shapes(name, recipe):
    batch = gen.make_batch(recipe, 21)
    adv, ref = oracle_case(batch, 0.2, 0.28, noise_scale=3.0)
    out = U.gpu_scores_fused(*device_inputs(batch, adv), 0.2, 0.28)
    check_all(out, ref, adv, batch, 0.2, 0.28)


def test_fused_with_a_minimal_workspace_runs_in_token_chunks():
    """A workspace for one 128-token panel: the batch goes through in chunks, sequences are cut
    by chunk boundaries and dW_head is accumulated over the chunks."""
    recipe = small_recipe(H=64, V=520, Q=4, length_law=("uniform", 60, 120))
    batch = gen.make_batch(recipe, 33)
    assert batch.T > 512
    adv, ref = oracle_case(batch, 0.2, 0.28, noise_scale=2.0)
    nbytes = B.sapo_workspace_bytes_min(B.WS_FUSED, batch.T, 64, 520, B.DTYPE_BF16)
    assert 0 < nbytes < B.sapo_workspace_bytes(B.WS_FUSED, batch.T, 64, 520, B.DTYPE_BF16)
    out = U.gpu_scores_fused(*device_inputs(batch, adv), 0.2, 0.28, workspace_bytes=nbytes)
    check_all(out, ref, adv, batch, 0.2, 0.28)
    # chunking changes the per-token outputs and dhidden by summation order at most
    whole = U.gpu_scores_fused(*device_inputs(batch, adv), 0.2, 0.28)
    for k in ("logp", "lse", "ratio", "surr", "gscale", "seq_surr", "loss", "dhidden"):
        assert torch.allclose(out[k], whole[k], rtol=1e-5, atol=1e-7), k


@pytest.mark.parametrize("loss_agg,kl_beta", [(1, 0.0), (1, 0.25)])
def test_fused_loss_variants(loss_agg, kl_beta):
    recipe = gen.Recipe("var", gen.DTYPE_BF16, 128, 2000, 4, 2, 2, ("uniform", 10, 90), ("bernoulli", 0.5))
    batch = gen.make_batch(recipe, 61)
    cur = U.oracle_current_logp(batch)
    rng = np.random.default_rng(3)
    ref_lp = (cur + rng.normal(size=batch.T).astype(np.float32) * np.float32(0.2)).astype(np.float32)
    adv, ref = oracle_case(batch, 0.2, 0.28, grad_scale=1.5, loss_agg=loss_agg, kl_beta=kl_beta,
                           ref_logp=ref_lp)
    out = U.gpu_scores_fused(*device_inputs(batch, adv), 0.2, 0.28, grad_scale=1.5, loss_agg=loss_agg,
                             kl_beta=kl_beta, ref_logp=U.to_torch(ref_lp) if kl_beta else None)
    check_all(out, ref, adv, batch, 0.2, 0.28, extra_scale=kl_beta)


@pytest.mark.parametrize("H,I", [(128, 2), (256, 8)], ids=["narrow_tiles", "wide_tiles_block_skipping"])
def test_fused_agrees_with_the_separate_calls_and_repeats_bit_for_bit(H, I):
    """A quarter of the questions have equal rewards (no gradient).  With H = 256 the wide-tile
    backward kernels run and whole 128-token blocks of such questions are left out of both
    contractions; the results must not change."""
    r = gen.config(3, length_div=16)
    recipe = gen.Recipe(**{**r.__dict__, "H": H, "V": 3000, "Q": 8, "I": I, "J": I})
    batch = gen.make_batch(recipe, 5)
    adv, ref = oracle_case(batch, 0.2, 0.2)
    check_all(U.gpu_scores_fused(*device_inputs(batch, adv), 0.2, 0.2), ref, adv, batch, 0.2, 0.2)
    args = device_inputs(batch, adv)
    a = U.gpu_scores_fused(*args, 0.2, 0.2)
    b = U.gpu_scores_fused(*args, 0.2, 0.2)
    for k in ("logp", "lse", "ratio", "surr", "gscale", "seq_surr", "loss", "dhidden", "dW"):
        assert torch.equal(a[k], b[k]), k
    sep = U.gpu_scores(*args, 0.2, 0.2)
    assert sep["status"] == 0 and a["status"] == 0
    assert (a["logp"] - sep["logp"]).abs().max().item() <= 1e-4
    assert U.rel_fro(a["dhidden"].cpu().numpy(), sep["dhidden"].double().cpu().numpy()) <= 1e-2
    assert U.rel_fro(a["dW"].cpu().numpy(), sep["dW"].double().cpu().numpy()) <= 1e-2
    # questions with equal rewards: no gradient from their tokens
    go, cu = batch.built.group_offsets, batch.built.cu_seqlens
    zero_q = [q for q in range(recipe.Q) if np.all(adv[go[q]:go[q + 1]] == 0)]
    assert zero_q
    for q in zero_q:
        assert torch.all(a["dhidden"][int(cu[go[q]]):int(cu[go[q + 1]])] == 0)


# Output widths around the tile shapes of the wide backward kernels (H >= 256: tiles of up to
# 2 x 256 columns, ragged last tile, columns past H clipped by the store) with token and vocabulary
# counts around the 128 / 256-row blocks.
EDGE = [
    ("h256_few_tokens", small_recipe(H=256, V=130, Q=2, length_law=("uniform", 2, 8))),
    ("h264_ragged_tile", small_recipe(H=264, V=1000, Q=4, length_law=("uniform", 10, 30))),
    ("h320_t_over_512", small_recipe(H=320, V=777, Q=6, length_law=("uniform", 20, 40))),
    ("h520_two_tiles", small_recipe(H=520, V=4100, Q=8, length_law=("uniform", 20, 45))),
    ("h1024_one_block", small_recipe(H=1024, V=2000, Q=2, length_law=("uniform", 20, 40))),
    ("h1032_three_tiles", small_recipe(H=1032, V=650, Q=4, length_law=("uniform", 30, 34))),
]


@pytest.mark.parametrize("name,recipe", EDGE, ids=[c[0] for c in EDGE])
def test_edge_shapes_of_the_wide_backward_kernels(name, recipe):
    """Both ways through the gradients (the separate backward uses the same wide kernels)."""
    batch = gen.make_batch(recipe, 77)
    adv, ref = oracle_case(batch, 0.2, 0.28, noise_scale=2.0)
    args = device_inputs(batch, adv)
    check_all(U.gpu_scores_fused(*args, 0.2, 0.28), ref, adv, batch, 0.2, 0.28)
    check_all(U.gpu_scores(*args, 0.2, 0.28), ref, adv, batch, 0.2, 0.28)
    # a one-panel workspace: token chunks, dW_head accumulated by TMA adds
    T, H, V = batch.T, recipe.H, recipe.V
    if T > 128:
        small = B.sapo_workspace_bytes_min(B.WS_FUSED, T, H, V, B.DTYPE_BF16)
        check_all(U.gpu_scores_fused(*args, 0.2, 0.28, workspace_bytes=small), ref, adv, batch, 0.2, 0.28)
        small_b = B.sapo_workspace_bytes_min(B.WS_BWD, T, H, V, B.DTYPE_BF16)
        check_all(U.gpu_scores(*args, 0.2, 0.28, bwd_workspace_bytes=small_b), ref, adv, batch, 0.2, 0.28)


@pytest.mark.parametrize("H", [256, 520])
@pytest.mark.parametrize("pattern", ["leading", "alternating", "all_zero"])
def test_blocks_of_zero_advantage_sequences_leave_no_trace(H, pattern):
    """Runs of sequences whose advantage is exactly zero that cover whole 128-token blocks: the
    forward writes no panel rows for them and the contractions leave them out.  The scratch is
    filled with NaN patterns beforehand, so anything read from an unwritten block would show;
    their log-probs must still be right and their dhidden rows exactly zero.  The patterns give
    256-token tiles with one written and one unwritten block, in either order."""
    recipe = small_recipe(H=H, V=1500, Q=8, I=2, J=2, length_law=("uniform", 100, 160))
    batch = gen.make_batch(recipe, 91)
    gen.install_old_logp(batch, U.oracle_current_logp(batch))
    b = batch.built
    S, T = batch.S, batch.T
    adv = np.linspace(-1.5, 1.5, S).astype(np.float32)
    adv[np.abs(adv) < 1e-3] = 0.25
    q_of = np.repeat(np.arange(8), 4)
    if pattern == "leading":
        adv[q_of < 3] = 0.0                    # 12 sequences, about 1500 tokens, then live ones
    elif pattern == "alternating":
        adv[q_of % 2 == 1] = 0.0               # about 500 dead tokens between live stretches
    else:
        adv[:] = 0.0
    h, W = gen.as_f32(b.hidden), gen.as_f32(batch.W)
    ref = orc.policy_loss_fwd(h, W, b.ids, b.old_logp, adv, b.cu_seqlens, 0.2, 0.28)
    ref.update(orc.policy_loss_bwd(h, W, b.ids, ref["lse"], ref["gscale"]))
    args = device_inputs(batch, adv)
    dead = np.repeat(adv == 0.0, np.diff(b.cu_seqlens))
    blocks = dead[: (T // 128) * 128].reshape(-1, 128).all(axis=1)
    assert pattern == "all_zero" or (blocks.any() and not blocks.all())
    small = B.sapo_workspace_bytes_min(B.WS_FUSED, T, H, 1500, B.DTYPE_BF16)
    three = small + 3 * 128 * (2 * 1536 + 2 * H + 4 + 2560)     # room for about three more blocks per chunk
    for nbytes in (None, small, three):      # one chunk; chunks of one block; chunks of a few blocks
        for out_dtype in (torch.float32, torch.bfloat16):
            kw = {} if nbytes is None else {"workspace_bytes": nbytes + (
                B.sapo_workspace_bytes_min(B.WS_FUSED | B.WS_OUT_BF16, T, H, 1500, B.DTYPE_BF16) - small
                if out_dtype == torch.bfloat16 else 0)}
            out = U.gpu_scores_fused(*args, 0.2, 0.28, out_dtype=out_dtype, **kw)
            assert out["status"] == 0
            U.check_forward(out, ref, adv.astype(np.float64), b.cu_seqlens, 0.2, 0.28)
            dH = out["dhidden"].float()
            assert torch.isfinite(dH).all() and torch.isfinite(out["dW"].float()).all()
            assert not dH[torch.from_numpy(dead).cuda()].any()
            if pattern == "all_zero":
                assert not out["dW"].float().any()
                continue
            tol = U.TOL_GRAD_FRO
            assert U.rel_fro(dH.cpu().numpy(), ref["dhidden"]) <= tol
            assert U.rel_fro(out["dW"].float().cpu().numpy(), ref["dW"]) <= tol


def _random_recipe(seed):
    rng = np.random.default_rng(1000 + seed)
    H = int(rng.choice([8, 16, 24, 64, 72, 248, 256, 264, 392, 512, 776, 1024, 1096]))
    V = int(rng.choice([1, 2, 63, 64, 65, 127, 129, 500, 1000, 2049, 4097]))
    Q = int(rng.integers(1, 7))
    lo = int(rng.choice([1, 1, 5, 30]))
    hi = lo + int(rng.choice([0, 3, 40, 90]))
    return small_recipe(H=H, V=V, Q=Q, I=int(rng.integers(1, 4)), J=int(rng.integers(0, 4)),
                        length_law=("uniform", lo, hi))


@pytest.mark.parametrize("seed", range(24))
def test_random_shapes_single_pass_against_separate_calls(seed):
    """Shapes drawn around the tile, block and box sizes of the kernels (hidden sizes on both
    sides of the wide-tile threshold, vocabularies of one entry and up, one token and up): the
    two ways through the loss and its gradients must agree with each other.  The old log-probs
    come from the separate forward itself, so no oracle pass is needed here."""
    recipe = _random_recipe(seed)
    batch = gen.make_batch(recipe, 300 + seed)
    b = batch.built
    hidden, W, ids = U.to_torch(b.hidden), U.to_torch(batch.W), U.to_torch(b.ids)
    cu = U.to_torch(b.cu_seqlens)
    adv_np = orc.group_advantages(b.rewards, b.group_offsets, adv_eps=1e-6)["adv"].astype(np.float32)
    adv = U.to_torch(adv_np)
    zero = torch.zeros(batch.T, device="cuda")
    cur = U.gpu_scores(hidden, W, ids, zero, adv, cu, 0.2, 0.28, want_bwd=False)["logp"]
    old = cur + U.to_torch(b.logp_noise.astype(np.float32)) * 2.0
    sep = U.gpu_scores(hidden, W, ids, old, adv, cu, 0.2, 0.28)
    one = U.gpu_scores_fused(hidden, W, ids, old, adv, cu, 0.2, 0.28)
    assert sep["status"] == 0 and one["status"] == 0, (recipe, sep["status"], one["status"])
    assert (one["logp"] - sep["logp"]).abs().max().item() <= 2e-4
    assert (one["lse"] - sep["lse"]).abs().max().item() <= 2e-4
    assert torch.allclose(one["ratio"], sep["ratio"], rtol=1e-3, atol=0)
    # the clip decision may differ for ratios within rounding of an edge
    rho = sep["ratio"]
    near = torch.minimum((rho - 0.8).abs(), (rho - 1.28).abs()) < 1e-3
    gmax = sep["gscale"].abs().max().item() + 1e-30
    assert ((one["gscale"] - sep["gscale"]).abs()[~near]).max().item() <= 2e-3 * gmax if (~near).any() else True
    if not near.any():
        scale = np.abs(adv_np).max() + 1e-30
        assert (one["seq_surr"] - sep["seq_surr"]).abs().max().item() <= 1e-3 * scale
        for k in ("dhidden", "dW"):
            ref = sep[k].double().cpu().numpy()
            diff = np.linalg.norm(one[k].double().cpu().numpy() - ref)
            # the floor covers degenerate cases (a vocabulary of one entry: both gradients are
            # rounding noise around zero)
            assert diff <= 1.5e-2 * np.linalg.norm(ref) + 1e-5 * gmax * np.sqrt(ref.size), (recipe, k)
    assert torch.isfinite(one["dhidden"]).all() and torch.isfinite(one["dW"]).all()


@pytest.mark.parametrize("H", [64, 256], ids=["narrow_tiles", "wide_tiles"])
def test_accumulate_dW_adds_to_what_the_caller_holds(H):
    """Gradient accumulation over micro-batches: with accumulate_dW set, both the separate
    backward and the single-pass call add this batch's dW_head to the buffer's contents."""
    recipe = small_recipe(H=H, V=700, Q=3, length_law=("uniform", 20, 60))
    batch = gen.make_batch(recipe, 12)
    adv, ref = oracle_case(batch, 0.2, 0.28)
    hidden, W, ids, old, advd, cu = device_inputs(batch, adv)
    T, V = batch.T, recipe.V
    base = torch.randn(V, H, device="cuda") * ref["dW"].std()
    want = base.double().cpu().numpy() + ref["dW"]
    # separate calls
    out = U.gpu_scores(hidden, W, ids, old, advd, cu, 0.2, 0.28, want_bwd=False)
    dH, dW = torch.empty(T, H, device="cuda"), base.clone()
    ws = torch.empty(B.sapo_workspace_bytes(B.WS_BWD, T, H, V, B.DTYPE_BF16), dtype=torch.uint8, device="cuda")
    status = B.new_status()
    B.sapo_policy_loss_bwd(hidden, W, ids, out["lse"], out["gscale"], dH, dW, True, ws, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert np.linalg.norm(dW.double().cpu().numpy() - want) <= U.TOL_GRAD_FRO * np.linalg.norm(ref["dW"])
    # single-pass call
    out2 = B.alloc_fwd_outputs(T, batch.S)
    dH2, dW2 = torch.empty(T, H, device="cuda"), base.clone()
    ws2 = torch.empty(B.sapo_workspace_bytes(B.WS_FUSED, T, H, V, B.DTYPE_BF16), dtype=torch.uint8, device="cuda")
    B.sapo_policy_loss_fwd_bwd(hidden, W, ids, old, advd, cu, 0.2, 0.28, 1.0, out2, dH2, dW2, True, ws2, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert np.linalg.norm(dW2.double().cpu().numpy() - want) <= U.TOL_GRAD_FRO * np.linalg.norm(ref["dW"])
    assert U.rel_fro(dH2.cpu().numpy(), ref["dhidden"]) <= U.TOL_GRAD_FRO


@pytest.mark.parametrize("H", [72, 264], ids=["narrow_tiles", "wide_tiles"])
def test_padded_leading_dimensions(H):
    """hidden and W_head as column slices of wider buffers (leading dimension > H)."""
    recipe = small_recipe(H=H, V=900, Q=3, length_law=("uniform", 20, 60))
    batch = gen.make_batch(recipe, 14)
    adv, ref = oracle_case(batch, 0.2, 0.28)
    hidden, W, ids, old, advd, cu = device_inputs(batch, adv)
    big_h = torch.full((batch.T, H + 40), 7.0, dtype=torch.bfloat16, device="cuda")
    big_W = torch.full((recipe.V, H + 16), -3.0, dtype=torch.bfloat16, device="cuda")
    big_h[:, :H] = hidden
    big_W[:, :H] = W
    hv, Wv = big_h[:, :H], big_W[:, :H]
    assert hv.stride(0) == H + 40 and Wv.stride(0) == H + 16
    check_all(U.gpu_scores_fused(hv, Wv, ids, old, advd, cu, 0.2, 0.28), ref, adv, batch, 0.2, 0.28)
    check_all(U.gpu_scores(hv, Wv, ids, old, advd, cu, 0.2, 0.28), ref, adv, batch, 0.2, 0.28)


@pytest.mark.parametrize("H", [64, 256], ids=["narrow_tiles", "wide_tiles"])
def test_peaked_distributions(H):
    """Logits with a standard deviation of about 8, as a trained head has, instead of the
    near-uniform softmax of a freshly drawn one: half of the chosen tokens are the arg-max
    (probability close to 1, so 1 - p is a difference of nearly equal numbers), the other half
    are random (log-probs of -20 and below)."""
    recipe = small_recipe(H=H, V=2000, Q=4, length_law=("uniform", 30, 60))
    batch = gen.make_batch(recipe, 41)
    rng = np.random.default_rng(5)
    batch.W = gen.draw_W(rng, recipe.V, H, recipe.dtype, std=8.0 / np.sqrt(H))
    b = batch.built
    z = gen.as_f32(b.hidden).astype(np.float64) @ gen.as_f32(batch.W).astype(np.float64).T
    top = z.argmax(axis=1).astype(np.int32)
    pick = rng.random(batch.T) < 0.5
    b.ids[pick] = top[pick]
    adv, ref = oracle_case(batch, 0.2, 0.28)
    assert np.exp(ref["logp"]).max() > 0.99 and ref["logp"].min() < -20
    args = device_inputs(batch, adv)
    check_all(U.gpu_scores(*args, 0.2, 0.28), ref, adv, batch, 0.2, 0.28)
    check_all(U.gpu_scores_fused(*args, 0.2, 0.28), ref, adv, batch, 0.2, 0.28)


def test_fused_flags_bad_ids_and_stale_old_logp():
    recipe = small_recipe(H=64, V=400, Q=2, length_law=("uniform", 20, 40))
    batch = gen.make_batch(recipe, 9)
    adv, ref = oracle_case(batch, 0.2, 0.28)
    hidden, W, ids, old, advd, cu = device_inputs(batch, adv)
    ids_bad = ids.clone(); ids_bad[3] = 400; ids_bad[7] = -1
    out = U.gpu_scores_fused(hidden, W, ids_bad, old, advd, cu, 0.2, 0.28)
    assert out["status"] == 0x10
    assert out["gscale"][3].item() == 0 and out["gscale"][7].item() == 0
    assert torch.all(out["dhidden"][3] == 0) and torch.all(out["dhidden"][7] == 0)
    assert torch.isfinite(out["dW"]).all() and torch.isfinite(out["dhidden"]).all()
    keep = np.ones(batch.T, dtype=bool); keep[[3, 7]] = False
    assert np.max(np.abs(out["logp"].cpu().numpy()[keep] - ref["logp"][keep])) <= U.TOL_LOGP_ABS
    # an old log-prob 200 nats below the current one: exp(z - c) leaves the safe range
    old_stale = old.clone(); old_stale[5] -= 200.0
    out = U.gpu_scores_fused(hidden, W, ids, old_stale, advd, cu, 0.2, 0.28)
    assert out["status"] == 0x80
    assert out["gscale"][5].item() == 0 and torch.all(out["dhidden"][5] == 0)
    assert torch.isfinite(out["dW"]).all() and torch.isfinite(out["dhidden"]).all()
    # and 200 nats above it: the exponentials overflow; the row is flagged and cleared, and the
    # other tokens' results are untouched
    old_stale = old.clone(); old_stale[6] += 200.0
    out = U.gpu_scores_fused(hidden, W, ids, old_stale, advd, cu, 0.2, 0.28)
    assert out["status"] == 0x80
    assert out["gscale"][6].item() == 0 and torch.all(out["dhidden"][6] == 0)
    assert torch.isfinite(out["dW"]).all() and torch.isfinite(out["dhidden"]).all()
    keep = np.ones(batch.T, dtype=bool); keep[6] = False
    assert np.max(np.abs(out["logp"].cpu().numpy()[keep] - ref["logp"][keep])) <= U.TOL_LOGP_ABS
    clean = U.gpu_scores_fused(hidden, W, ids, old, advd, cu, 0.2, 0.28)
    rows = torch.from_numpy(np.nonzero(keep)[0]).cuda()
    assert torch.equal(out["dhidden"][rows], clean["dhidden"][rows])


def test_fused_argument_errors():
    x = torch.zeros(8, 16, dtype=torch.float32, device="cuda")
    W = torch.zeros(16, 16, dtype=torch.float32, device="cuda")
    i = torch.zeros(8, dtype=torch.int32, device="cuda")
    f = torch.zeros(8, device="cuda")
    cu = torch.tensor([0, 8], dtype=torch.int32, device="cuda")
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    out = B.alloc_fwd_outputs(8, 1)
    dH, dW = torch.empty(8, 16, device="cuda"), torch.empty(16, 16, device="cuda")
    with pytest.raises(B.SapoError, match="unsupported shape"):      # fp32 operands
        B.sapo_policy_loss_fwd_bwd(x, W, i, f, f[:1], cu, 0.2, 0.2, 1.0, out, dH, dW, False, ws, B.new_status())
    xb, Wb = x.bfloat16(), W.bfloat16()
    with pytest.raises(B.SapoError, match="workspace too small"):
        B.sapo_policy_loss_fwd_bwd(xb, Wb, i, f, f[:1], cu, 0.2, 0.2, 1.0, out, dH, dW, False, ws[:1024],
                                   B.new_status())
    assert B.sapo_workspace_bytes(B.WS_FUSED, 8, 16, 16, B.DTYPE_F32) == 0


def test_steps_from_pinned_host_buffers_overlap_their_copies_and_repeat_bit_for_bit():
    """PolicyScorer.step_from_host keeps two sets of device input buffers and copies the next
    step's inputs while the current step computes: consecutive steps (which alternate between
    the sets) must give the bits of a step over device-resident inputs."""
    from paper_2509_08721_b200.pipeline import PolicyScorer
    recipe = small_recipe(H=256, V=3000, Q=6, length_law=("uniform", 40, 120))
    batch = gen.make_batch(recipe, 55)
    gen.install_old_logp(batch, U.oracle_current_logp(batch))
    scorer = PolicyScorer(U.to_torch(batch.W), batch.T, batch.S, recipe.Q, eps_low=0.2, eps_high=0.28,
                          backward="fused")
    scorer.make_host_batch(batch)
    first = scorer.step_from_host(batch.T, batch.S)
    torch.cuda.synchronize()
    want = {k: first.fwd[k].clone() for k in ("logp", "ratio", "gscale", "loss")}
    want_dW, want_dH = first.dW.clone(), first.dhidden.clone()
    for _ in range(4):
        res = scorer.step_from_host(batch.T, batch.S)
    torch.cuda.synchronize()
    scorer.check_status()
    for k, v in want.items():
        assert torch.equal(res.fwd[k], v), k
    assert torch.equal(res.dW, want_dW) and torch.equal(res.dhidden, want_dH)
    assert torch.equal(scorer._logp_host, want["logp"][:batch.T].cpu())
    # and against the oracle, so that "the same bits" are the right ones
    adv = orc.group_advantages(batch.built.rewards, batch.built.group_offsets,
                               adv_eps=float(np.float32(batch.adv_eps)))["adv"]
    ref = orc.policy_loss_fwd(gen.as_f32(batch.built.hidden), gen.as_f32(batch.W), batch.built.ids,
                              batch.built.old_logp, adv, batch.built.cu_seqlens, 0.2, 0.28)
    out = {k: res.fwd[k][:batch.T] for k in ("logp", "lse", "ratio", "surr", "gscale")}
    U.check_forward(out, ref, adv, batch.built.cu_seqlens, 0.2, 0.28)
