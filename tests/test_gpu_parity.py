"""Parity of the CUDA path (through the C ABI) with the fp64 oracle on the same seeded
inputs: bit-exact for pack, 2e-3 absolute on log-probs, 1e-3 relative on the loss,
2e-2 relative Frobenius on dhidden and dW_head."""
import numpy as np
import pytest
import torch

from oracle import sapo_oracle as orc
from paper_2509_08721_b200 import binding as B
from paper_2509_08721_b200 import inputs as gen
from tests import util as U

pytestmark = pytest.mark.gpu


def small_recipe(**kw):
    base = dict(name="small", dtype=gen.DTYPE_BF16, H=64, V=1000, Q=3, I=2, J=2,
                length_law=("uniform", 1, 40), reward_law=("bernoulli", 0.5))
    base.update(kw)
    return gen.Recipe(**base)


# ------------------------------------------------------------------------------------ pack
PACK_CASES = [
    ("ragged_groups", small_recipe(Q=5), [(2, 2), (0, 3), (4, 0), (1, 1), (3, 5)]),
    ("paper_granularity", small_recipe(Q=8, H=72), [(8, 0)] * 4 + [(0, 8)] * 4),
    ("fp32_rows", small_recipe(dtype=gen.DTYPE_F32, H=20), None),
    ("odd_row_bytes", small_recipe(H=13), None),
    ("cfg1", gen.config(1), None),
    ("cfg2_lite", gen.config(2, length_div=8), None),
    # the swarm-mix sweep: every external share, drawn from the pool of eight node buffers
    ("cfg5_lite_J0", gen.config(5, ext_fraction=0.0, length_div=16), None),
    ("cfg5_lite_J2", gen.config(5, ext_fraction=0.25, length_div=16), None),
    ("cfg5_lite_J4", gen.config(5, ext_fraction=0.5, length_div=16), None),
    ("cfg5_lite_J6", gen.config(5, ext_fraction=0.75, length_div=16), None),
]


@pytest.mark.parametrize("name,recipe,selections", PACK_CASES, ids=[c[0] for c in PACK_CASES])
def test_pack_is_bit_exact(name, recipe, selections):
    if recipe.V > 5000:
        recipe = gen.Recipe(**{**recipe.__dict__, "V": 512})     # W is irrelevant to pack
    batch = gen.make_batch(recipe, 11, selections=selections)
    ref = orc.pack_rollouts(U.buf_dict(batch.local), U.buf_dict(batch.ext), U.sel_dict(batch.sel))
    out, status = U.gpu_pack(batch, max_tokens=batch.T + 37, max_seqs=batch.S + 3)
    assert status == 0
    T, S = ref["n_tokens"], len(ref["seq_group"])
    assert int(out["n_tokens"].item()) == T and int(out["n_seqs"].item()) == S
    hid = U.to_numpy(out["hidden"])[:T]
    assert np.array_equal(hid.view(np.uint8), np.ascontiguousarray(ref["hidden"]).view(np.uint8))
    assert np.array_equal(U.to_numpy(out["ids"])[:T], ref["ids"])
    assert np.array_equal(U.to_numpy(out["old_logp"])[:T].view(np.uint32), ref["old_logp"].view(np.uint32))
    assert np.array_equal(U.to_numpy(out["rewards"])[:S].view(np.uint32), ref["rewards"].view(np.uint32))
    assert np.array_equal(U.to_numpy(out["cu_seqlens"])[:S + 1], ref["cu_seqlens"])
    for k in ("seq_group", "seq_is_ext", "seq_src"):
        assert np.array_equal(U.to_numpy(out[k])[:S], ref[k]), k
    assert np.array_equal(U.to_numpy(out["tok_seq"])[:T], ref["tok_seq"])
    assert np.array_equal(U.to_numpy(out["group_offsets"]), ref["group_offsets"])
    mask = U.to_numpy(out["tok_mask"])
    assert mask[:T].all() and not mask[T:].any()


def test_pack_reports_overflow_and_bad_indices():
    batch = gen.make_batch(small_recipe(), 3)
    out, status = U.gpu_pack(batch, max_tokens=batch.T - 5)
    assert status & 0x01 and int(out["n_tokens"].item()) == batch.T - 5
    ref = orc.pack_rollouts(U.buf_dict(batch.local), U.buf_dict(batch.ext), U.sel_dict(batch.sel))
    assert np.array_equal(U.to_numpy(out["ids"]), ref["ids"][:batch.T - 5])
    out, status = U.gpu_pack(batch, max_seqs=batch.S - 1)
    assert status & 0x02 and int(out["n_tokens"].item()) == 0
    batch.sel.local_idx[1] = batch.local.n_rollouts + 4          # outside the buffer
    out, status = U.gpu_pack(batch)
    assert status & 0x04
    cu = U.to_numpy(out["cu_seqlens"])
    assert cu[2] == cu[1]                                        # packed as an empty sequence


def test_pack_empty_selection():
    batch = gen.make_batch(small_recipe(Q=2), 3, selections=[(0, 0), (0, 0)])
    out, status = U.gpu_pack(batch, max_tokens=16, max_seqs=4)
    assert status == 0 and int(out["n_tokens"].item()) == 0 and int(out["n_seqs"].item()) == 0
    assert not U.to_numpy(out["tok_mask"]).any()


# ------------------------------------------------------------------------------ advantages
@pytest.mark.parametrize("ddof", [0, 1])
def test_advantages_match_oracle(ddof):
    rng = np.random.default_rng(5)
    sizes = [8, 16, 1, 3, 40, 8, 8, 0, 33]
    go = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    r = rng.choice([0.0, 0.5, 1.0], size=go[-1]).astype(np.float32)
    r[go[5]:go[6]] = 0.1                                         # all-equal, not exactly summable
    r[go[4]:go[5]] = rng.normal(size=40).astype(np.float32)
    eps = float(np.float32(1e-6))
    ref = orc.group_advantages(r, go, adv_eps=eps, ddof=ddof)
    adv = torch.empty(len(r), dtype=torch.float32, device="cuda")
    mean = torch.empty(len(sizes), dtype=torch.float32, device="cuda")
    std = torch.empty(len(sizes), dtype=torch.float32, device="cuda")
    status = B.new_status()
    B.sapo_group_advantages(U.to_torch(r), U.to_torch(go), eps, ddof, adv, mean, std, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    a = adv.cpu().numpy().astype(np.float64)
    assert np.allclose(a, ref["adv"], rtol=U.TOL_ADV_REL, atol=1e-9)
    assert np.all(a[go[5]:go[6]] == 0.0)
    assert np.allclose(mean.cpu().numpy(), ref["mean"], rtol=U.TOL_ADV_REL, atol=1e-12)
    assert np.allclose(std.cpu().numpy(), ref["std"], rtol=U.TOL_ADV_REL, atol=1e-12)
    for g in range(len(sizes)):
        assert abs(a[go[g]:go[g + 1]].sum()) < 1e-5


def test_advantages_with_many_questions_take_the_thread_per_question_path():
    """From 4096 questions on, one thread serves a question (float4 where alignment allows)."""
    rng = np.random.default_rng(6)
    sizes = rng.integers(0, 21, size=5003)
    sizes[:64] = 8
    go = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    r = rng.choice([0.0, 0.5, 1.0], size=go[-1]).astype(np.float32)
    eps = float(np.float32(1e-6))
    ref = orc.group_advantages(r, go, adv_eps=eps, ddof=0)
    adv = torch.empty(len(r), dtype=torch.float32, device="cuda")
    mean = torch.empty(len(sizes), dtype=torch.float32, device="cuda")
    std = torch.empty(len(sizes), dtype=torch.float32, device="cuda")
    status = B.new_status()
    B.sapo_group_advantages(U.to_torch(r), U.to_torch(go), eps, 0, adv, mean, std, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert np.allclose(adv.cpu().numpy(), ref["adv"], rtol=U.TOL_ADV_REL, atol=1e-9)
    assert np.allclose(mean.cpu().numpy(), ref["mean"], rtol=U.TOL_ADV_REL, atol=1e-12)
    assert np.allclose(std.cpu().numpy(), ref["std"], rtol=U.TOL_ADV_REL, atol=1e-12)


@pytest.mark.parametrize("warp_level", [False, True], ids=["thread_per_question", "warp_level"])
@pytest.mark.parametrize("G", [8, 16])
def test_advantages_stay_within_the_stated_ulps_whatever_the_offset(G, warp_level):
    """The kernels keep their sums in compensated fp32.  Against the fp64 oracle: binary and
    partial-credit rewards, real-valued rewards, and the same on top of a large common offset
    (where an uncompensated fp32 mean would lose the deviations) all stay within 6 fp32 ulp."""
    rng = np.random.default_rng(100 + G)
    Q = 6000
    go = (np.arange(Q + 1) * G).astype(np.int32)
    base = np.concatenate([
        rng.choice([0.0, 0.5, 1.0], size=(Q // 3, G)),
        rng.normal(size=(Q // 3, G)),
        rng.random(size=(Q - 2 * (Q // 3), G)) * 1e-3,
    ]).astype(np.float32)
    eps = float(np.float32(1e-6))
    worst = 0.0
    for offset in (0.0, 1000.0, -3.0e5):
        r = (base + np.float32(offset)).astype(np.float32).reshape(-1)
        ref = orc.group_advantages(r, go, adv_eps=eps, ddof=0)
        adv = torch.empty(len(r), dtype=torch.float32, device="cuda")
        std = torch.empty(Q, dtype=torch.float32, device="cuda")
        status = B.new_status()
        B.sapo_group_advantages(U.to_torch(r), U.to_torch(go), eps, 0, adv, None, std, status,
                                warp_level=warp_level)
        torch.cuda.synchronize()
        assert status.item() == 0
        a = adv.cpu().numpy().astype(np.float64)
        big = np.abs(ref["adv"]) > 1e-3                     # ulps of values that are not rounding residue
        ulp = np.abs(a - ref["adv"])[big] / np.spacing(np.abs(ref["adv"][big]).astype(np.float32))
        worst = max(worst, float(ulp.max()))
        assert np.allclose(a, ref["adv"], rtol=U.TOL_ADV_REL, atol=1e-9), (offset, float(ulp.max()))
        assert np.allclose(std.cpu().numpy(), ref["std"], rtol=U.TOL_ADV_REL, atol=1e-12)
    assert worst <= 6.5, worst                               # 6 ulp by the error analysis + the fp32 rounding of the result


def test_advantages_flag_nonfinite_rewards():
    r = torch.tensor([0.0, float("nan"), 1.0, 1.0], device="cuda")
    go = torch.tensor([0, 2, 4], dtype=torch.int32, device="cuda")
    adv = torch.empty(4, device="cuda")
    status = B.new_status()
    B.sapo_group_advantages(r, go, 1e-6, 0, adv, None, None, status)
    torch.cuda.synchronize()
    assert status.item() & 0x40
    assert adv[2:].abs().max().item() == 0.0


# ---------------------------------------------------------------------- loss forward/backward
def run_case(batch, eps_low=None, eps_high=None, grad_scale=1.0, bwd_ws=None, noise_scale=1.0):
    """pack -> advantages -> fwd -> bwd on the device, all of it against the oracle."""
    eps_low = batch.eps_low if eps_low is None else eps_low
    eps_high = batch.eps_high if eps_high is None else eps_high
    batch.built.logp_noise *= np.float32(noise_scale)
    gen.install_old_logp(batch, U.oracle_current_logp(batch))
    # oracle, end to end
    p = orc.pack_rollouts(U.buf_dict(batch.local), U.buf_dict(batch.ext), U.sel_dict(batch.sel))
    eps = float(np.float32(batch.adv_eps))
    a = orc.group_advantages(p["rewards"], p["group_offsets"], adv_eps=eps)
    h64, W64 = gen.as_f32(p["hidden"]), gen.as_f32(batch.W)
    ref = orc.policy_loss_fwd_bwd_rows(h64, W64, p["ids"], p["old_logp"], a["adv"], p["cu_seqlens"],
                                       eps_low, eps_high, grad_scale)
    # device, end to end
    packed, st = U.gpu_pack(batch)
    assert st == 0
    adv = torch.empty(batch.S, dtype=torch.float32, device="cuda")
    status = B.new_status()
    B.sapo_group_advantages(packed["rewards"], packed["group_offsets"], eps, 0, adv, None, None, status)
    out = U.gpu_scores(packed["hidden"], U.to_torch(batch.W), packed["ids"], packed["old_logp"], adv,
                       packed["cu_seqlens"], eps_low, eps_high, grad_scale, bwd_workspace_bytes=bwd_ws)
    assert out["status"] == 0 and status.item() == 0
    assert np.allclose(adv.cpu().numpy(), a["adv"], rtol=U.TOL_ADV_REL, atol=1e-9)
    U.check_forward(out, ref, a["adv"], p["cu_seqlens"], eps_low, eps_high)
    seq = out["seq_surr"].cpu().numpy().astype(np.float64)
    assert np.max(np.abs(seq - ref["seq_surr"])) <= 1e-3 * (np.abs(a["adv"]).max() + 1e-30)
    U.check_loss(float(out["loss"].item()), ref["loss"], a["adv"])
    e_h = U.rel_fro(out["dhidden"].cpu().numpy(), ref["dhidden"])
    e_w = U.rel_fro(out["dW"].cpu().numpy(), ref["dW"])
    assert e_h <= U.TOL_GRAD_FRO and e_w <= U.TOL_GRAD_FRO, (e_h, e_w)
    return out, ref, (e_h, e_w)


SHAPES = [
    # name, recipe, selections
    ("bf16_one_tile", small_recipe(H=64, V=200, Q=2, length_law=("uniform", 3, 20)), None),
    ("bf16_vocab_tail", small_recipe(H=64, V=1000), None),
    ("bf16_k_tail", small_recipe(H=72, V=777, Q=4, length_law=("uniform", 20, 90)), None),
    ("bf16_many_tiles", small_recipe(H=328, V=2500, Q=6, I=3, J=3, length_law=("uniform", 30, 120)), None),
    ("bf16_single_tokens", small_recipe(H=128, V=300, Q=4, length_law=("fixed", 1)), None),
    ("bf16_one_group", small_recipe(H=64, V=520, Q=1, I=3, J=0), None),
    ("fp32_small", small_recipe(dtype=gen.DTYPE_F32, H=40, V=333, Q=3), None),
    # two dH tiles with a long vocabulary contraction: the thin last wave is cut along K
    ("bf16_k_split", small_recipe(H=128, V=20000, Q=2, length_law=("uniform", 50, 90)), None),
    # about 48 dH tiles (fewer than CTA pairs, more than half of them), each cut in three along
    # the vocabulary: more parts than pairs, so pairs take several parts in turn
    ("bf16_k_split_rounds", small_recipe(H=512, V=8192, Q=8, length_law=("uniform", 150, 230)), None),
]


@pytest.mark.parametrize("name,recipe,selections", SHAPES, ids=[c[0] for c in SHAPES])
def test_loss_forward_backward_small_shapes(name, recipe, selections):
    batch = gen.make_batch(recipe, 21, selections=selections)
    run_case(batch, eps_low=0.2, eps_high=0.28, noise_scale=3.0)


def test_config1_tiny_fp32():
    batch = gen.make_batch(gen.config(1), 1001)
    out, ref, _ = run_case(batch)
    # fp32 operands are split into bf16 high and low parts: log-probs stay at fp32 accuracy
    assert np.max(np.abs(out["logp"].cpu().numpy() - ref["logp"])) < 2e-5


def test_backward_with_a_minimal_panel_accumulates_over_chunks():
    recipe = small_recipe(H=64, V=520, Q=4, length_law=("uniform", 60, 120))
    batch = gen.make_batch(recipe, 33)
    ws = B.sapo_workspace_bytes_min(B.WS_BWD, batch.T, 64, 520, B.DTYPE_BF16)
    assert batch.T > 256
    run_case(batch, bwd_ws=ws)


def test_zero_advantage_groups_and_repeatability():
    r = gen.config(3, length_div=16)
    recipe = gen.Recipe(**{**r.__dict__, "H": 128, "V": 3000, "Q": 8, "I": 2, "J": 2})
    batch = gen.make_batch(recipe, 3003)
    out, ref, _ = run_case(batch)
    cu = batch.built.cu_seqlens
    go = batch.built.group_offsets
    dh = out["dhidden"].cpu().numpy()
    for q in range(2):                                   # the all-equal-reward questions
        rows = slice(cu[go[q]], cu[go[q + 1]])
        assert np.all(dh[rows] == 0.0)
        assert np.all(out["gscale"].cpu().numpy()[rows] == 0.0)
    # fixed reduction order: a second run gives identical bits
    packed, _ = U.gpu_pack(batch)
    adv = U.to_torch(orc.group_advantages(batch.built.rewards, go, adv_eps=float(np.float32(1e-6)))["adv"]
                     .astype(np.float32))
    again = U.gpu_scores(packed["hidden"], U.to_torch(batch.W), packed["ids"], packed["old_logp"], adv,
                         packed["cu_seqlens"], batch.eps_low, batch.eps_high)
    for k in ("logp", "loss", "dhidden", "dW"):
        assert torch.equal(again[k], out[k]), k


def test_bad_token_id_is_flagged_and_masked():
    batch = gen.make_batch(small_recipe(H=64, V=300), 5)
    gen.install_old_logp(batch, U.oracle_current_logp(batch))
    b = batch.built
    ids = b.ids.copy()
    ids[3] = 300
    adv = np.ones(batch.S, np.float32)
    out = U.gpu_scores(U.to_torch(b.hidden), U.to_torch(batch.W), U.to_torch(ids), U.to_torch(b.old_logp),
                       U.to_torch(adv), U.to_torch(b.cu_seqlens), 0.2, 0.2, want_bwd=False)
    assert out["status"] & 0x10
    assert out["gscale"][3].item() == 0.0 and out["surr"][3].item() == 0.0


def test_argument_errors_are_reported_on_the_host():
    x = torch.zeros(8, 12, dtype=torch.bfloat16, device="cuda")       # H = 12 is not a multiple of 8
    W = torch.zeros(16, 12, dtype=torch.bfloat16, device="cuda")
    i = torch.zeros(8, dtype=torch.int32, device="cuda")
    f = torch.zeros(8, device="cuda")
    cu = torch.tensor([0, 8], dtype=torch.int32, device="cuda")
    out = B.alloc_fwd_outputs(8, 1)
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SapoError):
        B.sapo_policy_loss_fwd(x, W, i, f, f[:1], cu, 0.2, 0.2, 1.0, out, ws, B.new_status())
    x = torch.zeros(8, 16, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(16, 16, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.SapoError, match="workspace"):
        B.sapo_policy_loss_fwd(x, W, i, f, f[:1], cu, 0.2, 0.2, 1.0, out, ws[:16], B.new_status())
