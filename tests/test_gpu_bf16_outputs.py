"""Gradients asked for in bf16 (for a bf16 backward pass and optimiser).  The sums are formed in
fp32 exactly as for fp32 outputs and rounded once, so a bf16 result must equal the fp32 result
rounded to bf16, bit for bit, on every path: narrow and wide tiles, K-split tiles, several token
chunks (dW_head summed in fp32 scratch first) and the compacting backward; and it must meet the
oracle tolerance."""
import numpy as np
import pytest
import torch

from paper_2509_08721_b200 import binding as B
from paper_2509_08721_b200 import inputs as gen
from tests import util as U
from tests.test_gpu_fused import device_inputs, oracle_case
from tests.test_gpu_parity import small_recipe

pytestmark = pytest.mark.gpu

SHAPES = [
    ("narrow_tiles", small_recipe(H=64, V=1000)),
    ("narrow_k_split", small_recipe(H=128, V=20000, Q=2, length_law=("uniform", 50, 90))),
    ("wide_tiles_ragged", small_recipe(H=328, V=2500, Q=6, I=3, J=3, length_law=("uniform", 30, 120))),
    ("wide_k_split", small_recipe(H=512, V=8192, Q=8, length_law=("uniform", 150, 230))),
    ("wide_three_tiles", small_recipe(H=1032, V=650, Q=4, length_law=("uniform", 30, 34))),
]


def _check(out16, out32, ref):
    assert out16["status"] == 0 and out32["status"] == 0
    for k in ("dhidden", "dW"):
        assert out16[k].dtype == torch.bfloat16
        assert torch.equal(out16[k], out32[k].to(torch.bfloat16)), k
    assert U.rel_fro(out16["dhidden"].float().cpu().numpy(), ref["dhidden"]) <= U.TOL_GRAD_FRO
    assert U.rel_fro(out16["dW"].float().cpu().numpy(), ref["dW"]) <= U.TOL_GRAD_FRO


@pytest.mark.parametrize("fused", [False, True], ids=["separate_calls", "single_pass"])
@pytest.mark.parametrize("name,recipe", SHAPES, ids=[c[0] for c in SHAPES])
def test_bf16_gradients_are_the_fp32_ones_rounded_once(name, recipe, fused):
    batch = gen.make_batch(recipe, 21)
    adv, ref = oracle_case(batch, 0.2, 0.28, noise_scale=3.0)
    run = U.gpu_scores_fused if fused else U.gpu_scores
    args = device_inputs(batch, adv)
    _check(run(*args, 0.2, 0.28, out_dtype=torch.bfloat16), run(*args, 0.2, 0.28), ref)


@pytest.mark.parametrize("fused", [False, True], ids=["separate_calls", "single_pass"])
@pytest.mark.parametrize("H", [64, 320], ids=["narrow_tiles", "wide_tiles"])
def test_bf16_gradients_over_several_token_chunks(H, fused):
    """With a panel of 128 tokens the batch runs in chunks: dW_head is summed over them in fp32
    scratch (asked for with the OUT_BF16 flag of the workspace query) and rounded once."""
    recipe = small_recipe(H=H, V=520, Q=4, length_law=("uniform", 60, 120))
    batch = gen.make_batch(recipe, 33)
    assert batch.T > 512
    adv, ref = oracle_case(batch, 0.2, 0.28, noise_scale=2.0)
    kind = B.WS_FUSED if fused else B.WS_BWD
    small16 = B.sapo_workspace_bytes_min(kind | B.WS_OUT_BF16, batch.T, H, 520, B.DTYPE_BF16)
    small32 = B.sapo_workspace_bytes_min(kind, batch.T, H, 520, B.DTYPE_BF16)
    assert small16 == small32 + 520 * H * 4                    # the fp32 copy of dW_head
    run = U.gpu_scores_fused if fused else U.gpu_scores
    key = "workspace_bytes" if fused else "bwd_workspace_bytes"
    args = device_inputs(batch, adv)
    _check(run(*args, 0.2, 0.28, out_dtype=torch.bfloat16, **{key: small16}),
           run(*args, 0.2, 0.28, **{key: small32}), ref)


@pytest.mark.parametrize("chunks", [False, True], ids=["one_chunk", "several_chunks"])
def test_bf16_dW_can_be_added_to_what_the_caller_holds(chunks):
    recipe = small_recipe(H=320, V=520, Q=4, length_law=("uniform", 60, 120))
    batch = gen.make_batch(recipe, 34)
    adv, ref = oracle_case(batch, 0.2, 0.28)
    args = device_inputs(batch, adv)
    kw = {}
    if chunks:
        kw["workspace_bytes"] = B.sapo_workspace_bytes_min(B.WS_FUSED | B.WS_OUT_BF16, batch.T, 320, 520, B.DTYPE_BF16)
    g = torch.Generator(device="cuda").manual_seed(1)
    held = (torch.randn(520, 320, device="cuda", generator=g) * 1e-3).to(torch.bfloat16)
    plain = U.gpu_scores_fused(*args, 0.2, 0.28, **({"workspace_bytes": B.sapo_workspace_bytes_min(
        B.WS_FUSED, batch.T, 320, 520, B.DTYPE_BF16)} if chunks else {}))
    out = U.gpu_scores_fused(*args, 0.2, 0.28, out_dtype=torch.bfloat16, accumulate_into=held.clone(), **kw)
    assert out["status"] == 0
    want = (held.float() + plain["dW"]).to(torch.bfloat16)
    # one rounding of (held + fp32 sum): the sum is formed in fp32 scratch first
    assert torch.equal(out["dW"], want)


def test_bf16_gradients_from_the_compacting_backward():
    r = gen.config(3, length_div=16)
    recipe = gen.Recipe(**{**r.__dict__, "H": 128, "V": 3000, "Q": 8, "I": 2, "J": 2})
    batch = gen.make_batch(recipe, 3003)
    adv, ref = oracle_case(batch, 0.2, 0.2)
    hidden, W, ids, old, adv_d, cu = device_inputs(batch, adv)
    T, H, V, S = batch.T, 128, 3000, batch.S
    fwd = U.gpu_scores(hidden, W, ids, old, adv_d, cu, 0.2, 0.2, want_bwd=False)
    res = {}
    for dt in (torch.float32, torch.bfloat16):
        kind = B.WS_BWD_ACTIVE | (B.WS_OUT_BF16 if dt == torch.bfloat16 else 0)
        ws = torch.empty(B.sapo_workspace_bytes(kind, T, H, V, B.DTYPE_BF16), dtype=torch.uint8, device="cuda")
        dH = torch.full((T, H), 7.0, dtype=dt, device="cuda")
        dW = torch.empty(V, H, dtype=dt, device="cuda")
        status = B.new_status()
        B.sapo_policy_loss_bwd_active(hidden, W, ids, fwd["lse"], fwd["gscale"], dH, dW, False, ws, status)
        torch.cuda.synchronize()
        assert status.item() == 0
        res[dt] = (dH, dW)
    assert torch.equal(res[torch.bfloat16][0], res[torch.float32][0].to(torch.bfloat16))
    assert torch.equal(res[torch.bfloat16][1], res[torch.float32][1].to(torch.bfloat16))
    assert U.rel_fro(res[torch.bfloat16][1].float().cpu().numpy(), ref["dW"]) <= U.TOL_GRAD_FRO


def test_mismatched_or_unknown_output_types_are_rejected():
    x = torch.zeros(8, 16, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(16, 16, dtype=torch.bfloat16, device="cuda")
    i = torch.zeros(8, dtype=torch.int32, device="cuda")
    f = torch.zeros(8, device="cuda")
    ws = torch.empty(1 << 24, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SapoError):
        B.sapo_policy_loss_bwd(x, W, i, f, f, torch.zeros(8, 16, device="cuda"),
                               torch.zeros(16, 16, dtype=torch.bfloat16, device="cuda"), False, ws, B.new_status())
