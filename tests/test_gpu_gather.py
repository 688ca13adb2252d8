"""The single-pass call with the hidden states read in place from the two rollout stores
(sapo_policy_loss_fwd_bwd_gather): the pack writes, for every packed token, its row in the local
or external store and copies no hidden rows; the projection's row loads follow that map.
The map is index work and must be exact; the loss and gradients must equal, bit for bit, those of
the regular single-pass call on a packed copy (the same rows reach the same kernels), and meet the
oracle tolerances."""
import numpy as np
import pytest
import torch

from paper_2509_08721_b200 import binding as B
from paper_2509_08721_b200 import inputs as gen
from tests import util as U
from tests.test_gpu_fused import check_all, oracle_case
from tests.test_gpu_parity import small_recipe

pytestmark = pytest.mark.gpu

CASES = [
    # name, recipe, per-question (I, J) lists or None
    ("sequences_across_blocks", small_recipe(H=320, V=2500, Q=5, length_law=("uniform", 30, 110)), None),
    ("many_tiny_sequences", small_recipe(H=128, V=1000, Q=12, I=4, J=4, length_law=("uniform", 1, 5)), None),
    ("single_token_sequences", small_recipe(H=64, V=300, Q=20, I=4, J=4, length_law=("fixed", 1)), None),
    ("all_local", small_recipe(H=256, V=777, Q=4, I=4, J=0, length_law=("uniform", 20, 90)), None),
    ("all_external", small_recipe(H=256, V=777, Q=4, I=0, J=3, length_law=("uniform", 20, 90)), None),
    ("long_sequences", small_recipe(H=512, V=4100, Q=2, I=1, J=1, length_law=("uniform", 300, 500)), None),
]


def expected_tok_src(batch):
    """Row of every packed token in its store, from the generator's own construction."""
    b = batch.built
    out = np.zeros(batch.T, dtype=np.int64)
    for s in range(batch.S):
        side = int(b.seq_is_ext[s])
        off = (batch.ext if side else batch.local).offsets[b.seq_src[s]]
        a, e = int(b.cu_seqlens[s]), int(b.cu_seqlens[s + 1])
        out[a:e] = off + np.arange(e - a) + (side << 62)
    return out


def run_gather(batch, adv, capacity=None, workspace_bytes=None, **kw):
    local, ext, sel = U.dev_rollouts(batch.local), U.dev_rollouts(batch.ext), U.dev_selection(batch.sel)
    T, S, H, V = batch.T, batch.S, batch.H, batch.V
    cap = T if capacity is None else capacity
    packed = B.alloc_packed(cap, S, batch.sel.Q, H, torch.bfloat16, copy_hidden=False)
    status = B.new_status()
    B.sapo_pack_rollouts(local, ext, sel, packed, status)
    out = B.alloc_fwd_outputs(cap, S)
    nbytes = (B.sapo_workspace_bytes(B.WS_FUSED | B.WS_GATHER, cap, H, V, B.DTYPE_BF16)
              if workspace_bytes is None else workspace_bytes)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    out["dhidden"] = torch.empty(cap, H, device="cuda")
    out["dW"] = torch.empty(V, H, device="cuda")
    B.sapo_policy_loss_fwd_bwd_gather(local.hidden, ext.hidden, packed["tok_src"], U.to_torch(batch.W),
                                      packed["ids"], packed["old_logp"], U.to_torch(adv.astype(np.float32)),
                                      packed["cu_seqlens"], 0.2, 0.28, 1.0, out, out["dhidden"], out["dW"], False,
                                      ws, status, **kw)
    torch.cuda.synchronize()
    out["status"] = int(status.item())
    return packed, out


@pytest.mark.parametrize("name,recipe,selections", CASES, ids=[c[0] for c in CASES])
def test_hidden_rows_read_in_place_give_the_results_of_the_packed_copy(name, recipe, selections):
    batch = gen.make_batch(recipe, 91, selections=selections)
    adv, ref = oracle_case(batch, 0.2, 0.28, noise_scale=2.0)
    packed, out = run_gather(batch, adv)
    assert packed["hidden"] is None
    assert np.array_equal(packed["tok_src"].cpu().numpy(), expected_tok_src(batch))
    check_all(out, ref, adv, batch, 0.2, 0.28)
    b = batch.built
    plain = U.gpu_scores_fused(U.to_torch(b.hidden), U.to_torch(batch.W), U.to_torch(b.ids), U.to_torch(b.old_logp),
                               U.to_torch(adv.astype(np.float32)), U.to_torch(b.cu_seqlens), 0.2, 0.28)
    for k in ("logp", "lse", "ratio", "surr", "gscale", "seq_surr", "loss", "dhidden", "dW"):
        assert torch.equal(out[k], plain[k]), k


def test_in_place_rows_over_several_token_chunks_and_with_entropy():
    recipe = small_recipe(H=64, V=520, Q=4, length_law=("uniform", 60, 120))
    batch = gen.make_batch(recipe, 92)
    assert batch.T > 512
    adv, ref = oracle_case(batch, 0.2, 0.28, noise_scale=2.0)
    small = B.sapo_workspace_bytes_min(B.WS_FUSED | B.WS_GATHER, batch.T, 64, 520, B.DTYPE_BF16)
    ent = torch.empty(batch.T, device="cuda")
    _, out = run_gather(batch, adv, workspace_bytes=small, entropy=ent)
    check_all(out, ref, adv, batch, 0.2, 0.28)
    from oracle import sapo_oracle as orc
    ref_ent = orc.token_entropy(gen.as_f32(batch.built.hidden), gen.as_f32(batch.W))
    assert np.max(np.abs(ent.cpu().numpy() - ref_ent)) <= U.TOL_LOGP_ABS


def test_in_place_rows_with_the_whole_capacity_scored():
    """Slots past the last packed token have no source row: they are scored as masked and the
    rest is unchanged."""
    recipe = small_recipe(H=320, V=2500, Q=5, length_law=("uniform", 30, 110))
    batch = gen.make_batch(recipe, 93)
    adv, ref = oracle_case(batch, 0.2, 0.28)
    T = batch.T
    packed, out = run_gather(batch, adv, capacity=T + 300)
    assert out["status"] == 0
    assert (packed["tok_src"][T:] == -1).all()
    head = {k: out[k][:T] for k in ("logp", "lse", "ratio", "surr", "gscale")}
    U.check_forward(head, ref, adv, batch.built.cu_seqlens, 0.2, 0.28)
    for k in ("logp", "lse", "ratio", "surr", "gscale"):
        assert not out[k][T:].any(), k
    assert not out["dhidden"][T:].any()
    assert U.rel_fro(out["dhidden"][:T].cpu().numpy(), ref["dhidden"]) <= U.TOL_GRAD_FRO
    assert U.rel_fro(out["dW"].cpu().numpy(), ref["dW"]) <= U.TOL_GRAD_FRO
    assert torch.isfinite(out["dW"]).all()


def test_a_source_row_outside_its_store_is_reported_not_read():
    recipe = small_recipe(H=64, V=300, Q=2, length_law=("uniform", 10, 20))
    batch = gen.make_batch(recipe, 94)
    adv, _ = oracle_case(batch, 0.2, 0.28)
    local, ext = U.dev_rollouts(batch.local), U.dev_rollouts(batch.ext)
    b = batch.built
    T, S, H, V = batch.T, batch.S, batch.H, batch.V
    tok_src = torch.from_numpy(expected_tok_src(batch)).cuda()
    tok_src[5] = local.hidden.shape[0] + 7            # a row past the end of the local store
    out = B.alloc_fwd_outputs(T, S)
    ws = torch.empty(B.sapo_workspace_bytes(B.WS_FUSED | B.WS_GATHER, T, H, V, B.DTYPE_BF16), dtype=torch.uint8,
                     device="cuda")
    status = B.new_status()
    B.sapo_policy_loss_fwd_bwd_gather(local.hidden, ext.hidden, tok_src, U.to_torch(batch.W), U.to_torch(b.ids),
                                      U.to_torch(b.old_logp), U.to_torch(adv.astype(np.float32)),
                                      U.to_torch(b.cu_seqlens), 0.2, 0.28, 1.0, out, torch.empty(T, H, device="cuda"),
                                      torch.empty(V, H, device="cuda"), False, ws, status)
    torch.cuda.synchronize()
    assert status.item() & 0x04
