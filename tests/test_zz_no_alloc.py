"""The forward entry point that needs no caller-side scratch, sapo_policy_loss_fwd_static.

It serves hosts of the library that must not allocate device memory (for instance a component
inside a process whose memory pool was fixed at start-up): its scratch is an array built into
the library.  Here it is called through the C ABI twice in a row — the second call reuses the
array with the first call's leftovers in it — and each result is compared with the regular
entry point's on the same inputs, under the parity tolerances of the other tests.
This file sorts last on purpose, so a run that stops at the first failure has already run
every other test.
"""
import numpy as np
import pytest
import torch

from paper_2509_08721_b200 import binding as B
from paper_2509_08721_b200 import inputs as gen
from tests import util as U

pytestmark = pytest.mark.gpu


def _inputs(recipe, seed):
    batch = gen.make_batch(recipe, seed)
    b = batch.built
    rng = np.random.default_rng(seed)
    hidden, W, ids = U.to_torch(b.hidden), U.to_torch(batch.W), U.to_torch(b.ids)
    cur = U.torch_current_logp(hidden, W, ids)
    old = cur + torch.from_numpy(b.logp_noise).cuda()
    adv = torch.from_numpy(rng.normal(size=batch.S).astype(np.float32)).cuda()
    return batch, hidden, W, ids, old, adv, U.to_torch(b.cu_seqlens)


def _regular(hidden, W, ids, old, adv, cu):
    T, H, V, S = hidden.shape[0], hidden.shape[1], W.shape[0], cu.numel() - 1
    out, status = B.alloc_fwd_outputs(T, S), B.new_status()
    ws = torch.empty(B.sapo_workspace_bytes(B.WS_FWD, T, H, V, B.DTYPE_BF16), dtype=torch.uint8, device="cuda")
    B.sapo_policy_loss_fwd(hidden, W, ids, old, adv, cu, 0.2, 0.28, 1.0, out, ws, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    return out


def _static(hidden, W, ids, old, adv, cu):
    T, S = hidden.shape[0], cu.numel() - 1
    out, status = B.alloc_fwd_outputs(T, S), B.new_status()
    B.sapo_policy_loss_fwd_static(hidden, W, ids, old, adv, cu, 0.2, 0.28, 1.0, out, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    return out


def _same(a, b):
    for k in ("logp", "lse"):
        assert (a[k] - b[k]).abs().max().item() <= U.TOL_LOGP_ABS, k
    for k in ("ratio", "surr", "gscale", "seq_surr"):
        scale = b[k].abs().max().item() + 1e-30
        assert (a[k] - b[k]).abs().max().item() <= 4e-3 * scale, k
    la, lb = a["loss"].item(), b["loss"].item()
    assert abs(la - lb) <= U.TOL_LOSS_REL * abs(lb) + 1e-7


def test_static_scratch_forward_matches_the_regular_one_twice_in_a_row():
    # two different shapes back to back: the second call finds the first one's partials in the array
    first = gen.Recipe("na1", gen.DTYPE_BF16, 128, 3000, 4, 2, 2, ("uniform", 20, 90), ("bernoulli", 0.5))
    second = gen.Recipe("na2", gen.DTYPE_BF16, 72, 777, 3, 3, 1, ("uniform", 5, 40), ("bernoulli", 0.5))
    for recipe, seed in ((first, 41), (second, 42)):
        _, hidden, W, ids, old, adv, cu = _inputs(recipe, seed)
        ref = _regular(hidden, W, ids, old, adv, cu)
        _same(_static(hidden, W, ids, old, adv, cu), ref)
    # and once more on the last shape, immediately after itself
    _same(_static(hidden, W, ids, old, adv, cu), ref)


def test_static_scratch_rejects_what_does_not_fit():
    lib = B.load()
    cfg = B.LossCfgC(0.2, 0.2, 1.0, 0, 0.0, None)
    one = torch.zeros(256, dtype=torch.float32, device="cuda")
    # three floats of scratch per token (and per vocab split): two million tokens need 24 MB
    T, H, V = 2_000_000, 64, 512
    assert B.sapo_workspace_bytes(B.WS_FWD, T, H, V, B.DTYPE_BF16) > B.STATIC_SCRATCH_BYTES
    rc = lib.sapo_policy_loss_fwd_static(one.data_ptr(), one.data_ptr(), B.DTYPE_BF16, T, H, V, H, H,
                                         one.data_ptr(), one.data_ptr(), one.data_ptr(), one.data_ptr(), 1,
                                         cfg, *([one.data_ptr()] * 7), B.new_status().data_ptr(), None)
    assert rc == -5 and b"static scratch" in lib.sapo_status_string(rc)
    rc = lib.sapo_policy_loss_fwd_static(one.data_ptr(), one.data_ptr(), B.DTYPE_F32, 128, H, V, H, H,
                                         one.data_ptr(), one.data_ptr(), one.data_ptr(), one.data_ptr(), 1,
                                         cfg, *([one.data_ptr()] * 7), B.new_status().data_ptr(), None)
    assert rc == -2
