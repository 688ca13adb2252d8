"""The forward entry point that needs no caller-side scratch, sapo_policy_loss_fwd_static.

It serves hosts of the library that must not allocate device memory (for instance a component
inside a process whose memory pool was fixed at start-up): its scratch is an array built into
the library.  Here it is called through the C ABI twice in a row — the second call reuses the
array with the first call's leftovers in it — and each result is compared with the regular
entry point's on the same inputs.  Both run the same kernels with the same schedule and a fixed
summation order, so every output must be bit-identical; a read of stale scratch, even of a
low-order partial, shows.  One case is also compared with the fp64 oracle, and the free device
memory is read before and after the calls to show that nothing was allocated.
This file sorts last on purpose, so a run that stops at the first failure has already run
every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import sapo_oracle as orc
from paper_2509_08721_b200 import binding as B
from paper_2509_08721_b200 import inputs as gen
from tests import util as U

pytestmark = pytest.mark.gpu


def _inputs(recipe, seed):
    batch = gen.make_batch(recipe, seed)
    b = batch.built
    rng = np.random.default_rng(seed)
    gen.install_old_logp(batch, U.oracle_current_logp(batch))
    hidden, W, ids = U.to_torch(b.hidden), U.to_torch(batch.W), U.to_torch(b.ids)
    adv_np = rng.normal(size=batch.S).astype(np.float32)
    return batch, adv_np, (hidden, W, ids, U.to_torch(b.old_logp), U.to_torch(adv_np), U.to_torch(b.cu_seqlens))


def _regular(hidden, W, ids, old, adv, cu):
    T, H, V, S = hidden.shape[0], hidden.shape[1], W.shape[0], cu.numel() - 1
    out, status = B.alloc_fwd_outputs(T, S), B.new_status()
    ws = torch.empty(B.sapo_workspace_bytes(B.WS_FWD, T, H, V, B.DTYPE_BF16), dtype=torch.uint8, device="cuda")
    B.sapo_policy_loss_fwd(hidden, W, ids, old, adv, cu, 0.2, 0.28, 1.0, out, ws, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    return out


def _static_raw(hidden, W, ids, old, adv, cu, out, status, entropy=None):
    """The raw symbol, called through ctypes with plain pointers: no tensor is created here."""
    T, H, V, S = hidden.shape[0], hidden.shape[1], W.shape[0], cu.numel() - 1
    cfg = B.LossCfgC(0.2, 0.28, 1.0, 0, 0.0, None, None if entropy is None else entropy.data_ptr())
    rc = B.load().sapo_policy_loss_fwd_static(
        hidden.data_ptr(), W.data_ptr(), B.DTYPE_BF16, T, H, V, hidden.stride(0), W.stride(0),
        ids.data_ptr(), old.data_ptr(), adv.data_ptr(), cu.data_ptr(), S, C.byref(cfg),
        out["logp"].data_ptr(), out["lse"].data_ptr(), out["ratio"].data_ptr(), out["surr"].data_ptr(),
        out["gscale"].data_ptr(), out["seq_surr"].data_ptr(), out["loss"].data_ptr(), status.data_ptr(),
        torch.cuda.current_stream().cuda_stream)
    assert rc == 0, rc


def _identical(a, b):
    for k in ("logp", "lse", "ratio", "surr", "gscale", "seq_surr", "loss"):
        assert torch.equal(a[k], b[k]), k


def test_static_scratch_forward_matches_the_regular_one_twice_in_a_row():
    # two different shapes back to back: the second call finds the first one's partials in the array
    first = gen.Recipe("na1", gen.DTYPE_BF16, 128, 3000, 4, 2, 2, ("uniform", 20, 90), ("bernoulli", 0.5))
    second = gen.Recipe("na2", gen.DTYPE_BF16, 72, 777, 3, 3, 1, ("uniform", 5, 40), ("bernoulli", 0.5))
    cases = []
    for recipe, seed in ((first, 41), (second, 42)):
        batch, adv_np, dev = _inputs(recipe, seed)
        ref = _regular(*dev)
        T, S = dev[0].shape[0], dev[5].numel() - 1
        cases.append((batch, adv_np, dev, ref, B.alloc_fwd_outputs(T, S), B.alloc_fwd_outputs(T, S)))
    status = B.new_status()
    torch.cuda.synchronize()
    # first use on this device outside the measured window: it looks up the array's address
    _static_raw(*cases[0][2], cases[0][4], status)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    _static_raw(*cases[0][2], cases[0][4], status)
    _static_raw(*cases[1][2], cases[1][4], status)
    _static_raw(*cases[1][2], cases[1][5], status)     # and once more on the last shape, right after itself
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before                   # the calls took no device memory
    assert status.item() == 0
    _identical(cases[0][4], cases[0][3])
    _identical(cases[1][4], cases[1][3])
    _identical(cases[1][5], cases[1][3])
    # with the entropy output (one more partial array in the scratch): same values as the regular call's
    hidden, W, ids, old, adv, cu = cases[0][2]
    T, H, V = hidden.shape[0], hidden.shape[1], W.shape[0]
    ent_s, ent_r = torch.empty(T, device="cuda"), torch.empty(T, device="cuda")
    ws = torch.empty(B.sapo_workspace_bytes(B.WS_FWD, T, H, V, B.DTYPE_BF16), dtype=torch.uint8, device="cuda")
    B.sapo_policy_loss_fwd(hidden, W, ids, old, adv, cu, 0.2, 0.28, 1.0, B.alloc_fwd_outputs(T, cu.numel() - 1),
                           ws, status, entropy=ent_r)
    _static_raw(hidden, W, ids, old, adv, cu, cases[0][5], status, entropy=ent_s)
    torch.cuda.synchronize()
    assert status.item() == 0 and torch.equal(ent_s, ent_r)
    _identical(cases[0][5], cases[0][3])
    # the static path against the oracle, under the tolerances of the other parity tests
    batch, adv_np, dev, _, out, _ = cases[0]
    b = batch.built
    ref = orc.policy_loss_fwd(gen.as_f32(b.hidden), gen.as_f32(batch.W), b.ids, b.old_logp, adv_np,
                              b.cu_seqlens, 0.2, 0.28)
    U.check_forward(out, ref, adv_np.astype(np.float64), b.cu_seqlens, 0.2, 0.28)
    seq = out["seq_surr"].cpu().numpy().astype(np.float64)
    assert np.max(np.abs(seq - ref["seq_surr"])) <= 1e-3 * np.abs(adv_np).max()
    U.check_loss(float(out["loss"].item()), ref["loss"], adv_np.astype(np.float64))


def test_static_scratch_rejects_what_does_not_fit():
    lib = B.load()
    cfg = B.LossCfgC(0.2, 0.2, 1.0, 0, 0.0, None)
    one = torch.zeros(256, dtype=torch.float32, device="cuda")
    p = one.data_ptr()

    def call(dtype, T, H, V):
        return lib.sapo_policy_loss_fwd_static(p, p, dtype, T, H, V, H, H, p, p, p, p, 1, C.byref(cfg),
                                               *([p] * 7), B.new_status().data_ptr(), None)
    # 24 bytes of scratch per token: the array holds 174,762 tokens, whatever the other sizes are
    for H, V in ((64, 512), (896, 151936), (3584, 152064)):
        rc = call(B.DTYPE_BF16, 174_763, H, V)
        assert rc == -5 and b"static scratch" in lib.sapo_status_string(rc)
    assert call(B.DTYPE_BF16, 2_000_000, 64, 512) == -5
    # the common argument checks come first and give the regular call's codes
    assert call(B.DTYPE_F32, 128, 64, 512) == -2          # fp32 operands: unsupported here
    assert call(B.DTYPE_BF16, 128, 12, 512) == -2         # H not a multiple of 8: unsupported shape
    assert call(7, 128, 64, 512) == -1                    # no such element type
    assert lib.sapo_policy_loss_fwd_static(None, p, B.DTYPE_BF16, 2_000_000, 64, 512, 64, 64, p, p, p, p, 1,
                                           C.byref(cfg), *([p] * 7), B.new_status().data_ptr(), None) == -1


def test_static_scratch_with_fewer_vocab_splits_than_the_regular_call():
    """A batch whose preferred number of vocab splits does not fit the array still runs (with
    fewer splits) and agrees with the regular call up to fp32 summation order."""
    T, H, V, S = 60_000, 64, 4096, 40
    assert B.sapo_workspace_bytes(B.WS_FWD, T, H, V, B.DTYPE_BF16) > B.STATIC_SCRATCH_BYTES
    g = torch.Generator(device="cuda").manual_seed(3)
    hidden = torch.randn(T, H, device="cuda", generator=g).to(torch.bfloat16)
    W = (torch.randn(V, H, device="cuda", generator=g) * 0.05).to(torch.bfloat16)
    ids = torch.randint(0, V, (T,), device="cuda", generator=g, dtype=torch.int32)
    old = U.torch_current_logp(hidden, W, ids) + 0.05 * torch.randn(T, device="cuda", generator=g)
    adv = torch.randn(S, device="cuda", generator=g)
    cu = torch.arange(S + 1, device="cuda", dtype=torch.int32) * (T // S)
    ref = _regular(hidden, W, ids, old, adv, cu)
    out, status = B.alloc_fwd_outputs(T, S), B.new_status()
    _static_raw(hidden, W, ids, old, adv, cu, out, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert (out["lse"] - ref["lse"]).abs().max().item() <= 1e-5
    assert (out["logp"] - ref["logp"]).abs().max().item() <= 1e-5
    near = ((ref["ratio"] - 0.8).abs() < 1e-4) | ((ref["ratio"] - 1.28).abs() < 1e-4)
    assert torch.allclose(out["gscale"][~near], ref["gscale"][~near], rtol=1e-4, atol=1e-9)
    assert abs(out["loss"].item() - ref["loss"].item()) <= 1e-5 * adv.abs().mean().item()
