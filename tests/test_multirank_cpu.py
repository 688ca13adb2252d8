"""Two gloo ranks on CPU: the replica bookkeeping used by bench.py at N > 1 (slowest rank's
time, total tokens, distinct seeds per rank)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2509_08721_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, tok = replicas.aggregate(10.0 + 5.0 * rank, 1000.0 + rank, device="cpu")
    out[rank] = (ms, tok, replicas.rank_seed(2, rank))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_all_tokens():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][:2] == res[1][:2] == (15.0, 2001.0)
    assert res[0][2] != res[1][2]
    assert replicas.throughput(15.0, 2001.0, 3) == 2001.0 * 3 / 0.015


def test_single_process_is_the_identity():
    assert replicas.aggregate(7.0, 9.0) == (7.0, 9.0)


# ---------------------------------------------------------------------------------------------
# The vocabulary-sharded loss over two gloo ranks.  The compute steps are stood in for by the
# fp64 oracle (no GPU here), so what is tested is everything around them: the shard bounds, the
# token-id offsets, the layout of the gathered (max, sum, target logit) triples, the log-sum-exp
# merge over the parts as the tail is asked to do it, and the sum of the dhidden shares.
import numpy as np

from oracle import sapo_oracle as orc
from paper_2509_08721_b200 import vocab_parallel as vp

LOG2E = 1.4426950408889634


class OracleBackend:
    def lse_partial(self, hidden, W_shard, ids, vocab_offset, triple, status):
        z = orc.logits(hidden.numpy(), W_shard.numpy())
        m2 = z.max(axis=1) * LOG2E
        s = np.exp2(z * LOG2E - m2[:, None]).sum(axis=1)
        loc = ids.numpy().astype(np.int64) - vocab_offset
        inside = (loc >= 0) & (loc < z.shape[1])
        zy = np.where(inside, z[np.arange(z.shape[0]), np.clip(loc, 0, z.shape[1] - 1)], 0.0)
        triple.copy_(torch.from_numpy(np.stack([m2, s, zy]).astype(np.float32)))

    def loss_from_partials(self, triples, V, ids, old_logp, adv, cu, eps_low, eps_high, grad_scale, out, status):
        t = triples.numpy().astype(np.float64)                 # [P, 3, T]
        M = t[:, 0].max(axis=0)
        S = (t[:, 1] * np.exp2(t[:, 0] - M)).sum(axis=0)
        lse = (M + np.log2(S)) / LOG2E
        logp = t[:, 2].sum(axis=0) - lse
        r = orc.surrogate_from_logp(logp, old_logp.numpy(), adv.numpy(), cu.numpy(), eps_low, eps_high, grad_scale)
        r["logp"], r["lse"] = logp, lse
        for k in ("logp", "lse", "ratio", "surr", "gscale", "seq_surr"):
            out[k].copy_(torch.from_numpy(np.asarray(r[k], dtype=np.float32)))
        out["loss"].fill_(float(r["loss"]))

    def bwd_shard(self, hidden, W_shard, ids, vocab_offset, lse, gscale, dhidden, dW_shard, status):
        h, W = hidden.numpy().astype(np.float64), W_shard.numpy().astype(np.float64)
        z = orc.logits(h, W)
        dz = -np.exp(z - lse.numpy().astype(np.float64)[:, None])
        loc = ids.numpy().astype(np.int64) - vocab_offset
        inside = np.nonzero((loc >= 0) & (loc < z.shape[1]))[0]
        dz[inside, loc[inside]] += 1.0
        dz *= gscale.numpy().astype(np.float64)[:, None]
        dhidden.copy_(torch.from_numpy((dz @ W).astype(np.float32)))
        dW_shard.copy_(torch.from_numpy((dz.T @ h).astype(np.float32)))


def _sharded_case():
    rng = np.random.default_rng(8)
    T, H, V, S = 37, 6, 300, 4                      # 300 rows: shards of 256 and 44 at two ranks
    hidden = rng.normal(size=(T, H)).astype(np.float32)
    W = (rng.normal(size=(V, H)) * 0.5).astype(np.float32)
    ids = rng.integers(0, V, size=T).astype(np.int32)
    ids[:3] = [0, 255, 256]                         # both sides of the shard boundary
    cu = np.array([0, 9, 20, 21, 37], dtype=np.int32)
    adv = np.array([1.0, -0.5, 0.0, 2.0], dtype=np.float32)
    cur = orc.token_logprobs(hidden, W, ids)["logp"]
    old = (cur + rng.normal(size=T) * 0.2).astype(np.float32)
    return hidden, W, ids, old, adv, cu


def _sharded_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    hidden, W, ids, old, adv, cu = _sharded_case()
    lo, hi = vp.shard_bounds(W.shape[0], world, rank)
    loss = vp.VocabShardedLoss(torch.from_numpy(W[lo:hi].copy()), W.shape[0], lo, backend=OracleBackend())
    res = loss.step(torch.from_numpy(hidden), torch.from_numpy(ids), torch.from_numpy(old),
                    torch.from_numpy(adv), torch.from_numpy(cu))
    out[rank] = {"lo": lo, "hi": hi, "loss": float(res.out["loss"].item()), "logp": res.out["logp"].numpy().copy(),
                 "gscale": res.out["gscale"].numpy().copy(), "dhidden": res.dhidden.numpy().copy(),
                 "dW": res.dW_shard.numpy().copy()}
    dist.barrier()
    dist.destroy_process_group()


def test_vocab_sharded_loss_over_two_ranks_equals_the_unsharded_one():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_sharded_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    hidden, W, ids, old, adv, cu = _sharded_case()
    ref = orc.policy_loss_fwd(hidden, W, ids, old, adv, cu, 0.2, 0.28)
    grads = orc.policy_loss_bwd(hidden, W, ids, ref["lse"], ref["gscale"])
    assert (res[0]["lo"], res[0]["hi"], res[1]["lo"], res[1]["hi"]) == (0, 256, 256, 300)
    for r in (0, 1):
        assert abs(res[r]["loss"] - ref["loss"]) <= 1e-6 * max(1.0, abs(ref["loss"]))
        assert np.allclose(res[r]["logp"], ref["logp"], rtol=0, atol=2e-6)
        assert np.allclose(res[r]["gscale"], ref["gscale"], rtol=1e-5, atol=1e-9)
        assert np.allclose(res[r]["dhidden"], grads["dhidden"], rtol=1e-4, atol=1e-7)      # the summed shares
        assert np.allclose(res[r]["dW"], grads["dW"][res[r]["lo"]:res[r]["hi"]], rtol=1e-4, atol=1e-7)
    assert np.array_equal(res[0]["dhidden"], res[1]["dhidden"])                            # one all-reduce, same bits


def test_shard_bounds_cover_the_vocabulary_in_whole_tiles():
    for V, world in ((151936, 2), (152064, 8), (1000, 2), (100, 4), (129, 2)):
        spans = [vp.shard_bounds(V, world, r) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == V
        for (a, b), (c, d) in zip(spans, spans[1:]):
            assert b == c and a <= b
        assert all(lo % 128 == 0 or lo == V for lo, _ in spans)        # a rank past the end holds no rows
