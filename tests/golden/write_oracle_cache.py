#!/usr/bin/env python
"""Write the oracle's forward pass over ALL tokens of the full-size workloads 3, 4 and 5.

    python tests/golden/write_oracle_cache.py [--cases 3 4 5:0 5:0.75] [--out build/oracle_cache]

For each case it builds the seeded batch (seed = 1000 x workload, as the full-size parity tests
do), runs oracle.token_logprobs over every packed token in blocks of rows (rows are independent)
and stores lse, logp and the per-token entropy as float64 in <out>/<case>.npz together with a
key: a hash of the oracle functions used and a fingerprint of the inputs.  The tests recompute
the key and ignore a file whose key differs, so a change to the oracle or to the generator can
never be checked against stale values.

This is several minutes of host BLAS per case (2 T V H float64 flops: 7e13 to 1.6e14), which
is why it is not done inside every test run.  It imports the oracle and the input generator
only; nothing here comes from the CUDA library.
"""
from __future__ import annotations

import argparse
import hashlib
import inspect
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import sapo_oracle as orc                      # noqa: E402
from paper_2509_08721_b200 import inputs as gen            # noqa: E402

DEFAULT_DIR = os.path.join(ROOT, "build", "oracle_cache")
DEFAULT_CASES = ("3", "4", "5:0", "5:0.75")


def parse_case(case: str):
    number, _, frac = case.partition(":")
    return int(number), (float(frac) if frac else None)


def case_name(number: int, ext_fraction) -> str:
    return f"workload{number}" if ext_fraction is None else f"workload{number}_ext{int(round(100 * ext_fraction)):03d}"


def build_batch(number: int, ext_fraction):
    return gen.make_batch(gen.config(number, ext_fraction=ext_fraction), 1000 * number)


def cache_key(batch) -> str:
    """Hash of what the stored values depend on: the oracle code that produces them and the
    inputs (shapes, every 997th hidden row, all token ids, every 1009th weight row)."""
    h = hashlib.sha256()
    for fn in (orc.logits, orc.token_logprobs, orc.entropy_from_logits):
        h.update(inspect.getsource(fn).encode())
    b = batch.built
    h.update(np.asarray([batch.T, batch.S, batch.H, batch.V], dtype=np.int64).tobytes())
    h.update(np.ascontiguousarray(b.hidden[::997]).tobytes())
    h.update(np.ascontiguousarray(b.ids).tobytes())
    h.update(np.ascontiguousarray(batch.W[::1009]).tobytes())
    return h.hexdigest()


def forward_all_tokens(batch, rows_per_block: int = 512, progress: bool = False):
    T = batch.T
    h = gen.as_f32(batch.built.hidden)
    W64 = gen.as_f32(batch.W).astype(np.float64)
    lse, logp, ent = np.zeros(T), np.zeros(T), np.zeros(T)
    t0 = time.time()
    for a in range(0, T, rows_per_block):
        e = min(T, a + rows_per_block)
        lp = orc.token_logprobs(h[a:e], W64, batch.built.ids[a:e])
        lse[a:e], logp[a:e] = lp["lse"], lp["logp"]
        ent[a:e] = orc.entropy_from_logits(lp["z"], lp["lse"])
        if progress and (a // rows_per_block) % 20 == 0:
            print(f"  {e}/{T} tokens, {time.time() - t0:.0f} s", flush=True)
    return {"lse": lse, "logp": logp, "entropy": ent}


def load(number: int, ext_fraction, batch, directory: str = DEFAULT_DIR):
    """The stored forward pass of this case, or None when there is none for these inputs."""
    path = os.path.join(directory, case_name(number, ext_fraction) + ".npz")
    if not os.path.exists(path):
        return None
    with np.load(path) as f:
        if str(f["key"]) != cache_key(batch):
            return None
        return {k: f[k] for k in ("lse", "logp", "entropy")}


def write(number: int, ext_fraction, directory: str = DEFAULT_DIR, batch=None, progress: bool = True):
    batch = build_batch(number, ext_fraction) if batch is None else batch
    out = forward_all_tokens(batch, progress=progress)
    os.makedirs(directory, exist_ok=True)
    path = os.path.join(directory, case_name(number, ext_fraction) + ".npz")
    np.savez(path, key=np.asarray(cache_key(batch)), **out)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--cases", nargs="*", default=list(DEFAULT_CASES))
    ap.add_argument("--out", default=DEFAULT_DIR)
    args = ap.parse_args()
    for case in args.cases:
        number, frac = parse_case(case)
        t0 = time.time()
        batch = build_batch(number, frac)
        if load(number, frac, batch, args.out) is not None:
            print(case_name(number, frac), "up to date")
            continue
        print(case_name(number, frac), f"T={batch.T} H={batch.H} V={batch.V}", flush=True)
        write(number, frac, args.out, batch)
        print(f"  written in {time.time() - t0:.0f} s", flush=True)


if __name__ == "__main__":
    main()
