"""Seeded synthetic inputs shaped like one SAPO node's policy-update batch.

This module only draws random numbers and arranges them into rollout buffers and
selection lists; it contains none of the method's arithmetic (no soft-max, no
advantage, no loss), so both the CUDA path and the CPU oracle can consume its
output without sharing any computation.

A batch mirrors the training set of the paper's Section 3.2: a node holds a buffer
of locally generated rollouts and a buffer of rollouts received from the swarm; for
every question it selects some local and some external completions by index.

Everything is numpy; bf16 tensors are carried as uint16 bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

DTYPE_BF16 = 0
DTYPE_F32 = 1


# --------------------------------------------------------------------------- bf16 helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even) and return the uint16 bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + rounding) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen uint16 bfloat16 bit patterns to float32 exactly."""
    return (b.astype(np.uint32) << 16).view(np.float32)


# --------------------------------------------------------------------------- containers
@dataclass
class RolloutBuffer:
    """A rollout store: `n` completions laid end to end.

    hidden   [n_tokens, H]  final hidden state at the position that predicts ids[t]
                            (uint16 bf16 bits, or float32 for the fp32 configuration)
    ids      [n_tokens]     int32 token chosen at that position
    old_logp [n_tokens]     float32 log-prob of ids[t] under the pre-update policy
    offsets  [n+1]          int64 token offsets of each completion
    rewards  [n]            float32 reward of each completion
    """
    hidden: np.ndarray
    ids: np.ndarray
    old_logp: np.ndarray
    offsets: np.ndarray
    rewards: np.ndarray

    @property
    def n_rollouts(self) -> int:
        return int(self.offsets.shape[0] - 1)

    @property
    def n_tokens(self) -> int:
        return int(self.offsets[-1])


@dataclass
class Selection:
    """Per-question CSR lists of chosen rollouts (indices into the two buffers)."""
    q_offsets_local: np.ndarray   # int32 [Q+1]
    local_idx: np.ndarray         # int32 [sum I_q]
    q_offsets_ext: np.ndarray     # int32 [Q+1]
    ext_idx: np.ndarray           # int32 [sum J_q]

    @property
    def Q(self) -> int:
        return int(self.q_offsets_local.shape[0] - 1)

    @property
    def S(self) -> int:
        return int(self.q_offsets_local[-1] + self.q_offsets_ext[-1])


@dataclass
class Constructed:
    """The packed batch as the generator built it, before scattering it into buffers.

    Serves as an independent check of any pack implementation: packing the buffers
    with the selection must reproduce these arrays bit for bit.
    """
    hidden: np.ndarray
    ids: np.ndarray
    logp_noise: np.ndarray
    rewards: np.ndarray
    cu_seqlens: np.ndarray     # int32 [S+1]
    seq_group: np.ndarray      # int32 [S]
    seq_is_ext: np.ndarray     # uint8 [S]
    seq_src: np.ndarray        # int32 [S] index of the rollout inside its buffer
    group_offsets: np.ndarray  # int32 [Q+1]


@dataclass
class Batch:
    name: str
    H: int
    V: int
    dtype: int
    W: np.ndarray              # [V, H] uint16 bf16 bits or float32
    local: RolloutBuffer
    ext: RolloutBuffer
    sel: Selection
    built: Constructed
    eps_low: float = 0.2
    eps_high: float = 0.2
    adv_eps: float = 1e-6
    noise_sigma: float = 0.05
    meta: Dict = field(default_factory=dict)

    @property
    def T(self) -> int:
        return int(self.built.cu_seqlens[-1])

    @property
    def S(self) -> int:
        return int(self.built.seq_group.shape[0])


# --------------------------------------------------------------------------- recipes
@dataclass
class Recipe:
    """Shape and distribution parameters of one workload."""
    name: str
    dtype: int
    H: int
    V: int
    Q: int
    I: int
    J: int
    length_law: Tuple            # ("fixed", n) | ("uniform", lo, hi) | ("lognormal", median, sigma, lo, hi)
    reward_law: Tuple            # ("bernoulli", p) | ("discrete", values, probs)
    equal_reward_fraction: float = 0.0   # leading fraction of questions with all-equal rewards
    noise_sigma: float = 0.05
    eps_low: float = 0.2
    eps_high: float = 0.2
    n_nodes: int = 2             # simulated nodes (this one included); from 3 on the buffers are a swarm pool:
                                 # the local buffer holds this node's Q x (I+J) rollouts, the external buffer
                                 # the Q x (I+J) rollouts of each of the other n_nodes - 1 nodes, end to end
    distractor_fraction: float = 0.25    # n_nodes == 2: share of unselected rollouts mixed into each buffer


def config(number: int, *, ext_fraction: Optional[float] = None, length_div: int = 1) -> Recipe:
    """The five workloads, numbered 1..5.

    `length_div` shrinks every completion length by that factor (same H, V, group
    structure and distributions): the "lite" variant used when the full size is too
    expensive for the fp64 oracle.  `ext_fraction` selects the sweep point of workload 5.
    """
    def lens(law):
        if length_div == 1:
            return law
        if law[0] == "fixed":
            return ("fixed", max(1, law[1] // length_div))
        if law[0] == "uniform":
            return ("uniform", max(1, law[1] // length_div), max(1, law[2] // length_div))
        return ("lognormal", law[1] / length_div, law[2], max(1, law[3] // length_div),
                max(1, law[4] // length_div))

    if number == 1:
        return Recipe("cfg1_tiny_fp32", DTYPE_F32, 64, 1000, 4, 4, 4, lens(("fixed", 32)),
                      ("bernoulli", 0.5))
    if number == 2:
        return Recipe("cfg2_qwen0.5b", DTYPE_BF16, 896, 151936, 8, 4, 4,
                      lens(("uniform", 64, 512)), ("bernoulli", 0.4))
    if number == 3:
        return Recipe("cfg3_h1536", DTYPE_BF16, 1536, 151936, 16, 8, 8,
                      lens(("uniform", 128, 1024)), ("bernoulli", 0.5),
                      equal_reward_fraction=0.25, noise_sigma=0.1)
    if number == 4:
        return Recipe("cfg4_h3584", DTYPE_BF16, 3584, 152064, 32, 2, 6,
                      lens(("lognormal", 512.0, 0.5, 128, 2048)),
                      ("discrete", (0.0, 0.5, 1.0), (0.5, 0.2, 0.3)))
    if number == 5:
        f = 0.5 if ext_fraction is None else ext_fraction
        J = int(round(8 * f))
        return Recipe(f"cfg5_swarm_mix_J{J}", DTYPE_BF16, 896, 151936, 64, 8 - J, J,
                      lens(("uniform", 256, 1024)), ("bernoulli", 0.3), n_nodes=8)
    raise ValueError(f"unknown workload {number}")


def _draw_lengths(rng: np.random.Generator, law: Tuple, n: int) -> np.ndarray:
    if law[0] == "fixed":
        return np.full(n, law[1], dtype=np.int64)
    if law[0] == "uniform":
        return rng.integers(law[1], law[2] + 1, size=n, dtype=np.int64)
    if law[0] == "lognormal":
        _, median, sigma, lo, hi = law
        raw = np.exp(np.log(median) + sigma * rng.standard_normal(n))
        return np.clip(np.rint(raw), lo, hi).astype(np.int64)
    raise ValueError(law)


def _draw_rewards(rng: np.random.Generator, law: Tuple, n: int) -> np.ndarray:
    if law[0] == "bernoulli":
        return (rng.random(n) < law[1]).astype(np.float32)
    if law[0] == "discrete":
        vals = np.asarray(law[1], dtype=np.float32)
        return vals[rng.choice(len(vals), size=n, p=np.asarray(law[2], dtype=np.float64))]
    raise ValueError(law)


def _draw_hidden(rng: np.random.Generator, n_tokens: int, H: int, dtype: int) -> np.ndarray:
    out = np.empty((n_tokens, H), dtype=np.float32 if dtype == DTYPE_F32 else np.uint16)
    step = max(1, (1 << 24) // max(H, 1))
    for a in range(0, n_tokens, step):
        b = min(n_tokens, a + step)
        x = rng.standard_normal((b - a, H), dtype=np.float32)
        out[a:b] = x if dtype == DTYPE_F32 else f32_to_bf16_bits(x)
    return out


def draw_W(rng: np.random.Generator, V: int, H: int, dtype: int, std: float = 0.02) -> np.ndarray:
    out = np.empty((V, H), dtype=np.float32 if dtype == DTYPE_F32 else np.uint16)
    step = max(1, (1 << 24) // max(H, 1))
    for a in range(0, V, step):
        b = min(V, a + step)
        x = rng.standard_normal((b - a, H), dtype=np.float32) * np.float32(std)
        out[a:b] = x if dtype == DTYPE_F32 else f32_to_bf16_bits(x)
    return out


def make_batch(recipe: Recipe, seed: int, *, selections: Optional[List[Tuple[int, int]]] = None
               ) -> Batch:
    """Draw one batch.

    `selections` overrides the per-question (I_q, J_q) counts (default: recipe.I, recipe.J
    for every question), which lets tests build ragged groups, wholly-local or
    wholly-external questions and empty sides.
    """
    rng = np.random.default_rng(np.random.PCG64(seed))
    Q = recipe.Q
    per_q = selections if selections is not None else [(recipe.I, recipe.J)] * Q
    assert len(per_q) == Q
    G = np.array([i + j for i, j in per_q], dtype=np.int64)
    S = int(G.sum())
    group_offsets = np.zeros(Q + 1, dtype=np.int32)
    group_offsets[1:] = np.cumsum(G)

    # ---- the packed batch, in its final order
    lengths = _draw_lengths(rng, recipe.length_law, S)
    rewards = _draw_rewards(rng, recipe.reward_law, S)
    n_equal = int(round(recipe.equal_reward_fraction * Q))
    for q in range(n_equal):
        rewards[group_offsets[q]:group_offsets[q + 1]] = np.float32(q % 2)
    cu = np.zeros(S + 1, dtype=np.int64)
    cu[1:] = np.cumsum(lengths)
    T = int(cu[-1])
    hidden = _draw_hidden(rng, T, recipe.H, recipe.dtype)
    ids = rng.integers(0, recipe.V, size=T, dtype=np.int32)
    noise = (rng.standard_normal(T, dtype=np.float32) * np.float32(recipe.noise_sigma))
    seq_group = np.repeat(np.arange(Q, dtype=np.int32), G)
    seq_is_ext = np.zeros(S, dtype=np.uint8)
    for q, (i, j) in enumerate(per_q):
        seq_is_ext[group_offsets[q] + i:group_offsets[q + 1]] = 1

    # ---- scatter the sequences into a local and an external buffer among rollouts that are not
    # selected: a fixed share of distractors, or (swarm pool) whole node buffers of Q x (I+J)
    # rollouts each, in which the selected ones sit at seeded uniform slots
    pool = recipe.n_nodes >= 3
    per_node = int(G.max()) * Q if Q > 0 else 0

    def scatter(which: np.ndarray, n_node_buffers: int):
        n_sel = int(which.sum())
        if pool:
            n_all = max(n_sel, n_node_buffers * per_node)
        else:
            n_all = n_sel + int(np.ceil(recipe.distractor_fraction * max(n_sel, 1)))
        slot_of = rng.permutation(n_all)[:n_sel]                 # buffer slot of each selected seq
        d_len = _draw_lengths(rng, recipe.length_law, n_all)
        d_rew = _draw_rewards(rng, recipe.reward_law, n_all)
        sel_seqs = np.nonzero(which)[0]
        d_len[slot_of] = lengths[sel_seqs]
        d_rew[slot_of] = rewards[sel_seqs]
        off = np.zeros(n_all + 1, dtype=np.int64)
        off[1:] = np.cumsum(d_len)
        nt = int(off[-1])
        b_hidden = _draw_hidden(rng, nt, recipe.H, recipe.dtype)
        b_ids = rng.integers(0, recipe.V, size=nt, dtype=np.int32)
        b_old = rng.standard_normal(nt, dtype=np.float32) * np.float32(recipe.noise_sigma)
        for s, slot in zip(sel_seqs, slot_of):
            a, b = off[slot], off[slot + 1]
            b_hidden[a:b] = hidden[cu[s]:cu[s + 1]]
            b_ids[a:b] = ids[cu[s]:cu[s + 1]]
            b_old[a:b] = noise[cu[s]:cu[s + 1]]
        buf = RolloutBuffer(b_hidden, b_ids, b_old, off, d_rew.astype(np.float32))
        src = np.full(S, -1, dtype=np.int32)
        src[sel_seqs] = slot_of.astype(np.int32)
        return buf, src

    local, src_l = scatter(seq_is_ext == 0, 1)
    # the external buffer stands for the concatenated buffers of the other nodes
    ext, src_e = scatter(seq_is_ext == 1, max(1, recipe.n_nodes - 1))
    seq_src = np.where(seq_is_ext == 1, src_e, src_l).astype(np.int32)

    qol = np.zeros(Q + 1, dtype=np.int32)
    qoe = np.zeros(Q + 1, dtype=np.int32)
    qol[1:] = np.cumsum([i for i, _ in per_q])
    qoe[1:] = np.cumsum([j for _, j in per_q])
    sel = Selection(qol, seq_src[seq_is_ext == 0].copy(), qoe, seq_src[seq_is_ext == 1].copy())

    built = Constructed(hidden, ids, noise, rewards.astype(np.float32), cu.astype(np.int32),
                        seq_group, seq_is_ext, seq_src, group_offsets)
    W = draw_W(rng, recipe.V, recipe.H, recipe.dtype)
    return Batch(recipe.name, recipe.H, recipe.V, recipe.dtype, W, local, ext, sel, built,
                 eps_low=recipe.eps_low, eps_high=recipe.eps_high,
                 noise_sigma=recipe.noise_sigma,
                 meta={"seed": seed, "Q": Q, "I": recipe.I, "J": recipe.J})


def install_old_logp(batch: Batch, current_logp: np.ndarray) -> None:
    """Set old log-probs = current + the batch's drawn noise, in both views of the data.

    `current_logp` [T] float32 is the log-prob of each packed token under the policy,
    supplied by the caller (this module does not compute it).  The sum is taken in
    float32 so every consumer reads identical bits.  Writes `built.old_logp` and the
    matching slices of the two rollout buffers.
    """
    b = batch.built
    old = (np.asarray(current_logp, dtype=np.float32) + b.logp_noise).astype(np.float32)
    b.old_logp = old
    for s in range(batch.S):
        buf = batch.ext if b.seq_is_ext[s] else batch.local
        a = buf.offsets[b.seq_src[s]]
        n = b.cu_seqlens[s + 1] - b.cu_seqlens[s]
        buf.old_logp[a:a + n] = old[b.cu_seqlens[s]:b.cu_seqlens[s + 1]]


def as_f32(x: np.ndarray) -> np.ndarray:
    """Exact float32 view of a tensor that is either float32 or bf16 bits."""
    return bf16_bits_to_f32(x) if x.dtype == np.uint16 else x
