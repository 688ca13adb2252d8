"""fp64 CPU oracle for the SAPO policy-scoring path.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain definition the CUDA library is checked against.  Only the
test-suite, the smoke check and the benchmark's CPU-baseline leg may import it; the
product path never does.  It shares no code with the CUDA sources.

What it computes, and where the method states it:

  pack_rollouts       the training set T^n = {I local samples} U {J external samples}
                      (paper Section 3.2, training-set equation; Algorithm 1,
                      where the training set is put together), as a varlen token layout
  group_advantages    GRPO's group-relative advantage (paper Section 4.2 names GRPO);
                      A = (r - mean_group) / (std_group + eps)
  token_logprobs      log-prob of each chosen token under the policy's LM head
                      (Section 3.2: a node encodes any rollout, received or its own, and
                      scores its tokens under its own policy)
  token_entropy       entropy of that distribution per position (a logged by-product)
  policy_loss_fwd     the clipped-ratio surrogate with KL weight 0 and separate lower /
                      upper clip thresholds (Section 4.2)
  policy_loss_bwd     its gradient with respect to the final hidden states and the
                      LM-head weight (Algorithm 1 "Policy update")

All floating point is float64; inputs (bf16 or fp32 values) are widened exactly.
Every function here is pinned by tests/test_oracle_pins.py against closed forms,
library routines, invariants, finite differences and brute force; none is unpinned.
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np


# --------------------------------------------------------------------------------------
def pack_rollouts(local: Dict[str, np.ndarray], ext: Dict[str, np.ndarray],
                  sel: Dict[str, np.ndarray]) -> Dict[str, np.ndarray]:
    """Merge the selected local and external rollouts into one token-major batch.

    Section 3.2 builds the training set as the union of I samples of the node's own
    rollouts and J samples shared by the swarm.  The paper writes a set; the order used
    here (and required bit for bit of any implementation) is: questions in order, and
    inside a question first its local picks in list order, then its external picks in
    list order.

    `local` / `ext`: dicts with hidden [n_tok,H], ids [n_tok], old_logp [n_tok],
    offsets [n+1], rewards [n].  `sel`: q_offsets_local [Q+1], local_idx,
    q_offsets_ext [Q+1], ext_idx.
    """
    Q = len(sel["q_offsets_local"]) - 1
    rows_hidden, rows_ids, rows_old = [], [], []
    rewards, seq_group, seq_is_ext, seq_src, lengths = [], [], [], [], []
    group_offsets = [0]
    for q in range(Q):
        picks = [(0, int(sel["local_idx"][k]))
                 for k in range(sel["q_offsets_local"][q], sel["q_offsets_local"][q + 1])]
        picks += [(1, int(sel["ext_idx"][k]))
                  for k in range(sel["q_offsets_ext"][q], sel["q_offsets_ext"][q + 1])]
        for is_ext, idx in picks:
            buf = ext if is_ext else local
            a, b = int(buf["offsets"][idx]), int(buf["offsets"][idx + 1])
            rows_hidden.append(buf["hidden"][a:b])
            rows_ids.append(buf["ids"][a:b])
            rows_old.append(buf["old_logp"][a:b])
            rewards.append(buf["rewards"][idx])
            seq_group.append(q)
            seq_is_ext.append(is_ext)
            seq_src.append(idx)
            lengths.append(b - a)
        group_offsets.append(len(seq_group))
    S = len(lengths)
    cu = np.zeros(S + 1, dtype=np.int32)
    for s in range(S):
        cu[s + 1] = cu[s] + lengths[s]
    T = int(cu[S])
    tok_seq = np.zeros(T, dtype=np.int32)
    for s in range(S):
        tok_seq[cu[s]:cu[s + 1]] = s
    H = local["hidden"].shape[1]
    cat = lambda rows, like, shape: (np.concatenate(rows, axis=0) if rows
                                     else np.zeros(shape, dtype=like.dtype))
    return {
        "hidden": cat(rows_hidden, local["hidden"], (0, H)),
        "ids": cat(rows_ids, local["ids"], (0,)),
        "old_logp": cat(rows_old, local["old_logp"], (0,)),
        "rewards": np.asarray(rewards, dtype=np.float32),
        "cu_seqlens": cu,
        "seq_group": np.asarray(seq_group, dtype=np.int32),
        "seq_is_ext": np.asarray(seq_is_ext, dtype=np.uint8),
        "seq_src": np.asarray(seq_src, dtype=np.int32),
        "tok_seq": tok_seq,
        "group_offsets": np.asarray(group_offsets, dtype=np.int32),
        "n_tokens": T,
    }


# --------------------------------------------------------------------------------------
def group_advantages(rewards: np.ndarray, group_offsets: np.ndarray,
                     adv_eps: float = 1e-6, ddof: int = 0) -> Dict[str, np.ndarray]:
    """Group-relative advantage of GRPO (the update rule named in Section 4.2).

    For every question g with member rewards r_1..r_G:
        mean_g = (1/G) sum r,   std_g = sqrt( sum (r-mean_g)^2 / (G - ddof) ),
        A_s    = (r_s - mean_g) / (std_g + adv_eps).
    The group runs over every completion of the question, local or external.
    A group with G - ddof <= 0 has std 0.
    """
    r = np.asarray(rewards, dtype=np.float64)
    Q = len(group_offsets) - 1
    adv = np.zeros_like(r)
    mean = np.zeros(Q)
    std = np.zeros(Q)
    for g in range(Q):
        a, b = int(group_offsets[g]), int(group_offsets[g + 1])
        if b == a:
            continue
        mu = r[a:b].sum() / (b - a)
        denom = (b - a) - ddof
        sd = np.sqrt(((r[a:b] - mu) ** 2).sum() / denom) if denom > 0 else 0.0
        mean[g], std[g] = mu, sd
        adv[a:b] = (r[a:b] - mu) / (sd + adv_eps)
    return {"adv": adv, "mean": mean, "std": std}


# --------------------------------------------------------------------------------------
def logits(hidden: np.ndarray, W: np.ndarray) -> np.ndarray:
    """z[t, v] = sum_k hidden[t, k] * W[v, k]  (LM head, no bias, temperature 1)."""
    return np.asarray(hidden, dtype=np.float64) @ np.asarray(W, dtype=np.float64).T


def token_logprobs(hidden: np.ndarray, W: np.ndarray, ids: np.ndarray) -> Dict[str, np.ndarray]:
    """lse_t = log sum_v exp z[t,v];  logp_t = z[t, ids_t] - lse_t."""
    z = logits(hidden, W)
    m = z.max(axis=1)
    lse = m + np.log(np.exp(z - m[:, None]).sum(axis=1))
    zy = z[np.arange(z.shape[0]), np.asarray(ids, dtype=np.int64)]
    return {"lse": lse, "logp": zy - lse, "z": z}


def entropy_from_logits(z: np.ndarray, lse: np.ndarray) -> np.ndarray:
    """H_t = - sum_v p[t,v] log p[t,v] with log p[t,v] = z[t,v] - lse_t (in nats)."""
    logp_all = np.asarray(z, dtype=np.float64) - np.asarray(lse, dtype=np.float64)[:, None]
    return -(np.exp(logp_all) * logp_all).sum(axis=1)


def token_entropy(hidden: np.ndarray, W: np.ndarray) -> np.ndarray:
    """Entropy of the policy's next-token distribution at every scored position:
        p[t,v] = exp(z[t,v] - lse_t),   H_t = - sum_v p[t,v] log p[t,v].
    Not part of the loss: the quantity RL post-training runs log beside the reward (the paper's
    experiments track rewards only; Section 5), available from the same pass over the logits."""
    z = logits(hidden, W)
    m = z.max(axis=1)
    lse = m + np.log(np.exp(z - m[:, None]).sum(axis=1))
    return entropy_from_logits(z, lse)


def _seq_of_token(cu_seqlens: np.ndarray) -> np.ndarray:
    S = len(cu_seqlens) - 1
    return np.repeat(np.arange(S), np.diff(np.asarray(cu_seqlens, dtype=np.int64)))


def surrogate_from_logp(logp: np.ndarray, old_logp: np.ndarray, adv: np.ndarray,
                        cu_seqlens: np.ndarray, eps_low: float, eps_high: float,
                        grad_scale: float = 1.0, n_seqs_total: Optional[int] = None,
                        loss_agg: int = 0, kl_beta: float = 0.0,
                        ref_logp: Optional[np.ndarray] = None,
                        n_tokens_total: Optional[int] = None) -> Dict[str, np.ndarray]:
    """Clipped-ratio surrogate and its derivative with respect to logp (Section 4.2).

        rho_t = exp(logp_t - old_t)
        u_t   = min( rho_t * A_s , clip(rho_t, 1-eps_low, 1+eps_high) * A_s )
        o_t   = u_t - beta * kl_t,   kl_t = exp(ref_t - logp_t) - (ref_t - logp_t) - 1
        L     = - sum_t w_t o_t,     w_t = 1/(S*T_s)  (loss_agg 0: mean over sequences of the
                                     token mean)  or  1/T  (loss_agg 1: mean over all tokens)
        g_t   = dL/dlogp_t = -w_t * ( A_s * rho_t * [unclipped term is the min]
                                      - beta * (1 - exp(ref_t - logp_t)) )
    The paper's runs use beta = 0 (Section 4.2), the default; kl_t is the non-negative
    estimator GRPO uses for its penalty towards a reference policy.
    The min is taken as "unclipped <= clipped" (ties count as unclipped).
    `n_seqs_total` / `n_tokens_total` override S / T in the weights when the rows given are
    only part of a batch (used to score sampled sequences of a large batch).
    """
    logp = np.asarray(logp, dtype=np.float64)
    old = np.asarray(old_logp, dtype=np.float64)
    A = np.asarray(adv, dtype=np.float64)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    S = len(cu) - 1
    S_norm = S if n_seqs_total is None else n_seqs_total
    T_norm = int(cu[-1]) if n_tokens_total is None else n_tokens_total
    seq = _seq_of_token(cu)
    T_s = np.diff(cu).astype(np.float64)
    A_t = A[seq]
    rho = np.exp(logp - old)
    unclipped = rho * A_t
    clipped = np.clip(rho, 1.0 - eps_low, 1.0 + eps_high) * A_t
    u = np.minimum(unclipped, clipped)
    active = (unclipped <= clipped).astype(np.float64)
    if kl_beta != 0.0:
        d = np.asarray(ref_logp, dtype=np.float64) - logp
        kl = np.exp(d) - d - 1.0
        dkl = 1.0 - np.exp(d)                      # d kl_t / d logp_t
    else:
        kl = np.zeros_like(logp)
        dkl = np.zeros_like(logp)
    o = u - kl_beta * kl
    w = 1.0 / (S_norm * T_s[seq]) if loss_agg == 0 else np.full(len(logp), 1.0 / T_norm)
    seq_surr = np.zeros(S)
    for s in range(S):
        seq_surr[s] = o[cu[s]:cu[s + 1]].sum() / T_s[s]
    loss = -(w * o).sum()
    g = -w * (A_t * rho * active - kl_beta * dkl) * grad_scale
    return {"ratio": rho, "surr": u, "gscale": g, "seq_surr": seq_surr, "loss": loss,
            "active": active, "kl": kl}


def policy_loss_fwd(hidden, W, ids, old_logp, adv, cu_seqlens, eps_low=0.2, eps_high=0.2,
                    grad_scale=1.0, loss_agg=0, kl_beta=0.0, ref_logp=None) -> Dict[str, np.ndarray]:
    """Forward of the policy loss: log-probs at the LM head, then the surrogate."""
    lp = token_logprobs(hidden, W, ids)
    out = surrogate_from_logp(lp["logp"], old_logp, adv, cu_seqlens, eps_low, eps_high,
                              grad_scale, loss_agg=loss_agg, kl_beta=kl_beta, ref_logp=ref_logp)
    out["logp"], out["lse"] = lp["logp"], lp["lse"]
    return out


def dlogits(hidden, W, ids, lse, gscale) -> np.ndarray:
    """dz[t,v] = g_t * ( [v == ids_t] - exp(z[t,v] - lse_t) )."""
    z = logits(hidden, W)
    dz = -np.exp(z - np.asarray(lse, dtype=np.float64)[:, None])
    dz[np.arange(z.shape[0]), np.asarray(ids, dtype=np.int64)] += 1.0
    return dz * np.asarray(gscale, dtype=np.float64)[:, None]


def policy_loss_bwd(hidden, W, ids, lse, gscale) -> Dict[str, np.ndarray]:
    """dhidden[t,:] = sum_v dz[t,v] W[v,:];   dW[v,:] = sum_t dz[t,v] hidden[t,:]."""
    dz = dlogits(hidden, W, ids, lse, gscale)
    return {"dhidden": dz @ np.asarray(W, dtype=np.float64),
            "dW": dz.T @ np.asarray(hidden, dtype=np.float64)}


# --------------------------------------------------------------------------------------
def policy_loss_fwd_bwd_rows(hidden, W, ids, old_logp, adv, cu_seqlens, eps_low=0.2,
                             eps_high=0.2, grad_scale=1.0, rows_per_block: int = 1024,
                             want_dW: bool = True) -> Dict[str, np.ndarray]:
    """Same results as policy_loss_fwd + policy_loss_bwd, evaluated a block of token rows
    at a time so that the [tokens x vocab] float64 logits never exceed a few GB of host
    memory.  Rows are independent in every formula above except the sum over t in dW,
    which is accumulated block by block; nothing else is reordered.
    """
    T = hidden.shape[0]
    W64 = np.asarray(W, dtype=np.float64)
    lse = np.zeros(T)
    logp = np.zeros(T)
    for a in range(0, T, rows_per_block):
        b = min(T, a + rows_per_block)
        lp = token_logprobs(hidden[a:b], W64, ids[a:b])
        lse[a:b], logp[a:b] = lp["lse"], lp["logp"]
    out = surrogate_from_logp(logp, old_logp, adv, cu_seqlens, eps_low, eps_high, grad_scale)
    out["logp"], out["lse"] = logp, lse
    dH = np.zeros((T, hidden.shape[1]))
    dW = np.zeros_like(W64) if want_dW else None
    for a in range(0, T, rows_per_block):
        b = min(T, a + rows_per_block)
        dz = dlogits(hidden[a:b], W64, ids[a:b], lse[a:b], out["gscale"][a:b])
        dH[a:b] = dz @ W64
        if want_dW:
            dW += dz.T @ np.asarray(hidden[a:b], dtype=np.float64)
    out["dhidden"], out["dW"] = dH, dW
    return out


def dW_rows(hidden, W, ids, lse, gscale, rows) -> np.ndarray:
    """The rows `rows` of dW only: dW[v,:] = sum_t dz[t,v] hidden[t,:] with
    dz[t,v] = g_t ([v == ids_t] - exp(z[t,v] - lse_t)), z restricted to those vocab rows.
    Same definition as policy_loss_bwd; used where the full [tokens x vocab] matrix is too
    large for the host.  lse must cover every token (it depends on the whole vocabulary)."""
    rows = np.asarray(rows, dtype=np.int64)
    h = np.asarray(hidden, dtype=np.float64)
    z = h @ np.asarray(W, dtype=np.float64)[rows].T                     # [T, len(rows)]
    dz = -np.exp(z - np.asarray(lse, dtype=np.float64)[:, None])
    dz += (np.asarray(ids, dtype=np.int64)[:, None] == rows[None, :])
    dz *= np.asarray(gscale, dtype=np.float64)[:, None]
    return dz.T @ h


# --------------------------------------------------------------------------------------
# Filtering and sampling the shared pool (Section 3.2, last paragraph before Algorithm 1, and
# Section 5: nodes first discard rollouts with zero advantage, then sample uniformly from the
# rest).  A pool entry is one question's rollout, i.e. its group of completions; its
# advantages are all zero exactly when its rewards are all equal.
_PHILOX_M0, _PHILOX_M1 = 0xD2511F53, 0xCD9E8D57
_PHILOX_W0, _PHILOX_W1 = 0x9E3779B9, 0xBB67AE85


def philox4x32(counter, key, rounds: int = 10):
    """Philox-4x32 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
    SC'11): a counter-based generator, four 32-bit outputs per (128-bit counter, 64-bit key)."""
    c0, c1, c2, c3 = (int(x) & 0xFFFFFFFF for x in counter)
    k0, k1 = (int(x) & 0xFFFFFFFF for x in key)
    for _ in range(rounds):
        p0 = _PHILOX_M0 * c0
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> 32, p0 & 0xFFFFFFFF
        hi1, lo1 = p1 >> 32, p1 & 0xFFFFFFFF
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = (k0 + _PHILOX_W0) & 0xFFFFFFFF
        k1 = (k1 + _PHILOX_W1) & 0xFFFFFFFF
    return c0, c1, c2, c3


def select_external(rewards: np.ndarray, group_offsets: np.ndarray, J: int, seed: int
                    ) -> Dict[str, np.ndarray]:
    """Drop the pool entries whose rewards are all equal (zero advantage), then draw J of the
    rest uniformly without replacement: every candidate g gets the 64-bit key
    (philox4x32(counter=(g,0,0,0), key=(seed_lo, seed_hi))[0] << 32) | g and the J smallest keys
    win.  Returns the chosen entries in pool order, the candidate flags and counts.
    Fewer than J candidates: all of them are taken."""
    r = np.asarray(rewards)
    n = len(group_offsets) - 1
    cand = np.zeros(n, dtype=bool)
    for g in range(n):
        a, b = int(group_offsets[g]), int(group_offsets[g + 1])
        cand[g] = b > a and r[a:b].min() != r[a:b].max()
    keys = []
    for g in range(n):
        if cand[g]:
            x = philox4x32((g, 0, 0, 0), (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))[0]
            keys.append(((x << 32) | g, g))
    keys.sort()
    chosen = sorted(g for _, g in keys[:max(0, J)])
    return {"selected": np.asarray(chosen, dtype=np.int32), "candidates": cand,
            "n_candidates": int(cand.sum()), "n_selected": len(chosen)}


# --------------------------------------------------------------------------------------
def adam_step(theta, grad, m, v, step: int, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8):
    """One Adam update (Kingma & Ba, Algorithm 1) with the default hyper-parameters the paper's
    runs use (Section 4.2: Adam, learning rate 0.001), in float64:
        m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2;
        theta <- theta - lr * (m / (1-b1^t)) / (sqrt(v / (1-b2^t)) + eps).
    Returns the new (theta, m, v)."""
    theta = np.asarray(theta, dtype=np.float64)
    g = np.asarray(grad, dtype=np.float64)
    m = beta1 * np.asarray(m, dtype=np.float64) + (1.0 - beta1) * g
    v = beta2 * np.asarray(v, dtype=np.float64) + (1.0 - beta2) * g * g
    m_hat = m / (1.0 - beta1 ** step)
    v_hat = v / (1.0 - beta2 ** step)
    return theta - lr * m_hat / (np.sqrt(v_hat) + eps), m, v
