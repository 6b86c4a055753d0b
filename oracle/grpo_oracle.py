"""CPU oracle for the GRPO scoring path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 restatement of what the entry points of the scoring path compute.  It is what the CUDA
library is checked against; it is not a fallback and nothing in the product path may import
it.  It shares no code with the CUDA path (numpy only; bf16 tensors arrive as raw uint16 bit
patterns and are widened exactly to float64).

The paper (AsyncFlow) states the data flow -- a sample-indexed columnar store read by global
index (Section 4.3 "Data Plane"), micro-batches handed out as metadata and fetched by the
worker (Section 4.2 "Interaction Interface"), the ``compute_log_prob`` task (Appendix, Backend
-level interface listing), GRPO advantages taken from rewards relative to the other responses to
the same prompt (Section 7.1 "RL algorithms") -- but prints no formula.  The arithmetic is therefore the
textbook definition of each quantity, written out below with no blocking, fusion or reordering:

  log-softmax / entropy .... the definition over the full vocabulary row
  GRPO advantage ........... (r - mean_g) / (std_g + eps) per group
  PPO-clip surrogate ....... -min(rho*A, clip(rho, 1-lo, 1+hi)*A)
  k3 KL estimator .......... exp(delta) - delta - 1,  delta = ref - logp
  backward ................. dZ = g * (onehot(y) - softmax), dH = dZ W, dW = dZ^T H

Pins (tests/test_oracle_*.py): gather and write-back are inverse to each other and leave unlisted
rows alone; rows of exp(log-softmax) sum to one; brute-force enumeration
at V <= 16; closed forms (zero weights, V = 2, Bernoulli groups, four-quadrant clip table);
invariances (logit shift, reward affine maps, group order); central finite differences of the
whole fp64 chain for every gradient.  No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np


# ----------------------------------------------------------------------------------------
# helpers
# ----------------------------------------------------------------------------------------
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float64."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


# ----------------------------------------------------------------------------------------
# O1  pack: index list -> cu_seqlens-packed columns            (Sections 4.2, 4.3; Appendix
#     TransferQueue usage listing: a task names the columns it needs and gets (batch, index))
# ----------------------------------------------------------------------------------------
def pack_microbatch_ref(tok_offset, idx, columns, adv=None):
    """Gather the rows of the indexed samples, in list order, into contiguous arrays.

    tok_offset : [N+1] int64, sample i owns store rows tok_offset[i] .. tok_offset[i+1]-1
    idx        : [B] sample indices (duplicates allowed: gathered twice)
    columns    : dict name -> per-token array [sum L, ...] (any dtype; copied verbatim)
    adv        : optional per-sample array [N]
    returns    : dict with cu_seqlens [B+1] int32, seq_id [T] int32, each packed column,
                 adv_seq [B] (when adv is given)
    """
    tok_offset = np.asarray(tok_offset, dtype=np.int64)
    idx = np.asarray(idx, dtype=np.int64)
    B = idx.shape[0]
    cu = np.zeros(B + 1, dtype=np.int64)
    for j in range(B):
        cu[j + 1] = cu[j] + (tok_offset[idx[j] + 1] - tok_offset[idx[j]])
    T = int(cu[B])
    out = {"cu_seqlens": cu.astype(np.int32), "seq_id": np.zeros(T, dtype=np.int32)}
    for name, col in columns.items():
        packed = np.empty((T,) + col.shape[1:], dtype=col.dtype)
        for j in range(B):
            packed[cu[j]:cu[j + 1]] = col[tok_offset[idx[j]]:tok_offset[idx[j] + 1]]
        out[name] = packed
    for j in range(B):
        out["seq_id"][cu[j]:cu[j + 1]] = j
    if adv is not None:
        out["adv_seq"] = np.asarray(adv)[idx].copy()
    return out


def unpack_microbatch_ref(tok_offset, idx, packed_columns, store_columns):
    """Write a task's per-token results back to the store by metadata (Section 4.2: once the task
    has computed, it writes its results to the storage units according to the metadata): the
    inverse of the gather above, one column at a time, in place.

    tok_offset      : [N+1] int64
    idx             : [B] sample indices, each at most once (two writers of one row have no defined order)
    packed_columns  : dict name -> array [T, ...] in packed order (T = sum of the listed lengths)
    store_columns   : dict name -> array [sum L, ...]; rows of the listed samples are overwritten,
                      every other row is left as it is
    returns T
    """
    tok_offset = np.asarray(tok_offset, dtype=np.int64)
    idx = np.asarray(idx, dtype=np.int64)
    if len(set(idx.tolist())) != idx.shape[0]:
        raise ValueError("duplicate sample index in a write-back list")
    t = 0
    for j in range(idx.shape[0]):
        lo, hi = int(tok_offset[idx[j]]), int(tok_offset[idx[j] + 1])
        for name, packed in packed_columns.items():
            for r in range(lo, hi):
                store_columns[name][r] = packed[t + (r - lo)]
        t += hi - lo
    return t


# ----------------------------------------------------------------------------------------
# O2  per-token log-prob, entropy, logsumexp       (compute_log_prob task; LM head only)
# ----------------------------------------------------------------------------------------
def token_logprob_ref(H_bits, W_bits, y, return_rows=False):
    """z = H W^T; lse = log sum_v exp z_v; logp = z_y - lse; ent = -sum_v p_v log p_v.

    H_bits [T, d], W_bits [V, d] : bf16 bit patterns;  y [T] : target ids in [0, V)
    returns logp, ent, lse (float64 [T]) and, if asked, the full log-softmax rows [T, V].
    """
    H = bf16_bits_to_f64(H_bits)
    W = bf16_bits_to_f64(W_bits)
    y = np.asarray(y, dtype=np.int64)
    z = H @ W.T                                        # [T, V] all logits
    m = z.max(axis=1, keepdims=True)
    lse = m[:, 0] + np.log(np.exp(z - m).sum(axis=1))
    logp_rows = z - lse[:, None]                       # log-softmax rows
    p = np.exp(logp_rows)
    plogp = np.where(p > 0.0, p * logp_rows, 0.0)      # 0 * log 0 := 0
    ent = -plogp.sum(axis=1)
    logp = logp_rows[np.arange(z.shape[0]), y]
    if return_rows:
        return logp, ent, lse, logp_rows
    return logp, ent, lse


# ----------------------------------------------------------------------------------------
# O2b  the same scoring with the vocabulary sharded over model-parallel ranks: every rank sees
#      the rows [v_offset, v_offset + V_shard) of W and reports four numbers per token; one
#      exchange of those numbers and a merge give the full-vocabulary result.  (The paper names
#      tensor parallelism among the strategies its instances combine, Section 2.1; it does not
#      describe the head.  The four statistics are the ones a softmax needs.)
# ----------------------------------------------------------------------------------------
def token_logprob_shard_ref(H_bits, W_shard_bits, y, v_offset):
    """Per token over the shard's logits z_v = H W_shard^T:
         m = max_v z_v;  s = sum_v exp(z_v - m);  u = sum_v exp(z_v - m) z_v;
         zy = z at the target if the target id falls into the shard, else -inf.
    Returns float64 [T, 4] = (m, s, u, zy)."""
    H = bf16_bits_to_f64(H_bits)
    W = bf16_bits_to_f64(W_shard_bits)
    y = np.asarray(y, dtype=np.int64) - int(v_offset)
    z = H @ W.T
    m = z.max(axis=1)
    e = np.exp(z - m[:, None])
    out = np.empty((z.shape[0], 4), dtype=np.float64)
    out[:, 0] = m
    out[:, 1] = e.sum(axis=1)
    out[:, 2] = (e * z).sum(axis=1)
    inside = (y >= 0) & (y < z.shape[1])
    out[:, 3] = np.where(inside, z[np.arange(z.shape[0]), np.clip(y, 0, z.shape[1] - 1)], -np.inf)
    return out


def merge_logprob_shards_ref(partials):
    """partials [R, T, 4] from token_logprob_shard_ref -> logp, ent, lse over the whole vocabulary:
         M = max_r m_r;  S = sum_r s_r exp(m_r - M);  U = sum_r u_r exp(m_r - M)
         lse = M + log S;  logp = max_r zy_r - lse;  ent = lse - U / S."""
    P = np.asarray(partials, dtype=np.float64)
    M = P[:, :, 0].max(axis=0)
    w = np.exp(P[:, :, 0] - M[None, :])
    S = (P[:, :, 1] * w).sum(axis=0)
    U = (P[:, :, 2] * w).sum(axis=0)
    lse = M + np.log(S)
    return P[:, :, 3].max(axis=0) - lse, lse - U / S, lse


# ----------------------------------------------------------------------------------------
# O3  GRPO group-normalised advantage                       (Section 7.1 "RL algorithms")
# ----------------------------------------------------------------------------------------
def grpo_advantage_ref(reward, group_id, n_groups, eps_adv=1e-6, ddof=0):
    """A_i = (r_i - mean_g) / (std_g + eps_adv); std with divisor n_g - ddof; any id order."""
    r = np.asarray(reward, dtype=np.float64)
    gid = np.asarray(group_id, dtype=np.int64)
    adv = np.zeros_like(r)
    for g in range(n_groups):
        members = np.nonzero(gid == g)[0]
        n = members.size
        if n == 0:
            continue
        mu = r[members].sum() / n
        dev = r[members] - mu
        denom = n - ddof
        sigma = np.sqrt((dev * dev).sum() / denom) if denom > 0 else 0.0
        adv[members] = dev / (sigma + eps_adv)
    return adv


# ----------------------------------------------------------------------------------------
# O4  clipped-ratio policy loss + k3 KL penalty, and d loss / d logp
# ----------------------------------------------------------------------------------------
def policy_loss_ref(logp, old_logp, ref_logp, adv_seq, cu_seqlens, clip_lo=0.2, clip_hi=0.2,
                    kl_coef=0.04, agg_mode=0, loss_scale=1.0, entropy=None):
    """Per token t of sequence i (A = adv_seq[i]):
         rho = exp(logp - old);  s1 = rho A;  s2 = clip(rho, 1-lo, 1+hi) A;  pg = -min(s1, s2)
         clipped  <=>  s2 < s1 (strict);  delta = ref - logp;  k3 = exp(delta) - delta - 1
         l = pg + kl_coef k3
       agg_mode 0: mean over tokens inside a sequence, then mean over sequences;
       agg_mode 1: mean over all tokens.  Both times ``loss_scale``.
       g_t = w_t ( [not clipped] (-A rho) + kl_coef (1 - exp(delta)) ),  w_t the token's weight.
    """
    logp = np.asarray(logp, dtype=np.float64)
    old = np.asarray(old_logp, dtype=np.float64)
    ref = np.asarray(ref_logp, dtype=np.float64)
    A_seq = np.asarray(adv_seq, dtype=np.float64)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    B = cu.shape[0] - 1
    T = int(cu[B])
    lens = cu[1:] - cu[:-1]
    seq_of = np.repeat(np.arange(B), lens)
    A = A_seq[seq_of]

    rho = np.exp(logp - old)
    s1 = rho * A
    s2 = np.minimum(np.maximum(rho, 1.0 - clip_lo), 1.0 + clip_hi) * A
    pg = -np.minimum(s1, s2)
    clipped = s2 < s1
    delta = ref - logp
    k3 = np.exp(delta) - delta - 1.0
    tok = pg + kl_coef * k3

    if agg_mode == 0:
        w = loss_scale / (B * lens[seq_of].astype(np.float64))
    else:
        w = np.full(T, loss_scale / T)

    def agg(x):
        if agg_mode == 0:
            total = 0.0
            for i in range(B):
                if lens[i] > 0:
                    total += x[cu[i]:cu[i + 1]].sum() / lens[i]
            return loss_scale * total / B
        return loss_scale * x.sum() / T

    dlogp = w * (np.where(clipped, 0.0, -A * rho) + kl_coef * (1.0 - np.exp(delta)))
    out = {
        "loss": agg(tok), "pg_loss": agg(pg), "kl_mean": agg(k3),
        "clip_frac": clipped.sum() / T if T else 0.0,
        "entropy_mean": (np.asarray(entropy, dtype=np.float64).sum() / T) if entropy is not None and T else 0.0,
        "n_tokens": T, "dlogp": dlogp, "clipped": clipped, "rho": rho,
    }
    return out


# ----------------------------------------------------------------------------------------
# O5  backward through log-softmax and the LM head
# ----------------------------------------------------------------------------------------
def policy_loss_backward_ref(H_bits, W_bits, y, lse, g, vocab_rows=None):
    """dZ_tv = g_t (1{v = y_t} - exp(z_tv - lse_t));  dH = dZ W;  dW = dZ^T H   (all fp64).

    ``lse`` is an input of the stage (with the true logsumexp, exp(z - lse) is the softmax).
    vocab_rows: optional list of vocabulary ids; then only those rows of dW are formed (each
    is a sum over all tokens) and dH is not returned -- used where [T, V] is out of reach.
    """
    H = bf16_bits_to_f64(H_bits)
    y = np.asarray(y, dtype=np.int64)
    lse = np.asarray(lse, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    if vocab_rows is not None:
        vs = np.asarray(vocab_rows, dtype=np.int64)
        Wv = bf16_bits_to_f64(np.asarray(W_bits)[vs])
        z = H @ Wv.T                                             # [T, |vs|]
        dZ = g[:, None] * ((y[:, None] == vs[None, :]).astype(np.float64) - np.exp(z - lse[:, None]))
        return dZ.T @ H                                          # [|vs|, d]
    W = bf16_bits_to_f64(W_bits)
    z = H @ W.T
    onehot = np.zeros_like(z)
    onehot[np.arange(z.shape[0]), y] = 1.0
    dZ = g[:, None] * (onehot - np.exp(z - lse[:, None]))
    return dZ @ W, dZ.T @ H


def policy_loss_backward_shard_ref(H_bits, W_shard_bits, y, lse, g, v_offset):
    """The backward of one vocabulary shard of the head (rows [v_offset, v_offset + V_s) of W):
    dZ_tv = g_t (1{y_t = v_offset + v} - exp(z_tv - lse_t)) over the shard's columns only, with the
    logsumexp of the WHOLE vocabulary; returns (dZ W_shard, dZ^T H) = this shard's contribution to
    dH [T, d] (the shards' contributions add up) and its own rows of dW [V_s, d]."""
    H = bf16_bits_to_f64(H_bits)
    Ws = bf16_bits_to_f64(W_shard_bits)
    y = np.asarray(y, dtype=np.int64)
    lse = np.asarray(lse, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    z = H @ Ws.T
    onehot = np.zeros_like(z)
    for t in range(z.shape[0]):
        if v_offset <= y[t] < v_offset + z.shape[1]:
            onehot[t, y[t] - v_offset] = 1.0
    dZ = g[:, None] * (onehot - np.exp(z - lse[:, None]))
    return dZ @ Ws, dZ.T @ H

