"""CPU oracle for the DapQ eviction scorer.  TEST INFRASTRUCTURE, NOT A PRODUCT PATH.

A plain, slow, float64 numpy statement of what the scorer computes, written from
the paper's definitions so that it can be checked against them by eye.  It shares
no code with the CUDA library and is imported only by the tests, the smoke check
and the benchmark's CPU-baseline leg.

Every function is pinned by the CPU tests (library causal attention on tiny
inputs, closed forms, invariants, equivariances, hand-worked cases): no function
here is "parity unpinned".

Notation (paper, Section 4): L_p prompt length, N pseudo tokens placed at
positions L_p .. L_p+N-1, d_k head dimension, S(j) importance of prompt token j,
K the number of retained tokens.  G is the number of query heads that share one
KV head (grouped-query attention; the paper's models are GQA, its equations carry
no head index, so scores of a group are summed: Eq. 4 is a sum).
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np


# --------------------------------------------------------------------------------------
# Section 4.1: pseudo queries carry the positional encodings of positions L_p .. L_p+N-1
# --------------------------------------------------------------------------------------
def rope_inv_freq(head_dim: int, rope_base: float) -> np.ndarray:
    """theta_c = base^(-2c/d), c = 0 .. d/2-1 (rotary position embedding frequencies)."""
    c = np.arange(head_dim // 2, dtype=np.float64)
    return np.power(np.float64(rope_base), -2.0 * c / np.float64(head_dim))


def rope_inv_freq_llama3(head_dim: int, rope_base: float, factor: float = 8.0,
                         low_freq_factor: float = 1.0, high_freq_factor: float = 4.0,
                         original_context: int = 8192) -> np.ndarray:
    """Frequencies of the Llama-3.1 long-context RoPE scaling (the model of the paper's efficiency
    runs, Appendix B.6, is Llama-3.1-8B-Instruct).  The published rule, per channel pair c with
    theta_c = base^(-2c/d) and wavelength lambda_c = 2 pi / theta_c:
      lambda_c < original_context / high_freq_factor   -> theta_c unchanged (fast channels)
      lambda_c > original_context / low_freq_factor    -> theta_c / factor  (slow channels)
      in between                                       -> ((1 - s) / factor + s) * theta_c  with
          s = (original_context / lambda_c - low_freq_factor) / (high_freq_factor - low_freq_factor).
    """
    theta = rope_inv_freq(head_dim, rope_base)
    out = np.empty_like(theta)
    for c in range(theta.shape[0]):
        wavelen = 2.0 * math.pi / theta[c]
        if wavelen < original_context / high_freq_factor:
            out[c] = theta[c]
        elif wavelen > original_context / low_freq_factor:
            out[c] = theta[c] / factor
        else:
            s_ = (original_context / wavelen - low_freq_factor) / (high_freq_factor - low_freq_factor)
            out[c] = ((1.0 - s_) / factor + s_) * theta[c]
    return out


def rope_pseudo_q(q_pre: np.ndarray, pos_start: int, rope_base: float,
                  inv_freq: Optional[np.ndarray] = None, interleaved: bool = False) -> np.ndarray:
    """Rotate pseudo queries to positions pos_start + i (Section 4.1, position assignment).

    q_pre [..., N, d].  Rotate-half pairing: channel c is paired with channel c + d/2,
      out[c]       = q[c]     cos(p theta_c) - q[c+d/2] sin(p theta_c)
      out[c + d/2] = q[c+d/2] cos(p theta_c) + q[c]     sin(p theta_c).
    interleaved: the pair of frequency c is (2c, 2c + 1) instead (the paper only says "RoPE";
    rotate-half is what its Llama / Qwen models use, adjacent pairs the other common layout).
    """
    q = np.asarray(q_pre, dtype=np.float64)
    n, d = q.shape[-2], q.shape[-1]
    half = d // 2
    theta = rope_inv_freq(d, rope_base) if inv_freq is None else np.asarray(inv_freq, np.float64)
    pos = np.float64(pos_start) + np.arange(n, dtype=np.float64)
    ang = pos[:, None] * theta[None, :]                    # [N, d/2]
    cos, sin = np.cos(ang), np.sin(ang)
    out = np.empty_like(q)
    if interleaved:
        lo, hi = q[..., 0::2], q[..., 1::2]
        out[..., 0::2] = lo * cos - hi * sin
        out[..., 1::2] = hi * cos + lo * sin
        return out
    lo, hi = q[..., :half], q[..., half:]
    out[..., :half] = lo * cos - hi * sin
    out[..., half:] = hi * cos + lo * sin
    return out


# --------------------------------------------------------------------------------------
# Section 4.2, Eq. 4: S(j) = sum_i Attention(q_i, k_j),  Attention = softmax(q K^T / sqrt(d_k))
# --------------------------------------------------------------------------------------
def visible_logits(q_rot_h: np.ndarray, keys: np.ndarray, prompt_len: int,
                   scale: Optional[float] = None) -> np.ndarray:
    """Pre-softmax scores s_ij = q_i . k_j / sqrt(d_k) with unseen keys set to -inf.

    q_rot_h [N, d]; keys [L_p + N, d]: L_p prompt keys followed by the N synthetic
    keys.  Pseudo query i sits at position L_p + i, so under the causal mask of the
    extended prefill it sees every prompt key and synthetic keys 0 .. i (itself
    included).  (Appendix C, Step 1 for s_j; Section 6.3 for the causal mask.)
    """
    q = np.asarray(q_rot_h, dtype=np.float64)
    kk = np.asarray(keys, dtype=np.float64)
    n, d = q.shape
    L = int(prompt_len)
    assert kk.shape[0] == L + n
    sc = 1.0 / math.sqrt(d) if scale is None else float(scale)
    s = (q @ kk.T) * sc                                      # [N, L+N]
    col = np.arange(L + n)[None, :]
    row = np.arange(n)[:, None]
    visible = (col < L) | ((col - L) <= row)
    return np.where(visible, s, -np.inf)


def attention_rows(q_rot_h: np.ndarray, keys: np.ndarray, prompt_len: int,
                   scale: Optional[float] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Attention weights of one head's N pseudo queries, and their log-sum-exp.

    Returns P [N, L_p + N], each row softmax(s) over the visible span (masked entries
    exactly 0; weights >= 0 and summing to 1), and lse [N] = log sum_j exp(s_ij).
    """
    s = visible_logits(q_rot_h, keys, prompt_len, scale)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    z = e.sum(axis=1, keepdims=True)
    return e / z, (m + np.log(z))[:, 0]


def score_sequence(q_rot: np.ndarray, k_seq: np.ndarray, prompt_len: int, group: int,
                   scale: Optional[float] = None) -> Dict[str, np.ndarray]:
    """Importance scores of one sequence's prompt tokens, per KV head (Eq. 4 + GQA sum).

    q_rot [H_q, N, d] rotated pseudo queries; k_seq [H_kv, L_p + N, d] that sequence's
    keys (prompt rows then synthetic rows).  Query head h reads KV head h // G.
    Returns
      scores      [H_kv, L_p]  sum over the group's G heads and the N queries of P_ij
      lse         [H_q, N]     log sum_j exp(s_ij) over the visible span
      prompt_mass [H_q]        sum_i sum_{j < L_p} P_ij
      syn_mass    [H_q]        sum_i sum_{synthetic j} P_ij   (prompt + syn = N)
    """
    q = np.asarray(q_rot, dtype=np.float64)
    Hq, n, d = q.shape
    Hkv = k_seq.shape[0]
    L = int(prompt_len)
    assert Hq == Hkv * group
    scores = np.zeros((Hkv, L), dtype=np.float64)
    lse = np.zeros((Hq, n), dtype=np.float64)
    pm = np.zeros(Hq, dtype=np.float64)
    sm = np.zeros(Hq, dtype=np.float64)
    for h in range(Hq):
        kv = h // group
        P, lse[h] = attention_rows(q[h], k_seq[kv], L, scale)
        S_h = P[:, :L].sum(axis=0)                           # Eq. 4: sum over the N queries
        scores[kv] += S_h                                    # GQA: sum over the group
        pm[h] = S_h.sum()
        sm[h] = P[:, L:].sum()
    return {"scores": scores, "lse": lse, "prompt_mass": pm, "syn_mass": sm}


def score_prompt_window(q_win_rot: np.ndarray, k_seq: np.ndarray, group: int,
                        scale: Optional[float] = None) -> np.ndarray:
    """Scores of the SnapKV-style observation window the paper compares against (Section 5.1): the
    N queries are those of the LAST N prompt tokens (already rotated), window query i sits at
    position L - N + i and, under the causal mask, attends to keys 0 .. L - N + i.

    q_win_rot [H_q, N, d]; k_seq [H_kv, L, d] (the whole prompt, no synthetic rows).  Returns
    [H_kv, L - N]: sum over the window queries and the group's heads of the attention each token
    BEFORE the window receives (the window's own tokens are always kept by that method).
    """
    q = np.asarray(q_win_rot, dtype=np.float64)
    kk = np.asarray(k_seq, dtype=np.float64)
    Hq, n, d = q.shape
    Hkv, L, _ = kk.shape
    sc = 1.0 / math.sqrt(d) if scale is None else float(scale)
    out = np.zeros((Hkv, L - n), dtype=np.float64)
    key_pos = np.arange(L)[None, :]
    query_pos = (L - n + np.arange(n))[:, None]
    for h in range(Hq):
        s = (q[h] @ kk[h // group].T) * sc                      # [N, L]
        s = np.where(key_pos <= query_pos, s, -np.inf)
        e = np.exp(s - s.max(axis=1, keepdims=True))
        P = e / e.sum(axis=1, keepdims=True)
        out[h // group] += P[:, :L - n].sum(axis=0)
    return out


# --------------------------------------------------------------------------------------
# Optional pooling of the accumulated scores before selection.  The paper specifies none
# for DapQ; it describes the SnapKV / PyramidKV baselines as selecting on pooled accumulated
# attention scores (Sections 2 and 5.1), which this option reproduces.
# --------------------------------------------------------------------------------------
def pool_scores(scores: np.ndarray, kernel: int, mode: str) -> np.ndarray:
    """1-D pooling along one sequence's prompt positions: window of odd width `kernel`
    centred on each position, stride 1, clipped at the ends of the sequence.
    mode "max": largest score in the window; "avg": mean of the scores in the window
    (of the positions that exist, so the ends average fewer values); "none": unchanged."""
    s = np.asarray(scores, dtype=np.float64)
    if mode == "none" or kernel <= 1:
        return s.copy()
    assert kernel % 2 == 1 and mode in ("max", "avg")
    L, r = s.shape[-1], kernel // 2
    out = np.empty_like(s)
    for j in range(L):
        win = s[..., max(0, j - r):min(L, j + r + 1)]
        out[..., j] = win.max(axis=-1) if mode == "max" else win.mean(axis=-1)
    return out


# --------------------------------------------------------------------------------------
# Section 4.2, Eq. 5: M_retain = TopK_j S(j)
# --------------------------------------------------------------------------------------
def topk_select(scores: np.ndarray, k_keep: int) -> np.ndarray:
    """Indices of the k_keep largest scores, returned in ascending position order.

    Full sort on (score descending, index ascending): ties at the threshold go to
    the lower index.  k_keep larger than the length keeps everything.
    """
    s = np.asarray(scores, dtype=np.float64)
    L = s.shape[0]
    kk = min(int(k_keep), L)
    order = np.lexsort((np.arange(L), -s))                   # last key is the primary one
    return np.sort(order[:kk]).astype(np.int32)


# --------------------------------------------------------------------------------------
# Section 4.2, last paragraph: prune the cache to M_retain, drop every synthetic token
# --------------------------------------------------------------------------------------
def compact_kv(k_seq_head: np.ndarray, v_seq_head: np.ndarray,
               idx: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Rows idx of one head's K and V, copied unchanged (same rows for K and V)."""
    return k_seq_head[idx].copy(), v_seq_head[idx].copy()


# --------------------------------------------------------------------------------------
# Section 3.3, Eq. 1-3: recall of a predicted retained set against a gold one
# --------------------------------------------------------------------------------------
def recall(idx_gold: np.ndarray, idx_pred: np.ndarray) -> float:
    """|M_gold ∩ M_pred| / |M_gold| for two index sets of one head (Eq. 3)."""
    gold = set(int(x) for x in np.asarray(idx_gold).ravel())
    pred = set(int(x) for x in np.asarray(idx_pred).ravel())
    return len(gold & pred) / len(gold)


def evict(q_pre: np.ndarray, k: np.ndarray, v: np.ndarray, cu_rows: Sequence[int],
          prompt_len: Sequence[int], k_keep: Sequence[int], rope_base: float,
          scale: Optional[float] = None,
          pos_start: Optional[Sequence[int]] = None, pool_mode: str = "none",
          pool_kernel: int = 1, inv_freq: Optional[np.ndarray] = None,
          rope_interleaved: bool = False) -> Dict[str, object]:
    """The whole path for one layer (Figure 1): rotate, score, select, compact.

    q_pre [B, H_q, N, d] pre-RoPE pseudo queries (any float dtype; converted exactly
    to float64); k, v [H_kv, R, d] packed cache whose sequence b owns rows
    cu_rows[b] .. cu_rows[b+1] (L_b prompt rows, then N synthetic rows).
    inv_freq [d/2] replaces the frequencies base^(-2c/d) (models with scaled RoPE).
    With pool_mode "max" / "avg" the selection runs on the pooled scores (returned as
    "pooled"); "scores" are always the unpooled Eq. 4 sums.
    Returns per-sequence lists: scores [H_kv, L_b], idx [H_kv, K_b] (sequence-local),
    k_out / v_out [H_kv, K_b, d] in the dtype of k / v, plus lse and the two masses.
    """
    B, Hq, n, d = q_pre.shape
    Hkv = k.shape[0]
    G = Hq // Hkv
    out: Dict[str, List] = {key: [] for key in
                            ("q_rot", "scores", "pooled", "lse", "prompt_mass", "syn_mass",
                             "idx", "k_out", "v_out")}
    for b in range(B):
        L = int(prompt_len[b])
        r0 = int(cu_rows[b])
        assert int(cu_rows[b + 1]) - r0 == L + n
        p0 = L if pos_start is None else int(pos_start[b])
        q_rot = rope_pseudo_q(np.asarray(q_pre[b], dtype=np.float64), p0, rope_base, inv_freq, rope_interleaved)
        k_seq = k[:, r0:r0 + L + n]
        v_seq = v[:, r0:r0 + L + n]
        res = score_sequence(q_rot, k_seq, L, G, scale)
        kk = min(int(k_keep[b]), L)
        pooled = pool_scores(res["scores"], pool_kernel, pool_mode)
        idx = np.stack([topk_select(pooled[h], kk) for h in range(Hkv)])
        kept = [compact_kv(k_seq[h], v_seq[h], idx[h]) for h in range(Hkv)]
        ko = np.stack([kv[0] for kv in kept])
        vo = np.stack([kv[1] for kv in kept])
        out["q_rot"].append(q_rot)
        for key in ("scores", "lse", "prompt_mass", "syn_mass"):
            out[key].append(res[key])
        out["pooled"].append(pooled)
        out["idx"].append(idx)
        out["k_out"].append(ko)
        out["v_out"].append(vo)
    return out
