"""Helpers shared by the parity tests: oracle drivers and the pass criteria."""
from __future__ import annotations

import numpy as np
import torch

from gen import inputs as gi
from oracle import dapq_oracle as orc

SCORE_RTOL = 2e-3     # per-token scores: within 2e-3 relative of the oracle
BAND_RTOL = 2e-3      # index sets may differ only inside this band around the K-th oracle score


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact float64 image of a bf16 / fp32 tensor."""
    return t.detach().cpu().to(torch.float64).numpy()


def oracle_q_rot(w: gi.Workload, data) -> torch.Tensor:
    """Rotated pseudo queries [B, H_q, N, d] (float64) from the oracle."""
    q = to_f64(data["q_pre"])
    return torch.from_numpy(np.stack([orc.rope_pseudo_q(q[b], w.prompt_lens[b], w.rope_base)
                                      for b in range(w.batch)]))


def make_case(w: gi.Workload, layer: int = 0, device="cpu"):
    """Draw a layer and plant its needles / sinks with the oracle's rotated queries."""
    data = gi.draw_layer(w, layer, device)
    gi.plant_structure(w, data, oracle_q_rot(w, data))
    return data


def oracle_evict(w: gi.Workload, data):
    return orc.evict(to_f64(data["q_pre"]), to_f64(data["k"]), to_f64(data["v"]), w.cu_rows,
                     w.prompt_lens, w.keep, w.rope_base)


def assert_scores_close(got: np.ndarray, ref: np.ndarray, what=""):
    err = np.abs(got - ref)
    bad = err > SCORE_RTOL * np.abs(ref) + 1e-30
    assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} scores off by more than {SCORE_RTOL} rel; "
                           f"worst rel {np.max(err / np.maximum(np.abs(ref), 1e-300)):.3e}")


def assert_index_sets_match(got_idx: np.ndarray, ref_scores: np.ndarray, ref_idx: np.ndarray, L: int, what=""):
    """got_idx: GPU indices of one (sequence, head); identical to the oracle's set except for
    tokens whose oracle score lies within BAND_RTOL (relative) of the K-th oracle score."""
    K = len(ref_idx)
    assert got_idx.shape == (K,), f"{what}: {got_idx.shape} vs K={K}"
    assert np.all(np.diff(got_idx) > 0), f"{what}: indices not strictly ascending"
    assert got_idx.min() >= 0 and got_idx.max() < L, f"{what}: index out of the prompt range"
    kth = np.sort(ref_scores)[-K]
    diff = np.setxor1d(got_idx, ref_idx)
    if diff.size:
        off = np.abs(ref_scores[diff] - kth)
        assert np.all(off <= BAND_RTOL * kth), (f"{what}: {diff.size} tokens differ outside the band; "
                                                f"worst {np.max(off / kth):.3e}")
    return diff.size
