"""Seeded synthetic inputs for the DapQ eviction scorer.

This module only DRAWS data: Gaussian pseudo queries and K/V caches with the
shapes and structure of the paper's models and context lengths (GQA head
counts, head_dim 128, 2k-128k prompts, observation window 32-128, budgets from
a few dozen rows to a few thousand).  It holds none of the method's arithmetic:
no RoPE, no attention, no softmax, no top-k.  Structure that depends on the
rotated pseudo queries (planted needle keys, attention-sink rows) is added by
`plant_structure`, which receives the rotated queries from its caller - the
oracle in the tests, the CUDA library in the benchmark - and only averages and
rescales them.

Both the CPU oracle and the CUDA path read the tensors produced here after they
have been rounded to their storage dtype, so both sides see identical bits.
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass
from typing import Dict, Optional, Tuple

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration (shapes follow the paper's model families)."""

    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_pseudo: int                  # N, size of the pseudo-query window
    prompt_lens: Tuple[int, ...]   # L_b per sequence
    keep: Tuple[int, ...]          # K_b per sequence (rows kept per KV head)
    dtype: str                     # "bf16" or "f32" (storage type of q, K, V)
    rope_base: float
    seed: int
    n_needles: int = 0             # planted needle keys per KV head and sequence
    needle_rho: float = 3.0        # norm of a needle key in units of sqrt(d) (a typical key has 1)
    outlier_channels: int = 0      # channels per KV head scaled by outlier_scale
    outlier_scale: float = 8.0
    sink_rows: int = 0             # first rows of each head with a heavy-tailed bias

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def batch(self) -> int:
        return len(self.prompt_lens)

    @property
    def cu_rows(self) -> np.ndarray:
        """Row offsets of the packed cache: sequence b holds L_b + N rows."""
        rows = np.asarray(self.prompt_lens, dtype=np.int64) + self.n_pseudo
        return np.concatenate([[0], np.cumsum(rows)]).astype(np.int32)

    @property
    def cu_prompt(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.prompt_lens)]).astype(np.int32)

    @property
    def cu_keep(self) -> np.ndarray:
        kk = [min(k, l) for k, l in zip(self.keep, self.prompt_lens)]
        return np.concatenate([[0], np.cumsum(kk)]).astype(np.int32)

    @property
    def total_rows(self) -> int:
        return int(self.cu_rows[-1])

    @property
    def total_prompt(self) -> int:
        return int(sum(self.prompt_lens))

    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32


def _ragged_lengths(seed: int, batch: int, lo: int, hi: int) -> Tuple[int, ...]:
    rs = np.random.RandomState(seed)
    return tuple(int(x) for x in rs.randint(lo, hi + 1, size=batch))


def _serving_lengths() -> Tuple[int, ...]:
    return _ragged_lengths(3, 8, 4096, 32768)


_SERVING = _serving_lengths()

#: The five configurations the benchmark contract names, in its order.
WORKLOADS: Dict[str, Workload] = {
    "tiny": Workload(
        name="tiny", n_layers=1, n_q_heads=8, n_kv_heads=2, head_dim=128, n_pseudo=32,
        prompt_lens=(2048,), keep=(128,), dtype="f32", rope_base=1.0e4, seed=0,
        n_needles=4),
    "llama3_8b_32k": Workload(
        name="llama3_8b_32k", n_layers=32, n_q_heads=32, n_kv_heads=8, head_dim=128,
        n_pseudo=64, prompt_lens=(32768,), keep=(983,), dtype="bf16", rope_base=5.0e5,
        seed=1, n_needles=16, outlier_channels=4),
    "qwen25_7b_128k": Workload(
        name="qwen25_7b_128k", n_layers=28, n_q_heads=28, n_kv_heads=4, head_dim=128,
        n_pseudo=64, prompt_lens=(131072,), keep=(4096,), dtype="bf16", rope_base=1.0e6,
        seed=2, sink_rows=4),
    "batched_serving": Workload(
        name="batched_serving", n_layers=32, n_q_heads=32, n_kv_heads=8, head_dim=128,
        n_pseudo=32, prompt_lens=_SERVING, keep=tuple(l // 10 for l in _SERVING),
        dtype="bf16", rope_base=5.0e5, seed=3),
    "llama3_70b_128k": Workload(
        name="llama3_70b_128k", n_layers=80, n_q_heads=64, n_kv_heads=8, head_dim=128,
        n_pseudo=128, prompt_lens=(131072,), keep=(3932,), dtype="bf16", rope_base=5.0e5,
        seed=4, n_needles=32, outlier_channels=4),
}

WORKLOAD_ORDER = ("tiny", "llama3_8b_32k", "qwen25_7b_128k", "batched_serving",
                  "llama3_70b_128k")


def workload(name: str, **overrides) -> Workload:
    """Look a configuration up; keyword overrides give scaled-down test variants."""
    w = WORKLOADS[name]
    return dataclasses.replace(w, **overrides) if overrides else w


def _generator(device, seed: int, layer: int, stream: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1_000_003 + layer) * 16 + stream)
    return g


def draw_layer(w: Workload, layer: int = 0, device="cpu") -> Dict[str, object]:
    """Draw one layer's pseudo queries and packed K/V cache.

    Returns a dict with
      q_pre  [B, H_q, N, d]    pre-RoPE pseudo queries, storage dtype
      k, v   [H_kv, R, d]      packed cache, R = sum_b (L_b + N); sequence b owns rows
                               cu_rows[b] .. cu_rows[b+1]: L_b prompt rows then N
                               synthetic rows.  Keys are understood as already rotated
                               (an isotropic Gaussian is unchanged in law by a rotation).
      needle_pos [B, H_kv, n_needles]  int64 sequence-local rows reserved for needles
      outlier_ch [H_kv, outlier_channels] int64
    Needles and sink rows are NOT planted yet: see `plant_structure`.
    """
    dt = w.torch_dtype()
    B, Hq, Hkv, N, d = w.batch, w.n_q_heads, w.n_kv_heads, w.n_pseudo, w.head_dim
    R = w.total_rows
    q_pre = torch.randn((B, Hq, N, d), generator=_generator(device, w.seed, layer, 0),
                        device=device, dtype=torch.float32).to(dt)
    k = torch.randn((Hkv, R, d), generator=_generator(device, w.seed, layer, 1),
                    device=device, dtype=torch.float32)
    v = torch.randn((Hkv, R, d), generator=_generator(device, w.seed, layer, 2),
                    device=device, dtype=torch.float32).to(dt)

    rs = np.random.RandomState((w.seed * 7919 + layer * 104729 + 17) % (2 ** 31 - 1))
    outlier_ch = np.zeros((Hkv, w.outlier_channels), dtype=np.int64)
    for h in range(Hkv):
        if w.outlier_channels:
            outlier_ch[h] = np.sort(rs.choice(d, size=w.outlier_channels, replace=False))
            k[h][:, torch.as_tensor(outlier_ch[h], device=k.device)] *= w.outlier_scale
    needle_pos = np.zeros((B, Hkv, w.n_needles), dtype=np.int64)
    for b in range(B):
        lo = w.sink_rows
        for h in range(Hkv):
            if w.n_needles:
                needle_pos[b, h] = np.sort(
                    lo + rs.choice(w.prompt_lens[b] - lo, size=w.n_needles, replace=False))
    # heavy-tailed sink strengths: 6 + |t_2|, clipped at 30 (Student-t, 2 dof)
    sink_tau = 6.0 + np.minimum(np.abs(rs.standard_t(2, size=(B, Hkv, max(w.sink_rows, 1)))),
                                24.0)
    return {
        "q_pre": q_pre, "k": k.to(dt), "v": v,
        "needle_pos": needle_pos, "outlier_ch": outlier_ch,
        "sink_tau": sink_tau[:, :, :w.sink_rows],
    }


def plant_structure(w: Workload, data: Dict[str, object], q_rot: torch.Tensor) -> None:
    """Write needle keys and sink rows into data["k"], in place.

    q_rot [B, H_q, N, d] are the pseudo queries ALREADY rotated to their decode
    positions, supplied by the caller.  With qbar the mean of the G*N rotated
    queries of a KV head's group and u = qbar/|qbar|:
      needle row:  k = rho * sqrt(d) * u   (a scaled copy of the mean rotated query, rho = 3
                   times the norm of a typical key, so every window query's logit against
                   it is rho*(|qbar| + z), z ~ N(0,1): far above the bulk, yet a key norm
                   a bf16 cache can hold without swamping the other rows' precision);
      sink row j:  k += tau_j * u, tau_j = 6 + |t_2| clipped at 30 (heavy-tailed).
    Values are rounded to the storage dtype on assignment.
    """
    if not (w.n_needles or w.sink_rows):
        return
    k = data["k"]
    cu = w.cu_rows
    G, d = w.group, w.head_dim
    q = q_rot.to(device=k.device, dtype=torch.float64)
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            qbar = q[b, h * G:(h + 1) * G].reshape(-1, d).mean(dim=0)
            u = qbar / qbar.norm()
            if w.n_needles:
                rows = torch.as_tensor(data["needle_pos"][b, h] + int(cu[b]), device=k.device)
                k[h, rows] = (w.needle_rho * math.sqrt(d) * u).to(k.dtype).unsqueeze(0).expand(len(rows), d)
            for j in range(w.sink_rows):
                tau = float(data["sink_tau"][b, h, j])
                add = tau * u
                row = int(cu[b]) + j
                k[h, row] = (k[h, row].to(torch.float64) + add).to(k.dtype)


def scaled_down(name: str, prompt_scale: int, n_layers: Optional[int] = None) -> Workload:
    """A configuration with every prompt (and budget) divided by `prompt_scale`."""
    w = WORKLOADS[name]
    lens = tuple(max(1, l // prompt_scale) for l in w.prompt_lens)
    keep = tuple(max(1, k // prompt_scale) for k in w.keep)
    return dataclasses.replace(w, prompt_lens=lens, keep=keep,
                               n_layers=n_layers if n_layers is not None else w.n_layers)
