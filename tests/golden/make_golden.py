"""Writes tests/golden/evict_small.json: the oracle's outputs on two small seeded cases.

    python tests/golden/make_golden.py

Only `oracle/` is called (never the CUDA library).  The paper prints no worked value of the
importance scores S(j) (Section 4.2, Eq. 4) or of a retained set (Eq. 5), so these are
regression fixtures of the pinned oracle, not paper values: they catch an accidental change of
the oracle's arithmetic, and give the GPU tests stored expected values that no GPU produced."""
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import dapq_oracle as orc  # noqa: E402

CASES = {
    # name: (seed, H_q, H_kv, N, d, prompt lengths, keep, rope base)
    "d8": (101, 2, 1, 3, 8, (9,), (4,), 1.0e4),
    "d128": (102, 4, 2, 4, 128, (40, 7), (6, 3), 5.0e5),
}


def draw(seed, hq, hkv, n, d, lens):
    """Inputs of a case: float32 values (exactly representable in both storage types used)."""
    rng = np.random.default_rng(seed)
    rows = sum(l + n for l in lens)
    q = rng.standard_normal((len(lens), hq, n, d)).astype(np.float32)
    k = rng.standard_normal((hkv, rows, d)).astype(np.float32)
    v = rng.standard_normal((hkv, rows, d)).astype(np.float32)
    cu = np.concatenate([[0], np.cumsum([l + n for l in lens])]).astype(np.int32)
    return q, k, v, cu


def main():
    out = {}
    for name, (seed, hq, hkv, n, d, lens, keep, base) in CASES.items():
        q, k, v, cu = draw(seed, hq, hkv, n, d, lens)
        res = orc.evict(q.astype(np.float64), k.astype(np.float64), v.astype(np.float64), cu, lens, keep, base)
        out[name] = {
            "citation": "Section 4.2, Eq. 4 (scores) and Eq. 5 (idx); oracle output, not a paper value",
            "scores": [[[float(x) for x in row] for row in s] for s in res["scores"]],
            "idx": [[[int(x) for x in row] for row in s] for s in res["idx"]],
            "lse": [[[float(x) for x in row] for row in s] for s in res["lse"]],
        }
    with open(os.path.join(HERE, "evict_small.json"), "w") as f:
        json.dump(out, f, indent=1)
    print("wrote evict_small.json")


if __name__ == "__main__":
    main()
