"""Stored expected values (tests/golden/evict_small.json, written by make_golden.py from the
oracle alone): the oracle still reproduces them, and the CUDA path matches them."""
import importlib.util
import json
import os

import numpy as np
import pytest
import torch

from oracle import dapq_oracle as orc
from tests import util

HERE = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _mk():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


GOLD = json.load(open(os.path.join(HERE, "evict_small.json")))


@pytest.mark.parametrize("name", ["d8", "d128"])
def test_oracle_reproduces_the_stored_values(name):
    mk = _mk()
    seed, hq, hkv, n, d, lens, keep, base = mk.CASES[name]
    q, k, v, cu = mk.draw(seed, hq, hkv, n, d, lens)
    res = orc.evict(q.astype(np.float64), k.astype(np.float64), v.astype(np.float64), cu, lens, keep, base)
    for b in range(len(lens)):
        np.testing.assert_allclose(res["scores"][b], np.array(GOLD[name]["scores"][b]), rtol=1e-12)
        np.testing.assert_array_equal(res["idx"][b], np.array(GOLD[name]["idx"][b]))
        np.testing.assert_allclose(res["lse"][b], np.array(GOLD[name]["lse"][b]), rtol=1e-12)
        # invariant on the stored numbers themselves: prompt mass below N per head group
        assert np.all(np.array(GOLD[name]["scores"][b]).sum(axis=1) < (hq // hkv) * n)


@pytest.mark.gpu
def test_cuda_path_matches_the_stored_values():
    import paper_2603_11564_b200 as dq
    mk = _mk()
    seed, hq, hkv, n, d, lens, keep, base = mk.CASES["d128"]
    q, k, v, cu = mk.draw(seed, hq, hkv, n, d, lens)
    ctx = dq.dapq_create(hq, hkv, n, len(lens), int(cu[-1]), dq.DAPQ_F32, base)
    KT, T = sum(min(a, b) for a, b in zip(keep, lens)), sum(lens)
    k_out = torch.empty((hkv, KT, d), dtype=torch.float32, device="cuda")
    v_out = torch.empty_like(k_out)
    idx = torch.empty((hkv, KT), dtype=torch.int32, device="cuda")
    scores = torch.empty((hkv, T), dtype=torch.float32, device="cuda")
    dq.dapq_evict(ctx, torch.from_numpy(q).cuda(), torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), cu, lens,
                  keep, k_out, v_out, idx, scores)
    dq.dapq_poll_status(ctx)
    dq.dapq_destroy(ctx)
    p0 = k0 = 0
    for b, (L, K) in enumerate(zip(lens, keep)):
        for h in range(hkv):
            ref = np.array(GOLD["d128"]["scores"][b][h])
            util.assert_scores_close(scores[h, p0:p0 + L].cpu().double().numpy(), ref, f"golden b={b} h={h}")
            util.assert_index_sets_match(idx[h, k0:k0 + K].cpu().numpy(), ref, np.array(GOLD["d128"]["idx"][b][h]), L)
        p0 += L
        k0 += K
