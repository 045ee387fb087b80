"""GPU parity: every C-ABI entry point against the CPU oracle on the same seeded inputs.

Pass criteria: per-token scores within 2e-3 relative; index sets identical except inside
the 2e-3 band around the K-th oracle score; compacted K/V bit-exact given the indices."""
import dataclasses

import numpy as np
import pytest
import torch

from gen import inputs as gi
from oracle import dapq_oracle as orc
from tests import util

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dq():
    import paper_2603_11564_b200 as lib
    lib.load_library()
    return lib


def _ctx(dq, w: gi.Workload, **kw):
    return dq.dapq_create(w.n_q_heads, w.n_kv_heads, w.n_pseudo, w.batch, w.total_rows,
                          dq.DAPQ_BF16 if w.dtype == "bf16" else dq.DAPQ_F32, w.rope_base, **kw)


def _small(name="llama3_8b_32k", lens=(700,), keep=(40,), **kw) -> gi.Workload:
    return gi.workload(name, prompt_lens=tuple(lens), keep=tuple(keep), n_layers=1, **kw)


def _gpu_evict(dq, w, data, ctx=None):
    dev = "cuda"
    own = ctx is None
    ctx = ctx or _ctx(dq, w)
    q, k, v = (data[x].to(dev) for x in ("q_pre", "k", "v"))
    KT, T = int(w.cu_keep[-1]), w.total_prompt
    k_out = torch.empty((w.n_kv_heads, KT, w.head_dim), dtype=k.dtype, device=dev)
    v_out = torch.empty_like(k_out)
    idx = torch.empty((w.n_kv_heads, KT), dtype=torch.int32, device=dev)
    scores = torch.empty((w.n_kv_heads, T), dtype=torch.float32, device=dev)
    dq.dapq_evict(ctx, q, k, v, w.cu_rows, w.prompt_lens, w.keep, k_out, v_out, idx, scores)
    dq.dapq_poll_status(ctx)
    if own:
        dq.dapq_destroy(ctx)
    return dict(k_out=k_out.cpu(), v_out=v_out.cpu(), idx=idx.cpu().numpy(), scores=scores.cpu().double().numpy())


def _check_evict(w, data, got, ref):
    cu_p, cu_k, cu_r = w.cu_prompt, w.cu_keep, w.cu_rows
    n_band = 0
    for b in range(w.batch):
        L = w.prompt_lens[b]
        for h in range(w.n_kv_heads):
            tag = f"{w.name} b={b} kvh={h}"
            util.assert_scores_close(got["scores"][h, cu_p[b]:cu_p[b + 1]], ref["scores"][b][h], tag)
            gidx = got["idx"][h, cu_k[b]:cu_k[b + 1]]
            n_band += util.assert_index_sets_match(gidx, ref["scores"][b][h], ref["idx"][b][h], L, tag)
            # compaction is a bit-exact copy of the rows the GPU itself selected
            rows = torch.as_tensor(gidx.astype(np.int64) + int(cu_r[b]))
            assert torch.equal(got["k_out"][h, cu_k[b]:cu_k[b + 1]], data["k"][h].cpu()[rows]), tag
            assert torch.equal(got["v_out"][h, cu_k[b]:cu_k[b + 1]], data["v"][h].cpu()[rows]), tag
            for p in (data["needle_pos"][b, h] if w.n_needles else []):
                assert int(p) in set(gidx.tolist()), f"{tag}: planted needle {p} evicted"
    return n_band


# ------------------------------------------------------------------------- dapq_rope_pseudo_q
@pytest.mark.parametrize("interleaved", [False, True])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_rope_parity(dq, dtype, interleaved):
    w = _small(lens=(5, 131072, 4097), keep=(1, 1, 1), dtype=dtype, n_pseudo=33, rope_base=5.0e5, n_needles=0)
    ctx = _ctx(dq, w, flags=dq.DAPQ_FLAG_ROPE_INTERLEAVED if interleaved else 0)
    data = gi.draw_layer(dataclasses.replace(w, prompt_lens=(8, 8, 8)), 0, "cpu")
    q = data["q_pre"].cuda()
    out = torch.empty_like(q)
    pos = [5, 131072, 0]
    dq.dapq_rope_pseudo_q(ctx, q, pos, out)
    torch.cuda.synchronize()
    ref = np.stack([orc.rope_pseudo_q(util.to_f64(data["q_pre"][b]), pos[b], w.rope_base, interleaved=interleaved)
                    for b in range(3)])
    got = util.to_f64(out)
    tol = 2.0 ** -8 if dtype == "bf16" else 2.0 ** -22
    assert np.all(np.abs(got - ref) <= tol * np.abs(ref) + 1e-7)
    assert torch.equal(out[2, :, 0].cpu(), data["q_pre"][2, :, 0])      # position 0 is the identity
    dq.dapq_destroy(ctx)


# --------------------------------------------------------------------------------- dapq_score
SCORE_CASES = [
    # dtype, H_q, H_kv, N, prompt lengths
    ("f32", 8, 2, 32, (2048,)),
    ("f32", 2, 2, 1, (1,)),
    ("f32", 3, 1, 5, (63, 64, 65)),
    ("bf16", 8, 2, 64, (1500,)),
    ("bf16", 7, 1, 64, (513, 1, 127)),
    ("bf16", 8, 1, 128, (129, 1031)),
    ("bf16", 4, 4, 100, (777,)),
    ("bf16", 8, 2, 17, (512, 1024, 300, 5)),
    # more than 256 query rows per KV head: sweep 2 keeps up to 512 resident, the second job narrow (48 / 16 columns)
    ("bf16", 3, 1, 100, (600, 90)),
    ("bf16", 5, 1, 104, (700,)),
    # CUDA-core sweeps at every chunk size (512 / 256 / 128 keys on a 148-SM part; the shorter cases above take 64)
    ("f32", 8, 8, 8, (19000,)),
    ("bf16", 8, 8, 4, (9000, 700)),
    ("f32", 4, 4, 16, (9500,)),
]


@pytest.mark.parametrize("dtype,hq,hkv,n,lens", SCORE_CASES)
def test_score_parity(dq, dtype, hq, hkv, n, lens):
    w = _small(lens=lens, keep=tuple(1 for _ in lens), dtype=dtype, n_q_heads=hq, n_kv_heads=hkv, n_pseudo=n,
               n_needles=0, outlier_channels=2 if dtype == "bf16" else 0)
    data = gi.draw_layer(w, 0, "cpu")
    q_rot64 = util.oracle_q_rot(w, data)
    q_rot = q_rot64.to(w.torch_dtype())                   # the operand both sides read
    ctx = _ctx(dq, w)
    B = w.batch
    scores = torch.empty((hkv, w.total_prompt), dtype=torch.float32, device="cuda")
    lse = torch.empty((B, hq, n), dtype=torch.float32, device="cuda")
    syn = torch.empty((B, hq), dtype=torch.float32, device="cuda")
    k64 = util.to_f64(data["k"])
    refs = [orc.score_sequence(util.to_f64(q_rot[b]), k64[:, int(w.cu_rows[b]):int(w.cu_rows[b + 1])], lens[b], w.group)
            for b in range(B)]
    # without syn_mass the bf16 shapes with G*N >= 64 run on the tensor cores; asking for
    # syn_mass routes the same call through the CUDA-core kernels
    for want_syn in (False, True):
        scores.fill_(-1.0)
        lse.fill_(0.0)
        kw = dict(lse_out=lse, syn_mass=syn) if want_syn else dict(lse_out=lse)
        dq.dapq_score(ctx, q_rot.cuda(), data["k"].cuda(), w.cu_rows, w.prompt_lens, scores, **kw)
        dq.dapq_poll_status(ctx)
        first = scores.clone()
        # bit-identical when repeated (fixed reduction order, no float atomics)
        dq.dapq_score(ctx, q_rot.cuda(), data["k"].cuda(), w.cu_rows, w.prompt_lens, scores, **kw)
        dq.dapq_poll_status(ctx)
        assert torch.equal(first, scores)
        got = scores.cpu().double().numpy()
        for b in range(B):
            ref = refs[b]
            util.assert_scores_close(got[:, w.cu_prompt[b]:w.cu_prompt[b + 1]], ref["scores"], f"b={b} syn={want_syn}")
            np.testing.assert_allclose(lse[b].cpu().numpy(), ref["lse"], rtol=0, atol=2e-3)
            if want_syn:
                np.testing.assert_allclose(syn[b].cpu().numpy(), ref["syn_mass"], rtol=2e-3, atol=1e-6)
                # mass conservation on the GPU's own numbers: sum_j scores + sum_g syn = G * N
                tot = (got[:, w.cu_prompt[b]:w.cu_prompt[b + 1]].sum(axis=1)
                       + syn[b].cpu().double().numpy().reshape(hkv, -1).sum(axis=1))
                np.testing.assert_allclose(tot, np.full(hkv, w.group * n), rtol=1e-4)
    # the caller's own log-sum-exp (from the oracle) replaces the first sweep
    lse_ref = torch.from_numpy(np.stack([refs[b]["lse"] for b in range(B)])).float().cuda()
    scores2 = torch.empty_like(scores)
    dq.dapq_score(ctx, q_rot.cuda(), data["k"].cuda(), w.cu_rows, w.prompt_lens, scores2, lse_in=lse_ref)
    torch.cuda.synchronize()
    np.testing.assert_allclose(scores2.cpu().numpy(), got, rtol=1e-3)
    dq.dapq_destroy(ctx)


def test_score_strided_view_and_custom_scale(dq):
    w = _small(lens=(300, 90), keep=(1, 1), n_q_heads=4, n_kv_heads=2, n_pseudo=16, n_needles=0, outlier_channels=0)
    data = gi.draw_layer(w, 0, "cpu")
    q_rot = util.oracle_q_rot(w, data).to(torch.bfloat16)
    R = w.total_rows
    # cache stored as [R, H_kv, 2*d] (row-major over tokens, padded rows): heads interleaved
    big = torch.zeros((R, w.n_kv_heads, 256), dtype=torch.bfloat16, device="cuda")
    big[:, :, :128] = data["k"].cuda().transpose(0, 1)
    kview = big[:, :, :128].transpose(0, 1)
    assert kview.stride() == (256, 512, 1)
    ctx = _ctx(dq, w, softmax_scale=0.05)
    scores = torch.empty((w.n_kv_heads, w.total_prompt), dtype=torch.float32, device="cuda")
    dq.dapq_score(ctx, q_rot.cuda(), kview, w.cu_rows, w.prompt_lens, scores)
    torch.cuda.synchronize()
    k64 = util.to_f64(data["k"])
    for b in range(2):
        r0, L = int(w.cu_rows[b]), w.prompt_lens[b]
        ref = orc.score_sequence(util.to_f64(q_rot[b]), k64[:, r0:r0 + L + 16], L, w.group, scale=0.05)
        util.assert_scores_close(scores[:, w.cu_prompt[b]:w.cu_prompt[b + 1]].cpu().double().numpy(), ref["scores"])
    dq.dapq_destroy(ctx)


# -------------------------------------------------------------------------- dapq_topk_select
@pytest.mark.parametrize("lens,keep", [
    ((1, 33, 4096, 5000, 131072, 77), (1, 33, 1, 4999, 3932, 200)),
    ((400000, 9), (12345, 3)),       # slices too long for the shared-memory key cache
    ((200000, 130000), (7000, 129999)),   # 32 keys per thread
])
def test_topk_exact_with_ties(dq, lens, keep):
    rng = np.random.default_rng(5)
    w = _small(lens=lens, keep=keep, n_q_heads=3, n_kv_heads=3, n_pseudo=4, n_needles=0, outlier_channels=0)
    T = w.total_prompt
    s = rng.random((3, T)).astype(np.float32)
    s[1] = np.round(s[1] * 50) / 50                      # heavy ties
    s[2] = 0.25                                          # all equal
    s[0, ::7] = 0.0
    ctx = _ctx(dq, w)
    idx = torch.full((3, int(w.cu_keep[-1])), -1, dtype=torch.int32, device="cuda")
    dq.dapq_topk_select(ctx, torch.from_numpy(s).cuda(), w.cu_prompt, keep, idx)
    torch.cuda.synchronize()
    got = idx.cpu().numpy()
    for b in range(len(lens)):
        for h in range(3):
            ref = orc.topk_select(s[h, w.cu_prompt[b]:w.cu_prompt[b + 1]].astype(np.float64), keep[b])
            np.testing.assert_array_equal(got[h, w.cu_keep[b]:w.cu_keep[b + 1]], ref, err_msg=f"b={b} h={h}")
    # the select is integer work in a fixed order: every repeat gives the same indices
    for _ in range(20):
        again = torch.full_like(idx, -1)
        dq.dapq_topk_select(ctx, torch.from_numpy(s).cuda(), w.cu_prompt, keep, again)
        assert torch.equal(again, idx)
    dq.dapq_destroy(ctx)


@pytest.mark.parametrize("case", ["heavy_tail_128k", "heavy_tail_batch", "half_constant", "signed", "two_level", "many_heads"])
def test_topk_score_distributions(dq, case):
    """Score distributions that drive the selection through its different routes: few candidates in the
    threshold's bin (each CTA finishes on its copy of the cluster's candidates), a bin that holds thousands of
    one CTA's keys but few of another's (the cluster falls back to merged histograms), aligned and unaligned
    starts, negative scores."""
    rng = np.random.default_rng(11)
    if case == "heavy_tail_128k":
        lens, keep = (131072,), (3932,)
        s = rng.lognormal(0.0, 1.5, size=(2, sum(lens))).astype(np.float32)
    elif case == "heavy_tail_batch":
        lens, keep = (32768, 32768, 1000, 20001), (983, 100, 999, 600)
        s = rng.lognormal(-9.0, 1.0, size=(2, sum(lens))).astype(np.float32)
        s[1, 40000:40200] = s[1, 39999]                  # a run of ties that straddles the threshold or not
    elif case == "half_constant":
        lens, keep = (65536,), (40000,)
        s = rng.uniform(0.0, 2.0, size=(2, sum(lens))).astype(np.float32)
        s[0, :32768] = 1.0                               # the threshold falls inside 32768 equal scores
        s[1, 1::2] = 1.0
    elif case == "signed":
        lens, keep = (50000, 7), (25000, 3)
        s = rng.standard_normal((2, sum(lens))).astype(np.float32)
        s[1] = np.round(s[1] * 4) / 4 + 0.0              # ties on both sides of zero (no negative zeros)
        s[s == 0] = 0.0
    elif case == "two_level":
        lens, keep = (100000,), (5000,)
        s = np.where(rng.random((2, sum(lens))) < 0.04, 3.0, 1.0).astype(np.float32)   # two values only
        s[1] += (rng.random(sum(lens)) < 0.5) * np.float32(2 ** -22)                   # ... and a last-bit split
    else:                                                # 320 heads of 12k keys: one CTA per head, two per SM
        lens, keep = (12000,) * 20, tuple(range(100, 2100, 100))
        s = rng.lognormal(0.0, 0.5, size=(16, sum(lens))).astype(np.float32)
        s[3] = np.round(s[3] * 8) / 8
        s[5] = 1.0
    H = s.shape[0]
    w = _small(lens=lens, keep=keep, n_q_heads=H, n_kv_heads=H, n_pseudo=4, n_needles=0, outlier_channels=0)
    ctx = _ctx(dq, w)
    idx = torch.full((H, int(w.cu_keep[-1])), -1, dtype=torch.int32, device="cuda")
    dq.dapq_topk_select(ctx, torch.from_numpy(s).cuda(), w.cu_prompt, keep, idx)
    torch.cuda.synchronize()
    got = idx.cpu().numpy()
    for b in range(len(lens)):
        for h in range(H):
            ref = orc.topk_select(s[h, w.cu_prompt[b]:w.cu_prompt[b + 1]].astype(np.float64), keep[b])
            np.testing.assert_array_equal(got[h, w.cu_keep[b]:w.cu_keep[b + 1]], ref, err_msg=f"{case} b={b} h={h}")
    dq.dapq_destroy(ctx)


# --------------------------------------------------------------------------- dapq_compact_kv
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_compact_bit_exact_given_oracle_indices(dq, dtype):
    w = _small(lens=(300, 17, 1000), keep=(30, 40, 999), dtype=dtype, n_q_heads=4, n_kv_heads=2, n_pseudo=8,
               n_needles=0, outlier_channels=0)
    data = gi.draw_layer(w, 0, "cpu")
    ref = util.oracle_evict(w, data)
    idx = np.concatenate(ref["idx"], axis=1)             # [H_kv, KT]
    ctx = _ctx(dq, w)
    KT = idx.shape[1]
    k_out = torch.zeros((2, KT, 128), dtype=w.torch_dtype(), device="cuda")
    v_out = torch.zeros_like(k_out)
    dq.dapq_compact_kv(ctx, data["k"].cuda(), data["v"].cuda(), w.cu_rows, w.prompt_lens, torch.from_numpy(idx).cuda(),
                       w.keep, k_out, v_out)
    dq.dapq_poll_status(ctx)
    view = torch.int16 if dtype == "bf16" else torch.int32
    for b in range(w.batch):
        sl = slice(int(w.cu_keep[b]), int(w.cu_keep[b + 1]))
        for h in range(2):
            rows = torch.as_tensor(ref["idx"][b][h].astype(np.int64) + int(w.cu_rows[b]))
            assert torch.equal(k_out[h, sl].cpu().view(view), data["k"][h][rows].view(view))
            assert torch.equal(v_out[h, sl].cpu().view(view), data["v"][h][rows].view(view))
            np.testing.assert_array_equal(util.to_f64(k_out[h, sl]), ref["k_out"][b][h])
    # an index that points at a synthetic row is skipped and reported, never read
    bad = torch.from_numpy(idx).cuda().clone()
    bad[0, 0] = w.prompt_lens[0]
    dq.dapq_compact_kv(ctx, data["k"].cuda(), data["v"].cuda(), w.cu_rows, w.prompt_lens, bad, w.keep, k_out, v_out)
    with pytest.raises(dq.DapqError):
        dq.dapq_poll_status(ctx)
    dq.dapq_poll_status(ctx)                             # the word was cleared
    dq.dapq_destroy(ctx)


# -------------------------------------------------------------------------------- dapq_evict
def test_evict_tiny_config_in_full(dq):
    w = gi.workload("tiny")
    data = util.make_case(w)
    _check_evict(w, data, _gpu_evict(dq, w, data), util.oracle_evict(w, data))


SCORERS = {"fp16": 0, "cuda_core": 1, "bf16_pair": 8 | 16}   # dapq_shape.flags


@pytest.mark.parametrize("scorer", list(SCORERS))
@pytest.mark.parametrize("name,scale", [("llama3_8b_32k", 16), ("qwen25_7b_128k", 64), ("batched_serving", 16),
                                        ("llama3_70b_128k", 64)])
def test_evict_scaled_configs(dq, name, scale, scorer):
    """Every scorer the flags select (default fp16 tensor-core path, CUDA cores, the older tensor-core kernels
    with the two-part bf16 query operand in both sweeps) meets the same criteria."""
    w = gi.scaled_down(name, scale, n_layers=1)
    data = util.make_case(w)
    ctx = _ctx(dq, w, flags=SCORERS[scorer])
    _check_evict(w, data, _gpu_evict(dq, w, data, ctx), util.oracle_evict(w, data))
    dq.dapq_destroy(ctx)


def test_coarse_query_modes_are_close_but_worse_than_the_default(dq):
    """DAPQ_FLAG_Q_BF16 (one bf16 rounding of the rotated queries) and the two-part operand in one sweep only are
    the documented coarse modes: on a cache with outlier channels their scores stay within 2e-2 of the oracle
    but are measurably worse than the default's."""
    w = gi.scaled_down("llama3_8b_32k", 8, n_layers=1)
    data = util.make_case(w)
    ref = util.oracle_evict(w, data)["scores"][0]
    worst = {}
    for name, flags in (("fp16", 0), ("bf16", dq.DAPQ_FLAG_Q_BF16), ("pair_sweep1", dq.DAPQ_FLAG_Q_LO_SWEEP1),
                        ("pair_sweep2", dq.DAPQ_FLAG_Q_LO_SWEEP2)):
        ctx = _ctx(dq, w, flags=flags)
        got = _gpu_evict(dq, w, data, ctx)["scores"]
        dq.dapq_destroy(ctx)
        worst[name] = float(np.max(np.abs(got - ref) / ref))
    assert worst["fp16"] < 1e-3, worst
    for name in ("bf16", "pair_sweep1", "pair_sweep2"):
        assert worst["fp16"] < worst[name] < 2e-2, worst


def test_score_with_the_older_kernels(dq):
    """A context that asks for the two-part operand sends dapq_score (whose bf16 queries have no low-order
    part) through the older tensor-core kernels as well; several query groups, ragged lengths."""
    for hq, hkv, n, lens in [(8, 1, 128, (129, 1031)), (8, 2, 64, (1500,)), (4, 4, 32, (700, 64))]:
        w = _small(lens=lens, keep=tuple(1 for _ in lens), n_q_heads=hq, n_kv_heads=hkv, n_pseudo=n, n_needles=0,
                   outlier_channels=2)
        data = gi.draw_layer(w, 0, "cpu")
        q_rot = util.oracle_q_rot(w, data).to(torch.bfloat16)
        ctx = _ctx(dq, w, flags=dq.DAPQ_FLAG_Q_LO_SWEEP1 | dq.DAPQ_FLAG_Q_LO_SWEEP2)
        scores = torch.empty((hkv, w.total_prompt), dtype=torch.float32, device="cuda")
        dq.dapq_score(ctx, q_rot.cuda(), data["k"].cuda(), w.cu_rows, w.prompt_lens, scores)
        dq.dapq_poll_status(ctx)
        dq.dapq_destroy(ctx)
        got, k64 = scores.cpu().double().numpy(), util.to_f64(data["k"])
        for b in range(w.batch):
            ref = orc.score_sequence(util.to_f64(q_rot[b]), k64[:, int(w.cu_rows[b]):int(w.cu_rows[b + 1])], lens[b], w.group)
            util.assert_scores_close(got[:, w.cu_prompt[b]:w.cu_prompt[b + 1]], ref["scores"], f"older kernels b={b}")


def test_evict_edge_shapes(dq):
    # K_b >= L_b keeps everything; L_b = 1; K_b = 1; lengths around the tile sizes
    w = _small(lens=(1, 64, 65, 511, 513, 2), keep=(5, 64, 1, 510, 100, 1), n_q_heads=4, n_kv_heads=2,
               n_pseudo=3, n_needles=0)
    data = util.make_case(w)
    got = _gpu_evict(dq, w, data)
    _check_evict(w, data, got, util.oracle_evict(w, data))
    np.testing.assert_array_equal(got["idx"][0, 1:65], np.arange(64))


@pytest.mark.parametrize("pinned", [True, False])
def test_evict_host_matches_device_call(dq, pinned):
    """Host buffers in, host buffers out.  Pinned V is gathered by the compaction kernel straight from host
    memory; pageable V is staged on the device first."""
    w = gi.scaled_down("batched_serving", 32, n_layers=1)
    data = util.make_case(w)
    ctx = _ctx(dq, w)
    dev = _gpu_evict(dq, w, data, ctx)
    KT = int(w.cu_keep[-1])
    pin = (lambda t: t.contiguous().pin_memory()) if pinned else (lambda t: t.contiguous().clone())
    k_out = torch.empty((w.n_kv_heads, KT, 128), dtype=torch.bfloat16).pin_memory()
    v_out = torch.empty_like(k_out).pin_memory()
    idx = torch.empty((w.n_kv_heads, KT), dtype=torch.int32).pin_memory()
    dq.dapq_evict_host(ctx, pin(data["q_pre"]), pin(data["k"]), pin(data["v"]), w.cu_rows, w.prompt_lens, w.keep,
                       k_out, v_out, idx)
    assert torch.equal(k_out, dev["k_out"]) and torch.equal(v_out, dev["v_out"])
    np.testing.assert_array_equal(idx.numpy(), dev["idx"])
    dq.dapq_destroy(ctx)


@pytest.mark.parametrize("pinned", [True, False])
def test_evict_layers_host_pipelines_five_layers(dq, pinned):
    """The multi-layer host call (two staging sets, copies of one layer beside the kernels of the layer
    before) equals a device call per layer, with per-layer budgets; layers 2..4 reuse the staging sets."""
    lens, budgets = (900, 333), [(90, 33), (45, 10), (200, 60), (9, 3), (120, 50)]
    ws, datas = _layer_cases(5, lens, budgets, n_q_heads=8, n_kv_heads=2, n_pseudo=32, n_needles=0)
    ctx = _ctx(dq, ws[0])
    pin = (lambda t: t.contiguous().pin_memory()) if pinned else (lambda t: t.contiguous().clone())   # pageable: V is staged too
    q, k, v = ([pin(d[x]) for d in datas] for x in ("q_pre", "k", "v"))
    ko = [torch.empty((w.n_kv_heads, int(w.cu_keep[-1]), 128), dtype=torch.bfloat16).pin_memory() for w in ws]
    vo = [torch.empty_like(t).pin_memory() for t in ko]
    idx = [torch.empty((w.n_kv_heads, int(w.cu_keep[-1])), dtype=torch.int32).pin_memory() for w in ws]
    dq.dapq_evict_layers_host(ctx, q, k, v, ws[0].cu_rows, ws[0].prompt_lens, budgets, ko, vo, idx)
    dq.dapq_poll_status(ctx)
    for l, (w, data) in enumerate(zip(ws, datas)):
        one = _gpu_evict(dq, w, data, ctx)
        np.testing.assert_array_equal(idx[l].numpy(), one["idx"])
        assert torch.equal(ko[l], one["k_out"]) and torch.equal(vo[l], one["v_out"]), f"layer {l}"
    dq.dapq_destroy(ctx)


def test_argument_errors_launch_nothing(dq):
    w = _small(lens=(100,), keep=(10,), n_needles=0)
    data = gi.draw_layer(w, 0, "cuda")
    ctx = _ctx(dq, w)
    n0 = dq.dapq_launch_count(ctx)
    scores = torch.empty((w.n_kv_heads, 100), dtype=torch.float32, device="cuda")
    with pytest.raises(dq.DapqError) as e:       # rows do not add up to L + N
        dq.dapq_score(ctx, data["q_pre"], data["k"], [0, 150], [100], scores)
    assert e.value.status == dq.DAPQ_ERR_INVALID_ARG
    with pytest.raises(dq.DapqError) as e:       # larger than the workspace
        dq.dapq_score(ctx, data["q_pre"], data["k"], [0, 264], [200], scores)
    assert e.value.status == dq.DAPQ_ERR_WORKSPACE
    with pytest.raises(dq.DapqError) as e:       # misaligned row stride
        dq.dapq_score(ctx, data["q_pre"], data["k"].as_strided((2, 164, 128), (164 * 132, 132, 1)),
                      w.cu_rows, w.prompt_lens, scores)
    assert e.value.status == dq.DAPQ_ERR_UNSUPPORTED
    with pytest.raises(dq.DapqError):
        dq.dapq_topk_select(ctx, scores, [0, 100], [0], torch.empty(8, 10, dtype=torch.int32, device="cuda"))
    assert dq.dapq_launch_count(ctx) == n0
    dq.dapq_destroy(ctx)


# ------------------------------------------------------ full-size configurations, sampled heads
@pytest.mark.parametrize("name,heads", [("llama3_8b_32k", (0, 3, 7)), ("qwen25_7b_128k", (2,)),
                                        ("batched_serving", (5,)), ("llama3_70b_128k", (6,))])
def test_evict_full_size_sampled_heads(dq, name, heads):
    """One layer of each benchmark configuration at its full size, through dapq_evict exactly as
    bench.py launches it; the oracle checks the sampled KV heads (all sequences of the batch)."""
    w = gi.workload(name)
    data = gi.draw_layer(w, 0, "cuda")
    ctx = _ctx(dq, w)
    # structure is planted with the library's own rotation, as in the benchmark
    q_rot = torch.empty_like(data["q_pre"])
    dq.dapq_rope_pseudo_q(ctx, data["q_pre"], list(w.prompt_lens), q_rot)
    torch.cuda.synchronize()
    gi.plant_structure(w, data, q_rot)
    got = _gpu_evict(dq, w, data, ctx)
    dq.dapq_destroy(ctx)
    G, N = w.group, w.n_pseudo
    cu_p, cu_k, cu_r = w.cu_prompt, w.cu_keep, w.cu_rows
    q64 = util.to_f64(data["q_pre"])
    for h in heads:
        k_h = data["k"][h].cpu()
        v_h = data["v"][h].cpu()
        k64 = util.to_f64(k_h)
        for b in range(w.batch):
            L, r0 = w.prompt_lens[b], int(cu_r[b])
            qr = orc.rope_pseudo_q(q64[b, h * G:(h + 1) * G], L, w.rope_base)
            ref = orc.score_sequence(qr, k64[None, r0:r0 + L + N], L, G)["scores"][0]
            ref_idx = orc.topk_select(ref, w.keep[b])
            tag = f"{name} b={b} kvh={h}"
            util.assert_scores_close(got["scores"][h, cu_p[b]:cu_p[b + 1]], ref, tag)
            gidx = got["idx"][h, cu_k[b]:cu_k[b + 1]]
            util.assert_index_sets_match(gidx, ref, ref_idx, L, tag)
            rows = torch.as_tensor(gidx.astype(np.int64) + r0)
            assert torch.equal(got["k_out"][h, cu_k[b]:cu_k[b + 1]], k_h[rows]), tag
            assert torch.equal(got["v_out"][h, cu_k[b]:cu_k[b + 1]], v_h[rows]), tag
            for p in (data["needle_pos"][b, h] if w.n_needles else []):
                assert int(p) in set(gidx.tolist()), f"{tag}: planted needle {p} evicted"


# ------------------------------------------------------------------ optional pooling
@pytest.mark.parametrize("mode,kernel", [("max", 7), ("avg", 5), ("max", 127), ("avg", 3)])
def test_pooled_selection_matches_oracle(dq, mode, kernel):
    code = dq.DAPQ_POOL_MAX if mode == "max" else dq.DAPQ_POOL_AVG
    w = gi.scaled_down("batched_serving", 16, n_layers=1)
    data = util.make_case(w)
    ref = orc.evict(util.to_f64(data["q_pre"]), util.to_f64(data["k"]), util.to_f64(data["v"]), w.cu_rows,
                    w.prompt_lens, w.keep, w.rope_base, pool_mode=mode, pool_kernel=kernel)
    ctx = _ctx(dq, w, pool_mode=code, pool_kernel=kernel)
    got = _gpu_evict(dq, w, data, ctx)
    cu_p, cu_k, cu_r = w.cu_prompt, w.cu_keep, w.cu_rows
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            tag = f"pool {mode}{kernel} b={b} kvh={h}"
            # the scores handed out stay the unpooled Eq. 4 sums
            util.assert_scores_close(got["scores"][h, cu_p[b]:cu_p[b + 1]], ref["scores"][b][h], tag)
            gidx = got["idx"][h, cu_k[b]:cu_k[b + 1]]
            util.assert_index_sets_match(gidx, ref["pooled"][b][h], ref["idx"][b][h], w.prompt_lens[b], tag)
            rows = torch.as_tensor(gidx.astype(np.int64) + int(cu_r[b]))
            assert torch.equal(got["k_out"][h, cu_k[b]:cu_k[b + 1]], data["k"][h].cpu()[rows]), tag
    # dapq_topk_select alone pools too: max pooling of fp32 scores is exact, so the sets are equal
    if mode == "max":
        rng = np.random.default_rng(9)
        s = rng.random((w.n_kv_heads, w.total_prompt)).astype(np.float32)
        idx = torch.empty((w.n_kv_heads, int(cu_k[-1])), dtype=torch.int32, device="cuda")
        dq.dapq_topk_select(ctx, torch.from_numpy(s).cuda(), cu_p, w.keep, idx)
        torch.cuda.synchronize()
        for b in range(w.batch):
            for h in range(w.n_kv_heads):
                pooled = orc.pool_scores(s[h, cu_p[b]:cu_p[b + 1]].astype(np.float64), kernel, "max")
                np.testing.assert_array_equal(idx[h, cu_k[b]:cu_k[b + 1]].cpu().numpy(), orc.topk_select(pooled, w.keep[b]))
    dq.dapq_destroy(ctx)


# ------------------------------------------------------------------ recall (Section 3.3, Eq. 1-3)
def test_recall_matches_oracle(dq):
    rng = np.random.default_rng(12)
    lens, keep = (900, 17, 5000), (64, 17, 1)
    w = _small(lens=lens, keep=keep, n_q_heads=4, n_kv_heads=2, n_pseudo=4, n_needles=0, outlier_channels=0)
    KT = int(w.cu_keep[-1])
    gold = np.zeros((2, KT), dtype=np.int32)
    pred = np.zeros((2, KT), dtype=np.int32)
    for h in range(2):
        for b, (L, K) in enumerate(zip(lens, keep)):
            sl = slice(int(w.cu_keep[b]), int(w.cu_keep[b + 1]))
            gold[h, sl] = np.sort(rng.choice(L, K, replace=False))
            pred[h, sl] = np.sort(rng.choice(L, K, replace=False)) if (h + b) % 2 else gold[h, sl]
    ctx = _ctx(dq, w)
    out = torch.full((3, 2), -1.0, dtype=torch.float32, device="cuda")
    dq.dapq_recall(ctx, torch.from_numpy(gold).cuda(), torch.from_numpy(pred).cuda(), lens, keep, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    for h in range(2):
        for b in range(3):
            sl = slice(int(w.cu_keep[b]), int(w.cu_keep[b + 1]))
            assert got[b, h] == pytest.approx(orc.recall(gold[h, sl], pred[h, sl]), abs=1e-7), (b, h)
    dq.dapq_destroy(ctx)


# ------------------------------------------------- caller-supplied RoPE frequencies, shifted positions
def test_evict_with_scaled_rope_frequencies(dq):
    """Frequencies of a scaled-RoPE model (long wavelengths divided by 8, as Llama-3.1 does) go in
    through inv_freq; the oracle rotates with the same table."""
    w = _small(lens=(900, 333), keep=(50, 20), n_q_heads=8, n_kv_heads=2, n_pseudo=32, n_needles=0)
    inv = orc.rope_inv_freq(128, w.rope_base)
    inv = np.where(2 * np.pi / inv > 8192, inv / 8.0, inv)
    data = gi.draw_layer(w, 0, "cpu")
    ref = orc.evict(util.to_f64(data["q_pre"]), util.to_f64(data["k"]), util.to_f64(data["v"]), w.cu_rows,
                    w.prompt_lens, w.keep, w.rope_base, inv_freq=inv)
    plain = util.oracle_evict(w, data)
    assert not np.allclose(ref["scores"][0], plain["scores"][0], rtol=1e-3)       # the table matters
    ctx = _ctx(dq, w, inv_freq=list(inv))
    _check_evict(w, data, _gpu_evict(dq, w, data, ctx), ref)
    dq.dapq_destroy(ctx)


def test_evict_with_interleaved_rope_pairs(dq):
    """DAPQ_FLAG_ROPE_INTERLEAVED through the whole path, on the tensor cores and on the CUDA cores."""
    w = _small(lens=(800, 77), keep=(60, 9), n_q_heads=8, n_kv_heads=2, n_pseudo=32, n_needles=0)
    data = gi.draw_layer(w, 0, "cpu")
    ref = orc.evict(util.to_f64(data["q_pre"]), util.to_f64(data["k"]), util.to_f64(data["v"]), w.cu_rows,
                    w.prompt_lens, w.keep, w.rope_base, rope_interleaved=True)
    assert not np.allclose(ref["scores"][0], util.oracle_evict(w, data)["scores"][0], rtol=1e-3)   # the pairing matters
    for extra in (0, dq.DAPQ_FLAG_CUDA_CORE_SCORER):
        ctx = _ctx(dq, w, flags=dq.DAPQ_FLAG_ROPE_INTERLEAVED | extra)
        _check_evict(w, data, _gpu_evict(dq, w, data, ctx), ref)
        dq.dapq_destroy(ctx)


def test_shifted_positions_through_rope_and_score(dq):
    """The paper's position ablation (Section 6.3: pseudo queries placed at L_p + offset) through the
    separate entry points: dapq_rope_pseudo_q with pos_start = L_b + offset, then dapq_score."""
    w = _small(lens=(700,), keep=(1,), n_q_heads=8, n_kv_heads=2, n_pseudo=32, n_needles=0)
    data = gi.draw_layer(w, 0, "cpu")
    offset = 4096
    ctx = _ctx(dq, w)
    q_rot = torch.empty_like(data["q_pre"]).cuda()
    dq.dapq_rope_pseudo_q(ctx, data["q_pre"].cuda(), [700 + offset], q_rot)
    scores = torch.empty((2, 700), dtype=torch.float32, device="cuda")
    dq.dapq_score(ctx, q_rot, data["k"].cuda(), w.cu_rows, w.prompt_lens, scores)
    dq.dapq_poll_status(ctx)
    # both sides score the rotated queries as stored (bf16)
    q_ref = util.to_f64(q_rot[0])
    ref = orc.score_sequence(q_ref, util.to_f64(data["k"]), 700, w.group)["scores"]
    util.assert_scores_close(scores.cpu().double().numpy(), ref, "shifted positions")
    want = orc.rope_pseudo_q(util.to_f64(data["q_pre"][0]), 700 + offset, w.rope_base)
    assert np.all(np.abs(q_ref - want) <= 2.0 ** -8 * np.abs(want) + 1e-7)
    dq.dapq_destroy(ctx)


# ------------------------------------------------------------- every layer in one call, budgets per layer
def _layer_cases(n_layers, lens, budgets, **kw):
    ws = [_small(lens=lens, keep=budgets[l], **kw) for l in range(n_layers)]
    return ws, [gi.draw_layer(ws[l], l, "cpu") for l in range(n_layers)]


def _layer_buffers(ws, datas):
    dev = "cuda"
    q, k, v = ([d[x].to(dev) for d in datas] for x in ("q_pre", "k", "v"))
    ko = [torch.empty((w.n_kv_heads, int(w.cu_keep[-1]), w.head_dim), dtype=k[0].dtype, device=dev) for w in ws]
    vo = [torch.empty_like(t) for t in ko]
    idx = [torch.empty((w.n_kv_heads, int(w.cu_keep[-1])), dtype=torch.int32, device=dev) for w in ws]
    return q, k, v, ko, vo, idx


def test_evict_layers_with_per_layer_budgets(dq):
    """dapq_evict_layers with a budget row per layer (layer-wise budgets as in the PyramidKV baseline of
    Section 5.1): every layer equals its own dapq_evict call bit for bit and the oracle's retained set."""
    lens, budgets = (600, 210), [(60, 21), (120, 40), (17, 3)]
    ws, datas = _layer_cases(3, lens, budgets, n_q_heads=8, n_kv_heads=2, n_pseudo=32, n_needles=0)
    q, k, v, ko, vo, idx = _layer_buffers(ws, datas)
    ctx = _ctx(dq, ws[0])
    dq.dapq_evict_layers(ctx, q, k, v, ws[0].cu_rows, ws[0].prompt_lens, budgets, ko, vo, idx)
    dq.dapq_poll_status(ctx)
    for l, (w, data) in enumerate(zip(ws, datas)):
        one = _gpu_evict(dq, w, data, ctx)
        assert np.array_equal(idx[l].cpu().numpy(), one["idx"]), f"layer {l}"
        assert torch.equal(ko[l].cpu(), one["k_out"]) and torch.equal(vo[l].cpu(), one["v_out"]), f"layer {l}"
        _check_evict(w, data, one, util.oracle_evict(w, data))
    # one budget row shared by all layers
    ws1, datas1 = _layer_cases(2, lens, [budgets[0]] * 2, n_q_heads=8, n_kv_heads=2, n_pseudo=32, n_needles=0)
    q, k, v, ko, vo, idx = _layer_buffers(ws1, datas1)
    dq.dapq_evict_layers(ctx, q, k, v, ws1[0].cu_rows, ws1[0].prompt_lens, budgets[0], ko, vo, idx)
    dq.dapq_poll_status(ctx)
    for l, (w, data) in enumerate(zip(ws1, datas1)):
        assert np.array_equal(idx[l].cpu().numpy(), _gpu_evict(dq, w, data, ctx)["idx"]), f"shared budgets, layer {l}"
    dq.dapq_destroy(ctx)


def test_evict_layers_replays_from_a_cuda_graph(dq):
    """The multi-layer call only issues launches, so it can be captured once and replayed on new cache
    contents: the replay equals an eager call on the same contents."""
    lens, budgets = (500, 1300), [(50, 130)] * 3
    ws, datas = _layer_cases(3, lens, budgets, n_needles=0)
    q, k, v, ko, vo, idx = _layer_buffers(ws, datas)
    ctx = _ctx(dq, ws[0])
    args = (ws[0].cu_rows, ws[0].prompt_lens, budgets[0])
    dq.dapq_evict_layers(ctx, q, k, v, *args, ko, vo, idx)                  # warm-up outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        dq.dapq_evict_layers(ctx, q, k, v, *args, ko, vo, idx)
    # new contents in the captured buffers: the layers of another draw
    fresh = [gi.draw_layer(ws[l], l + 7, "cpu") for l in range(3)]
    for l in range(3):
        for dst, name in ((q, "q_pre"), (k, "k"), (v, "v")):
            dst[l].copy_(fresh[l][name])
        ko[l].zero_(); vo[l].zero_(); idx[l].zero_()
    graph.replay()
    torch.cuda.synchronize()
    dq.dapq_poll_status(ctx)
    for l in range(3):
        one = _gpu_evict(dq, ws[l], fresh[l], ctx)
        assert np.array_equal(idx[l].cpu().numpy(), one["idx"]), f"layer {l}"
        assert torch.equal(ko[l].cpu(), one["k_out"]) and torch.equal(vo[l].cpu(), one["v_out"]), f"layer {l}"
    dq.dapq_destroy(ctx)


# --------------------------------------------------- observation window taken from the prompt itself
def test_prompt_window_variant_uses_the_same_entry_points(dq):
    """The SnapKV-style window of Section 5.1's baselines (queries = the last N prompt tokens, query i sees
    keys up to its own position, window rows always kept) is the same computation with prompt_len = L - N:
    the window's rows play the part of the synthetic rows.  Reference: the oracle's score_prompt_window."""
    L, N, hq, hkv, keep = 1500, 32, 8, 2, 200
    w = _small(lens=(L - N,), keep=(keep - N,), n_q_heads=hq, n_kv_heads=hkv, n_pseudo=N, n_needles=0)
    data = gi.draw_layer(w, 0, "cpu")                            # k: [H_kv, L, d]; q_pre stands for the window's rotated queries
    q_win, k = data["q_pre"], data["k"]
    assert k.shape[1] == L
    ref = torch.from_numpy(orc.score_prompt_window(util.to_f64(q_win[0]), util.to_f64(k), hq // hkv))
    ctx = _ctx(dq, w)
    scores = torch.empty((hkv, L - N), dtype=torch.float32, device="cuda")
    dq.dapq_score(ctx, q_win.cuda(), k.cuda(), w.cu_rows, w.prompt_lens, scores)
    idx = torch.empty((hkv, keep - N), dtype=torch.int32, device="cuda")
    dq.dapq_topk_select(ctx, scores, w.cu_prompt, w.keep, idx)
    dq.dapq_poll_status(ctx)
    util.assert_scores_close(scores.cpu().double().numpy(), ref.numpy(), "prompt window")
    for h in range(hkv):
        ref_idx = np.sort(np.argsort(-ref[h].numpy(), kind="stable")[:keep - N])
        util.assert_index_sets_match(idx[h].cpu().numpy(), ref[h].numpy(), ref_idx, L - N, f"window kvh={h}")
        kept = np.concatenate([idx[h].cpu().numpy(), np.arange(L - N, L)])      # the caller appends the window rows
        assert len(np.unique(kept)) == keep
    dq.dapq_destroy(ctx)


# ------------------------------------------------------------------- seeded random shapes, end to end
def _random_cases(n_cases, seed=20260311):
    rng = np.random.default_rng(seed)
    cases = []
    for _ in range(n_cases):
        hkv = int(rng.choice([1, 2, 4, 8]))
        group = int(rng.choice([1, 2, 4, 7, 8]))
        n = int(rng.choice([1, 3, 16, 17, 32, 33, 64, 100, 128]))
        batch = int(rng.integers(1, 5))
        lens = tuple(int(x) for x in np.maximum(1, (rng.pareto(1.2, batch) * 150).astype(np.int64) % 2600 + rng.integers(1, 40, batch)))
        keep = tuple(int(rng.integers(1, L + 1)) for L in lens)
        dtype = "bf16" if rng.random() < 0.75 else "f32"
        cases.append((dtype, hkv * group, hkv, n, lens, keep))
    return cases


@pytest.mark.parametrize("dtype,hq,hkv,n,lens,keep", _random_cases(16))
def test_evict_random_shapes(dq, dtype, hq, hkv, n, lens, keep):
    """Seeded random head counts, window sizes, ragged batches and budgets through the whole path (both
    scorers, both geometries of the tensor-core sweeps, every top-k cluster size that these lengths reach)."""
    w = _small(lens=lens, keep=keep, dtype=dtype, n_q_heads=hq, n_kv_heads=hkv, n_pseudo=n, n_needles=0,
               outlier_channels=2 if dtype == "bf16" else 0)
    data = gi.draw_layer(w, 0, "cpu")
    _check_evict(w, data, _gpu_evict(dq, w, data), util.oracle_evict(w, data))


@pytest.mark.parametrize("hq,n", [(3, 100), (5, 104), (7, 64), (6, 128)])
def test_evict_more_than_256_query_rows_per_kv_head(dq, hq, n):
    """300, 520, 448 and 768 query rows on one KV head: sweep 1 cuts them into groups of up to 256 rows, sweep 2
    into groups of up to 512 whose second job is 48, 16, 192 or 128 columns wide (default fp16 queries)."""
    w = _small(lens=(900, 130, 1), keep=(90, 130, 1), dtype="bf16", n_q_heads=hq, n_kv_heads=1, n_pseudo=n, n_needles=0,
               outlier_channels=2)
    data = gi.draw_layer(w, 0, "cpu")
    _check_evict(w, data, _gpu_evict(dq, w, data), util.oracle_evict(w, data))


def test_evict_largest_batch(dq):
    """DAPQ_MAX_BATCH sequences in one call (1 to 300 tokens each, some keeping every row)."""
    rng = np.random.default_rng(77)
    lens = tuple(int(x) for x in rng.integers(1, 301, 128))
    keep = tuple(int(min(L, max(1, rng.integers(1, 2 * L)))) for L in lens)
    w = _small(lens=lens, keep=keep, n_q_heads=8, n_kv_heads=2, n_pseudo=16, n_needles=0)
    data = gi.draw_layer(w, 0, "cpu")
    _check_evict(w, data, _gpu_evict(dq, w, data), util.oracle_evict(w, data))


# ----------------------------------------------------------------- precision of the query operand
@pytest.mark.parametrize("name,heads,bound", [("llama3_8b_32k", (0, 3), 1e-3), ("llama3_70b_128k", (6,), 1e-3)])
def test_default_precision_full_size_within_half_the_budget(dq, name, heads, bound):
    """The default query precision (fp16, K converted on the fly) keeps the worst per-token error of the two
    configurations with outlier channels, at full size, below 1e-3: half of the 2e-3 budget."""
    w = gi.workload(name)
    data = gi.draw_layer(w, 0, "cuda")
    ctx = _ctx(dq, w)
    q_rot = torch.empty_like(data["q_pre"])
    dq.dapq_rope_pseudo_q(ctx, data["q_pre"], list(w.prompt_lens), q_rot)
    torch.cuda.synchronize()
    gi.plant_structure(w, data, q_rot)
    got = _gpu_evict(dq, w, data, ctx)["scores"]
    dq.dapq_destroy(ctx)
    G, N, L = w.group, w.n_pseudo, w.prompt_lens[0]
    q64 = util.to_f64(data["q_pre"])
    for h in heads:
        qr = orc.rope_pseudo_q(q64[0, h * G:(h + 1) * G], L, w.rope_base)
        ref = orc.score_sequence(qr, util.to_f64(data["k"][h].cpu())[None, :L + N], L, G)["scores"][0]
        worst = float(np.max(np.abs(got[h] - ref) / ref))
        assert worst < bound, f"{name} kvh={h}: worst relative error {worst:.3e}"


# ----------------------------------------------------------------------- Llama-3.1 scaled RoPE
def test_evict_with_llama31_rope_preset(dq):
    """The frequency table of Llama-3.1's long-context scaling (the model of the paper's efficiency runs),
    produced by the library's helper, through the whole path; the oracle rotates with its own statement
    of the same rule."""
    w = _small(lens=(1200, 410), keep=(60, 25), n_q_heads=8, n_kv_heads=2, n_pseudo=32, n_needles=0, rope_base=5.0e5)
    inv = np.array(dq.dapq_rope_inv_freq_llama3(5.0e5, 8.0, 1.0, 4.0, 8192))
    ref_inv = orc.rope_inv_freq_llama3(128, 5.0e5, 8.0, 1.0, 4.0, 8192)
    np.testing.assert_allclose(inv, ref_inv, rtol=1e-14)
    data = gi.draw_layer(w, 0, "cpu")
    ref = orc.evict(util.to_f64(data["q_pre"]), util.to_f64(data["k"]), util.to_f64(data["v"]), w.cu_rows,
                    w.prompt_lens, w.keep, w.rope_base, inv_freq=ref_inv)
    assert not np.allclose(ref["scores"][0], util.oracle_evict(w, data)["scores"][0], rtol=1e-3)   # the scaling matters
    for flags in (0, dq.DAPQ_FLAG_CUDA_CORE_SCORER):
        ctx = _ctx(dq, w, inv_freq=list(inv), flags=flags)
        _check_evict(w, data, _gpu_evict(dq, w, data, ctx), ref)
        dq.dapq_destroy(ctx)


# ------------------------------------------------------------ the call the benchmark times, at full size
def test_evict_layers_full_size_sampled_heads(dq):
    """Two layers of the Llama-3-8B-shaped cache at full size through dapq_evict_layers (the call bench.py
    steps through), sampled KV heads against the oracle."""
    w = gi.workload("llama3_8b_32k")
    ctx = _ctx(dq, w)
    datas = []
    for l in range(2):
        d = gi.draw_layer(w, l, "cuda")
        q_rot = torch.empty_like(d["q_pre"])
        dq.dapq_rope_pseudo_q(ctx, d["q_pre"], list(w.prompt_lens), q_rot)
        torch.cuda.synchronize()
        gi.plant_structure(w, d, q_rot)
        datas.append(d)
    KT, L, G, N = int(w.cu_keep[-1]), w.prompt_lens[0], w.group, w.n_pseudo
    ko = [torch.empty((w.n_kv_heads, KT, 128), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    vo = [torch.empty_like(t) for t in ko]
    idx = [torch.empty((w.n_kv_heads, KT), dtype=torch.int32, device="cuda") for _ in range(2)]
    dq.dapq_evict_layers(ctx, [d["q_pre"] for d in datas], [d["k"] for d in datas], [d["v"] for d in datas], w.cu_rows,
                         w.prompt_lens, w.keep, ko, vo, idx)
    dq.dapq_poll_status(ctx)
    dq.dapq_destroy(ctx)
    for l, h in ((0, 2), (1, 5)):
        d = datas[l]
        k_h, v_h = d["k"][h].cpu(), d["v"][h].cpu()
        qr = orc.rope_pseudo_q(util.to_f64(d["q_pre"])[0, h * G:(h + 1) * G], L, w.rope_base)
        ref = orc.score_sequence(qr, util.to_f64(k_h)[None, :L + N], L, G)["scores"][0]
        gidx = idx[l][h].cpu().numpy()
        util.assert_index_sets_match(gidx, ref, orc.topk_select(ref, w.keep[0]), L, f"layer {l} kvh={h}")
        rows = torch.as_tensor(gidx.astype(np.int64))
        assert torch.equal(ko[l][h].cpu(), k_h[rows]) and torch.equal(vo[l][h].cpu(), v_h[rows])
        for p in d["needle_pos"][0, h]:
            assert int(p) in set(gidx.tolist())


# ------------------------------------------------------------------ a device-side wait that runs out
@pytest.mark.parametrize("flags", [0, 8 | 16])
def test_wait_limit_gives_up_reports_timeout_and_recovers(dq, flags):
    """With the wait bound set to one cycle, the first wait of every score CTA that is not satisfied at once
    runs out: the kernels return normally, dapq_poll_status reports DAPQ_ERR_TIMEOUT once and clears the
    status word, and the same context then computes the right answer again.  Both tensor-core scorers (flags 0:
    fp16 queries; 8 | 16: the older kernels with the two-part bf16 operand)."""
    w = gi.scaled_down("llama3_8b_32k", 8, n_layers=1)
    data = util.make_case(w)
    ref = util.oracle_evict(w, data)
    ctx = _ctx(dq, w, flags=flags)
    good = _gpu_evict(dq, w, data, ctx)
    dq.dapq_set_wait_limit(ctx, 1)
    q, k, v = (data[x].cuda() for x in ("q_pre", "k", "v"))
    KT = int(w.cu_keep[-1])
    k_out = torch.empty((w.n_kv_heads, KT, 128), dtype=torch.bfloat16, device="cuda")
    v_out = torch.empty_like(k_out)
    dq.dapq_evict(ctx, q, k, v, w.cu_rows, w.prompt_lens, w.keep, k_out, v_out)
    with pytest.raises(dq.DapqError) as e:
        dq.dapq_poll_status(ctx)
    assert e.value.status == dq.DAPQ_ERR_TIMEOUT
    dq.dapq_poll_status(ctx)                                     # the word was cleared by the poll above
    dq.dapq_set_wait_limit(ctx, 0)
    again = _gpu_evict(dq, w, data, ctx)
    np.testing.assert_array_equal(again["scores"], good["scores"])
    np.testing.assert_array_equal(again["idx"], good["idx"])
    _check_evict(w, data, again, ref)
    dq.dapq_destroy(ctx)


# --------------------------------------------------- logits far from the row's reference (sweep 1)
@pytest.mark.parametrize("where", [3, 700, 1290])
def test_logits_far_above_and_below_the_first_key(dq, where):
    """Sweep 1 measures every logit of a row against the row's logit for the first key of the sequence and sums
    2^(difference) without tracking a maximum; a key whose logit lies more than the float range above that
    reference has to take the careful per-job path.  One key aligned with a query (logit about +150 for that
    row, tens above or below the bulk for the others), early, in the middle and among the last tiles."""
    w = _small(lens=(1300,), keep=(40,), n_q_heads=8, n_kv_heads=2, n_pseudo=64, n_needles=0, outlier_channels=0)
    data = gi.draw_layer(w, 0, "cpu")
    q_rot = util.oracle_q_rot(w, data)[0]                               # [H_q, N, d] float64
    for h in range(w.n_kv_heads):
        u = q_rot[h * w.group + 1, 7]
        data["k"][h, where] = (150.0 * np.sqrt(128.0) * u / (u.norm() ** 2)).to(torch.bfloat16)
    ref = util.oracle_evict(w, data)
    lg = (q_rot[1] @ data["k"][0].double().T) / np.sqrt(128.0)
    assert float(lg[7, where] - lg[7, 0]) > 120.0                        # beyond 2^127 in base 2 for that row
    for flags in (0, dq.DAPQ_FLAG_Q_LO_SWEEP1 | dq.DAPQ_FLAG_Q_LO_SWEEP2):
        ctx = _ctx(dq, w, flags=flags)
        _check_evict(w, data, _gpu_evict(dq, w, data, ctx), ref)
        dq.dapq_destroy(ctx)
