"""dapq_score_static: the scorer for callers that cannot allocate device memory (no context,
scratch in a fixed array inside the library).  Its scores must equal those of the ordinary
dapq_score entry point and lie within the oracle's tolerance, call after call, although every
call reuses the same scratch area; and after the first (warm-up) call on a device no later call
may take device memory, whatever its shape or dtype.  Collected last on purpose: a failure here
never hides another test."""
import numpy as np
import pytest
import torch

from gen import inputs as gi
from oracle import dapq_oracle as orc
from tests import util


def _case(seed, lens, n_pseudo, hq, hkv, dtype):
    w = gi.workload("llama3_8b_32k", prompt_lens=tuple(lens), keep=tuple(1 for _ in lens), n_layers=1,
                    n_q_heads=hq, n_kv_heads=hkv, n_pseudo=n_pseudo, dtype=dtype, seed=seed, n_needles=0,
                    outlier_channels=0)
    data = gi.draw_layer(w, 0, "cpu")
    q_rot = util.oracle_q_rot(w, data).to(w.torch_dtype())
    return w, data, q_rot


def _static(dq, L, hq=32, hkv=8, n=64):
    """Call the entry point with tensors that are never touched (the call is refused before any launch)."""
    dq.dapq_score_static(hq, hkv, n, dq.DAPQ_BF16, torch.zeros(8, dtype=torch.bfloat16),
                         torch.zeros((hkv, 1, 128), dtype=torch.bfloat16), [0, L + n], [L], torch.zeros(64), stream=0)


def test_size_limit_is_rejected_without_a_device():
    import paper_2603_11564_b200 as dq
    dq.load_library()
    # 1M prompt tokens at H_q = 32, N = 64 need far more than the fixed 2 MiB of scratch
    with pytest.raises(dq.DapqError) as e:
        _static(dq, 1 << 20)
    assert e.value.status == dq.DAPQ_ERR_WORKSPACE and "scratch" in str(e.value)
    # the documented edge: 64512 tokens is the longest single prompt that fits at H_q = 32, N = 64; one
    # token more needs another chunk of partials (8192 + 128 * 16384 bytes > 2 MiB)
    with pytest.raises(dq.DapqError) as e:
        _static(dq, 64513)
    assert e.value.status == dq.DAPQ_ERR_WORKSPACE
    with pytest.raises(dq.DapqError) as e:
        _static(dq, 65536)
    assert e.value.status == dq.DAPQ_ERR_WORKSPACE


@pytest.mark.gpu
def test_static_scorer_matches_dapq_score_and_the_oracle_twice_in_a_row():
    import paper_2603_11564_b200 as dq
    dq.load_library()
    # two different problems back to back: the second must not see the first one's partials
    cases = [_case(11, (1500, 70), 32, 8, 2, "bf16"), _case(12, (300,), 17, 4, 4, "f32")]
    mem = None
    for rep in range(2):
        for w, data, q_rot in cases:
            code = dq.DAPQ_BF16 if w.dtype == "bf16" else dq.DAPQ_F32
            q, k = q_rot.cuda(), data["k"].cuda()
            got = torch.full((w.n_kv_heads, w.total_prompt), -1.0, dtype=torch.float32, device="cuda")
            ref = torch.empty_like(got)
            torch.cuda.synchronize()
            if mem is not None:
                # (free device memory as the driver sees it, and what torch's caching allocator holds: the
                # former moves when anybody in this process allocates from the driver)
                mem = (torch.cuda.mem_get_info()[0], torch.cuda.memory_reserved())
            dq.dapq_score_static(w.n_q_heads, w.n_kv_heads, w.n_pseudo, code, q, k, w.cu_rows, w.prompt_lens, got)
            torch.cuda.synchronize()
            if mem is not None:
                # after the warm-up call no call takes device memory, also not one of another shape and dtype
                # (which runs other kernel instantiations)
                assert (torch.cuda.mem_get_info()[0], torch.cuda.memory_reserved()) == mem, (rep, w.dtype)
            mem = True
            # the existing entry point, kept on the same CUDA-core kernels
            ctx = dq.dapq_create(w.n_q_heads, w.n_kv_heads, w.n_pseudo, w.batch, w.total_rows, code, w.rope_base,
                                 flags=dq.DAPQ_FLAG_CUDA_CORE_SCORER)
            dq.dapq_score(ctx, q, k, w.cu_rows, w.prompt_lens, ref)
            dq.dapq_poll_status(ctx)
            dq.dapq_destroy(ctx)
            g, r = got.cpu().double().numpy(), ref.cpu().double().numpy()
            k64 = util.to_f64(data["k"])
            for h in range(w.n_kv_heads):
                util.assert_scores_close(g[h], r[h], f"rep {rep} {w.dtype} kvh={h}")
            for b in range(w.batch):
                want = orc.score_sequence(util.to_f64(q_rot[b]), k64[:, int(w.cu_rows[b]):int(w.cu_rows[b + 1])],
                                          w.prompt_lens[b], w.group)["scores"]
                util.assert_scores_close(g[:, w.cu_prompt[b]:w.cu_prompt[b + 1]], want, f"rep {rep} {w.dtype} b={b} vs oracle")
            assert np.all(g > 0)


@pytest.mark.gpu
def test_static_scorer_just_under_the_scratch_limit():
    """A prompt of 64000 tokens at H_q = 32, N = 64 needs 8192 + 126 * 16384 bytes: all but one chunk of the
    fixed area, so the launcher cannot cut the work finer than 512-key chunks.  One KV head against the oracle."""
    import paper_2603_11564_b200 as dq
    dq.load_library()
    w, data, q_rot = _case(13, (64000,), 64, 32, 8, "bf16")
    q, k = q_rot.cuda(), data["k"].cuda()
    got = torch.empty((w.n_kv_heads, w.total_prompt), dtype=torch.float32, device="cuda")
    dq.dapq_score_static(w.n_q_heads, w.n_kv_heads, w.n_pseudo, dq.DAPQ_BF16, q, k, w.cu_rows, w.prompt_lens, got)
    torch.cuda.synchronize()
    h, G = 5, w.group
    want = orc.score_sequence(util.to_f64(q_rot[0, h * G:(h + 1) * G]), util.to_f64(data["k"][h:h + 1]), 64000, G)["scores"][0]
    util.assert_scores_close(got[h].cpu().double().numpy(), want, "near the scratch limit")
