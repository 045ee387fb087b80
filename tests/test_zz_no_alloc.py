"""dapq_score_static: the scorer for callers that cannot allocate device memory (no context,
scratch in a fixed array inside the library).  Its scores must equal those of the ordinary
dapq_score entry point on the same inputs, call after call, although every call reuses the
same scratch area.  Collected last on purpose: a failure here never hides another test."""
import numpy as np
import pytest
import torch

from gen import inputs as gi
from tests import util


def _case(seed, lens, n_pseudo, hq, hkv, dtype):
    w = gi.workload("llama3_8b_32k", prompt_lens=tuple(lens), keep=tuple(1 for _ in lens), n_layers=1,
                    n_q_heads=hq, n_kv_heads=hkv, n_pseudo=n_pseudo, dtype=dtype, seed=seed, n_needles=0,
                    outlier_channels=0)
    data = gi.draw_layer(w, 0, "cpu")
    q_rot = util.oracle_q_rot(w, data).to(w.torch_dtype())
    return w, data, q_rot


def test_size_limit_is_rejected_without_a_device():
    import paper_2603_11564_b200 as dq
    dq.load_library()
    # 1M prompt tokens at H_q = 32, N = 64 need far more than the fixed 2 MiB of scratch
    L = 1 << 20
    k = torch.zeros(64)             # never touched: the call is refused before anything is launched
    with pytest.raises(dq.DapqError) as e:
        dq.dapq_score_static(32, 8, 64, dq.DAPQ_BF16, torch.zeros(8, dtype=torch.bfloat16),
                             torch.zeros((8, 1, 128), dtype=torch.bfloat16), [0, L + 64], [L], k, stream=0)
    assert e.value.status == dq.DAPQ_ERR_WORKSPACE and "scratch" in str(e.value)


@pytest.mark.gpu
def test_static_scorer_matches_dapq_score_twice_in_a_row():
    import paper_2603_11564_b200 as dq
    dq.load_library()
    # two different problems back to back: the second must not see the first one's partials
    cases = [_case(11, (1500, 70), 32, 8, 2, "bf16"), _case(12, (300,), 17, 4, 4, "f32")]
    for rep in range(2):
        for w, data, q_rot in cases:
            code = dq.DAPQ_BF16 if w.dtype == "bf16" else dq.DAPQ_F32
            q, k = q_rot.cuda(), data["k"].cuda()
            got = torch.full((w.n_kv_heads, w.total_prompt), -1.0, dtype=torch.float32, device="cuda")
            dq.dapq_score_static(w.n_q_heads, w.n_kv_heads, w.n_pseudo, code, q, k, w.cu_rows, w.prompt_lens, got)
            torch.cuda.synchronize()
            # the existing entry point, kept on the same CUDA-core kernels
            ctx = dq.dapq_create(w.n_q_heads, w.n_kv_heads, w.n_pseudo, w.batch, w.total_rows, code, w.rope_base,
                                 flags=dq.DAPQ_FLAG_CUDA_CORE_SCORER)
            ref = torch.empty_like(got)
            dq.dapq_score(ctx, q, k, w.cu_rows, w.prompt_lens, ref)
            dq.dapq_poll_status(ctx)
            dq.dapq_destroy(ctx)
            g, r = got.cpu().double().numpy(), ref.cpu().double().numpy()
            for h in range(w.n_kv_heads):
                util.assert_scores_close(g[h], r[h], f"rep {rep} {w.dtype} kvh={h}")
            assert np.all(g > 0)
