"""CPU checks of the boundary: the library loads, exports every declared symbol, and
rejects bad shapes before touching a device (no compute calls here)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__ as ge
    ge.build()
    import paper_2603_11564_b200 as pkg
    return pkg


def _declared():
    text = open(os.path.join(ROOT, "include", "dapq.h")).read()
    return sorted(set(re.findall(r"DAPQ_API[^;(]*?\b(dapq_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 11
    cdll = lib.load_library()
    for n in names:
        assert hasattr(cdll, n), n
    assert sorted(lib.EXPORTS) == names
    for n in names:                      # the binding carries the same names
        assert callable(getattr(lib, n))


def test_struct_layouts_match_the_header(lib):
    assert C.sizeof(lib.dapq_shape) == 64
    assert lib.dapq_shape.max_total_rows.offset == 24 and lib.dapq_shape.inv_freq_host.offset == 40
    assert C.sizeof(lib.dapq_cache_view) == 72 and lib.dapq_cache_view.batch.offset == 64


@pytest.mark.parametrize("kw,status", [
    (dict(head_dim=64), 2), (dict(n_pseudo=129), 2), (dict(n_pseudo=0), 2), (dict(n_kv_heads=3), 1),
    (dict(max_batch=0), 1), (dict(max_batch=129), 2), (dict(dtype=7), 1), (dict(rope_base=0.0), 1),
    (dict(softmax_scale=-1.0), 1), (dict(max_total_rows=0), 1), (dict(pool_mode=5), 1),
    (dict(pool_mode=1, pool_kernel=4), 2), (dict(pool_mode=2, pool_kernel=129), 2), (dict(flags=32), 1),
])
def test_create_rejects_bad_shapes_without_a_device(lib, kw, status):
    args = dict(n_q_heads=8, n_kv_heads=2, n_pseudo=32, max_batch=1, max_total_rows=1000, dtype=0, rope_base=1e4)
    args.update(kw)
    with pytest.raises(lib.DapqError) as e:
        lib.dapq_create(**args)
    assert e.value.status == status
    assert "dapq_create" in str(e.value)


def test_null_context_is_an_error_not_a_crash(lib):
    cdll = lib.load_library()
    assert cdll.dapq_poll_status(None, None) == lib.DAPQ_ERR_INVALID_ARG
    assert cdll.dapq_launch_count(None) == 0
    assert cdll.dapq_evict_layers(None, 0, None, None, None, 0, None, None, None, None) == lib.DAPQ_ERR_INVALID_ARG
    assert cdll.dapq_evict_layers_host(None, 0, None, None, None, 0, None, None, None, None) == lib.DAPQ_ERR_INVALID_ARG
    cdll.dapq_destroy(None)


def test_llama3_frequency_helper_matches_the_oracle(lib):
    """Host arithmetic of the C helper against the oracle's statement of the published rule."""
    import numpy as np
    from oracle import dapq_oracle as orc
    for args in [(5.0e5, 8.0, 1.0, 4.0, 8192), (1.0e4, 32.0, 1.0, 4.0, 8192), (1.0e6, 4.0, 2.0, 8.0, 4096)]:
        got = np.array(lib.dapq_rope_inv_freq_llama3(*args))
        np.testing.assert_allclose(got, orc.rope_inv_freq_llama3(128, *args), rtol=1e-14)
    with pytest.raises(lib.DapqError):
        lib.dapq_rope_inv_freq_llama3(5.0e5, 8.0, 4.0, 1.0, 8192)       # high must exceed low
