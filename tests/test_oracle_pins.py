"""CPU pins for the oracle: every oracle function is checked against something other
than itself - a library routine, a closed form, an invariant, a hand-worked case or
brute force on tiny inputs - before any CUDA result is compared with it."""
import math

import numpy as np
import pytest
import torch

from oracle import dapq_oracle as orc


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


# ------------------------------------------------------------------ RoPE (Section 4.1)
def test_rope_quarter_and_half_turns():
    # Plane rotations by 90 and 180 degrees have exact images: pair (1,3) -> (-3,1),
    # pair (2,4) -> (-2,-4).  Pairs are (c, c + d/2).
    q = np.array([[1.0, 2.0, 3.0, 4.0]])
    out = orc.rope_pseudo_q(q, pos_start=1, rope_base=1.0,
                            inv_freq=np.array([math.pi / 2, math.pi]))
    np.testing.assert_allclose(out, [[-3.0, -2.0, 1.0, -4.0]], atol=1e-14)


def test_rope_positions_advance_by_one_per_pseudo_query():
    # Query i sits at pos_start + i: with theta = pi/2 and q = e_0 the four queries
    # at positions 4,5,6,7 point along +x, +y, -x, -y of the (0, 1) pair.
    q = np.tile(np.array([[1.0, 0.0]]), (4, 1))
    out = orc.rope_pseudo_q(q, pos_start=4, rope_base=1.0, inv_freq=np.array([math.pi / 2]))
    np.testing.assert_allclose(out, [[1, 0], [0, 1], [-1, 0], [0, -1]], atol=1e-14)


def test_rope_inv_freq_closed_form():
    # base^(-2c/d): for d = 8, base = 10^4 the frequencies are 1, 0.1, 0.01, 0.001.
    np.testing.assert_allclose(orc.rope_inv_freq(8, 1.0e4), [1.0, 0.1, 0.01, 0.001], rtol=1e-14)


def test_rope_matches_transformers_llama():
    tf = pytest.importorskip("transformers.models.llama.modeling_llama")
    from transformers import LlamaConfig
    d, n, pos0 = 16, 5, 37
    cfg = LlamaConfig(hidden_size=4 * d, num_attention_heads=4, head_dim=d, rope_theta=5.0e5)
    rot = tf.LlamaRotaryEmbedding(cfg)
    q = _rand((1, 4, n, d), 1)
    qt = torch.from_numpy(q)
    cos, sin = rot(qt, torch.arange(pos0, pos0 + n)[None])
    lib, _ = tf.apply_rotary_pos_emb(qt, qt, cos.double(), sin.double())
    mine = orc.rope_pseudo_q(q[0], pos0, 5.0e5)
    # the library builds its table in float32
    np.testing.assert_allclose(mine, lib[0].numpy(), atol=2e-5)


def test_llama3_scaled_frequencies_match_transformers_and_the_rule():
    """rope_inv_freq_llama3 against the library routine for the "llama3" rope type, and against what
    the rule fixes by itself: fast channels untouched, slow channels divided by the factor, the band
    in between strictly inside the two, frequencies still decreasing."""
    ru = pytest.importorskip("transformers.modeling_rope_utils")
    from transformers import LlamaConfig
    for d, base, factor, lo, hi, orig in [(128, 5.0e5, 8.0, 1.0, 4.0, 8192), (64, 1.0e4, 32.0, 1.0, 4.0, 8192),
                                          (128, 1.0e6, 4.0, 2.0, 8.0, 4096)]:
        cfg = LlamaConfig(hidden_size=4 * d, num_attention_heads=4, head_dim=d, rope_theta=base,
                          max_position_embeddings=16 * orig,
                          rope_scaling={"rope_type": "llama3", "factor": factor, "low_freq_factor": lo,
                                        "high_freq_factor": hi, "original_max_position_embeddings": orig})
        lib, att = ru.ROPE_INIT_FUNCTIONS["llama3"](cfg, "cpu")
        mine = orc.rope_inv_freq_llama3(d, base, factor, lo, hi, orig)
        assert att == 1.0
        np.testing.assert_allclose(mine, lib.double().numpy(), rtol=2e-6)      # the library works in float32
        plain = orc.rope_inv_freq(d, base)
        wl = 2 * np.pi / plain
        fast, slow = wl < orig / hi, wl > orig / lo
        assert fast.any() and slow.any() and (~fast & ~slow).any()
        np.testing.assert_array_equal(mine[fast], plain[fast])
        np.testing.assert_allclose(mine[slow], plain[slow] / factor, rtol=1e-15)
        mid = ~fast & ~slow
        assert np.all(mine[mid] < plain[mid]) and np.all(mine[mid] > plain[mid] / factor)
        assert np.all(np.diff(mine) < 0)
    # factor 1 is no scaling at all
    np.testing.assert_allclose(orc.rope_inv_freq_llama3(128, 5.0e5, 1.0), orc.rope_inv_freq(128, 5.0e5), rtol=1e-15)


def test_rope_identity_norm_and_relative_property():
    q, k = _rand((3, 6, 32), 2), _rand((3, 6, 32), 3)
    np.testing.assert_array_equal(orc.rope_pseudo_q(q[:, :1], 0, 1.0e4), q[:, :1])
    r = orc.rope_pseudo_q(q, 1000, 1.0e4)
    np.testing.assert_allclose(np.linalg.norm(r, axis=-1), np.linalg.norm(q, axis=-1), rtol=1e-13)
    # <R_m q, R_n k> depends on m - n only
    for shift in (1, 77, 4096):
        a = np.einsum("hnd,hnd->hn", orc.rope_pseudo_q(q, 50, 1.0e4), orc.rope_pseudo_q(k, 20, 1.0e4))
        b = np.einsum("hnd,hnd->hn", orc.rope_pseudo_q(q, 50 + shift, 1.0e4),
                      orc.rope_pseudo_q(k, 20 + shift, 1.0e4))
        np.testing.assert_allclose(a, b, atol=1e-9)


def test_rope_interleaved_pairs_hand_case_and_library():
    # Adjacent pairs: (1,2) by 90 degrees -> (-2,1); (3,4) by 180 degrees -> (-3,-4).
    q = np.array([[1.0, 2.0, 3.0, 4.0]])
    out = orc.rope_pseudo_q(q, pos_start=1, rope_base=1.0, inv_freq=np.array([math.pi / 2, math.pi]),
                            interleaved=True)
    np.testing.assert_allclose(out, [[-2.0, 1.0, -3.0, -4.0]], atol=1e-14)
    # As complex numbers x[2c] + i x[2c+1], the rotation is a multiplication by exp(i p theta_c).
    q = _rand((2, 7, 16), 11)
    z = torch.view_as_complex(torch.from_numpy(q).reshape(2, 7, 8, 2).contiguous())
    theta = torch.from_numpy(orc.rope_inv_freq(16, 1.0e4))
    pos = torch.arange(300, 307, dtype=torch.float64)
    rot = torch.polar(torch.ones(7, 8, dtype=torch.float64), pos[:, None] * theta[None, :])
    want = torch.view_as_real(z * rot).reshape(2, 7, 16).numpy()
    np.testing.assert_allclose(orc.rope_pseudo_q(q, 300, 1.0e4, interleaved=True), want, atol=1e-12)
    # and it is the rotate-half form seen through the channel permutation 2c -> c, 2c + 1 -> c + d/2
    perm = np.concatenate([np.arange(0, 16, 2), np.arange(1, 16, 2)])
    half = orc.rope_pseudo_q(q[..., perm], 300, 1.0e4)
    np.testing.assert_allclose(orc.rope_pseudo_q(q, 300, 1.0e4, interleaved=True)[..., perm], half, atol=1e-13)


def test_rope_angle_precision_at_128k():
    # double-precision angles at the largest position used (131072 + 127) agree with
    # extended precision to far below the scorer's tolerance
    d, base, pos = 128, 5.0e5, 131072 + 127
    c = np.arange(d // 2, dtype=np.longdouble)
    theta = np.power(np.longdouble(base), -2 * c / np.longdouble(d))
    ang = np.longdouble(pos) * theta
    q = np.ones((1, d))
    out = orc.rope_pseudo_q(q, pos, base)[0]
    ref_lo = (np.cos(ang) - np.sin(ang)).astype(np.float64)
    ref_hi = (np.cos(ang) + np.sin(ang)).astype(np.float64)
    np.testing.assert_allclose(out[:d // 2], ref_lo, atol=1e-9)
    np.testing.assert_allclose(out[d // 2:], ref_hi, atol=1e-9)


# ------------------------------------------------ scorer (Eq. 4) vs library causal attention
def sdpa_scores(q_rot, k_seq, L, G, scale=None):
    """Column sums from textbook causal attention over the whole extended sequence.

    torch's scaled_dot_product_attention with V = identity returns the attention
    matrix itself; rows L.. are the pseudo queries (rows < L carry arbitrary
    queries, their outputs are ignored)."""
    Hq, n, d = q_rot.shape
    Hkv = k_seq.shape[0]
    T = L + n
    out = np.zeros((Hkv, L))
    eye = torch.eye(T, dtype=torch.float64)[None, None]
    for h in range(Hq):
        qfull = np.concatenate([_rand((L, d), 100 + h), q_rot[h]], axis=0)
        P = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(qfull)[None, None], torch.from_numpy(np.ascontiguousarray(k_seq[h // G]))[None, None],
            eye, is_causal=True, scale=scale)[0, 0].numpy()
        out[h // G] += P[L:, :L].sum(axis=0)
    return out


@pytest.mark.parametrize("L,n,d,Hkv,G", [(1, 1, 4, 1, 1), (5, 3, 8, 2, 2), (17, 3, 128, 1, 4),
                                         (64, 8, 16, 2, 1), (33, 7, 32, 3, 3)])
def test_score_equals_library_causal_attention(L, n, d, Hkv, G):
    q = _rand((Hkv * G, n, d), 5)
    k = _rand((Hkv, L + n, d), 6)
    got = orc.score_sequence(q, k, L, G)["scores"]
    np.testing.assert_allclose(got, sdpa_scores(q, k, L, G), rtol=1e-11, atol=1e-14)


def test_score_custom_scale_matches_library():
    q, k = _rand((2, 3, 8), 7), _rand((1, 9 + 3, 8), 8)
    got = orc.score_sequence(q, k, 9, 2, scale=0.7)["scores"]
    np.testing.assert_allclose(got, sdpa_scores(q, k, 9, 2, scale=0.7), rtol=1e-11)


def test_pins_catch_planted_mistakes(monkeypatch):
    """The library pin must fail for plausible mistakes in the oracle (planted here)."""
    q, k = _rand((4, 3, 8), 9), _rand((2, 12 + 3, 8), 10)
    ref = sdpa_scores(q, k, 12, 2)
    good = orc.visible_logits

    def strict_causal(qh, keys, L, scale=None):          # self not visible
        s = good(qh, keys, L, scale).copy()
        n = qh.shape[0]
        for i in range(1, n):
            s[i, L + i] = -np.inf
        return s

    def no_scale(qh, keys, L, scale=None):               # dropped 1/sqrt(d)
        return good(qh, keys, L, 1.0)

    def prompt_only(qh, keys, L, scale=None):            # synthetic keys left out of the span
        s = good(qh, keys, L, scale).copy()
        s[:, L + 1:] = -np.inf
        return s

    for bad in (strict_causal, no_scale, prompt_only):
        monkeypatch.setattr(orc, "visible_logits", bad)
        got = orc.score_sequence(q, k, 12, 2)["scores"]
        assert not np.allclose(got, ref, rtol=1e-6), bad.__name__
    monkeypatch.setattr(orc, "visible_logits", good)
    # wrong head -> KV head map (interleaved instead of blocked groups)
    got = orc.score_sequence(q[[0, 2, 1, 3]], k, 12, 2)["scores"]
    assert not np.allclose(got, ref, rtol=1e-6)
    np.testing.assert_allclose(orc.score_sequence(q, k, 12, 2)["scores"], ref, rtol=1e-11)


# ------------------------------------------------------------------------- closed forms
def test_identical_keys_give_harmonic_scores():
    # all keys equal -> every row is uniform over its L + i + 1 visible keys
    L, n, d = 11, 6, 8
    k = np.tile(_rand((1, 1, d), 11), (1, L + n, 1))
    q = _rand((1, n, d), 12)
    res = orc.score_sequence(q, k, L, 1)
    expect = sum(1.0 / (L + i + 1) for i in range(n))
    np.testing.assert_allclose(res["scores"][0], np.full(L, expect), rtol=1e-13)
    np.testing.assert_allclose(res["lse"][0], [math.log(L + i + 1) + float(q[0, i] @ k[0, 0]) / math.sqrt(d)
                                               for i in range(n)], rtol=1e-12)


def test_single_query_single_head_is_one_softmax_row():
    scipy_special = pytest.importorskip("scipy.special")
    L, d = 23, 16
    q, k = _rand((1, 1, d), 13), _rand((1, L + 1, d), 14)
    row = scipy_special.softmax((k[0] @ q[0, 0]) / math.sqrt(d))
    res = orc.score_sequence(q, k, L, 1)
    np.testing.assert_allclose(res["scores"][0], row[:L], rtol=1e-12)
    np.testing.assert_allclose(res["syn_mass"][0], row[L], rtol=1e-12)
    np.testing.assert_allclose(res["lse"][0, 0], scipy_special.logsumexp((k[0] @ q[0, 0]) / math.sqrt(d)),
                               rtol=1e-13)


# --------------------------------------------------------------------------- invariants
def test_rows_sum_to_one_and_mass_is_conserved():
    L, n, d, Hkv, G = 300, 16, 64, 2, 4
    q, k = _rand((Hkv * G, n, d), 15) * 2.0, _rand((Hkv, L + n, d), 16) * 2.0
    for h in range(Hkv * G):
        P, _ = orc.attention_rows(q[h], k[h // G], L)
        assert (P >= 0).all()
        np.testing.assert_allclose(P.sum(axis=1), np.ones(n), rtol=1e-12)
        # causal span: query i never sees synthetic key i' > i
        assert np.all(np.triu(P[:, L:], k=1) == 0.0) and np.all(np.diagonal(P[:, L:]) > 0)
    res = orc.score_sequence(q, k, L, G)
    np.testing.assert_allclose(res["prompt_mass"] + res["syn_mass"], np.full(Hkv * G, n), rtol=1e-12)
    np.testing.assert_allclose(res["scores"].sum(axis=1) + res["syn_mass"].reshape(Hkv, G).sum(axis=1),
                               np.full(Hkv, G * n), rtol=1e-12)


def test_equivariances():
    L, n, d, Hkv, G = 40, 5, 16, 2, 3
    q, k = _rand((Hkv * G, n, d), 17), _rand((Hkv, L + n, d), 18)
    base = orc.score_sequence(q, k, L, G)["scores"]
    # permuting heads inside a group changes nothing; swapping groups swaps KV heads
    perm = np.array([2, 0, 1, 4, 5, 3])
    np.testing.assert_allclose(orc.score_sequence(q[perm], k, L, G)["scores"], base, rtol=1e-12)
    swap = np.array([3, 4, 5, 0, 1, 2])
    np.testing.assert_allclose(orc.score_sequence(q[swap], k[::-1], L, G)["scores"], base[::-1], rtol=1e-12)
    # permuting prompt rows (keys are stored post-RoPE) permutes the scores
    p = np.random.default_rng(19).permutation(L)
    kp = k.copy()
    kp[:, :L] = k[:, p]
    np.testing.assert_allclose(orc.score_sequence(q, kp, L, G)["scores"], base[:, p], rtol=1e-12)
    # adding one vector to every key shifts each row's logits by a constant
    shift = _rand((d,), 20)
    np.testing.assert_allclose(orc.score_sequence(q, k + shift, L, G)["scores"], base, rtol=1e-10)


def test_theorem_bounds_hold():
    # Appendix C, inequalities (4) and (5): for unit q, q' the largest logit gap and the
    # L1 gap of the attention rows are bounded by K_max * |q - q'| / sqrt(d_k)
    rng = np.random.default_rng(21)
    d, L = 32, 200
    k = rng.standard_normal((1, L + 1, d))
    kmax = np.linalg.norm(k[0], axis=1).max()
    for _ in range(20):
        q = rng.standard_normal(d)
        q /= np.linalg.norm(q)
        q2 = q + 0.3 * rng.standard_normal(d)
        q2 /= np.linalg.norm(q2)
        bound = kmax * math.sqrt(2 * (1 - float(q @ q2))) / math.sqrt(d)
        a, _ = orc.attention_rows(q[None], k[0], L)
        b, _ = orc.attention_rows(q2[None], k[0], L)
        sa = orc.visible_logits(q[None], k[0], L)
        sb = orc.visible_logits(q2[None], k[0], L)
        assert np.abs(sa - sb).max() <= bound + 1e-12
        assert np.abs(a - b).sum() <= bound + 1e-12


# ------------------------------------------------------------------- top-K (Eq. 5)
def test_topk_hand_cases():
    s = np.array([0.5, 0.2, 0.5, 0.1, 0.2])
    np.testing.assert_array_equal(orc.topk_select(s, 1), [0])          # tie -> lower index
    np.testing.assert_array_equal(orc.topk_select(s, 2), [0, 2])
    np.testing.assert_array_equal(orc.topk_select(s, 3), [0, 1, 2])    # tie at threshold -> index 1
    np.testing.assert_array_equal(orc.topk_select(s, 4), [0, 1, 2, 4])
    np.testing.assert_array_equal(orc.topk_select(s, 5), [0, 1, 2, 3, 4])
    np.testing.assert_array_equal(orc.topk_select(s, 9), [0, 1, 2, 3, 4])  # clamp
    np.testing.assert_array_equal(orc.topk_select(np.zeros(4), 2), [0, 1])
    assert orc.topk_select(s, 3).dtype == np.int32


def test_topk_properties_and_library_agreement():
    rng = np.random.default_rng(22)
    for L, K in [(1, 1), (100, 7), (1000, 999), (4097, 128)]:
        s = rng.random(L)
        idx = orc.topk_select(s, K)
        assert len(idx) == K and np.all(np.diff(idx) > 0) and idx.min() >= 0 and idx.max() < L
        rest = np.setdiff1d(np.arange(L), idx)
        assert rest.size == 0 or s[idx].min() >= s[rest].max()
        lib = torch.topk(torch.from_numpy(s), K).indices.numpy()      # distinct values: unique set
        np.testing.assert_array_equal(idx, np.sort(lib))


# --------------------------------------------------------------- compaction / full path
def test_compaction_is_a_bit_exact_row_copy_without_synthetic_rows():
    rng = np.random.default_rng(23)
    B, Hq, Hkv, n, d = 2, 4, 2, 3, 8
    Ls, Ks = [19, 7], [5, 9]
    cu = np.concatenate([[0], np.cumsum([l + n for l in Ls])])
    q = rng.standard_normal((B, Hq, n, d))
    k = rng.standard_normal((Hkv, cu[-1], d)).astype(np.float32)
    v = rng.standard_normal((Hkv, cu[-1], d)).astype(np.float32)
    res = orc.evict(q, k, v, cu, Ls, Ks, 1.0e4)
    for b in range(B):
        idx = res["idx"][b]
        kk = min(Ks[b], Ls[b])
        assert idx.shape == (Hkv, kk) and idx.max() < Ls[b]          # never a synthetic row
        for h in range(Hkv):
            assert res["k_out"][b][h].tobytes() == k[h, cu[b] + idx[h]].tobytes()
            assert res["v_out"][b][h].tobytes() == v[h, cu[b] + idx[h]].tobytes()
            assert res["k_out"][b].dtype == np.float32
    # K_b >= L_b keeps every prompt row, in order
    np.testing.assert_array_equal(res["idx"][1][0], np.arange(7))


def test_evict_uses_decode_positions():
    # the path rotates sequence b's queries to L_b .. L_b+N-1 (Section 4.1)
    rng = np.random.default_rng(24)
    q = rng.standard_normal((1, 2, 4, 16))
    k = rng.standard_normal((1, 30 + 4, 16))
    res = orc.evict(q, k, k, [0, 34], [30], [5], 1.0e4)
    np.testing.assert_array_equal(res["q_rot"][0], orc.rope_pseudo_q(q[0], 30, 1.0e4))
    direct = orc.score_sequence(orc.rope_pseudo_q(q[0], 30, 1.0e4), k, 30, 2)["scores"]
    np.testing.assert_array_equal(res["scores"][0], direct)
    other = orc.evict(q, k, k, [0, 34], [30], [5], 1.0e4, pos_start=[31])
    assert not np.allclose(other["scores"][0], direct)


def test_planted_needles_are_retained():
    from gen import inputs as gi
    w = gi.workload("tiny")
    data = gi.draw_layer(w, 0, "cpu")
    q_rot = np.stack([orc.rope_pseudo_q(data["q_pre"][b].double().numpy(), w.prompt_lens[b], w.rope_base)
                      for b in range(w.batch)])
    gi.plant_structure(w, data, torch.from_numpy(q_rot))
    res = orc.evict(data["q_pre"].double().numpy(), data["k"].double().numpy(), data["v"].double().numpy(),
                    w.cu_rows, w.prompt_lens, w.keep, w.rope_base)
    for h in range(w.n_kv_heads):
        idx = set(res["idx"][0][h].tolist())
        sc = res["scores"][0][h]
        kth = np.sort(sc)[-w.keep[0]]
        for p in data["needle_pos"][0, h]:
            assert int(p) in idx
            assert sc[p] >= 10 * kth


# ------------------------------------------------------------------ optional pooling
@pytest.mark.parametrize("L,kernel", [(1, 3), (2, 5), (7, 7), (50, 5), (33, 13)])
def test_pooling_matches_library_pooling(L, kernel):
    s = np.abs(_rand((3, L), 30)) + 0.1
    t = torch.from_numpy(s)[None]
    r = kernel // 2
    # max: the library pads with -inf, which is clipping the window
    lib_max = torch.nn.functional.max_pool1d(t, kernel, stride=1, padding=r)[0].numpy()
    np.testing.assert_array_equal(orc.pool_scores(s, kernel, "max"), lib_max)
    # avg over the positions that exist = the library's count_include_pad=False
    lib_avg = torch.nn.functional.avg_pool1d(t, kernel, stride=1, padding=r, count_include_pad=False)[0].numpy()
    np.testing.assert_allclose(orc.pool_scores(s, kernel, "avg"), lib_avg, rtol=1e-13)


def test_pooling_hand_case_and_identity():
    s = np.array([1.0, 5.0, 2.0, 0.0, 3.0])
    np.testing.assert_array_equal(orc.pool_scores(s, 3, "max"), [5, 5, 5, 3, 3])
    np.testing.assert_allclose(orc.pool_scores(s, 3, "avg"), [3.0, 8 / 3, 7 / 3, 5 / 3, 1.5])
    np.testing.assert_array_equal(orc.pool_scores(s, 1, "max"), s)
    np.testing.assert_array_equal(orc.pool_scores(s, 7, "none"), s)


def test_evict_selects_on_pooled_scores():
    rng = np.random.default_rng(31)
    q = rng.standard_normal((1, 2, 4, 16))
    k = rng.standard_normal((1, 40 + 4, 16))
    plain = orc.evict(q, k, k, [0, 44], [40], [6], 1.0e4)
    pooled = orc.evict(q, k, k, [0, 44], [40], [6], 1.0e4, pool_mode="max", pool_kernel=5)
    np.testing.assert_array_equal(pooled["scores"][0], plain["scores"][0])      # Eq. 4 sums are untouched
    np.testing.assert_array_equal(pooled["pooled"][0], orc.pool_scores(plain["scores"][0], 5, "max"))
    np.testing.assert_array_equal(pooled["idx"][0][0], orc.topk_select(pooled["pooled"][0][0], 6))
    # max pooling spreads the top score over its window: its neighbours are kept (ties -> lower index)
    top = int(np.argmax(plain["scores"][0][0]))
    assert {max(0, top - 2), top}.issubset(set(pooled["idx"][0][0].tolist()))


# ------------------------------------------------------------------ recall (Section 3.3)
def test_recall_hand_cases_and_library_agreement():
    assert orc.recall([1, 2, 3, 4], [1, 2, 3, 4]) == 1.0
    assert orc.recall([1, 2, 3, 4], [5, 6, 7, 8]) == 0.0
    assert orc.recall([0, 2, 4, 6], [1, 2, 3, 4]) == 0.5            # {2, 4} of four gold tokens
    rng = np.random.default_rng(40)
    for _ in range(5):
        a = np.sort(rng.choice(500, 60, replace=False))
        b = np.sort(rng.choice(500, 60, replace=False))
        assert orc.recall(a, b) == pytest.approx(np.intersect1d(a, b).size / 60)


def test_recall_of_a_smaller_window_against_a_larger_one():
    # Eq. 1-3 on one cache: gold = top-K under all 16 queries, pred = top-K under the last 4;
    # identical windows give 1, and the value is a fraction with denominator K
    rng = np.random.default_rng(41)
    q = rng.standard_normal((1, 1, 16, 16))
    k = rng.standard_normal((1, 60 + 16, 16))
    gold = orc.evict(q, k, k, [0, 76], [60], [10], 1.0e4)["idx"][0][0]
    assert orc.recall(gold, gold) == 1.0
    k4 = np.concatenate([k[:, :60], k[:, 72:]], axis=1)
    pred = orc.evict(q[:, :, 12:], k4, k4, [0, 64], [60], [10], 1.0e4, pos_start=[72])["idx"][0][0]
    r = orc.recall(gold, pred)
    assert 0.0 <= r <= 1.0 and abs(r * 10 - round(r * 10)) < 1e-12


def test_prompt_window_scores_match_library_causal_attention():
    """score_prompt_window against torch's scaled_dot_product_attention over the L-token prompt (value
    matrix = identity, so the output rows ARE the attention weights), and against the identity that
    ties it to the pseudo-query scorer: a window cut from the prompt is the same computation with
    prompt_len = L - N and the window's rows in the place of the synthetic rows."""
    rng = np.random.default_rng(5)
    for Hq, Hkv, n, L, d in [(4, 2, 3, 17, 8), (2, 2, 5, 40, 16), (6, 2, 1, 9, 4)]:
        G = Hq // Hkv
        q = rng.standard_normal((Hq, n, d))
        k = rng.standard_normal((Hkv, L, d))
        got = orc.score_prompt_window(q, k, G)
        qt, kt = torch.from_numpy(q), torch.from_numpy(k).repeat_interleave(G, dim=0)
        mask = torch.arange(L)[None, :] <= (L - n + torch.arange(n))[:, None]
        P = torch.nn.functional.scaled_dot_product_attention(qt[None], kt[None], torch.eye(L, dtype=torch.float64).expand(1, Hq, L, L),
                                                             attn_mask=mask)[0]
        want = P[:, :, :L - n].sum(dim=1).reshape(Hkv, G, L - n).sum(dim=1).numpy()
        np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(got, orc.score_sequence(q, k, L - n, G)["scores"], rtol=1e-12, atol=1e-15)
    # a planted mistake (strictly causal window: a query that does not see its own key) fails the pin
    q, k = rng.standard_normal((2, 3, 8)), rng.standard_normal((1, 12, 8))
    good = orc.score_prompt_window(q, k, 2)
    s = np.einsum("hnd,ld->hnl", q, k[0]) / np.sqrt(8.0)
    s = np.where(np.arange(12)[None, None, :] < (9 + np.arange(3))[None, :, None], s, -np.inf)
    e = np.exp(s - s.max(-1, keepdims=True))
    bad = (e / e.sum(-1, keepdims=True))[:, :, :9].sum(axis=(0, 1))
    assert not np.allclose(good[0], bad, rtol=1e-3)
