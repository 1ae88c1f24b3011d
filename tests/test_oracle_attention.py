"""Pins of the oracle's attention routines against things other than the oracle:
a library attention, closed forms, and a hand-worked example."""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


def _sdpa_causal(q, k, v, scale, offset=0):
    """Library attention (torch, fp64).  q [n_q,Hq,D], k/v [n_kv,Hkv,D]; row p sees keys t <= p + offset."""
    Hq, Hkv = q.shape[1], k.shape[1]
    G = Hq // Hkv
    qt = torch.from_numpy(q).double().permute(1, 0, 2)[None]
    kt = torch.from_numpy(k).double().permute(1, 0, 2)[None].repeat_interleave(G, 1)
    vt = torch.from_numpy(v).double().permute(1, 0, 2)[None].repeat_interleave(G, 1)
    n_q, n_kv = q.shape[0], k.shape[0]
    mask = torch.arange(n_kv)[None, :] <= (torch.arange(n_q)[:, None] + offset)
    o = F.scaled_dot_product_attention(qt, kt, vt, attn_mask=mask, scale=scale)
    return o[0].permute(1, 0, 2).numpy()


@pytest.mark.parametrize("n,Hq,Hkv,D", [(37, 4, 2, 16), (64, 7, 1, 8), (5, 6, 3, 32), (1, 2, 2, 4)])
def test_full_causal_matches_library_attention(n, Hq, Hkv, D):
    q, k, v = _rand((n, Hq, D), 1), _rand((n, Hkv, D), 2), _rand((n, Hkv, D), 3)
    scale = 1.0 / math.sqrt(D)
    got = oracle.full_causal_attn(q, k, v, scale)
    ref = _sdpa_causal(q, k, v, scale)
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)
    # the important-token stage is the same operator on packed rows
    got2 = oracle.important_attn(q, k, v, scale)
    np.testing.assert_allclose(got2, ref, rtol=0, atol=1e-12)


@pytest.mark.parametrize("L_d,L_q,Hq,Hkv,D", [(29, 6, 4, 2, 16), (8, 1, 3, 1, 8), (3, 9, 2, 2, 4)])
def test_question_attention_matches_library_attention(L_d, L_q, Hq, Hkv, D):
    N = L_d + L_q
    qq, k, v = _rand((L_q, Hq, D), 4), _rand((N, Hkv, D), 5), _rand((N, Hkv, D), 6)
    scale = 0.37
    got = oracle.qd_attn(qq, k, v, L_d, scale)
    ref = _sdpa_causal(qq, k, v, scale, offset=L_d)
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)


def test_question_rows_equal_tail_of_full_attention():
    L_d, L_q, Hq, Hkv, D = 21, 7, 6, 2, 8
    N = L_d + L_q
    q, k, v = _rand((N, Hq, D), 7), _rand((N, Hkv, D), 8), _rand((N, Hkv, D), 9)
    full = oracle.full_causal_attn(q, k, v, 0.25)
    qd = oracle.qd_attn(q[L_d:], k, v, L_d, 0.25)
    np.testing.assert_allclose(qd, full[L_d:], rtol=0, atol=1e-13)


def test_hand_worked_rational_example():
    rows = np.loadtxt(os.path.join(GOLDEN, "softmax_rational.txt"))
    a = np.array([1.0, 2.0, 5.0, 8.0])
    q = np.tile(np.array([2.0, 0, 0, 0], dtype=np.float32), (4, 1)).reshape(4, 1, 4)
    k = np.stack([np.log(a), np.full(4, 7.0), np.full(4, -3.0), np.full(4, 1.0)], axis=1).astype(np.float32)
    v = np.array([[1, 0, 0, -1], [0, 1, 0, 2], [2, 2, 0, 0], [-4, 0, 8, 1]], dtype=np.float32)
    out, lse = oracle.full_causal_attn(q, k.reshape(4, 1, 4), v.reshape(4, 1, 4), 0.5, return_lse=True)
    # ln a_t is rounded to fp32 on input, hence 1e-6 rather than 1e-15
    np.testing.assert_allclose(out[:, 0, :], rows[:, 1:5], rtol=0, atol=1e-6)
    np.testing.assert_allclose(lse[:, 0], rows[:, 5], rtol=0, atol=1e-6)


def test_zero_keys_give_running_mean_of_values():
    n, Hq, Hkv, D = 50, 4, 2, 8
    q, v = _rand((n, Hq, D), 10), _rand((n, Hkv, D), 11)
    k = np.zeros((n, Hkv, D), dtype=np.float32)
    out, lse = oracle.important_attn(q, k, v, 0.3, return_lse=True)
    mean = np.cumsum(v.astype(np.float64), axis=0) / np.arange(1, n + 1)[:, None, None]
    for h in range(Hq):
        np.testing.assert_allclose(out[:, h], mean[:, h // 2], rtol=0, atol=1e-13)
    np.testing.assert_allclose(lse, np.log(np.arange(1, n + 1))[:, None].repeat(Hq, 1), atol=1e-13)
    # same closed form for the question stage: mean over the L_d + i + 1 visible keys
    L_d, L_q = 40, 10
    oq = oracle.qd_attn(q[L_d:], k, v, L_d, 0.3)
    for h in range(Hq):
        np.testing.assert_allclose(oq[:, h], mean[L_d:, h // 2], rtol=0, atol=1e-13)


def test_constant_values_and_first_row():
    n, Hq, Hkv, D = 33, 2, 1, 16
    q, k = _rand((n, Hq, D), 12), _rand((n, Hkv, D), 13)
    v = np.full((n, Hkv, D), 1.75, dtype=np.float32)
    out = oracle.full_causal_attn(q, k, v, 1.0)
    np.testing.assert_allclose(out, 1.75, rtol=0, atol=1e-13)
    v2 = _rand((n, Hkv, D), 14)
    out2 = oracle.full_causal_attn(q, k, v2, 1.0)
    # row 0 sees one key: the output is that value row exactly
    assert np.array_equal(out2[0, 0], v2[0, 0].astype(np.float64))
    assert np.array_equal(out2[0, 1], v2[0, 0].astype(np.float64))


def test_dominant_logit_selects_its_value_row():
    n, D = 20, 8
    q = np.zeros((n, 1, D), dtype=np.float32)
    q[:, 0, 0] = 1.0
    k = np.zeros((n, 1, D), dtype=np.float32)
    k[7, 0, 0] = 200.0
    v = _rand((n, 1, D), 15)
    out = oracle.full_causal_attn(q, k, v, 1.0)
    np.testing.assert_allclose(out[7:, 0], np.tile(v[7, 0], (n - 7, 1)), atol=1e-12)
    # before key 7 becomes visible the rows are plain running means
    mean = np.cumsum(v.astype(np.float64), axis=0) / np.arange(1, n + 1)[:, None, None]
    np.testing.assert_allclose(out[:7, 0], mean[:7, 0], atol=1e-13)


def test_softmax_rows_sum_to_one_via_lse():
    n, Hq, Hkv, D = 40, 4, 4, 8
    q, k, v = _rand((n, Hq, D), 16), _rand((n, Hkv, D), 17), _rand((n, Hkv, D), 18)
    scale = 0.9
    _, lse = oracle.full_causal_attn(q, k, v, scale, return_lse=True)
    logits = np.einsum("phd,thd->pht", q.astype(np.float64), k.astype(np.float64)) * scale
    for p in range(n):
        s = np.exp(logits[p, :, : p + 1] - lse[p][:, None]).sum(axis=1)
        np.testing.assert_allclose(s, 1.0, atol=1e-12)


def test_row_subset_equals_full_rows():
    n, Hq, Hkv, D = 45, 4, 2, 8
    q, k, v = _rand((n, Hq, D), 19), _rand((n, Hkv, D), 20), _rand((n, Hkv, D), 21)
    full = oracle.full_causal_attn(q, k, v, 0.5)
    rows = [44, 0, 17, 3]
    sub = oracle.full_causal_attn(q, k, v, 0.5, rows=rows)
    assert np.array_equal(sub, full[rows])


def test_future_keys_do_not_matter():
    n, Hq, Hkv, D = 30, 2, 1, 8
    q, k, v = _rand((n, Hq, D), 22), _rand((n, Hkv, D), 23), _rand((n, Hkv, D), 24)
    a = oracle.full_causal_attn(q, k, v, 0.5, rows=[11])
    k2, v2 = k.copy(), v.copy()
    k2[12:] += 5.0
    v2[12:] -= 3.0
    b = oracle.full_causal_attn(q, k2, v2, 0.5, rows=[11])
    assert np.array_equal(a, b)
    k2[11] += 1.0
    c = oracle.full_causal_attn(q, k2, v2, 0.5, rows=[11])
    assert not np.array_equal(a, c)
