"""Pins of the oracle's selection, gather, hybrid-cache and fusion steps."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_num_important_golden():
    rows = np.loadtxt(os.path.join(GOLDEN, "num_important.txt"))
    for L_d, r, k in rows:
        assert oracle.num_important(int(L_d), float(r)) == int(k), (L_d, r, k)
    assert oracle.num_important(100, 0.0) == 0
    assert oracle.num_important(0, 0.5) == 0
    assert oracle.num_important(10, 2.0) == 10
    # r stored as fp32 (as the C ABI passes it) still gives the stated counts
    assert oracle.num_important(1024, float(np.float32(0.15))) == 154
    assert oracle.num_important(32768, float(np.float32(0.2))) == 6554
    assert oracle.num_important(1000, float(np.float32(0.1))) == 100


def _rank_count_select(s, k):
    """O(n^2) definition: i is kept iff fewer than k tokens come before it in (score desc, index asc)."""
    n = len(s)
    keep = []
    for i in range(n):
        before = 0
        for j in range(n):
            if s[j] > s[i] or (s[j] == s[i] and j < i):
                before += 1
        if before < k:
            keep.append(i)
    return np.array(keep, dtype=np.int32)


@pytest.mark.parametrize("n,k,seed", [(64, 16, 0), (97, 1, 1), (50, 50, 2), (33, 0, 3), (200, 61, 4)])
def test_select_matches_rank_count_and_stable_argsort(n, k, seed):
    rng = np.random.default_rng(seed)
    s = np.exp(rng.standard_normal(n)).astype(np.float32)
    s[rng.integers(0, n, n // 4)] = s[0]  # plant ties
    got = oracle.select(s, k)
    assert np.array_equal(got, _rank_count_select(s, k))
    lib = np.sort(np.argsort(-s.astype(np.float64), kind="stable")[:k]).astype(np.int32)
    assert np.array_equal(got, lib)
    assert np.all(np.diff(got) > 0)


def test_select_known_permutation_and_ties():
    n, k = 40, 7
    perm = np.random.default_rng(5).permutation(n)
    s = perm.astype(np.float32)  # token i has score perm[i]; the top 7 are where perm >= 33
    assert np.array_equal(oracle.select(s, k), np.sort(np.nonzero(perm >= n - k)[0]).astype(np.int32))
    assert np.array_equal(oracle.select(np.full(n, 3.0, np.float32), k), np.arange(k, dtype=np.int32))
    assert np.array_equal(oracle.select(s, n), np.arange(n, dtype=np.int32))


def test_select_special_values():
    s = np.array([0.0, -0.0, np.nan, 1.0, -np.inf, np.inf, np.nan, -1.0], dtype=np.float32)
    # order: inf(5), 1(3), +0(0), -0(1) [equal, index order], -1(7), -inf(4), nan(2), nan(6)
    assert list(oracle.select(s, 3)) == [0, 3, 5]
    assert list(oracle.select(s, 4)) == [0, 1, 3, 5]
    assert list(oracle.select(s, 6)) == [0, 1, 3, 4, 5, 7]
    assert list(oracle.select(s, 7)) == [0, 1, 2, 3, 4, 5, 7]


def test_aggregate_is_fp32_sum_in_row_order():
    S = np.array([[1e8, 1.0], [1.0, 1.0], [-1e8, 1.0]], dtype=np.float32)
    got = oracle.aggregate(S)
    exp0 = np.float32(np.float32(np.float32(1e8) + np.float32(1.0)) + np.float32(-1e8))  # 0.0: the 1 is absorbed
    assert got[0] == exp0 == 0.0 and got[1] == 3.0
    # selection sees the aggregated signal
    S2 = np.array([[1.0, 5.0, 2.0, 0.0], [4.0, 0.0, 2.5, 0.0], [1.0, 0.0, 1.0, 0.0]], dtype=np.float32)
    assert list(oracle.select(S2, 2)) == [0, 2]  # sums 6, 5, 5.5, 0


def test_gather_hybrid_and_fuse_placement():
    rng = np.random.default_rng(6)
    L_d, L_q, H, D = 12, 3, 2, 4
    N = L_d + L_q
    fresh = rng.standard_normal((N, H, D)).astype(np.float32)
    cached = rng.standard_normal((L_d, H, D)).astype(np.float32)
    idx = np.array([0, 4, 5, 11], dtype=np.int32)
    assert np.array_equal(oracle.gather_rows(fresh, idx), fresh[idx])
    hyb = oracle.hybrid_kv(cached, fresh, idx, L_d, L_q)
    exp = np.concatenate([cached, fresh[L_d:]], 0)
    exp[idx] = fresh[idx]
    assert np.array_equal(hyb, exp)
    hyb0 = oracle.hybrid_kv(cached, fresh, idx, L_d, L_q, overwrite=False)
    assert np.array_equal(hyb0, np.concatenate([cached, fresh[L_d:]], 0))
    o_imp = rng.standard_normal((4, H, D))
    o_q = rng.standard_normal((L_q, H, D))
    hid, pos = oracle.fuse(o_imp, o_q, idx, L_d, mode=0)
    assert np.array_equal(hid, np.concatenate([o_imp, o_q], 0))
    assert list(pos) == [0, 4, 5, 11, 12, 13, 14]
    base = np.full((N, H, D), -7.0)
    hid1, pos1 = oracle.fuse(o_imp, o_q, idx, L_d, mode=1, hidden=base)
    exp1 = np.full((N, H, D), -7.0)
    exp1[idx] = o_imp
    exp1[L_d:] = o_q
    assert np.array_equal(hid1, exp1) and list(pos1) == list(pos)


def test_deviation_scores_closed_forms_and_library_sum():
    rng = np.random.default_rng(8)
    L_d, H, D = 9, 2, 4
    kf = rng.standard_normal((L_d + 3, H, D)).astype(np.float32)   # fresh tensors carry question rows too
    vf = rng.standard_normal((L_d + 3, H, D)).astype(np.float32)
    kc, vc = kf[:L_d].copy(), vf[:L_d].copy()
    assert np.all(oracle.deviation_scores(kf, vf, kc, vc, L_d) == 0.0)          # equal tensors: no deviation
    kc[4, 1, 2] += 0.5                                                           # one element off by c: c^2
    vc[6, 0, 0] -= 2.0
    s = oracle.deviation_scores(kf, vf, kc, vc, L_d)
    want = np.zeros(L_d)
    want[4], want[6] = 0.25, 4.0
    np.testing.assert_allclose(s, want, atol=1e-6)
    # hand-worked: K differs by (1,2,...,8), V by (1,1,...,1) on token 0 -> 204 + 8
    kc2, vc2 = kf[:L_d].copy(), vf[:L_d].copy()
    kc2[0] -= np.arange(1, 9, dtype=np.float32).reshape(H, D)
    vc2[0] -= 1.0
    assert abs(oracle.deviation_scores(kf, vf, kc2, vc2, L_d)[0] - 212.0) < 1e-4
    # library sum of squares on random tensors
    kc3 = rng.standard_normal((L_d, H, D)).astype(np.float32)
    vc3 = rng.standard_normal((L_d, H, D)).astype(np.float32)
    lib = ((kf[:L_d].astype(np.float64) - kc3) ** 2 + (vf[:L_d].astype(np.float64) - vc3) ** 2).sum(axis=(1, 2))
    np.testing.assert_allclose(oracle.deviation_scores(kf, vf, kc3, vc3, L_d), lib, rtol=1e-12)
