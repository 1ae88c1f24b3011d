"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by
element on the same seeded inputs.  Integer and byte results must be identical;
attention outputs must be within max-abs 2e-2 and mean-abs 2e-3 of the oracle
(bf16 operands and output, fp32 accumulation), plus a relative Frobenius bound
that stays meaningful where outputs are small."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2607_21599_b200 import api, build
from paper_2607_21599_b200 import workloads as W

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS, REL_FRO = 2e-2, 2e-3, 1e-2


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    build.build()
    api.lib()
    yield
    torch.cuda.synchronize()


def _f(t):
    return t.float().cpu().numpy()


def _assert_close(got_bf16, ref_f64, what):
    got = got_bf16.float().cpu().numpy().astype(np.float64)
    assert got.shape == ref_f64.shape, (what, got.shape, ref_f64.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - ref_f64)
    fro = np.linalg.norm(got - ref_f64) / max(np.linalg.norm(ref_f64), 1e-30)
    assert err.max() <= MAX_ABS, f"{what}: max-abs {err.max():.3e}"
    assert err.mean() <= MEAN_ABS, f"{what}: mean-abs {err.mean():.3e}"
    assert fro <= REL_FRO, f"{what}: relative Frobenius {fro:.3e}"


def _ok(status, workspace, what):
    api.check(status, what)
    torch.cuda.synchronize()
    api.check(api.daf_poll_status(workspace), what + " (device status)")


def _normal(shape, seed, scale=1.0):
    return (W.normal_bf16(shape, seed).float() * scale).to(torch.bfloat16)


# --------------------------------------------------------------------------- selection
@pytest.mark.parametrize("L_d,r,n_sig,kind", [
    (1024, 0.15, 1, "lognormal"), (6144, 0.15, 1, "lognormal"), (16384, 0.10, 3, "lognormal"),
    (32768, 0.20, 1, "pareto"), (1000, 0.1, 2, "ties"), (777, 1.0, 1, "lognormal"), (130, 0.5, 1, "special"),
    (50000, 0.07, 1, "lognormal"), (33, 0.03, 1, "ties"), (4096, 0.25, 1, "constant"),
    (16384, 0.10, 1, "constant"), (20000, 0.3, 2, "ties"), (40960, 0.2, 1, "lognormal"), (40961, 0.2, 1, "lognormal"),
    (7, 0.5, 1, "lognormal"), (1, 1.0, 1, "lognormal"), (12000, 0.2, 1, "special"), (16384, 0.5, 1, "ties"),
    (16385, 0.5, 1, "ties"), (2048, 0.05, 1, "narrow"),
    # either side of the size at which the cluster kernel takes over; a cluster-sized problem whose keys differ
    # only in their last byte (every radix pass is needed) and one whose keys differ only in the first two
    (8192, 0.15, 1, "lognormal"), (8193, 0.15, 1, "lognormal"), (20000, 0.2, 1, "lowbyte"), (24000, 0.1, 1, "highbytes"),
    (30000, 1.0, 1, "lognormal"), (30000, 0.0, 1, "lognormal"),
    # sums of two signal rows that are subnormal in fp32: the aggregation must keep them apart, not flush them to 0
    (3000, 0.2, 2, "denormal"), (12000, 0.1, 3, "denormal"),
])
def test_select_indices_bit_exact(L_d, r, n_sig, kind):
    if kind == "pareto":
        w = W.Workload("t", 3, 4, 2, 128, 1, L_d, 512, 0, r, "pareto_clustered", n_sig)
        S = W.importance_scores(w, 1)
    else:
        w = W.Workload("t", 7, 4, 2, 128, 1, L_d, L_d, 0, r, "lognormal", n_sig)
        S = W.importance_scores(w, 2)
        if kind == "ties":
            S = torch.round(S * 2) / 2
        if kind == "constant":
            S = torch.full_like(S, 1.5)
        if kind == "narrow":      # scores within a few ulps of each other: the key range needs only a few bits
            S = 1.0 + torch.floor(S * 4) * 2.0 ** -22
        if kind == "lowbyte":     # 256 distinct values one ulp apart: many ties, decided by the last byte only
            S = (1.0 + torch.floor(S * 37).remainder(256) * 2.0 ** -23).float()
        if kind == "highbytes":   # powers of two times {1, 1.5}: the low two bytes of every key are zero
            S = torch.pow(2.0, torch.floor(S * 3).remainder(40) - 20) * (1.0 + 0.5 * (torch.floor(S * 11).remainder(2)))
        if kind == "denormal":    # distinct multiples of the smallest subnormal, a few normal values among them
            S = (torch.floor(S * 1000).remainder(4000) * 2.0 ** -149).float()
            S[0, ::97] = 1.0e-37
        if kind == "special":
            S[0, 3] = float("nan"); S[0, 4] = float("inf"); S[0, 5] = -float("inf")
            S[0, 6] = 0.0; S[0, 7] = -0.0; S[0, 8] = float("nan"); S[0, 9:40] = -S[0, 9:40]
    p = api.make_params(L_d, 0, r, 4, 2)
    k = api.daf_num_important(L_d, r)
    assert k == oracle.num_important(L_d, r)
    ws = api.alloc_workspace(p)
    dev = "cuda"
    H = 4
    qf = torch.zeros(L_d, H, 128, dtype=torch.bfloat16, device=dev)
    kf = torch.zeros(L_d, 2, 128, dtype=torch.bfloat16, device=dev)
    kvk, kvv = torch.zeros_like(kf), torch.zeros_like(kf)
    idx_out = torch.full((max(k, 1),), -1, dtype=torch.int32, device=dev)
    qp = torch.zeros(max(k, 1), H, 128, dtype=torch.bfloat16, device=dev)
    kp = torch.zeros(max(k, 1), 2, 128, dtype=torch.bfloat16, device=dev)
    vp = torch.zeros_like(kp)
    _ok(api.daf_select(p, S.to(dev), n_sig, None, qf, kf, kf.clone(), kvk, kvv, idx_out, qp, kp, vp, ws), ws, "daf_select")
    ref = oracle.select(S.numpy(), k)
    assert np.array_equal(idx_out[:k].cpu().numpy(), ref)


# --------------------------------------------------------------------------- deviation signal
@pytest.mark.parametrize("L_d,L_q,Hkv", [(1024, 32, 4), (777, 0, 8), (6144, 64, 4), (5, 3, 1), (40000, 16, 8)])
def test_deviation_scores_match_oracle(L_d, L_q, Hkv):
    N = L_d + L_q
    kf, vf = _normal((N, Hkv, 128), 71), _normal((N, Hkv, 128), 72)
    kc, vc = _normal((L_d, Hkv, 128), 73), _normal((L_d, Hkv, 128), 74)
    kc[: min(3, L_d)] = kf[: min(3, L_d)]          # tokens whose K did not move
    p = api.make_params(L_d, L_q, 0.1, 4 * Hkv, Hkv)
    s = torch.full((L_d + 1,), -1.0, dtype=torch.float32, device="cuda")
    api.check(api.daf_deviation_scores(p, kf.cuda(), vf.cuda(), kc.cuda(), vc.cuda(), s), "daf_deviation_scores")
    torch.cuda.synchronize()
    ref = oracle.deviation_scores(_f(kf), _f(vf), _f(kc), _f(vc), L_d)
    # fp32 accumulation of Hkv*256 non-negative terms against the fp64 oracle
    np.testing.assert_allclose(s[:L_d].cpu().numpy().astype(np.float64), ref, rtol=2e-5, atol=0)
    assert float(s[L_d]) == -1.0, "wrote past the end"
    # the selection that follows ranks exactly these fp32 scores: the rows it keeps must dominate the rest
    # in the oracle's scores up to the fp32 rounding of the signal
    k = api.daf_num_important(L_d, 0.1)
    if k > 0 and k < L_d:
        ws = api.alloc_workspace(p)
        z = torch.zeros(N, 4 * Hkv, 128, dtype=torch.bfloat16, device="cuda")
        kk = torch.zeros(N, Hkv, 128, dtype=torch.bfloat16, device="cuda")
        idx_out = torch.zeros(k, dtype=torch.int32, device="cuda")
        qp = torch.zeros(k, 4 * Hkv, 128, dtype=torch.bfloat16, device="cuda")
        kp = torch.zeros(k, Hkv, 128, dtype=torch.bfloat16, device="cuda")
        _ok(api.daf_select(p, s[:L_d].contiguous(), 1, None, z, kk, kk.clone(), kk.clone(), kk.clone(), idx_out, qp, kp,
                           kp.clone(), ws), ws, "daf_select on deviation scores")
        sel = np.zeros(L_d, dtype=bool)
        sel[idx_out.cpu().numpy()] = True
        assert sel.sum() == k
        assert ref[sel].min() >= ref[~sel].max() * (1 - 1e-4)


@pytest.mark.parametrize("L_d,L_q,Hkv,n_sig,r", [(1024, 32, 4, 3, 0.15), (6144, 64, 4, 3, 0.15), (777, 0, 8, 1, 0.3),
                                                 (20000, 16, 8, 2, 0.1), (40, 3, 1, 8, 0.5)])
def test_selection_straight_from_the_signal_layers_kv(L_d, L_q, Hkv, n_sig, r):
    """daf_select_from_kv: the aggregated signal equals the per-layer signals of daf_deviation_scores added in
    ascending layer order in fp32 (bit for bit), agrees with the fp64 oracle within the signal's tolerance, and the
    selected positions are exactly what the oracle's selection gives on those fp32 sums; gather and cache update
    as in daf_select."""
    dev = "cuda"
    N, Hq = L_d + L_q, 2 * Hkv
    layers = []
    for l in range(n_sig):
        kf, vf = _normal((N, Hkv, 128), 500 + 10 * l).to(dev), _normal((N, Hkv, 128), 501 + 10 * l).to(dev)
        # offline rows: the fresh ones plus a perturbation whose size varies from token to token
        g = W.standard_normal(L_d, 600 + l).float().abs().view(L_d, 1, 1).to(dev)
        kc = (kf[:L_d].float() + 0.2 * g * _normal((L_d, Hkv, 128), 502 + 10 * l).to(dev).float()).to(torch.bfloat16)
        vc = (vf[:L_d].float() + 0.1 * g * _normal((L_d, Hkv, 128), 503 + 10 * l).to(dev).float()).to(torch.bfloat16)
        layers.append((kf, vf, kc, vc))
    p = api.make_params(L_d, L_q, r, Hq, Hkv)
    k = api.daf_num_important(L_d, r)
    ws = api.alloc_workspace(p)
    # the layer being processed
    q_fresh, k_fresh, v_fresh = _normal((N, Hq, 128), 700).to(dev), _normal((N, Hkv, 128), 701).to(dev), _normal((N, Hkv, 128), 702).to(dev)
    k_cached, v_cached = _normal((L_d, Hkv, 128), 703).to(dev), _normal((L_d, Hkv, 128), 704).to(dev)
    kv_k = torch.cat([k_cached, torch.zeros(L_q, Hkv, 128, dtype=torch.bfloat16, device=dev)])
    kv_v = torch.cat([v_cached, torch.zeros(L_q, Hkv, 128, dtype=torch.bfloat16, device=dev)])
    idx_out = torch.full((max(k, 1),), -1, dtype=torch.int32, device=dev)
    qp = torch.zeros(max(k, 1), Hq, 128, dtype=torch.bfloat16, device=dev)
    kp = torch.zeros(max(k, 1), Hkv, 128, dtype=torch.bfloat16, device=dev)
    vp = torch.zeros_like(kp)
    sums = torch.full((L_d + 4,), -1.0, dtype=torch.float32, device=dev)
    _ok(api.daf_select_from_kv(p, [x[0] for x in layers], [x[1] for x in layers], [x[2] for x in layers],
                               [x[3] for x in layers], q_fresh, k_fresh, v_fresh, kv_k, kv_v, idx_out, qp, kp, vp, sums, ws),
        ws, "daf_select_from_kv")
    assert torch.all(sums[L_d:] == -1.0), "wrote past the end of the sums"
    got = sums[:L_d].cpu().numpy()
    # (1) per-layer signals from the stand-alone kernel, added in ascending order in fp32
    rows = []
    for kf, vf, kc, vc in layers:
        row = torch.zeros(L_d, dtype=torch.float32, device=dev)
        api.check(api.daf_deviation_scores(p, kf, vf, kc, vc, row), "daf_deviation_scores")
        rows.append(row.cpu().numpy())
    acc = rows[0].copy()
    for row in rows[1:]:
        acc = (acc + row).astype(np.float32)
    assert np.array_equal(got.view(np.uint32), acc.view(np.uint32)), "aggregate differs from the per-layer rows added in order"
    # (2) against the oracle's fp64 signal
    ref = sum(oracle.deviation_scores(_f(kf), _f(vf), _f(kc), _f(vc), L_d) for kf, vf, kc, vc in layers)
    np.testing.assert_allclose(got.astype(np.float64), ref, rtol=2e-5, atol=0)
    # (3) positions: the oracle's selection on the same fp32 sums, bit-exact; and the oracle's aggregation of
    #     the per-layer rows gives the same sums
    assert np.array_equal(oracle.aggregate(np.stack(rows)).view(np.uint32), got.view(np.uint32))
    idx = oracle.select(got[None, :], k)
    assert np.array_equal(idx_out[:k].cpu().numpy(), idx)
    # (4) gather and hybrid cache, byte-exact
    it = torch.from_numpy(idx).long().to(dev)
    assert torch.equal(qp[:k], q_fresh[it]) and torch.equal(kp[:k], k_fresh[it]) and torch.equal(vp[:k], v_fresh[it])
    exp_k = torch.cat([k_cached, k_fresh[L_d:]]); exp_k[it] = k_fresh[it]
    exp_v = torch.cat([v_cached, v_fresh[L_d:]]); exp_v[it] = v_fresh[it]
    assert torch.equal(kv_k, exp_k) and torch.equal(kv_v, exp_v)


# --------------------------------------------------------------------------- gather / hybrid cache / fusion
@pytest.mark.parametrize("name,Hq,Hkv,L_d,L_q,r", [("c0", 28, 4, 1024, 32, 0.15), ("x", 8, 8, 300, 7, 0.4),
                                                  ("y", 40, 8, 513, 0, 0.2), ("z", 4, 1, 64, 5, 0.0)])
def test_gather_hybrid_cache_and_fuse_bit_exact(name, Hq, Hkv, L_d, L_q, r):
    w = W.Workload(name, 11, Hq, Hkv, 128, 1, L_d, L_d, L_q, r, "lognormal")
    L = W.make_layer(w, 0)
    dev = "cuda"
    p = api.make_params(L_d, L_q, r, Hq, Hkv)
    k = api.daf_num_important(L_d, r)
    ws = api.alloc_workspace(p)
    N = L_d + L_q
    g = {n: L[n].to(dev) for n in ("q_fresh", "k_fresh", "v_fresh")}
    kvk = torch.zeros(N, Hkv, 128, dtype=torch.bfloat16, device=dev)
    kvv = torch.zeros_like(kvk)
    kvk[:L_d], kvv[:L_d] = L["k_cached"].to(dev), L["v_cached"].to(dev)
    kvk[L_d:], kvv[L_d:] = 7.0, 7.0  # stale question rows must be replaced
    idx_out = torch.full((max(k, 1),), -1, dtype=torch.int32, device=dev)
    qp = torch.full((max(k, 1), Hq, 128), 3.0, dtype=torch.bfloat16, device=dev)
    kp = torch.full((max(k, 1), Hkv, 128), 3.0, dtype=torch.bfloat16, device=dev)
    vp = torch.full_like(kp, 3.0)
    _ok(api.daf_select(p, L["scores"].to(dev), 1, None, g["q_fresh"], g["k_fresh"], g["v_fresh"], kvk, kvv, idx_out,
                       qp, kp, vp, ws), ws, "daf_select")
    idx = oracle.select(L["scores"].numpy(), k)
    assert np.array_equal(idx_out[:k].cpu().numpy(), idx)
    assert np.array_equal(_f(qp[:k]), oracle.gather_rows(_f(L["q_fresh"]), idx))
    assert np.array_equal(_f(kp[:k]), oracle.gather_rows(_f(L["k_fresh"]), idx))
    assert np.array_equal(_f(vp[:k]), oracle.gather_rows(_f(L["v_fresh"]), idx))
    assert np.array_equal(_f(kvk), oracle.hybrid_kv(_f(L["k_cached"]), _f(L["k_fresh"]), idx, L_d, L_q))
    assert np.array_equal(_f(kvv), oracle.hybrid_kv(_f(L["v_cached"]), _f(L["v_fresh"]), idx, L_d, L_q))
    # the same call with given indices and without overwriting the document rows
    p0 = api.make_params(L_d, L_q, r, Hq, Hkv, overwrite_doc_kv=0)
    kvk0 = torch.zeros_like(kvk)
    kvk0[:L_d] = L["k_cached"].to(dev)
    kvv0 = kvk0.clone()
    idx_in = torch.from_numpy(idx).to(dev) if k else None
    idx_out2 = torch.full((max(k, 1),), -1, dtype=torch.int32, device=dev)
    _ok(api.daf_select(p0, None, 0, idx_in, g["q_fresh"], g["k_fresh"], g["v_fresh"], kvk0, kvv0, idx_out2, qp, kp,
                       vp, ws), ws, "daf_select(idx_in)")
    assert np.array_equal(idx_out2[:k].cpu().numpy(), idx)
    assert np.array_equal(_f(kvk0), oracle.hybrid_kv(_f(L["k_cached"]), _f(L["k_fresh"]), idx, L_d, L_q, overwrite=False))
    # stand-alone fusion: compact and scatter placement, canary rows untouched
    o_imp = _normal((max(k, 1), Hq, 128), 5).to(dev)
    o_q = _normal((max(L_q, 1), Hq, 128), 6).to(dev)
    for mode in (0, 1):
        pm = api.make_params(L_d, L_q, r, Hq, Hkv, fuse_mode=mode)
        rows = k + L_q if mode == 0 else N
        hidden = torch.full((rows + 2, Hq, 128), -9.0, dtype=torch.bfloat16, device=dev)  # 2 canary rows
        row_pos = torch.full((max(k + L_q, 1),), -1, dtype=torch.int32, device=dev)
        api.check(api.daf_fuse(pm, k, idx_in, o_imp, o_q, hidden, row_pos), "daf_fuse")
        torch.cuda.synchronize()
        base = np.full((rows, Hq, 128), -9.0)
        ref, ref_pos = oracle.fuse(_f(o_imp[:k]).astype(np.float64), _f(o_q[:L_q]).astype(np.float64), idx, L_d,
                                   mode, hidden=base if mode == 1 else None)
        assert np.array_equal(_f(hidden[:rows]).astype(np.float64), ref)
        assert np.all(_f(hidden[rows:]) == -9.0)
        assert np.array_equal(row_pos[: k + L_q].cpu().numpy(), ref_pos)


# --------------------------------------------------------------------------- attention stages
@pytest.mark.parametrize("n,Hq,Hkv,qscale", [(154, 28, 4, 1.0), (1, 4, 2, 1.0), (128, 4, 4, 1.0), (129, 8, 2, 1.0),
                                             (300, 40, 8, 1.0), (257, 4, 1, 4.0), (922, 28, 4, 1.0)])
def test_important_attention_matches_oracle(n, Hq, Hkv, qscale):
    q, k, v = _normal((n, Hq, 128), 21, qscale), _normal((n, Hkv, 128), 22), _normal((n, Hkv, 128), 23)
    p = api.make_params(max(n, 1), 0, 1.0, Hq, Hkv)
    ws = api.alloc_workspace(p)
    out = torch.full((n + 1, Hq, 128), 5.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(Hq, n, dtype=torch.float32, device="cuda")
    _ok(api.daf_important_attn(p, n, q.cuda(), k.cuda(), v.cuda(), out, Hq * 256, None, lse, ws), ws, "daf_important_attn")
    scale = 1.0 / math.sqrt(128)
    ref, ref_lse = oracle.important_attn(_f(q), _f(k), _f(v), scale, return_lse=True)
    _assert_close(out[:n], ref, f"important attention n={n}")
    assert torch.all(out[n] == 5.0), "row past the end was written"
    np.testing.assert_allclose(lse.cpu().numpy().T, ref_lse, atol=2e-3, rtol=0)
    # first packed row sees one key: its output is that value row exactly
    assert np.array_equal(_f(out[0]), np.repeat(_f(v[0]), Hq // Hkv, axis=0))


def test_important_attention_scatters_rows_through_dst_rows():
    n, Hq, Hkv = 200, 4, 2
    q, k, v = _normal((n, Hq, 128), 31), _normal((n, Hkv, 128), 32), _normal((n, Hkv, 128), 33)
    dst = torch.randperm(400, generator=torch.Generator().manual_seed(1))[:n].sort().values.to(torch.int32)
    p = api.make_params(n, 0, 1.0, Hq, Hkv)
    ws = api.alloc_workspace(p)
    out = torch.full((400, Hq, 128), 5.0, dtype=torch.bfloat16, device="cuda")
    _ok(api.daf_important_attn(p, n, q.cuda(), k.cuda(), v.cuda(), out, Hq * 256, dst.cuda(), None, ws), ws, "imp")
    ref = oracle.important_attn(_f(q), _f(k), _f(v), 1.0 / math.sqrt(128))
    _assert_close(out[dst.long().cuda()], ref, "scattered rows")
    others = np.setdiff1d(np.arange(400), dst.numpy())
    assert torch.all(out[torch.from_numpy(others).cuda()] == 5.0)


@pytest.mark.parametrize("L_d,L_q,r,Hq,Hkv,mode", [(1024, 32, 0.15, 28, 4, 0), (1024, 32, 0.15, 28, 4, 1), (3000, 130, 0.3, 8, 2, 1),
                                                  (700, 9, 0.5, 5, 5, 0)])
def test_fused_epilogue_rows_equal_unfused_rows_plus_daf_fuse_bit_for_bit(L_d, L_q, r, Hq, Hkv, mode):
    """State fusion done by the attention epilogues (out / dst_rows of the two stand-alone attention calls)
    gives exactly the bytes of the same two calls writing their own buffers followed by daf_fuse."""
    dev = "cuda"
    N = L_d + L_q
    p = api.make_params(L_d, L_q, r, Hq, Hkv, fuse_mode=mode)
    k = api.daf_num_important(L_d, r)
    ws = api.alloc_workspace(p)
    qp, kp, vp = (_normal((k, h, 128), 70 + i).to(dev) for i, h in enumerate((Hq, Hkv, Hkv)))
    qq, kk, vv = _normal((L_q, Hq, 128), 80).to(dev), _normal((N, Hkv, 128), 81).to(dev), _normal((N, Hkv, 128), 82).to(dev)
    idx = torch.randperm(L_d, generator=torch.Generator().manual_seed(3))[:k].sort().values.to(torch.int32).to(dev)
    row = Hq * 256
    # unfused: each stage into its own buffer, then the stand-alone fusion
    o_imp = torch.zeros(k, Hq, 128, dtype=torch.bfloat16, device=dev)
    o_q = torch.zeros(L_q, Hq, 128, dtype=torch.bfloat16, device=dev)
    _ok(api.daf_important_attn(p, k, qp, kp, vp, o_imp, row, None, None, ws), ws, "imp")
    _ok(api.daf_qd_attn(p, qq, kk, vv, o_q, row, None, None, ws), ws, "qd")
    rows_total = N if mode == 1 else k + L_q
    unfused = torch.full((rows_total, Hq, 128), 3.0, dtype=torch.bfloat16, device=dev)
    api.check(api.daf_fuse(p, k, idx, o_imp, o_q, unfused, None), "daf_fuse")
    # fused: the same two calls write the final rows themselves
    fused = torch.full((rows_total, Hq, 128), 3.0, dtype=torch.bfloat16, device=dev)
    if mode == 0:
        _ok(api.daf_important_attn(p, k, qp, kp, vp, fused, row, None, None, ws), ws, "imp fused")
        _ok(api.daf_qd_attn(p, qq, kk, vv, fused, row, None, None, ws, out_offset_bytes=k * row), ws, "qd fused")
    else:
        dst_q = torch.arange(L_d, N, dtype=torch.int32, device=dev)
        _ok(api.daf_important_attn(p, k, qp, kp, vp, fused, row, idx, None, ws), ws, "imp fused")
        _ok(api.daf_qd_attn(p, qq, kk, vv, fused, row, dst_q, None, ws), ws, "qd fused")
    torch.cuda.synchronize()
    assert torch.equal(fused.view(torch.int16), unfused.view(torch.int16))


@pytest.mark.parametrize("L_d,L_q,Hq,Hkv,qscale", [(1024, 32, 28, 4, 1.0), (1000, 1, 4, 4, 1.0), (333, 17, 8, 2, 1.0),
                                                   (2048, 128, 40, 8, 1.0), (640, 64, 32, 8, 4.0), (100, 130, 4, 1, 1.0),
                                                   (6144, 64, 28, 4, 1.0)])
def test_question_attention_matches_oracle(L_d, L_q, Hq, Hkv, qscale):
    N = L_d + L_q
    q, k, v = _normal((L_q, Hq, 128), 41, qscale), _normal((N, Hkv, 128), 42), _normal((N, Hkv, 128), 43)
    p = api.make_params(L_d, L_q, 0.1, Hq, Hkv)
    ws = api.alloc_workspace(p)
    out = torch.full((L_q + 1, Hq, 128), 5.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(Hq, L_q, dtype=torch.float32, device="cuda")
    _ok(api.daf_qd_attn(p, q.cuda(), k.cuda(), v.cuda(), out, Hq * 256, None, lse, ws), ws, "daf_qd_attn")
    ref, ref_lse = oracle.qd_attn(_f(q), _f(k), _f(v), L_d, 1.0 / math.sqrt(128), return_lse=True)
    _assert_close(out[:L_q], ref, f"question attention L_d={L_d} L_q={L_q}")
    assert torch.all(out[L_q] == 5.0)
    np.testing.assert_allclose(lse.cpu().numpy().T, ref_lse, atol=2e-3, rtol=0)


@pytest.mark.parametrize("n,Hq,Hkv", [(1056, 28, 4), (513, 8, 8)])
def test_full_causal_attention_matches_oracle(n, Hq, Hkv):
    q, k, v = _normal((n, Hq, 128), 51), _normal((n, Hkv, 128), 52), _normal((n, Hkv, 128), 53)
    p = api.make_params(n, 0, 1.0, Hq, Hkv)
    ws = api.alloc_workspace(p)
    out = torch.zeros(n, Hq, 128, dtype=torch.bfloat16, device="cuda")
    _ok(api.daf_full_causal_attn(p, n, q.cuda(), k.cuda(), v.cuda(), out, None, ws), ws, "daf_full_causal_attn")
    ref = oracle.full_causal_attn(_f(q), _f(k), _f(v), 1.0 / math.sqrt(128))
    _assert_close(out, ref, f"full causal n={n}")


@pytest.mark.parametrize("L_d,L_q,r,Hq,Hkv", [(1024, 32, 0.15, 28, 4), (700, 5, 0.3, 8, 2), (2048, 128, 0.05, 40, 8),
                                               (300, 0, 1.0, 4, 4)])
def test_full_context_variant_matches_oracle(L_d, L_q, r, Hq, Hkv):
    w = W.Workload("b", 31, Hq, Hkv, 128, 1, L_d, L_d, L_q, r, "lognormal")
    L = W.make_layer(w, 0)
    k = api.daf_num_important(L_d, r)
    idx = oracle.select(L["scores"].numpy(), k)
    pos = np.concatenate([idx, np.arange(L_d, L_d + L_q, dtype=np.int32)]).astype(np.int32)
    kv_k = torch.cat([L["k_cached"], L["k_fresh"][L_d:]], 0)
    kv_v = torch.cat([L["v_cached"], L["v_fresh"][L_d:]], 0)
    it = torch.from_numpy(idx).long()
    kv_k[it], kv_v[it] = L["k_fresh"][it], L["v_fresh"][it]
    q_rows = L["q_fresh"][torch.from_numpy(pos).long()].contiguous()
    p = api.make_params(L_d, L_q, r, Hq, Hkv)
    ws = api.alloc_workspace(p)
    n = len(pos)
    out = torch.full((n + 1, Hq, 128), 5.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(Hq, n, dtype=torch.float32, device="cuda")
    _ok(api.daf_blend_attn(p, n, q_rows.cuda(), kv_k.cuda(), kv_v.cuda(), torch.from_numpy(pos).cuda(), out, Hq * 256,
                           lse, ws), ws, "daf_blend_attn")
    ref, ref_lse = oracle.blend_attn(_f(q_rows), _f(kv_k), _f(kv_v), pos, 1.0 / math.sqrt(128), return_lse=True)
    _assert_close(out[:n], ref, f"full-context variant L_d={L_d}")
    assert torch.all(out[n] == 5.0)
    np.testing.assert_allclose(lse.cpu().numpy().T, ref_lse, atol=2e-3, rtol=0)


def test_closed_forms_on_the_gpu():
    """Zero keys give the running mean of the values; constant values come back unchanged."""
    n, Hq, Hkv = 260, 4, 2
    q, v = _normal((n, Hq, 128), 61), _normal((n, Hkv, 128), 62)
    k = torch.zeros(n, Hkv, 128, dtype=torch.bfloat16)
    p = api.make_params(n, 0, 1.0, Hq, Hkv)
    ws = api.alloc_workspace(p)
    out = torch.zeros(n, Hq, 128, dtype=torch.bfloat16, device="cuda")
    _ok(api.daf_important_attn(p, n, q.cuda(), k.cuda(), v.cuda(), out, Hq * 256, None, None, ws), ws, "imp")
    mean = np.cumsum(_f(v).astype(np.float64), axis=0) / np.arange(1, n + 1)[:, None, None]
    _assert_close(out, np.repeat(mean, 2, axis=1), "running mean")
    vc = torch.full((n, Hkv, 128), 1.75, dtype=torch.bfloat16)
    _ok(api.daf_important_attn(p, n, q.cuda(), _normal((n, Hkv, 128), 63).cuda(), vc.cuda(), out, Hq * 256, None, None, ws), ws, "imp")
    assert torch.all((out.float() - 1.75).abs() <= 1.75 * 2 ** -7)


# --------------------------------------------------------------------------- whole layer
def _run_layer(w, layer, fuse_mode, host=False):
    L = W.make_layer(w, layer)
    dev = "cuda"
    p = api.make_params(w.L_d, w.L_q, w.r, w.n_q_heads, w.n_kv_heads, fuse_mode=fuse_mode)
    k = api.daf_num_important(w.L_d, w.r)
    N, Hq, Hkv = w.N, w.n_q_heads, w.n_kv_heads
    rows = k + w.L_q if fuse_mode == 0 else N
    kv_k = torch.zeros(N, Hkv, 128, dtype=torch.bfloat16)
    kv_v = torch.zeros_like(kv_k)
    kv_k[: w.L_d], kv_v[: w.L_d] = L["k_cached"], L["v_cached"]
    n_sig = 0 if L["scores"] is None else L["scores"].shape[0]
    if host:
        arena = torch.zeros(api.daf_layer_host_arena_bytes(p), dtype=torch.uint8, device=dev)
        hidden = torch.full((rows, Hq, 128), -9.0, dtype=torch.bfloat16).pin_memory()
        idx_out = torch.full((max(k, 1),), -1, dtype=torch.int32)
        pin = lambda t: None if t is None else t.pin_memory()  # noqa: E731
        st = api.daf_layer_host(p, pin(L["scores"]), n_sig, pin(L["idx_in"]), pin(L["q_fresh"]), pin(L["k_fresh"]),
                                pin(L["v_fresh"]), kv_k, kv_v, 1, hidden, idx_out, arena)
        api.check(st, "daf_layer_host")
        return L, hidden, idx_out[:k].numpy(), None, kv_k, kv_v
    g = {n: (None if t is None else t.to(dev)) for n, t in L.items()}
    kv_k, kv_v = kv_k.to(dev), kv_v.to(dev)
    ws = api.alloc_workspace(p)
    idx_out = torch.full((max(k, 1),), -1, dtype=torch.int32, device=dev)
    qp = torch.zeros(max(k, 1), Hq, 128, dtype=torch.bfloat16, device=dev)
    kp = torch.zeros(max(k, 1), Hkv, 128, dtype=torch.bfloat16, device=dev)
    vp = torch.zeros_like(kp)
    hidden = torch.full((rows, Hq, 128), -9.0, dtype=torch.bfloat16, device=dev)
    row_pos = torch.full((max(k + w.L_q, 1),), -1, dtype=torch.int32, device=dev)
    _ok(api.daf_layer(p, g["scores"], n_sig, g["idx_in"], g["q_fresh"], g["k_fresh"], g["v_fresh"], kv_k, kv_v,
                      idx_out, qp, kp, vp, hidden, row_pos, ws), ws, "daf_layer")
    return L, hidden.cpu(), idx_out[:k].cpu().numpy(), row_pos[: k + w.L_q].cpu().numpy(), kv_k.cpu(), kv_v.cpu()


def _oracle_layer(w, L, fuse_mode, overwrite=1):
    base = np.full((w.N, w.n_q_heads, 128), -9.0) if fuse_mode == 1 else None
    return oracle.daf_layer(_f(L["q_fresh"]), _f(L["k_fresh"]), _f(L["v_fresh"]), _f(L["k_cached"]), _f(L["v_cached"]),
                            w.L_d, w.L_q, w.softmax_scale,
                            scores=None if L["scores"] is None else L["scores"].numpy(),
                            idx=None if L["idx_in"] is None else L["idx_in"].numpy(), r=w.r, fuse_mode=fuse_mode,
                            overwrite=bool(overwrite), hidden=base)


def test_host_layer_from_pageable_and_from_pinned_fresh_tensors_agree():
    """daf_layer_host reads the needed fresh rows straight from pinned host tensors and copies pageable ones whole:
    the same bits either way."""
    w = W.Workload("t", 37, 8, 2, 128, 1, 1100, 500, 33, 0.3, "lognormal", 1)
    dev = "cuda"
    p = api.make_params(w.L_d, w.L_q, w.r, w.n_q_heads, w.n_kv_heads)
    k = api.daf_num_important(w.L_d, w.r)
    L = W.make_layer(w, 0)
    arena = torch.zeros(api.daf_layer_host_arena_bytes(p), dtype=torch.uint8, device=dev)
    outs = []
    for pinned in (True, False):
        fresh = {n: (L[n].pin_memory() if pinned else L[n].clone()) for n in ("q_fresh", "k_fresh", "v_fresh")}
        assert all(t.is_pinned() == pinned for t in fresh.values())
        kv_k = torch.zeros(w.N, w.n_kv_heads, 128, dtype=torch.bfloat16)
        kv_v = torch.zeros_like(kv_k)
        kv_k[: w.L_d], kv_v[: w.L_d] = L["k_cached"], L["v_cached"]
        hidden = torch.full((k + w.L_q, w.n_q_heads, 128), -9.0, dtype=torch.bfloat16).pin_memory()
        idx_out = torch.full((k,), -1, dtype=torch.int32)
        api.check(api.daf_layer_host(p, L["scores"], 1, None, fresh["q_fresh"], fresh["k_fresh"], fresh["v_fresh"], kv_k, kv_v, 1,
                                     hidden, idx_out, arena), "daf_layer_host")
        outs.append((hidden.clone(), idx_out, kv_k, kv_v))
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a, b)
    ref = _oracle_layer(w, L, 0)
    assert np.array_equal(outs[0][1].numpy(), ref["idx"])
    assert np.array_equal(_f(outs[0][2]), ref["kv_k"]) and np.array_equal(_f(outs[0][3]), ref["kv_v"])
    _assert_close(outs[0][0], ref["hidden"], "hidden rows from pinned host tensors")


def test_host_layers_pipelined_on_two_arenas_match_the_plain_host_call():
    """daf_layer_host_begin / _end with two arenas and two streams (layer i + 1 begun before layer i is ended) give,
    layer by layer, exactly what daf_layer_host gives."""
    w = W.Workload("t", 31, 8, 2, 128, 5, 1200, 500, 40, 0.25, "lognormal", 2)
    dev = "cuda"
    p = api.make_params(w.L_d, w.L_q, w.r, w.n_q_heads, w.n_kv_heads)
    k = api.daf_num_important(w.L_d, w.r)
    pin = lambda t: None if t is None else t.pin_memory()  # noqa: E731

    def host_layer(i):
        L = W.make_layer(w, i)
        h = {n: pin(t) for n, t in L.items()}
        for n, src in (("kv_k", "k_cached"), ("kv_v", "v_cached")):
            h[n] = torch.zeros(w.N, w.n_kv_heads, 128, dtype=torch.bfloat16).pin_memory()
            h[n][: w.L_d] = L[src]
        h["hidden"] = torch.full((k + w.L_q, w.n_q_heads, 128), -9.0, dtype=torch.bfloat16).pin_memory()
        h["idx_out"] = torch.full((k,), -1, dtype=torch.int32).pin_memory()
        return h

    def args(h, arena):
        return (p, h["scores"], 2, h["idx_in"], h["q_fresh"], h["k_fresh"], h["v_fresh"], h["kv_k"], h["kv_v"], 1,
                h["hidden"], h["idx_out"], arena)

    plain = [host_layer(i) for i in range(w.layers)]
    arena = torch.zeros(api.daf_layer_host_arena_bytes(p), dtype=torch.uint8, device=dev)
    for h in plain:
        api.check(api.daf_layer_host(*args(h, arena)), "daf_layer_host")
    piped = [host_layer(i) for i in range(w.layers)]
    arenas = [torch.zeros_like(arena) for _ in range(2)]
    lanes = [torch.cuda.Stream(), torch.cuda.Stream()]
    pending = None
    for i, h in enumerate(piped):
        api.check(api.daf_layer_host_begin(*args(h, arenas[i & 1]), stream=lanes[i & 1]), "begin")
        if pending is not None:
            api.check(api.daf_layer_host_end(p, arenas[pending], stream=lanes[pending]), "end")
        pending = i & 1
    api.check(api.daf_layer_host_end(p, arenas[pending], stream=lanes[pending]), "end")
    for a, b in zip(plain, piped):
        for n in ("hidden", "idx_out", "kv_k", "kv_v"):
            assert torch.equal(a[n], b[n]), n
    assert not torch.equal(plain[0]["hidden"], plain[1]["hidden"])   # the layers do differ


@pytest.mark.parametrize("fuse_mode", [0, 1])
def test_layer_smallest_configuration(fuse_mode):
    w = W.CONFIGS["c0"]
    L, hidden, idx, row_pos, kv_k, kv_v = _run_layer(w, 0, fuse_mode)
    ref = _oracle_layer(w, L, fuse_mode)
    assert np.array_equal(idx, ref["idx"])
    assert np.array_equal(row_pos, ref["row_pos"])
    assert np.array_equal(_f(kv_k), ref["kv_k"]) and np.array_equal(_f(kv_v), ref["kv_v"])
    if fuse_mode == 0:
        _assert_close(hidden, ref["hidden"], "fused hidden rows (compact)")
    else:
        rows = ref["row_pos"]
        _assert_close(hidden[rows], ref["hidden"][rows], "fused hidden rows (scatter)")
        others = np.setdiff1d(np.arange(w.N), rows)
        assert torch.all(hidden[others] == -9.0), "a row that is neither important nor a question row was written"
    # fused epilogues and the stand-alone stages + fusion pass agree up to the last bf16 bit or two: the
    # layer cuts the key axis into different ranges than the stand-alone stages, so the fp32 sums are
    # associated differently before the final rounding
    p = api.make_params(w.L_d, w.L_q, w.r, w.n_q_heads, w.n_kv_heads, fuse_mode=fuse_mode)
    ws = api.alloc_workspace(p)
    k = len(idx)
    dev = "cuda"
    idx_d = torch.from_numpy(idx).to(dev)
    Hq = w.n_q_heads
    o_imp = torch.zeros(k, Hq, 128, dtype=torch.bfloat16, device=dev)
    o_q = torch.zeros(w.L_q, Hq, 128, dtype=torch.bfloat16, device=dev)
    qp = L["q_fresh"][idx].to(dev); kp = L["k_fresh"][idx].to(dev); vp = L["v_fresh"][idx].to(dev)
    _ok(api.daf_important_attn(p, k, qp, kp, vp, o_imp, Hq * 256, None, None, ws), ws, "imp")
    _ok(api.daf_qd_attn(p, L["q_fresh"][w.L_d:].to(dev), kv_k.to(dev), kv_v.to(dev), o_q, Hq * 256, None, None, ws), ws, "qd")
    h2 = torch.full(hidden.shape, -9.0, dtype=torch.bfloat16, device=dev)
    api.check(api.daf_fuse(p, k, idx_d, o_imp, o_q, h2, None), "daf_fuse")
    torch.cuda.synchronize()
    assert torch.allclose(h2.cpu().float(), hidden.float(), rtol=2.0 ** -6, atol=2e-3)
    assert torch.equal(h2.cpu() == -9.0, hidden == -9.0)


def test_layer_with_selection_and_three_signal_rows():
    w = W.Workload("m", 21, 8, 2, 128, 1, 2000, 500, 48, 0.13, "lognormal", 3)
    L, hidden, idx, row_pos, kv_k, kv_v = _run_layer(w, 0, 0)
    ref = _oracle_layer(w, L, 0)
    assert np.array_equal(idx, ref["idx"]) and np.array_equal(row_pos, ref["row_pos"])
    assert np.array_equal(_f(kv_k), ref["kv_k"])
    _assert_close(hidden, ref["hidden"], "layer m")


def test_layer_host_buffers():
    w = W.Workload("h", 22, 8, 2, 128, 1, 1500, 500, 40, 0.2, "pareto_clustered", 1)
    L, hidden, idx, _, kv_k, kv_v = _run_layer(w, 0, 0, host=True)
    ref = _oracle_layer(w, L, 0)
    assert np.array_equal(idx, ref["idx"])
    assert np.array_equal(_f(kv_k), ref["kv_k"]) and np.array_equal(_f(kv_v), ref["kv_v"])
    _assert_close(hidden, ref["hidden"], "layer through host buffers")


def test_degenerate_sizes():
    # r = 1 and no question: the layer is full causal attention
    w = W.Workload("d1", 23, 4, 2, 128, 1, 200, 100, 0, 1.0, "lognormal", 1)
    L, hidden, idx, _, _, _ = _run_layer(w, 0, 0)
    assert np.array_equal(idx, np.arange(200))
    ref_full = oracle.full_causal_attn(_f(L["q_fresh"]), _f(L["k_fresh"]), _f(L["v_fresh"]), w.softmax_scale)
    _assert_close(hidden, ref_full, "r=1, L_q=0")
    # r = 0: only the question stage runs
    w0 = W.Workload("d0", 24, 4, 2, 128, 1, 200, 100, 9, 0.0, "lognormal", 1)
    L0, hidden0, idx0, row_pos0, kv_k0, _ = _run_layer(w0, 0, 0)
    ref0 = _oracle_layer(w0, L0, 0)
    assert len(idx0) == 0 and np.array_equal(row_pos0, ref0["row_pos"])
    _assert_close(hidden0, ref0["hidden"], "r=0")


def test_fresh_change_at_non_important_row_is_invisible():
    """The hybrid-cache reading: only important rows of the document cache are replaced."""
    w = W.CONFIGS["c0"]
    L, hidden, idx, _, _, _ = _run_layer(w, 0, 0)
    non_imp = int(np.setdiff1d(np.arange(w.L_d), idx)[0])
    orig = W.make_layer

    def patched(wl, layer, device="cpu"):
        out = orig(wl, layer, device)
        out["k_fresh"][non_imp] += 3.0
        out["v_fresh"][non_imp] -= 2.0
        return out

    W.make_layer = patched
    try:
        _, hidden2, idx2, _, _, _ = _run_layer(w, 0, 0)
    finally:
        W.make_layer = orig
    assert np.array_equal(idx, idx2) and torch.equal(hidden, hidden2)


# --------------------------------------------------------------------------- device-side status, edge shapes
def test_status_word_makes_kernels_stand_down_and_is_reported_once():
    """A failure recorded in the workspace makes later attention kernels return without touching their
    outputs; daf_poll_status reports it once and clears it (no GPU fault is involved anywhere)."""
    n, Hq, Hkv = 300, 4, 2
    q, k, v = _normal((n, Hq, 128), 81), _normal((n, Hkv, 128), 82), _normal((n, Hkv, 128), 83)
    p = api.make_params(n, 0, 1.0, Hq, Hkv)
    ws = api.alloc_workspace(p)
    ws.view(torch.int32)[0] = api.DAF_ERR_TIMEOUT          # as a CTA whose bounded wait ran out would leave it
    out = torch.full((n, Hq, 128), 5.0, dtype=torch.bfloat16, device="cuda")
    api.check(api.daf_important_attn(p, n, q.cuda(), k.cuda(), v.cuda(), out, Hq * 256, None, None, ws), "launch")
    torch.cuda.synchronize()
    assert torch.all(out == 5.0), "a kernel ran although the workspace carried a failure"
    assert api.daf_poll_status(ws) == api.DAF_ERR_TIMEOUT
    assert api.daf_poll_status(ws) == api.DAF_OK            # reported once, then cleared
    _ok(api.daf_important_attn(p, n, q.cuda(), k.cuda(), v.cuda(), out, Hq * 256, None, None, ws), ws, "after clearing")
    _assert_close(out, oracle.important_attn(_f(q), _f(k), _f(v), 1.0 / math.sqrt(128)), "after clearing")


def test_bounded_wait_runs_out_reports_and_leaves_the_context_usable():
    """The wait every kernel relies on, pointed at a barrier that nothing signals: it gives up after the
    limit, the status word says so, nothing faults, and the next call computes as usual."""
    import time
    n, Hq, Hkv = 200, 4, 2
    p = api.make_params(n, 0, 1.0, Hq, Hkv)
    ws = api.alloc_workspace(p)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    api.check(api.daf_selftest_bounded_wait(ws, 50), "self-test launch")
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    assert 0.04 <= waited < 5.0, f"the wait took {waited:.3f} s for a 50 ms limit"
    assert api.daf_poll_status(ws) == api.DAF_ERR_TIMEOUT
    assert api.daf_poll_status(ws) == api.DAF_OK
    q, k, v = _normal((n, Hq, 128), 91), _normal((n, Hkv, 128), 92), _normal((n, Hkv, 128), 93)
    out = torch.zeros((n, Hq, 128), dtype=torch.bfloat16, device="cuda")
    _ok(api.daf_important_attn(p, n, q.cuda(), k.cuda(), v.cuda(), out, Hq * 256, None, None, ws), ws, "after the self-test")
    _assert_close(out, oracle.important_attn(_f(q), _f(k), _f(v), 1.0 / math.sqrt(128)), "after the self-test")


def test_out_of_range_index_is_skipped_and_reported():
    L_d, L_q, Hq, Hkv = 64, 2, 4, 2
    p = api.make_params(L_d, L_q, 4 / 64, Hq, Hkv)
    assert api.daf_num_important(L_d, 4 / 64) == 4
    ws = api.alloc_workspace(p)
    dev = "cuda"
    qf = _normal((L_d + L_q, Hq, 128), 84).to(dev)
    kf, vf = _normal((L_d + L_q, Hkv, 128), 85).to(dev), _normal((L_d + L_q, Hkv, 128), 86).to(dev)
    kvk, kvv = torch.zeros_like(kf), torch.zeros_like(kf)
    idx_in = torch.tensor([3, 9, 1000, 40], dtype=torch.int32, device=dev)     # 1000 is outside [0, L_d)
    idx_out = torch.zeros(4, dtype=torch.int32, device=dev)
    qp = torch.full((4, Hq, 128), 3.0, dtype=torch.bfloat16, device=dev)
    kp = torch.full((4, Hkv, 128), 3.0, dtype=torch.bfloat16, device=dev)
    vp = torch.full_like(kp, 3.0)
    api.check(api.daf_select(p, None, 0, idx_in, qf, kf, vf, kvk, kvv, idx_out, qp, kp, vp, ws), "daf_select")
    torch.cuda.synchronize()
    assert api.daf_poll_status(ws) == api.DAF_ERR_BOUNDS
    assert torch.all(qp[2] == 3.0) and torch.equal(qp[0], qf[3]) and torch.equal(qp[3], qf[40])


@pytest.mark.parametrize("L_d,r,n_sig", [(6144, 0.15, 1), (20000, 0.1, 3), (300, 1.0, 2), (300, 0.0, 1), (8193, 0.5, 1)])
def test_selection_alone_gives_the_positions_of_the_full_call(L_d, r, n_sig):
    """daf_select_topk writes what daf_select writes to idx_out (and the oracle's selection), and a layer run
    from those positions through idx_in reproduces the layer run from the scores bit for bit."""
    dev = "cuda"
    L_q, Hq, Hkv = 9, 4, 2
    w = W.Workload("st", 13, Hq, Hkv, 128, 1, L_d, L_d, L_q, r, "lognormal", n_sig).with_k(api.daf_num_important)
    L = W.make_layer(w, 0, dev)
    p = api.make_params(L_d, L_q, r, Hq, Hkv)
    k = w.k
    ws = api.alloc_workspace(p)
    idx_sel = torch.full((max(k, 1),), -1, dtype=torch.int32, device=dev)
    _ok(api.daf_select_topk(p, L["scores"], n_sig, idx_sel, ws), ws, "daf_select_topk")
    assert np.array_equal(idx_sel[:k].cpu().numpy(), oracle.select(L["scores"].cpu().numpy(), k))
    if k == 0:
        assert int(idx_sel[0]) == -1
        return
    bf = torch.bfloat16

    def run(scores, idx_in):
        o = dict(kv_k=torch.cat([L["k_cached"], torch.zeros(L_q, Hkv, 128, dtype=bf, device=dev)]),
                 kv_v=torch.cat([L["v_cached"], torch.zeros(L_q, Hkv, 128, dtype=bf, device=dev)]),
                 idx=torch.full((k,), -1, dtype=torch.int32, device=dev), qp=torch.zeros(k, Hq, 128, dtype=bf, device=dev),
                 kp=torch.zeros(k, Hkv, 128, dtype=bf, device=dev), vp=torch.zeros(k, Hkv, 128, dtype=bf, device=dev),
                 hidden=torch.zeros(k + L_q, Hq, 128, dtype=bf, device=dev))
        _ok(api.daf_layer(p, scores, n_sig if scores is not None else 0, idx_in, L["q_fresh"], L["k_fresh"], L["v_fresh"],
                          o["kv_k"], o["kv_v"], o["idx"], o["qp"], o["kp"], o["vp"], o["hidden"], None, ws), ws, "daf_layer")
        return o

    a, b = run(L["scores"], None), run(None, idx_sel)
    for name in a:
        x, y = a[name], b[name]
        assert torch.equal(x.view(torch.int16) if x.dtype == bf else x, y.view(torch.int16) if y.dtype == bf else y), name


@pytest.mark.parametrize("idx,expect", [([3, 9, 40, 63], 0), ([3, 9, 9, 40], -7), ([3, 40, 9, 50], -7), ([0, 1, 2, 64], -7),
                                        ([-1, 1, 2, 3], -7), (list(range(0, 64)), 0), ([5], 0)])
def test_positions_given_by_the_caller_can_be_checked_on_the_device(idx, expect):
    p = api.make_params(64, 2, 0.5, 4, 2)
    ws = api.alloc_workspace(p)
    t = torch.tensor(idx, dtype=torch.int32, device="cuda")
    api.check(api.daf_check_indices(p, len(idx), t, ws), "daf_check_indices")
    torch.cuda.synchronize()
    assert api.daf_poll_status(ws) == expect
    assert api.daf_poll_status(ws) == api.DAF_OK      # reported once


@pytest.mark.parametrize("L_d,L_q,r,Hq,Hkv,n_sig", [(900, 300, 0.2, 4, 4, 1), (512, 40, 1.0, 16, 2, 8),
                                                     (1500, 130, 0.1, 8, 1, 2), (257, 129, 0.5, 12, 4, 3)])
def test_layer_edge_shapes(L_d, L_q, r, Hq, Hkv, n_sig):
    """More than one question token block, group sizes 1 and 8, r = 1 with a question, several signal rows."""
    w = W.Workload("e", 41, Hq, Hkv, 128, 1, L_d, L_d, L_q, r, "lognormal", n_sig)
    for fuse_mode in (0, 1):
        L, hidden, idx, row_pos, kv_k, kv_v = _run_layer(w, 0, fuse_mode)
        ref = _oracle_layer(w, L, fuse_mode)
        assert np.array_equal(idx, ref["idx"]) and np.array_equal(row_pos, ref["row_pos"])
        assert np.array_equal(_f(kv_k), ref["kv_k"]) and np.array_equal(_f(kv_v), ref["kv_v"])
        rows = np.arange(len(ref["row_pos"])) if fuse_mode == 0 else ref["row_pos"]
        _assert_close(hidden[rows], ref["hidden"][rows], f"edge shape L_d={L_d} L_q={L_q} mode={fuse_mode}")


@pytest.mark.parametrize("k,L_d,L_q,Hq,Hkv,fuse_mode", [(700, 2000, 70, 8, 2, 0), (922, 3000, 64, 28, 4, 1),
                                                        (129, 400, 1, 4, 4, 0), (1300, 1300, 260, 4, 1, 1)])
def test_both_attention_stages_from_one_work_list(k, L_d, L_q, Hq, Hkv, fuse_mode):
    """daf_imp_qd_attn (the two stages as one launch, ranges merged afterwards) against the oracle of
    each stage, element by element: ragged last tiles, causal chains long enough to be cut into ranges,
    several token blocks of question rows, compact and scattered output rows."""
    dev = "cuda"
    N = L_d + L_q
    r = k / L_d
    p = api.make_params(L_d, L_q, r, Hq, Hkv, fuse_mode=fuse_mode)
    assert api.daf_num_important(L_d, r) == k
    ws = api.alloc_workspace(p)
    qp, kp, vp = _normal((k, Hq, 128), 11), _normal((k, Hkv, 128), 12), _normal((k, Hkv, 128), 13)
    qq = _normal((L_q, Hq, 128), 14)
    kv_k, kv_v = _normal((N, Hkv, 128), 15), _normal((N, Hkv, 128), 16)
    idx = torch.from_numpy(np.sort(np.random.default_rng(5).choice(L_d, k, replace=False)).astype(np.int32))
    rows = k + L_q if fuse_mode == 0 else N
    hidden = torch.full((rows, Hq, 128), -9.0, dtype=torch.bfloat16, device=dev)
    _ok(api.daf_imp_qd_attn(p, qp.to(dev), None, kp.to(dev), vp.to(dev), qq.to(dev), kv_k.to(dev), kv_v.to(dev),
                            idx.to(dev), hidden, ws), ws, "daf_imp_qd_attn")
    # the same with the Q rows read in place: q_fresh holds packed row j at position idx[j], noise elsewhere
    q_fresh = _normal((L_d, Hq, 128), 17)
    q_fresh[idx.long()] = qp
    hidden2 = torch.full((rows, Hq, 128), -9.0, dtype=torch.bfloat16, device=dev)
    _ok(api.daf_imp_qd_attn(p, None, q_fresh.to(dev), kp.to(dev), vp.to(dev), qq.to(dev), kv_k.to(dev), kv_v.to(dev),
                            idx.to(dev), hidden2, ws), ws, "daf_imp_qd_attn (Q in place)")
    assert torch.equal(hidden2, hidden), "reading Q in place must give the same bits as reading the packed copy"
    scale = 1.0 / math.sqrt(128)
    ref_i = oracle.important_attn(_f(qp), _f(kp), _f(vp), scale)
    ref_q = oracle.qd_attn(_f(qq), _f(kv_k), _f(kv_v), L_d, scale)
    h = hidden.cpu()
    if fuse_mode == 0:
        _assert_close(h[:k], ref_i, "important rows")
        _assert_close(h[k:], ref_q, "question rows")
    else:
        _assert_close(h[idx.long()], ref_i, "important rows (scattered)")
        _assert_close(h[L_d:], ref_q, "question rows")
        others = np.setdiff1d(np.arange(L_d), idx.numpy())
        assert torch.all(h[others] == -9.0), "a row that is neither important nor a question row was written"


@pytest.mark.parametrize("fuse_mode", [0, 1])
def test_layer_without_packed_q_buffer(fuse_mode):
    """daf_layer with q_pack = NULL (step 2 reads its Q rows in place) gives the same bits as with the buffer,
    and daf_select with q_pack = NULL still packs K/V and updates the cache."""
    w = W.Workload("t", 11, 8, 2, 128, 1, 1500, 500, 70, 0.3, "lognormal", 2)
    L = W.make_layer(w, 0)
    dev = "cuda"
    p = api.make_params(w.L_d, w.L_q, w.r, w.n_q_heads, w.n_kv_heads, fuse_mode=fuse_mode)
    k = api.daf_num_important(w.L_d, w.r)
    g = {n: (None if t is None else t.to(dev)) for n, t in L.items()}
    rows = k + w.L_q if fuse_mode == 0 else w.N
    outs = []
    for with_q in (True, False):
        ws = api.alloc_workspace(p)
        kv_k = torch.zeros(w.N, w.n_kv_heads, 128, dtype=torch.bfloat16, device=dev)
        kv_v = torch.zeros_like(kv_k)
        kv_k[: w.L_d], kv_v[: w.L_d] = g["k_cached"], g["v_cached"]
        idx_out = torch.full((k,), -1, dtype=torch.int32, device=dev)
        qp = torch.full((k, w.n_q_heads, 128), 7.0, dtype=torch.bfloat16, device=dev)
        kp = torch.zeros(k, w.n_kv_heads, 128, dtype=torch.bfloat16, device=dev)
        vp = torch.zeros_like(kp)
        hidden = torch.full((rows, w.n_q_heads, 128), -9.0, dtype=torch.bfloat16, device=dev)
        _ok(api.daf_layer(p, g["scores"], 2, None, g["q_fresh"], g["k_fresh"], g["v_fresh"], kv_k, kv_v, idx_out,
                          qp if with_q else None, kp, vp, hidden, None, ws), ws, "daf_layer")
        outs.append((hidden.cpu(), idx_out.cpu(), kp.cpu(), vp.cpu(), kv_k.cpu(), kv_v.cpu()))
        if with_q:
            assert torch.equal(qp.cpu(), L["q_fresh"][idx_out.cpu().long()])
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a, b)
    ref = _oracle_layer(w, L, fuse_mode)
    hid = outs[1][0]
    if fuse_mode == 0:
        _assert_close(hid, ref["hidden"], "hidden rows (compact), Q read in place")
    else:
        _assert_close(hid[ref["row_pos"]], ref["hidden"][ref["row_pos"]], "hidden rows (scatter), Q read in place")
    # the selection step alone, without a packed-Q buffer
    ws = api.alloc_workspace(p)
    kv_k = torch.zeros(w.N, w.n_kv_heads, 128, dtype=torch.bfloat16, device=dev)
    kv_v = torch.zeros_like(kv_k)
    kv_k[: w.L_d], kv_v[: w.L_d] = g["k_cached"], g["v_cached"]
    idx_out = torch.full((k,), -1, dtype=torch.int32, device=dev)
    kp = torch.zeros(k, w.n_kv_heads, 128, dtype=torch.bfloat16, device=dev)
    vp = torch.zeros_like(kp)
    _ok(api.daf_select(p, g["scores"], 2, None, g["q_fresh"], g["k_fresh"], g["v_fresh"], kv_k, kv_v, idx_out, None, kp, vp,
                       ws), ws, "daf_select")
    assert torch.equal(idx_out.cpu(), outs[0][1]) and torch.equal(kp.cpu(), outs[0][2]) and torch.equal(vp.cpu(), outs[0][3])
    assert torch.equal(kv_k.cpu(), outs[0][4]) and torch.equal(kv_v.cpu(), outs[0][5])


@pytest.mark.parametrize("fuse_mode,overwrite,with_q", [(0, 1, True), (1, 1, False), (0, 0, False), (1, 0, True)])
@pytest.mark.parametrize("shape", [(1500, 70, 0.3, 8, 2), (3000, 64, 0.31, 28, 4), (700, 140, 0.9, 4, 4), (260, 3, 0.5, 8, 1)])
def test_layer_without_packed_kv_buffers(shape, fuse_mode, overwrite, with_q):
    """daf_layer with k_pack = v_pack = NULL: the attention kernel fetches the important rows' K/V in place (rows idx
    of the fresh tensors, ragged last sub-step zero-filled) and the kernel before it only updates the cache.  Same
    bits as with the packed copies, in both fusion modes, with and without the cache overwrite, with and without
    a packed Q; and against the oracle."""
    L_d, L_q, r, Hq, Hkv = shape
    w = W.Workload("t", 23, Hq, Hkv, 128, 1, L_d, 500, L_q, r, "lognormal", 2)
    L = W.make_layer(w, 0)
    dev = "cuda"
    p = api.make_params(w.L_d, w.L_q, w.r, Hq, Hkv, fuse_mode=fuse_mode, overwrite_doc_kv=overwrite)
    k = api.daf_num_important(w.L_d, w.r)
    g = {n: (None if t is None else t.to(dev)) for n, t in L.items()}
    rows = k + w.L_q if fuse_mode == 0 else w.N
    outs = []
    for with_kv in (True, False):
        ws = api.alloc_workspace(p)
        kv_k = torch.zeros(w.N, Hkv, 128, dtype=torch.bfloat16, device=dev)
        kv_v = torch.zeros_like(kv_k)
        kv_k[: w.L_d], kv_v[: w.L_d] = g["k_cached"], g["v_cached"]
        idx_out = torch.full((k,), -1, dtype=torch.int32, device=dev)
        qp = torch.zeros(k, Hq, 128, dtype=torch.bfloat16, device=dev) if with_q else None
        kp = torch.zeros(k, Hkv, 128, dtype=torch.bfloat16, device=dev) if with_kv else None
        vp = torch.zeros(k, Hkv, 128, dtype=torch.bfloat16, device=dev) if with_kv else None
        hidden = torch.full((rows, Hq, 128), -9.0, dtype=torch.bfloat16, device=dev)
        _ok(api.daf_layer(p, g["scores"], 2, None, g["q_fresh"], g["k_fresh"], g["v_fresh"], kv_k, kv_v, idx_out,
                          qp, kp, vp, hidden, None, ws), ws, "daf_layer")
        outs.append((hidden.cpu(), idx_out.cpu(), kv_k.cpu(), kv_v.cpu()))
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a, b), "reading K/V in place must give the same bits as reading the packed copies"
    ref = _oracle_layer(w, L, fuse_mode, overwrite=overwrite)
    hid = outs[1][0]
    assert np.array_equal(outs[1][1].numpy(), ref["idx"])
    assert np.array_equal(_f(outs[1][2]), ref["kv_k"]) and np.array_equal(_f(outs[1][3]), ref["kv_v"])
    sel = np.arange(len(ref["row_pos"])) if fuse_mode == 0 else ref["row_pos"]
    _assert_close(hid[sel], ref["hidden"][sel], "hidden rows, K/V read in place")


def test_layer_rejects_half_a_pair_of_packed_kv_buffers():
    """k_pack and v_pack go together; without a question there is no joint launch to read rows in place."""
    dev = "cuda"
    w = W.Workload("t", 3, 4, 2, 128, 1, 300, 100, 20, 0.3, "lognormal", 1)
    L = {n: (None if t is None else t.to(dev)) for n, t in W.make_layer(w, 0).items()}
    p = api.make_params(w.L_d, w.L_q, w.r, 4, 2)
    k = api.daf_num_important(w.L_d, w.r)
    ws = api.alloc_workspace(p)
    kv = torch.zeros(w.N, 2, 128, dtype=torch.bfloat16, device=dev)
    kv2 = torch.zeros_like(kv)
    idx_out = torch.zeros(k, dtype=torch.int32, device=dev)
    kp = torch.zeros(k, 2, 128, dtype=torch.bfloat16, device=dev)
    hidden = torch.zeros(k + w.L_q, 4, 128, dtype=torch.bfloat16, device=dev)
    for a, b in ((kp, None), (None, kp)):
        assert api.daf_layer(p, L["scores"], 1, None, L["q_fresh"], L["k_fresh"], L["v_fresh"], kv, kv2, idx_out, None, a, b,
                             hidden, None, ws) == api.DAF_ERR_INVALID_ARG
    p0 = api.make_params(w.L_d, 0, w.r, 4, 2)
    ws0 = api.alloc_workspace(p0)
    qp = torch.zeros(k, 4, 128, dtype=torch.bfloat16, device=dev)
    assert api.daf_layer(p0, L["scores"], 1, None, L["q_fresh"][: w.L_d], L["k_fresh"][: w.L_d], L["v_fresh"][: w.L_d],
                         kv[: w.L_d], kv2[: w.L_d], idx_out, qp, None, None, hidden, None, ws0) == api.DAF_ERR_INVALID_ARG


def test_layers_drawn_at_random():
    """Seeded random layers through daf_layer against the oracle: group sizes 1-8, document lengths that leave ragged
    tiles, one to a few hundred question tokens, r from 0.05 to 1, both fusion modes, with and without the cache
    overwrite, with and without packed Q and packed K/V buffers."""
    rng = np.random.default_rng(20261125)
    dev = "cuda"
    for case in range(24):
        Hkv = int(rng.choice([1, 2, 4, 8]))
        Hq = min(Hkv * int(rng.choice([1, 2, 4, 7, 8])), 32 // Hkv * Hkv)
        L_d, L_q = int(rng.integers(130, 2600)), int(rng.integers(1, 200))
        r = float(rng.choice([0.05, 0.1, 0.2, 0.3, 0.5, 0.9, 1.0]))
        fuse, ow = int(rng.integers(0, 2)), int(rng.integers(0, 2))
        with_q, with_kv = bool(rng.integers(0, 2)), bool(rng.integers(0, 2))
        w = W.Workload("f", int(rng.integers(1, 1000)), Hq, Hkv, 128, 1, L_d, 500, L_q, r, "lognormal", int(rng.integers(1, 4)))
        L = W.make_layer(w, 0)
        p = api.make_params(L_d, L_q, r, Hq, Hkv, fuse_mode=fuse, overwrite_doc_kv=ow)
        k = api.daf_num_important(L_d, r)
        g = {n: (None if t is None else t.to(dev)) for n, t in L.items()}
        ws = api.alloc_workspace(p)
        kv_k = torch.zeros(w.N, Hkv, 128, dtype=torch.bfloat16, device=dev)
        kv_v = torch.zeros_like(kv_k)
        kv_k[:L_d], kv_v[:L_d] = g["k_cached"], g["v_cached"]
        idx_out = torch.full((k,), -1, dtype=torch.int32, device=dev)
        qp = torch.zeros(k, Hq, 128, dtype=torch.bfloat16, device=dev) if with_q else None
        kp = torch.zeros(k, Hkv, 128, dtype=torch.bfloat16, device=dev) if with_kv else None
        vp = torch.zeros(k, Hkv, 128, dtype=torch.bfloat16, device=dev) if with_kv else None
        rows = k + L_q if fuse == 0 else w.N
        hidden = torch.full((rows, Hq, 128), -9.0, dtype=torch.bfloat16, device=dev)
        what = f"case {case}: L_d={L_d} L_q={L_q} r={r} Hq={Hq} Hkv={Hkv} fuse={fuse} overwrite={ow} q_pack={with_q} kv_pack={with_kv}"
        _ok(api.daf_layer(p, g["scores"], L["scores"].shape[0], None, g["q_fresh"], g["k_fresh"], g["v_fresh"], kv_k, kv_v,
                          idx_out, qp, kp, vp, hidden, None, ws), ws, what)
        ref = _oracle_layer(w, L, fuse, overwrite=ow)
        assert np.array_equal(idx_out.cpu().numpy(), ref["idx"]), what
        assert np.array_equal(_f(kv_k), ref["kv_k"]) and np.array_equal(_f(kv_v), ref["kv_v"]), what
        sel = np.arange(len(ref["row_pos"])) if fuse == 0 else ref["row_pos"]
        _assert_close(hidden.cpu()[sel], ref["hidden"][sel], what)


def test_work_list_shapes_drawn_at_random():
    """Seeded random shapes through daf_imp_qd_attn: group sizes 1-8, condensed sequences around multiples of
    the 128-row tile and of the 64-key sub-step, question blocks that see different numbers of key tiles."""
    rng = np.random.default_rng(20260721)
    dev = "cuda"
    scale = 1.0 / math.sqrt(128)
    for case in range(10):
        Hkv = int(rng.choice([1, 2, 4]))
        G = int(rng.choice([1, 2, 4, 7, 8]))
        Hq = Hkv * G
        k = int(rng.choice([1, 63, 64, 65, 127, 128, 129, 191, 257, 500, 640]))
        L_d = k + int(rng.integers(0, 700))
        L_q = int(rng.choice([1, 2, 17, 64, 130, 300]))
        fuse_mode = int(rng.integers(0, 2))
        N = L_d + L_q
        r = k / L_d
        p = api.make_params(L_d, L_q, r, Hq, Hkv, fuse_mode=fuse_mode)
        if api.daf_num_important(L_d, r) != k:
            continue
        ws = api.alloc_workspace(p)
        qp, kp, vp = _normal((k, Hq, 128), 100 + case), _normal((k, Hkv, 128), 200 + case), _normal((k, Hkv, 128), 300 + case)
        qq = _normal((L_q, Hq, 128), 400 + case)
        kv_k, kv_v = _normal((N, Hkv, 128), 500 + case), _normal((N, Hkv, 128), 600 + case)
        idx = torch.from_numpy(np.sort(rng.choice(L_d, k, replace=False)).astype(np.int32))
        rows = k + L_q if fuse_mode == 0 else N
        hidden = torch.full((rows, Hq, 128), -9.0, dtype=torch.bfloat16, device=dev)
        what = f"case {case}: k={k} L_d={L_d} L_q={L_q} Hq={Hq} Hkv={Hkv} fuse={fuse_mode}"
        _ok(api.daf_imp_qd_attn(p, qp.to(dev), None, kp.to(dev), vp.to(dev), qq.to(dev), kv_k.to(dev), kv_v.to(dev),
                                idx.to(dev), hidden, ws), ws, what)
        ref_i = oracle.important_attn(_f(qp), _f(kp), _f(vp), scale)
        ref_q = oracle.qd_attn(_f(qq), _f(kv_k), _f(kv_v), L_d, scale)
        h = hidden.cpu()
        if fuse_mode == 0:
            _assert_close(h[:k], ref_i, what + " important rows")
            _assert_close(h[k:], ref_q, what + " question rows")
        else:
            _assert_close(h[idx.long()], ref_i, what + " important rows")
            _assert_close(h[L_d:], ref_q, what + " question rows")
