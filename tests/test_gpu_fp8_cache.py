"""Offline cache stored in fp8: the expansion is bit-exact against the oracle, the layer run from an fp8 cache equals
the bf16 layer run from the widened cache bit for bit, and it matches the oracle within the attention tolerance."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_21599_b200 import api, build
from paper_2607_21599_b200 import workloads as W

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS, REL_FRO = 2e-2, 2e-3, 1e-2


def _f(t):
    return t.float().cpu().numpy()


def _fp8_cache(shape, seed, dev):
    """Seeded N(0,1) values rounded to the 8-bit format by the library conversion (input generation only)."""
    x = W.normal_bf16(shape, seed).float()
    b = x.to(torch.float8_e4m3fn).view(torch.uint8)
    assert not bool(((b & 0x7F) == 0x7F).any())
    return b.to(dev)


@pytest.mark.parametrize("L_d,Hkv,scaled", [(1024, 4, False), (777, 8, True), (5, 1, True), (6144, 4, True)])
def test_expansion_is_bit_exact(L_d, Hkv, scaled):
    build.build()
    dev = "cuda"
    k8, v8 = _fp8_cache((L_d, Hkv, 128), 11, dev), _fp8_cache((L_d, Hkv, 128), 12, dev)
    # every byte value occurs at least once (NaN patterns included: they must stay NaN)
    if L_d * Hkv * 128 >= 256:
        k8.view(-1)[:256] = torch.arange(256, dtype=torch.uint8, device=dev)
    ks = (0.25 + torch.arange(Hkv, dtype=torch.float32) * 0.37).to(dev) if scaled else None
    vs = (1.5 - torch.arange(Hkv, dtype=torch.float32) * 0.11).to(dev) if scaled else None
    p = api.make_params(L_d, 3, 0.1, 2 * Hkv, Hkv)
    kv_k = torch.full((L_d + 3, Hkv, 128), 7.0, dtype=torch.bfloat16, device=dev)
    kv_v = torch.full_like(kv_k, 7.0)
    api.check(api.daf_expand_fp8_cache(p, k8, v8, ks, vs, kv_k, kv_v), "daf_expand_fp8_cache")
    torch.cuda.synchronize()
    ref_k = oracle.dequant_fp8(k8.cpu().numpy(), None if ks is None else ks.cpu().numpy())
    ref_v = oracle.dequant_fp8(v8.cpu().numpy(), None if vs is None else vs.cpu().numpy())
    got_k, got_v = _f(kv_k[:L_d]), _f(kv_v[:L_d])
    assert np.array_equal(np.isnan(got_k), np.isnan(ref_k))
    assert np.array_equal(np.nan_to_num(got_k).view(np.uint32), np.nan_to_num(ref_k).view(np.uint32))
    assert np.array_equal(got_v.view(np.uint32), ref_v.view(np.uint32))
    assert torch.all(kv_k[L_d:] == 7.0) and torch.all(kv_v[L_d:] == 7.0), "question rows were touched"


@pytest.mark.parametrize("L_d,L_q,r,Hq,Hkv,scaled,given", [(1024, 32, 0.15, 28, 4, False, False), (1500, 70, 0.3, 8, 2, True, False),
                                                           (900, 17, 0.2, 8, 8, True, True), (640, 0, 0.25, 4, 2, True, False),
                                                           (640, 12, 0.0, 4, 2, False, False)])
def test_layer_from_an_fp8_cache(L_d, L_q, r, Hq, Hkv, scaled, given):
    build.build()
    dev = "cuda"
    N = L_d + L_q
    w = W.Workload("f8", 21, Hq, Hkv, 128, 1, L_d, L_d, L_q, r, "lognormal").with_k(api.daf_num_important)
    L = W.make_layer(w, 0, dev)
    k = w.k
    k8, v8 = _fp8_cache((L_d, Hkv, 128), 31, dev), _fp8_cache((L_d, Hkv, 128), 32, dev)
    ks = (0.5 + torch.arange(Hkv, dtype=torch.float32) * 0.21).to(dev) if scaled else None
    vs = (1.25 - torch.arange(Hkv, dtype=torch.float32) * 0.07).to(dev) if scaled else None
    p = api.make_params(L_d, L_q, r, Hq, Hkv)
    ws = api.alloc_workspace(p)
    scores = None if given else L["scores"]
    idx_in = W.given_indices(w).to(dev) if given else None
    n_sig = 0 if given else scores.shape[0]
    bf = torch.bfloat16

    def outputs():
        return dict(kv_k=torch.zeros(N, Hkv, 128, dtype=bf, device=dev), kv_v=torch.zeros(N, Hkv, 128, dtype=bf, device=dev),
                    idx=torch.full((k,), -1, dtype=torch.int32, device=dev), qp=torch.zeros(k, Hq, 128, dtype=bf, device=dev),
                    kp=torch.zeros(k, Hkv, 128, dtype=bf, device=dev), vp=torch.zeros(k, Hkv, 128, dtype=bf, device=dev),
                    hidden=torch.zeros(k + L_q, Hq, 128, dtype=bf, device=dev))

    a = outputs()
    api.check(api.daf_layer_fp8(p, scores, n_sig, idx_in, L["q_fresh"], L["k_fresh"], L["v_fresh"], k8, v8, ks, vs, a["kv_k"],
                                a["kv_v"], a["idx"], a["qp"], a["kp"], a["vp"], a["hidden"], None, ws), "daf_layer_fp8")
    torch.cuda.synchronize()
    api.check(api.daf_poll_status(ws), "fp8 layer")
    # the same layer through the bf16 entry point, from the cache the oracle expands
    wide_k = oracle.dequant_fp8(k8.cpu().numpy(), None if ks is None else ks.cpu().numpy())
    wide_v = oracle.dequant_fp8(v8.cpu().numpy(), None if vs is None else vs.cpu().numpy())
    b = outputs()
    b["kv_k"][:L_d] = torch.from_numpy(wide_k).to(bf).to(dev)
    b["kv_v"][:L_d] = torch.from_numpy(wide_v).to(bf).to(dev)
    api.check(api.daf_layer(p, scores, n_sig, idx_in, L["q_fresh"], L["k_fresh"], L["v_fresh"], b["kv_k"], b["kv_v"], b["idx"],
                            b["qp"], b["kp"], b["vp"], b["hidden"], None, ws), "daf_layer")
    torch.cuda.synchronize()
    api.check(api.daf_poll_status(ws), "bf16 layer")
    for name in a:
        assert torch.equal(a[name].view(torch.int16) if a[name].dtype == bf else a[name],
                           b[name].view(torch.int16) if b[name].dtype == bf else b[name]), name
    # and against the oracle run on the expanded cache
    ref = oracle.daf_layer(_f(L["q_fresh"]), _f(L["k_fresh"]), _f(L["v_fresh"]), wide_k, wide_v, L_d, L_q, w.softmax_scale,
                           scores=None if given else scores.cpu().numpy(), idx=None if given else None if not given else None,
                           r=r) if not given else \
        oracle.daf_layer(_f(L["q_fresh"]), _f(L["k_fresh"]), _f(L["v_fresh"]), wide_k, wide_v, L_d, L_q, w.softmax_scale,
                         idx=idx_in.cpu().numpy())
    assert np.array_equal(a["idx"].cpu().numpy(), ref["idx"])
    assert np.array_equal(_f(a["kv_k"]), ref["kv_k"]) and np.array_equal(_f(a["kv_v"]), ref["kv_v"])
    got = _f(a["hidden"]).astype(np.float64)
    err = np.abs(got - ref["hidden"])
    fro = np.linalg.norm(got - ref["hidden"]) / np.linalg.norm(ref["hidden"])
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS and fro <= REL_FRO, (err.max(), err.mean(), fro)
