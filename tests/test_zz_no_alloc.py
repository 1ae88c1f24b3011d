"""The workspace-free question-document entry point (daf_qd_attn_static).

It serves callers that cannot obtain device memory when they need this step (their
pool already owns the GPU, or an allocation would stall their streams), so its
scratch is a fixed array inside the library.  The check: called through the C ABI,
twice in a row on different problems, it reproduces daf_qd_attn, and the array's
leftovers from the first call do not leak into the second.

This file sorts last on purpose: a run that stops at the first failure has then
already covered every other test.
"""
import numpy as np
import pytest
import torch

from paper_2607_21599_b200 import api, build
from paper_2607_21599_b200 import workloads as W

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3


def _run_both(L_d, L_q, Hq, Hkv, seed, warm=True):
    N = L_d + L_q
    dev = "cuda"
    q = W.normal_bf16((L_q, Hq, 128), seed).to(dev)
    k = W.normal_bf16((N, Hkv, 128), seed + 1).to(dev)
    v = W.normal_bf16((N, Hkv, 128), seed + 2).to(dev)
    p = api.make_params(L_d, L_q, 0.1, Hq, Hkv)
    ws = api.alloc_workspace(p)
    ref = torch.zeros(L_q, Hq, 128, dtype=torch.bfloat16, device=dev)
    ref_lse = torch.zeros(Hq, L_q, dtype=torch.float32, device=dev)
    api.check(api.daf_qd_attn(p, q, k, v, ref, Hq * 256, None, ref_lse, ws), "daf_qd_attn")
    got = torch.full((L_q + 1, Hq, 128), 5.0, dtype=torch.bfloat16, device=dev)
    got_lse = torch.zeros(Hq, L_q, dtype=torch.float32, device=dev)
    if warm:
        # lazy loading of the library's device image happens at the first launch; it is not the call's doing
        api.check(api.daf_qd_attn_static(p, q, k, v, got, Hq * 256, None, got_lse), "daf_qd_attn_static (warm-up)")
        torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    free_before, _ = torch.cuda.mem_get_info()
    api.check(api.daf_qd_attn_static(p, q, k, v, got, Hq * 256, None, got_lse), "daf_qd_attn_static")
    assert torch.cuda.memory_allocated() == before, "the call went through torch's allocator"
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after >= free_before, "the call took device memory from the driver"
    api.check(api.daf_poll_status(ws), "device status (workspace call)")
    api.check(api.daf_qd_attn_static_poll_status(), "device status (static call)")
    return ref, ref_lse, got, got_lse, L_q


def _compare(ref, ref_lse, got, got_lse, L_q):
    err = (got[:L_q].float() - ref.float()).abs()
    assert torch.isfinite(got[:L_q].float()).all()
    assert err.max().item() <= MAX_ABS and err.mean().item() <= MEAN_ABS, (err.max().item(), err.mean().item())
    assert torch.all(got[L_q] == 5.0), "row past the end was written"
    np.testing.assert_allclose(got_lse.cpu().numpy(), ref_lse.cpu().numpy(), atol=2e-3, rtol=0)


def test_static_scratch_entry_point_matches_workspace_entry_point_twice():
    assert torch.cuda.is_available()
    build.build()
    assert api.daf_qd_attn_static_max_bytes() >= 1 << 20
    # first call: many KV splits, so the fixed array is filled with partial results
    first = _run_both(6144, 64, 28, 4, seed=101)
    _compare(*first)
    # second call, right after, on a different shape: must not be disturbed by the first call's leftovers
    second = _run_both(2000, 33, 8, 2, seed=202)
    _compare(*second)
    # and the first problem once more gives the first result again
    third = _run_both(6144, 64, 28, 4, seed=101)
    _compare(*third)
    assert torch.equal(third[2], first[2])


def test_static_scratch_entry_point_rejects_oversized_problems():
    build.build()
    # 128 question rows x 64 heads split four ways over the context needs a little more than the array holds
    p = api.make_params(8192, 128, 0.1, 64, 8)
    assert api.daf_workspace_bytes(p) > api.daf_qd_attn_static_max_bytes()
    dummy = torch.zeros(16, dtype=torch.uint8, device="cuda")
    assert api.daf_qd_attn_static(p, dummy, dummy, dummy, dummy, 64 * 256, None, None) == api.DAF_ERR_WORKSPACE
    bad = api.make_params(1024, 8, 0.1, 4, 2, head_dim=64)
    assert api.daf_qd_attn_static(bad, dummy, dummy, dummy, dummy, 1024, None, None) == api.DAF_ERR_UNSUPPORTED
