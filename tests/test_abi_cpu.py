"""CPU-side checks of the C-ABI library: it builds for sm_100a, loads, exports every
symbol the header declares, and rejects bad arguments on the host before any launch."""
import ctypes
import os
import re

import pytest
import torch

from paper_2607_21599_b200 import api, build


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.lib()


def test_header_symbols_are_exported(lib, repo_root):
    header = open(os.path.join(repo_root, "include", "daf.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(daf_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(api.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_layout_matches_header():
    # int32 int32 double int32 int32 int32 float int32 int32 -> 40 bytes with natural alignment
    assert ctypes.sizeof(api.daf_params) == 40
    assert api.daf_params.r.offset == 8 and api.daf_params.n_q_heads.offset == 16


def test_num_important_matches_stated_counts(lib):
    assert api.daf_num_important(1024, 0.15) == 154
    assert api.daf_num_important(6144, 0.15) == 922
    assert api.daf_num_important(16384, 0.10) == 1639
    assert api.daf_num_important(32768, 0.20) == 6554
    assert api.daf_num_important(1000, float(torch.tensor(0.1, dtype=torch.float32))) == 100
    assert api.daf_num_important(10, 0.0) == 0 and api.daf_num_important(10, 1.0) == 10


def test_workspace_bytes_and_arena(lib):
    p = api.make_params(16384, 128, 0.1, 32, 8)
    ws = api.daf_workspace_bytes(p)
    assert ws >= 256
    assert api.daf_layer_host_arena_bytes(p) > ws
    bad = api.make_params(16384, 128, 0.1, 32, 8, head_dim=64)
    assert api.daf_workspace_bytes(bad) == 0


def test_host_side_argument_validation(lib):
    """Every error code that argument checking can produce, without a GPU: a failing call launches nothing."""
    ok = api.make_params(256, 16, 0.25, 4, 2)
    ws = torch.zeros(api.daf_workspace_bytes(ok) + 16, dtype=torch.uint8)
    base = ws.data_ptr()
    assert base % 16 == 0

    def sel(p, workspace=ws, **kw):
        a = dict(scores=None, n_sig=1, idx_in=None, q_fresh=None, k_fresh=None, v_fresh=None, kv_k=None, kv_v=None,
                 idx_out=None, q_pack=None, k_pack=None, v_pack=None)
        a.update(kw)
        return api.daf_select(p, a["scores"], a["n_sig"], a["idx_in"], a["q_fresh"], a["k_fresh"], a["v_fresh"],
                              a["kv_k"], a["kv_v"], a["idx_out"], a["q_pack"], a["k_pack"], a["v_pack"], workspace)

    assert sel(api.make_params(256, 16, 0.25, 4, 2, head_dim=64)) == api.DAF_ERR_UNSUPPORTED
    assert sel(api.make_params(256, 16, 0.25, 5, 2)) == api.DAF_ERR_UNSUPPORTED
    assert sel(api.make_params(-1, 16, 0.25, 4, 2)) == api.DAF_ERR_INVALID_ARG
    assert sel(api.make_params(256, 16, 1.5, 4, 2)) == api.DAF_ERR_INVALID_ARG
    assert sel(api.make_params(256, 16, float("nan"), 4, 2)) == api.DAF_ERR_INVALID_ARG
    assert sel(api.make_params(256, 16, 0.25, 4, 2, fuse_mode=3)) == api.DAF_ERR_INVALID_ARG
    assert sel(ok, workspace=None) == api.DAF_ERR_WORKSPACE
    assert sel(ok, workspace=ws[:64]) == api.DAF_ERR_WORKSPACE
    assert sel(ok, workspace=ws[8:]) in (api.DAF_ERR_ALIGNMENT, api.DAF_ERR_WORKSPACE)
    assert sel(ok) == api.DAF_ERR_INVALID_ARG  # no scores, no indices, no tensors
    # the attention entry points validate the same way
    assert api.daf_important_attn(ok, 300, None, None, None, None, 1024, None, None, ws) == api.DAF_ERR_INVALID_ARG
    assert api.daf_important_attn(ok, 8, None, None, None, None, 1024, None, None, ws) == api.DAF_ERR_INVALID_ARG
    assert api.daf_important_attn(ok, 0, None, None, None, None, 1024, None, None, ws) == api.DAF_OK  # k = 0: no-op
    assert api.daf_qd_attn(ok, None, None, None, None, 1024, None, None, ws) == api.DAF_ERR_INVALID_ARG
    assert api.daf_full_causal_attn(ok, -5, None, None, None, None, None, ws) == api.DAF_ERR_INVALID_ARG
    assert api.daf_fuse(ok, 4, None, None, None, None, None) == api.DAF_ERR_INVALID_ARG
    buf = torch.zeros(4096, dtype=torch.uint8)
    # a row stride that is not a multiple of 16 bytes, and one smaller than a row
    assert api.daf_important_attn(ok, 2, buf, buf, buf, buf, 1000, None, None, ws) == api.DAF_ERR_ALIGNMENT
    assert api.daf_important_attn(ok, 2, buf, buf, buf, buf, 512, None, None, ws) == api.DAF_ERR_INVALID_ARG
    assert api.daf_important_attn(ok, 2, buf[8:], buf, buf, buf, 1024, None, None, ws) == api.DAF_ERR_ALIGNMENT
    # both stages from one work list: needs packed K/V, the question rows, the cache, and either packed Q
    # rows or (q_fresh, idx); idx also for scattered output rows
    both = lambda p, q_pack, q_fresh, idx, hidden=buf: api.daf_imp_qd_attn(p, q_pack, q_fresh, buf, buf, buf, buf, buf, idx,  # noqa: E731
                                                                         hidden, ws)
    assert both(ok, None, None, None) == api.DAF_ERR_INVALID_ARG            # no Q rows at all
    assert both(ok, None, buf, None) == api.DAF_ERR_INVALID_ARG             # Q in place needs idx
    assert both(ok, buf, None, None, hidden=None) == api.DAF_ERR_INVALID_ARG
    assert both(ok, buf[8:], None, None) == api.DAF_ERR_ALIGNMENT
    assert both(api.make_params(256, 16, 0.25, 4, 2, fuse_mode=1), buf, None, None) == api.DAF_ERR_INVALID_ARG
    assert both(api.make_params(256, 0, 0.25, 4, 2), buf, None, None) == api.DAF_ERR_INVALID_ARG   # no question rows
    assert both(api.make_params(256, 16, 0.0, 4, 2), buf, None, None) == api.DAF_ERR_INVALID_ARG   # no important rows
    # a layer without question rows cannot read Q in place (only the joint launch does)
    no_q = api.make_params(256, 0, 0.25, 4, 2)
    assert api.daf_layer(no_q, buf, 1, None, buf, buf, buf, buf, buf, buf, None, buf, buf, buf, None, ws) == api.DAF_ERR_INVALID_ARG
    # nothing selected (r = 0) but question rows present: they are read from q_fresh, so it is required
    r0 = api.make_params(256, 16, 0.0, 4, 2)
    assert api.daf_layer(r0, None, 0, None, None, buf, buf, buf, buf, None, None, None, None, buf, None, ws) == api.DAF_ERR_INVALID_ARG
    assert api.daf_layer(r0, None, 0, None, buf[8:], buf, buf, buf, buf, None, None, None, None, buf, None, ws) == api.DAF_ERR_ALIGNMENT
    assert api.daf_layer(r0, None, 0, None, buf, buf, buf, None, buf, None, None, None, None, buf, None, ws) == api.DAF_ERR_INVALID_ARG
    # important rows without packed K/V buffers
    assert api.daf_layer(ok, buf, 1, None, buf, buf, buf, buf, buf, buf, buf, None, buf, buf, None, ws) == api.DAF_ERR_INVALID_ARG
    # selection straight from the signal layers' K/V: the number of layers and every pointer are checked first
    sig = lambda n: [buf] * n  # noqa: E731
    skv = lambda n, kf=None, wsp=ws: api.daf_select_from_kv(ok, kf if kf is not None else sig(n), sig(n), sig(n), sig(n), buf, buf, buf,  # noqa: E731
                                                           buf, buf, buf, buf, buf, buf, None, wsp)
    assert skv(0) == api.DAF_ERR_INVALID_ARG and skv(9) == api.DAF_ERR_INVALID_ARG
    assert skv(2, kf=[buf, None]) == api.DAF_ERR_INVALID_ARG
    assert skv(2, kf=[buf, buf[8:]]) == api.DAF_ERR_ALIGNMENT
    assert skv(2, wsp=None) == api.DAF_ERR_WORKSPACE
    assert api.daf_check_indices(ok, 300, buf, ws) == api.DAF_ERR_INVALID_ARG
    assert api.daf_check_indices(ok, 4, None, ws) == api.DAF_ERR_INVALID_ARG
    assert api.daf_check_indices(ok, 4, buf, None) == api.DAF_ERR_WORKSPACE
    assert api.daf_check_indices(ok, 0, None, ws) == api.DAF_OK
    # the self-test of the bounded wait checks its arguments before it launches anything
    assert api.daf_selftest_bounded_wait(None, 50) == api.DAF_ERR_WORKSPACE
    assert api.daf_selftest_bounded_wait(ws[:64], 50) == api.DAF_ERR_WORKSPACE
    assert api.daf_selftest_bounded_wait(ws, 0) == api.DAF_ERR_INVALID_ARG
    assert api.daf_selftest_bounded_wait(ws, 5000) == api.DAF_ERR_INVALID_ARG
    assert api.daf_launch_count() == 0
    assert "workspace" in api.daf_strerror(api.DAF_ERR_WORKSPACE)
    assert api.daf_layer_host(ok, None, 1, None, None, None, None, None, None, 0, None, None, None) == api.DAF_ERR_WORKSPACE
    assert api.daf_layer_host_begin(ok, None, 1, None, None, None, None, None, None, 0, None, None, None) == api.DAF_ERR_WORKSPACE
    assert api.daf_layer_host_end(ok, None) == api.DAF_ERR_WORKSPACE


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="missing"):
        api.daf_num_important(10, 0.5)
