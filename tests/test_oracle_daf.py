"""Pins of the whole DAF layer of the oracle: brute-force masked attention over the
concatenated context, the r = 1 reduction to full causal attention, and the
hybrid-cache reading."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_21599_b200 import workloads as W


def _np(t):
    return t.float().numpy()


def _brute_force(q, kh, vh, idx, L_d, scale):
    """One N x N masked softmax attention.  Row p attends key t iff
    (p and t important, t <= p) or (p is a question row and t <= p)."""
    N, Hq, D = q.shape
    Hkv = kh.shape[1]
    G = Hq // Hkv
    imp = np.zeros(N, dtype=bool)
    imp[idx] = True
    pos = np.arange(N)
    mask = ((imp[:, None] & imp[None, :]) | (pos[:, None] >= L_d)) & (pos[None, :] <= pos[:, None])
    out = np.full((N, Hq, D), np.nan)
    for h in range(Hq):
        logits = (q[:, h].astype(np.float64) @ kh[:, h // G].astype(np.float64).T) * scale
        logits = np.where(mask, logits, -np.inf)
        rows = mask.any(axis=1)
        lg = logits[rows]
        p = np.exp(lg - lg.max(axis=1, keepdims=True))
        p /= p.sum(axis=1, keepdims=True)
        out[rows, h] = p @ vh[:, h // G].astype(np.float64)
    return out, mask


@pytest.mark.parametrize("seed_layer,L_d,L_q,r,Hq,Hkv", [(0, 48, 5, 0.25, 4, 2), (1, 64, 1, 0.1, 6, 2),
                                                         (2, 32, 9, 0.5, 7, 1), (3, 40, 4, 1.0, 2, 2)])
def test_layer_equals_brute_force_masked_attention(seed_layer, L_d, L_q, r, Hq, Hkv):
    w = W.tiny(L_d=L_d, doc_len=8, L_q=L_q, r=r, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=8, n_sig=3, num_important=oracle.num_important)
    L = W.make_layer(w, seed_layer)
    q, kf, vf, kc, vc = (_np(L[n]) for n in ("q_fresh", "k_fresh", "v_fresh", "k_cached", "v_cached"))
    res = oracle.daf_layer(q, kf, vf, kc, vc, L_d, L_q, w.softmax_scale, scores=L["scores"].numpy(), r=r)
    idx = res["idx"]
    assert len(idx) == oracle.num_important(L_d, r)
    # hybrid cache built here by plain indexing, independently of the oracle's routine
    kh = np.concatenate([kc, kf[L_d:]], 0)
    vh = np.concatenate([vc, vf[L_d:]], 0)
    kh[idx], vh[idx] = kf[idx], vf[idx]
    bf, mask = _brute_force(q, kh, vh, idx, L_d, w.softmax_scale)
    rows = np.concatenate([idx, np.arange(L_d, L_d + L_q)])
    assert np.array_equal(res["row_pos"], rows)
    np.testing.assert_allclose(res["hidden"], bf[rows], rtol=0, atol=1e-12)
    # rows that are neither important nor question rows have no output at all
    others = np.setdiff1d(np.arange(L_d), idx)
    assert not mask[others].any()
    # scatter mode puts the same rows at their original positions and leaves the rest alone
    base = np.full((L_d + L_q, Hq, 8), 42.0)
    res1 = oracle.daf_layer(q, kf, vf, kc, vc, L_d, L_q, w.softmax_scale, idx=idx, fuse_mode=1, hidden=base)
    np.testing.assert_allclose(res1["hidden"][rows], bf[rows], rtol=0, atol=1e-12)
    assert np.all(res1["hidden"][others] == 42.0)


def test_r_one_without_question_is_full_causal_attention():
    w = W.tiny(L_d=40, doc_len=8, L_q=0, r=1.0, n_q_heads=4, n_kv_heads=2, head_dim=8, num_important=oracle.num_important)
    L = W.make_layer(w, 0)
    q, kf, vf, kc, vc = (_np(L[n]) for n in ("q_fresh", "k_fresh", "v_fresh", "k_cached", "v_cached"))
    res = oracle.daf_layer(q, kf, vf, kc, vc, 40, 0, w.softmax_scale, scores=L["scores"].numpy(), r=1.0)
    assert np.array_equal(res["idx"], np.arange(40))
    # library attention, not the oracle, is the reference here
    qt = torch.from_numpy(q).double().permute(1, 0, 2)[None]
    kt = torch.from_numpy(kf).double().permute(1, 0, 2)[None].repeat_interleave(2, 1)
    vt = torch.from_numpy(vf).double().permute(1, 0, 2)[None].repeat_interleave(2, 1)
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(res["hidden"], ref, rtol=0, atol=1e-12)
    # with r = 1 the hybrid cache is entirely fresh
    assert np.array_equal(res["kv_k"], kf) and np.array_equal(res["kv_v"], vf)


def test_question_stage_equals_full_recompute_when_cache_is_fresh():
    w = W.tiny(L_d=48, doc_len=16, L_q=6, r=0.25, num_important=oracle.num_important)
    L = W.make_layer(w, 4)
    q, kf, vf = (_np(L[n]) for n in ("q_fresh", "k_fresh", "v_fresh"))
    res = oracle.daf_layer(q, kf, vf, kf[:48], vf[:48], 48, 6, w.softmax_scale, scores=L["scores"].numpy(), r=0.25)
    full = oracle.full_causal_attn(q, kf, vf, w.softmax_scale)
    np.testing.assert_allclose(res["o_q"], full[48:], rtol=0, atol=1e-13)


def test_hybrid_cache_reading_important_rows_are_overwritten():
    w = W.tiny(L_d=48, doc_len=16, L_q=4, r=0.25, num_important=oracle.num_important)
    L = W.make_layer(w, 5)
    q, kf, vf, kc, vc = (_np(L[n]) for n in ("q_fresh", "k_fresh", "v_fresh", "k_cached", "v_cached"))
    sc = L["scores"].numpy()
    base = oracle.daf_layer(q, kf, vf, kc, vc, 48, 4, w.softmax_scale, scores=sc, r=0.25)
    idx = base["idx"]
    non_imp = int(np.setdiff1d(np.arange(48), idx)[0])
    # a fresh K/V change at a non-important document row is invisible everywhere
    kf2, vf2 = kf.copy(), vf.copy()
    kf2[non_imp] += 3.0
    vf2[non_imp] -= 2.0
    r2 = oracle.daf_layer(q, kf2, vf2, kc, vc, 48, 4, w.softmax_scale, scores=sc, r=0.25)
    assert np.array_equal(r2["hidden"], base["hidden"])
    # at an important row it reaches the question rows (through the overwritten cache row)
    kf3 = kf.copy()
    kf3[idx[0]] += 3.0
    r3 = oracle.daf_layer(q, kf3, vf, kc, vc, 48, 4, w.softmax_scale, scores=sc, r=0.25)
    assert not np.array_equal(r3["o_q"], base["o_q"])
    # and a cached-row change at an important position is invisible (the row was replaced)
    kc4 = kc.copy()
    kc4[idx[0]] += 3.0
    r4 = oracle.daf_layer(q, kf, vf, kc4, vc, 48, 4, w.softmax_scale, scores=sc, r=0.25)
    assert np.array_equal(r4["hidden"], base["hidden"])
    # ablation switch: without overwriting, the cached row is what the question sees
    r5 = oracle.daf_layer(q, kf, vf, kc4, vc, 48, 4, w.softmax_scale, scores=sc, r=0.25, overwrite=False)
    r6 = oracle.daf_layer(q, kf, vf, kc, vc, 48, 4, w.softmax_scale, scores=sc, r=0.25, overwrite=False)
    assert not np.array_equal(r5["o_q"], r6["o_q"])


def test_flop_model_matches_complexity_terms():
    # visible pairs: k(k+1)/2 + L_q*L_d + L_q(L_q+1)/2, i.e. the r^2 L_d^2 and L_q (L_d + L_q) terms
    for name, w in W.CONFIGS.items():
        p = W.attention_pairs(w)
        assert p["important"] == w.k * (w.k + 1) // 2
        assert p["question"] == sum(w.L_d + i + 1 for i in range(w.L_q))
        assert p["full"] == sum(i + 1 for i in range(w.N))
    gf = {n: (W.attention_flops(W.CONFIGS[n])["important"] + W.attention_flops(W.CONFIGS[n])["question"]) / 1e9
          for n in W.CONFIGS}
    assert abs(gf["c0"] - 0.648) < 0.001 and abs(gf["c1"] - 11.77) < 0.01
    assert abs(gf["c2"] - 56.5) < 0.1 and abs(gf["c3"] - 368.2) < 0.1


def test_full_context_variant_against_masked_library_attention():
    """Rows at positions row_pos attend every key up to their position (selective recomputation over the
    full context): pinned by a library attention with an explicit mask, by the identity position map
    (plain causal attention) and by the question rows of the DAF layer."""
    w = W.tiny(L_d=40, doc_len=8, L_q=4, r=0.25, n_q_heads=6, n_kv_heads=2, head_dim=8, num_important=oracle.num_important)
    L = W.make_layer(w, 7)
    q, kf, vf, kc, vc = (_np(L[n]) for n in ("q_fresh", "k_fresh", "v_fresh", "k_cached", "v_cached"))
    base = oracle.daf_layer(q, kf, vf, kc, vc, 40, 4, w.softmax_scale, scores=L["scores"].numpy(), r=0.25)
    pos = base["row_pos"]
    q_rows = q[pos]
    got = oracle.blend_attn(q_rows, base["kv_k"], base["kv_v"], pos, w.softmax_scale)
    qt = torch.from_numpy(q_rows).double().permute(1, 0, 2)[None]
    kt = torch.from_numpy(base["kv_k"]).double().permute(1, 0, 2)[None].repeat_interleave(3, 1)
    vt = torch.from_numpy(base["kv_v"]).double().permute(1, 0, 2)[None].repeat_interleave(3, 1)
    mask = torch.arange(44)[None, :] <= torch.from_numpy(pos.astype(np.int64))[:, None]
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=mask, scale=w.softmax_scale)
    np.testing.assert_allclose(got, ref[0].permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)
    # the question rows of this variant are the question stage of DAF
    np.testing.assert_allclose(got[len(base["idx"]):], base["o_q"], rtol=0, atol=1e-13)
    # identity position map: plain causal attention
    ident = oracle.blend_attn(q, kf, vf, np.arange(44), w.softmax_scale)
    np.testing.assert_allclose(ident, oracle.full_causal_attn(q, kf, vf, w.softmax_scale), rtol=0, atol=1e-13)
    # a row subset is the same rows
    sub = oracle.blend_attn(q_rows, base["kv_k"], base["kv_v"], pos, w.softmax_scale, rows=[0, 5, len(pos) - 1])
    assert np.array_equal(sub, got[[0, 5, len(pos) - 1]])
