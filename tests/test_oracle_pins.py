"""Pins of the fp64 CPU oracle against things other than itself: closed forms,
library routines (torch softmax / scaled_dot_product_attention in fp64), a
hand-worked example, invariants the definitions force, and a dense-mask brute
force on tiny inputs.  Chosen so that a dropped term, a wrong sign or index, a
wrong head mapping or a transposed operand fails at least one test.
"""
import os

import numpy as np
import pytest
import torch

from oracle import relaxkv_oracle as orc
from paper_2609_33503_b200 import inputs
from tests import bruteforce as bf

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits(t: torch.Tensor) -> np.ndarray:
    return inputs.bf16_bits(t.to(torch.bfloat16))


def rand_bits(rng, *shape, scale=1.0):
    g = torch.Generator().manual_seed(int(rng.integers(1 << 30)))
    return bits(torch.randn(*shape, generator=g) * scale)


def t64(b: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bf.f64(b))


# ---------------------------------------------------------------- scores ----

@pytest.mark.parametrize("H,Hkv,D,Q,T", [(4, 1, 64, 5, 37), (6, 3, 32, 3, 50), (8, 8, 16, 2, 19)])
def test_raw_scores_match_bruteforce_and_sum_to_one(H, Hkv, D, Q, T):
    rng = np.random.default_rng(1)
    q, k = rand_bits(rng, Q, H, D), rand_bits(rng, T, Hkv, D)
    scale = 1.0 / np.sqrt(D)
    raw = orc.raw_scores(q, k, scale)
    np.testing.assert_allclose(raw, bf.raw_scores(q, k, scale), rtol=1e-12, atol=1e-15)
    assert abs(raw.sum() - 1.0) < 1e-12          # each softmax row sums to one
    a = orc.minmax(raw)
    assert a.min() == 0.0 and a.max() == 1.0 and np.all((a >= 0) & (a <= 1))
    np.testing.assert_allclose(a, bf.minmax(raw), rtol=1e-13)


def test_raw_scores_single_row_is_library_softmax():
    rng = np.random.default_rng(2)
    D, T = 64, 129
    q, k = rand_bits(rng, 1, 1, D), rand_bits(rng, T, 1, D)
    scale = 0.37
    logits = (t64(k)[:, 0, :] @ t64(q)[0, 0, :]) * scale
    np.testing.assert_allclose(orc.raw_scores(q, k, scale), torch.softmax(logits, 0).numpy(), rtol=1e-12)


def test_raw_scores_head_mapping_and_strided_cache():
    """Query head h must read KV head h // G (not h % H_kv); the cache may be a
    strided view ([H_kv, T, D] storage seen as [T, H_kv, D])."""
    rng = np.random.default_rng(3)
    H, Hkv, D, Q, T = 6, 2, 32, 4, 41
    q = rand_bits(rng, Q, H, D)
    k_store = rand_bits(rng, Hkv, T, D)                      # head-major storage
    k_view = k_store.transpose(1, 0, 2)                      # [T,Hkv,D] strided view
    scale = 1 / np.sqrt(D)
    kx = t64(np.ascontiguousarray(k_view)).repeat_interleave(H // Hkv, dim=1)     # [T,H,D]
    s = torch.einsum("thd,ihd->hti", t64(q), kx) * scale
    ref = torch.softmax(s, dim=-1).mean(dim=(0, 1)).numpy()
    np.testing.assert_allclose(orc.raw_scores(q, k_view, scale), ref, rtol=1e-12)
    wrong = torch.softmax(torch.einsum("thd,ihd->hti", t64(q), t64(np.ascontiguousarray(k_view)).repeat(1, H // Hkv, 1)) * scale, -1).mean(dim=(0, 1)).numpy()
    assert np.abs(wrong - ref).max() > 1e-4                   # the other mapping is really different


def test_raw_scores_closed_forms():
    rng = np.random.default_rng(4)
    H, Hkv, D, Q, T = 4, 2, 16, 3, 23
    q = rand_bits(rng, Q, H, D)
    k = np.broadcast_to(rand_bits(rng, 1, Hkv, D), (T, Hkv, D)).copy()      # all keys equal
    raw = orc.raw_scores(q, k, 0.25)
    np.testing.assert_allclose(raw, np.full(T, 1.0 / T), rtol=1e-13)
    assert np.all(orc.minmax(np.full(T, 0.3)) == 0.0)                         # constant -> zeros
    k2 = rand_bits(rng, T, Hkv, D)
    k2[7] = k2[3]                                                             # duplicated key -> equal score
    raw2 = orc.raw_scores(q, k2, 0.25)
    assert raw2[7] == raw2[3]
    perm = rng.permutation(Q)                                                 # query order is irrelevant
    np.testing.assert_allclose(orc.raw_scores(q[perm], k2, 0.25), raw2, rtol=1e-13)


def test_raw_scores_with_supplied_lse_is_wider_softmax_restricted_to_context():
    rng = np.random.default_rng(5)
    H, Hkv, D, Q, T, X = 4, 2, 32, 3, 31, 6
    q, k, kx = rand_bits(rng, Q, H, D), rand_bits(rng, T, Hkv, D), rand_bits(rng, X, Hkv, D)
    scale = 1 / np.sqrt(D)
    kall = t64(np.concatenate([k, kx], 0)).repeat_interleave(H // Hkv, dim=1)
    s = torch.einsum("thd,ihd->hti", t64(q), kall) * scale                   # [H,Q,T+X]
    lse = torch.logsumexp(s, dim=-1).numpy()
    ref = torch.softmax(s, -1)[..., :T].mean(dim=(0, 1)).numpy()
    got = orc.raw_scores(q, k, scale, lse=lse)
    np.testing.assert_allclose(got, ref, rtol=1e-12)
    assert got.sum() < 1.0
    np.testing.assert_allclose(orc.row_lse(q, k, scale), torch.logsumexp(s[..., :T], -1).numpy(), rtol=1e-13)


# ------------------------------------------------------------ count, top-k ----

def test_anchor_count_golden():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "anchor_counts.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) >= 15
    for T, r, k in rows:
        assert orc.anchor_count(int(T), float(r)) == int(k), (T, r, k)


def test_topk_ties_and_bruteforce():
    assert orc.topk(np.array([1.0, 3.0, 3.0, 2.0, 3.0]), 2).tolist() == [1, 2]     # ties -> lower index
    assert orc.topk(np.array([1.0, 3.0, 3.0, 2.0, 3.0]), 4).tolist() == [1, 2, 3, 4]
    assert orc.topk(np.array([5.0, 1.0, 2.0]), 3).tolist() == [0, 1, 2]             # k = T
    rng = np.random.default_rng(6)
    for T, k in [(100, 15), (257, 1), (64, 64), (300, 123)]:
        s = rng.integers(0, 20, size=T).astype(np.float64) / 7.0                   # many ties
        got = orc.topk(s, k)
        assert got.tolist() == bf.topk(s, k).tolist()
        assert len(set(got.tolist())) == k and np.all(np.diff(got) > 0)
        thr = np.sort(s)[::-1][k - 1]
        assert np.all(s[got] >= thr) and np.all(np.delete(s, got) <= thr)


# -------------------------------------------------------------------- sets ----

def _golden_sets():
    d = {}
    for l in open(os.path.join(GOLDEN, "active_sets_example.txt")):
        if l.strip() and l[0] != "#":
            p = l.split()
            d[p[0]] = [int(x) for x in p[1:]]
    return d


def test_active_sets_hand_example():
    g = _golden_sets()
    T = g["T"][0]
    anchors = np.array([g["S0"], g["S1"], g["S2"]], dtype=np.int32)
    s = orc.active_sets(anchors, T)
    assert s.h.tolist() == g["h"]
    assert s.u_pos.tolist() == g["U"]
    for l in range(3):
        assert s.positions(l).tolist() == g[f"R{l}"]
        assert orc.edges(s.ranks(l)) == g["E"][l]
    # causal context of the target at position 2 = first (rank+1) entries of U
    r2 = s.u_rank[2]
    assert s.u_pos[:r2 + 1].tolist() == g["C2"]
    assert [s.u_rank[p] for p in g["U"]] == list(range(len(g["U"])))
    assert s.u_rank[3] == -1 and s.u_rank[5] == -1


@pytest.mark.parametrize("L,T,k,seed", [(1, 40, 7, 0), (5, 64, 9, 1), (12, 200, 30, 2), (3, 16, 16, 3)])
def test_active_sets_invariants_and_bruteforce(L, T, k, seed):
    rng = np.random.default_rng(seed)
    anchors = np.stack([np.sort(rng.choice(T, size=k, replace=False)) for _ in range(L)]).astype(np.int32)
    s = orc.active_sets(anchors, T)
    U, h, R = bf.sets(anchors, T)
    assert s.u_pos.tolist() == U
    assert all(s.h[i] == h.get(i, -1) for i in range(T))
    for l in range(L):
        assert s.positions(l).tolist() == R[l]
        assert set(anchors[l].tolist()) <= set(R[l])                      # S_l subset of R_l
        if l + 1 < L:
            assert set(R[l + 1]) <= set(R[l])                             # monotone across layers
    assert s.positions(0).tolist() == U                                   # R_0 = U
    assert s.positions(L - 1).tolist() == sorted(anchors[L - 1].tolist()) # R_{L-1} = S_{L-1}
    assert len(U) <= min(T, L * k)
    assert s.r_cu[L] == sum(h[i] + 1 for i in U)                          # sum_l |R_l| = sum_i (h_i + 1)
    same = np.tile(anchors[:1], (L, 1))
    s2 = orc.active_sets(same, T)
    for l in range(L):
        assert s2.positions(l).tolist() == sorted(anchors[0].tolist())    # identical S_l -> R_l = U


# --------------------------------------------------------------- attention ----

def sdpa_causal(q_bits, k_bits, v_bits, scale):
    q, k, v = t64(q_bits), t64(k_bits), t64(v_bits)                       # [n,H,D], [n,Hkv,D]
    G = q.shape[1] // k.shape[1]
    qh = q.permute(1, 0, 2).unsqueeze(0)
    kh = k.repeat_interleave(G, dim=1).permute(1, 0, 2).unsqueeze(0)
    vh = v.repeat_interleave(G, dim=1).permute(1, 0, 2).unsqueeze(0)
    o = torch.nn.functional.scaled_dot_product_attention(qh, kh, vh, is_causal=True, scale=scale)
    return o[0].permute(1, 0, 2).numpy()


@pytest.mark.parametrize("H,Hkv,D,T", [(4, 1, 64, 48), (6, 2, 32, 33)])
def test_full_ratio_equals_dense_causal_attention(H, Hkv, D, T):
    """Anchor ratio 100 %: U = R_l = every position, so the result is plain causal
    attention over the fresh K/V (library SDPA in fp64).  Same for the full-prefix mode."""
    rng = np.random.default_rng(7)
    ck, cv = rand_bits(rng, T, Hkv, D), rand_bits(rng, T, Hkv, D)
    qn, kn, vn = rand_bits(rng, T, H, D), rand_bits(rng, T, Hkv, D), rand_bits(rng, T, Hkv, D)
    scale = 1 / np.sqrt(D)
    allpos = np.arange(T, dtype=np.int32)
    ref = sdpa_causal(qn, kn, vn, scale)
    out, lse = orc.repair_attention(ck, cv, qn, kn, vn, allpos, allpos, scale)
    np.testing.assert_allclose(out, ref, rtol=1e-10, atol=1e-12)
    out2, _ = orc.repair_attention(ck, cv, qn, kn, vn, allpos, allpos, scale, full_prefix=True)
    np.testing.assert_allclose(out2, ref, rtol=1e-10, atol=1e-12)
    # one chunk: the fresh states equal the cached ones -> prefix recompute over the cache
    out3, _ = orc.repair_attention(ck, cv, qn, ck, cv, allpos, allpos, scale)
    np.testing.assert_allclose(out3, sdpa_causal(qn, ck, cv, scale), rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("seed,full_prefix", [(0, False), (1, False), (2, True), (3, True)])
def test_attention_matches_dense_mask_bruteforce(seed, full_prefix):
    rng = np.random.default_rng(100 + seed)
    H, Hkv, D, T, L, k = 6, 2, 32, 61, 3, 11
    ck, cv = rand_bits(rng, T, Hkv, D), rand_bits(rng, T, Hkv, D)
    anchors = np.stack([np.sort(rng.choice(T, size=k, replace=False)) for _ in range(L)]).astype(np.int32)
    s = orc.active_sets(anchors, T)
    scale = 1 / np.sqrt(D)
    for l in range(L):
        ranks, pos = s.ranks(l), s.positions(l)
        qn = rand_bits(rng, len(pos), H, D)
        kn, vn = rand_bits(rng, len(pos), Hkv, D), rand_bits(rng, len(pos), Hkv, D)
        out, lse = orc.repair_attention(ck, cv, qn, kn, vn, s.u_pos, ranks, scale, full_prefix=full_prefix)
        ref, ref_lse, n_edges = bf.attention(ck, cv, qn, kn, vn, s.u_pos, pos, scale, full_prefix=full_prefix)
        np.testing.assert_allclose(out, ref, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(lse, ref_lse, rtol=1e-12)
        limit = pos if full_prefix else ranks
        assert orc.edges(limit) == n_edges                                 # edge-count formula
        # row subset = same rows of the full result
        rows = np.array([len(pos) - 1, 0], dtype=np.int32)
        sub, _ = orc.repair_attention(ck, cv, qn, kn, vn, s.u_pos, ranks, scale, full_prefix=full_prefix, rows=rows)
        np.testing.assert_array_equal(sub, out[rows])


def test_attention_special_cases():
    rng = np.random.default_rng(8)
    H, Hkv, D, T = 4, 2, 16, 40
    ck, cv = rand_bits(rng, T, Hkv, D), rand_bits(rng, T, Hkv, D)
    anchors = np.stack([np.sort(rng.choice(T, size=9, replace=False)) for _ in range(2)]).astype(np.int32)
    s = orc.active_sets(anchors, T)
    ranks, pos = s.ranks(1), s.positions(1)
    n = len(pos)
    qn, kn, vn = rand_bits(rng, n, H, D), rand_bits(rng, n, Hkv, D), rand_bits(rng, n, Hkv, D)
    scale = 0.3
    # V == 1 everywhere -> every output is exactly a convex combination of ones
    ones = np.full((T, Hkv, D), 0x3F80, dtype=np.uint16)
    out, _ = orc.repair_attention(ck, ones, qn, kn, ones[:n], s.u_pos, ranks, scale)
    np.testing.assert_allclose(out, 1.0, rtol=1e-13)
    # a target that is the first member of U sees only itself -> output = its fresh V
    s0 = orc.active_sets(anchors[:1], T)
    r0 = s0.ranks(0)
    n0 = len(r0)
    q0, k0, v0 = rand_bits(rng, n0, H, D), rand_bits(rng, n0, Hkv, D), rand_bits(rng, n0, Hkv, D)
    out0, _ = orc.repair_attention(ck, cv, q0, k0, v0, s0.u_pos, r0, scale)
    np.testing.assert_allclose(out0[0], np.repeat(bf.f64(v0[0]), H // Hkv, axis=0), rtol=1e-13)
    # fresh == cached -> mixing is a no-op (same as reading the cache only)
    same_k, same_v = ck[pos], cv[pos]
    a, _ = orc.repair_attention(ck, cv, qn, same_k, same_v, s.u_pos, ranks, scale)
    b, _ = orc.repair_attention(ck, cv, qn, None, None, s.u_pos, ranks, scale)
    np.testing.assert_array_equal(a, b)
    # tokens of U that are not active at this layer contribute their *cached* states
    mk, mv = orc.mix_context(ck, cv, kn, vn, s.u_pos, ranks)
    inactive = np.setdiff1d(np.arange(len(s.u_pos)), ranks)
    assert len(inactive) > 0
    np.testing.assert_array_equal(mk[inactive], ck[s.u_pos[inactive]])
    np.testing.assert_array_equal(mv[ranks], vn)


# ------------------------------------------ controlled configurations (explicit lists) ----

def test_list_attention_reduces_to_the_method_and_matches_bruteforce():
    rng = np.random.default_rng(21)
    H, Hkv, D, T, L, k = 4, 2, 16, 57, 3, 10
    ck, cv = rand_bits(rng, T, Hkv, D), rand_bits(rng, T, Hkv, D)
    anchors = np.stack([np.sort(rng.choice(T, size=k, replace=False)) for _ in range(L)]).astype(np.int32)
    s = orc.active_sets(anchors, T)
    scale = 0.25
    l = 1
    pos = s.positions(l)
    qn, kn, vn = rand_bits(rng, len(pos), H, D), rand_bits(rng, len(pos), Hkv, D), rand_bits(rng, len(pos), Hkv, D)
    # context = U, targets = R_l  ->  the method itself; context = everything -> the full-prefix control
    a, la = orc.list_attention(ck, cv, qn, kn, vn, s.u_pos, pos, scale)
    b, lb = orc.repair_attention(ck, cv, qn, kn, vn, s.u_pos, s.ranks(l), scale)
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(orc.limits(s.u_pos, pos), s.ranks(l))
    c, _ = orc.list_attention(ck, cv, qn, kn, vn, np.arange(T), pos, scale)
    d, _ = orc.repair_attention(ck, cv, qn, kn, vn, s.u_pos, s.ranks(l), scale, full_prefix=True)
    np.testing.assert_array_equal(c, d)
    # arbitrary targets that need not lie in the context list (global targets, sparse context variants)
    for trial in range(4):
        ctx = np.sort(rng.choice(np.arange(3, T), size=15, replace=False)).astype(np.int32)
        tgt = np.sort(rng.choice(T, size=12, replace=False)).astype(np.int32)
        tgt[0] = 1                                   # before every context position: empty context
        tgt = np.unique(tgt)
        q2, k2, v2 = rand_bits(rng, len(tgt), H, D), rand_bits(rng, len(tgt), Hkv, D), rand_bits(rng, len(tgt), Hkv, D)
        out, lse = orc.list_attention(ck, cv, q2, k2, v2, ctx, tgt, scale)
        ref, ref_lse, _ = bf.attention(ck, cv, q2, k2, v2, ctx, tgt, scale)
        np.testing.assert_allclose(out, ref, rtol=1e-10, atol=1e-12)
        assert np.all(out[0] == 0) and np.all(np.isneginf(lse[0]))          # the reading for an empty context
        np.testing.assert_allclose(lse[1:], ref_lse[1:], rtol=1e-12)
        lim = orc.limits(ctx, tgt)
        assert lim[0] == -1 and all(lim[i] == np.searchsorted(ctx, tgt[i], side="right") - 1 for i in range(len(tgt)))


def test_mean_scores():
    rng = np.random.default_rng(22)
    a = rng.random((5, 33))
    np.testing.assert_allclose(orc.mean_scores(a), a.mean(axis=0), rtol=1e-15)


# ------------------------------------------------------------------ update ----

def test_scatter_semantics_and_order_equivalence():
    rng = np.random.default_rng(9)
    H, Hkv, D, T = 4, 2, 16, 50
    store_k, store_v = rand_bits(rng, Hkv, T, D), rand_bits(rng, Hkv, T, D)      # head-major storage
    ck, cv = store_k.transpose(1, 0, 2), store_v.transpose(1, 0, 2)              # strided views
    anchors = np.stack([np.sort(rng.choice(T, size=12, replace=False)) for _ in range(2)]).astype(np.int32)
    s = orc.active_sets(anchors, T)
    ranks, pos = s.ranks(1), s.positions(1)
    n = len(pos)
    qn, kn, vn = rand_bits(rng, n, H, D), rand_bits(rng, n, Hkv, D), rand_bits(rng, n, Hkv, D)
    before, _ = orc.repair_attention(ck, cv, qn, kn, vn, s.u_pos, ranks, 0.25)
    k0, v0 = ck.copy(), cv.copy()
    orc.scatter(ck, cv, kn, vn, pos)
    rest = np.setdiff1d(np.arange(T), pos)
    np.testing.assert_array_equal(ck[rest], k0[rest])
    np.testing.assert_array_equal(cv[rest], v0[rest])
    np.testing.assert_array_equal(ck[pos], kn)
    np.testing.assert_array_equal(cv[pos], vn)
    k1 = ck.copy()
    orc.scatter(ck, cv, kn, vn, pos)                                              # idempotent
    np.testing.assert_array_equal(ck, k1)
    after, _ = orc.repair_attention(ck, cv, qn, None, None, s.u_pos, ranks, 0.25)  # update first, then attend
    np.testing.assert_array_equal(before, after)


# ------------------------------------------------------- input recipe sanity ----

def test_tiny_workload_scores_are_peaked_on_the_planted_chunk():
    w = inputs.tiny()
    q, k, v = inputs.layer_qkv(w, 0, 0)
    raw = orc.raw_scores(inputs.bf16_bits(q), inputs.bf16_bits(k), 1 / np.sqrt(w.head_dim))
    kk = orc.anchor_count(w.ctx_lens[0], w.ratio)
    assert kk == 154
    sel = orc.topk(raw, kk)
    in_planted = np.sum((sel >= 512) & (sel < 768))
    assert in_planted > 120
    assert abs(raw.sum() - 1) < 1e-12
