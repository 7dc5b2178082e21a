"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the
Llama-3.1-8B-shaped 16K layer in full, and the Qwen3-14B-shaped 32K context (two layers of the
stack: the oracle scores every context position of both).  Scores and anchors are compared in full;
attention on sampled target rows the oracle computes one by one - whole first and last query tiles
plus rows spread over the staircase."""
import numpy as np
import pytest
import torch

from paper_2609_33503_b200 import inputs
from tests.harness import Case, attention_errors, check_anchor_band

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3


def sampled_rows(n, tile_rows, n_spread, seed):
    rng = np.random.default_rng(seed)
    rows = set(range(min(n, tile_rows))) | set(range(max(0, n - 2 * tile_rows), n))
    rows |= set(int(x) for x in np.linspace(0, n - 1, n_spread))
    rows |= set(int(x) for x in rng.integers(0, n, size=n_spread))
    return np.array(sorted(rows), dtype=np.int32)


def run_full(w, tile_targets, n_spread):
    from paper_2609_33503_b200 import binding as B
    case = Case(w)
    s = case.make_session(want_norm=True)
    views = case.cache_views()
    s.score_select(case.q_layers, views)
    raw = s.raw.cpu().numpy().astype(np.float64)
    anchors = s.anchors.cpu().numpy()
    T = w.ctx_lens[0]
    for l in range(w.n_layers):
        ref = case.raw[(l, 0)]
        assert np.all(np.abs(raw[l] - ref) <= 1e-3 * ref + 1e-6 / T), np.abs(raw[l] / ref - 1).max()
        check_anchor_band(ref, case.k[0], anchors[l])
    # downstream on the oracle's own sets
    s.build_active_sets(case.anchors_tensor())
    n_u, n_r = s.counts()
    assert n_u[0] == len(case.sets[0].u_pos)
    for l in range(w.n_layers):
        assert n_r[l][0] == len(case.sets[0].ranks(l))
        f = case.fresh[l]
        for mode, full_prefix in ((B.CTX_UNION, False), (B.CTX_FULL_PREFIX, True)):
            out = torch.zeros_like(f.q_new)
            s.attention(l, views[l], f.q_new, f.k_new, f.v_new, out, case.max_targets(l), case.max_ctx(), mode=mode)
            st, detail = B.relaxkv_read_device_status()
            assert st == 0, (st, detail)
            rows = sampled_rows(f.q_new.shape[0], 2 * tile_targets, n_spread, seed=l)
            if full_prefix:
                rows = rows[:: 4]                       # the full-prefix oracle rows are several times longer
            ref, _ = case.oracle_attention(l, 0, full_prefix=full_prefix, rows=rows)
            mx, mean = attention_errors(out[torch.from_numpy(rows.astype(np.int64)).to(out.device)], ref)
            assert mx <= MAX_ABS and mean <= MEAN_ABS, (l, full_prefix, mx, mean)
        # cache update, bit-exact
        k2, v2 = case.k_cache[l].clone(), case.v_cache[l].clone()
        s.scatter(l, B.CacheView(k2, v2, [0]), f.k_new, f.v_new, case.max_targets(l))
        pos = torch.from_numpy(case.sets[0].positions(l).astype(np.int64)).to(k2.device)
        assert torch.equal(k2[pos], f.k_new) and torch.equal(v2[pos], f.v_new)
        keep = torch.ones(T, dtype=torch.bool, device=k2.device)
        keep[pos] = False
        assert torch.equal(k2[keep], case.k_cache[l][keep]) and torch.equal(v2[keep], case.v_cache[l][keep])


def test_llama8b_16k_full_size():
    run_full(inputs.llama8b_16k(), tile_targets=32, n_spread=48)


@pytest.mark.parametrize("ratio", [0.05, 0.15, 0.30])
def test_qwen14b_32k_full_context_two_layers(ratio):
    """The 32K context at the end points and the default of the anchor-ratio sweep, each with its Full-Prefix
    Control (run_full checks both context modes on the same targets)."""
    run_full(inputs.qwen14b_32k("calibrated", ratio, n_layers=2), tile_targets=25, n_spread=24 if ratio == 0.15 else 12)


def test_persistent_form_at_32k_equals_the_one_shot_kernel():
    """A 32K layer (3 600 query-tile pairs x heads) through the persistent form, one block per SM as in production:
    bit-identical to the one-shot kernel's output, and sampled rows against the oracle."""
    from paper_2609_33503_b200 import binding as B
    w = inputs.qwen14b_32k("calibrated", 0.15, n_layers=1)
    case = Case(w)
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    f = case.fresh[0]
    outs = []
    for persistent in (2, 1):
        s.shape.set_tuning(attention_persistent=persistent)
        out = torch.zeros_like(f.q_new)
        lse = torch.zeros(w.n_q_heads, f.q_new.shape[0], dtype=torch.float32, device=out.device)
        s.attention(0, case.cache_views()[0], f.q_new, f.k_new, f.v_new, out, case.max_targets(0), case.max_ctx(), lse_out=lse)
        st, detail = B.relaxkv_read_device_status()
        assert st == 0, (st, detail)
        outs.append((out, lse))
    s.shape.set_tuning()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    rows = sampled_rows(f.q_new.shape[0], 50, 16, seed=3)
    ref, _ = case.oracle_attention(0, 0, full_prefix=False, rows=rows)
    mx, mean = attention_errors(outs[1][0][torch.from_numpy(rows.astype(np.int64)).to(out.device)], ref)
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)


def test_decode_attention_at_32k():
    """One decode token per request over 32K-token caches at the Qwen3-14B head layout, in the launch configuration the
    time-to-first-token benchmark uses (automatic split: one wave of blocks): output and log-sum-exp against the oracle."""
    from paper_2609_33503_b200 import binding as B
    import oracle.relaxkv_oracle as orc
    H, Hkv, D = 40, 8, 128
    lens, pos = (32768, 20000), (32767, 12345)
    offs = [0, 32768 + 64]
    rows = offs[1] + lens[1] + 64
    g = torch.Generator(device="cpu").manual_seed(21)
    k_all = torch.randn(rows, Hkv, D, generator=g).to(torch.bfloat16).cuda()
    v_all = torch.randn(rows, Hkv, D, generator=g).to(torch.bfloat16).cuda()
    q = torch.randn(2, H, D, generator=g).to(torch.bfloat16).cuda()
    shape = B.Shape(H, Hkv, D, list(lens), None, D ** -0.5)
    ws = torch.empty(B.relaxkv_workspace_bytes(shape, 1) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    out = torch.zeros_like(q)
    lse = torch.zeros(H, 2, dtype=torch.float32, device="cuda")
    B.relaxkv_cache_attention(shape, B.CacheView(k_all, v_all, offs), q, torch.tensor(pos, dtype=torch.int32).cuda(),
                              torch.tensor([0, 1, 2], dtype=torch.int32).cuda(), [1, 1], out, ws, lse_out=lse)
    st, detail = B.relaxkv_read_device_status()
    assert st == 0, (st, detail)
    for b in range(2):
        kb = inputs.bf16_bits(k_all[offs[b]:offs[b] + lens[b]].contiguous())
        vb = inputs.bf16_bits(v_all[offs[b]:offs[b] + lens[b]].contiguous())
        ref, ref_lse = orc.list_attention(kb, vb, inputs.bf16_bits(q[b:b + 1]), None, None, np.arange(lens[b]),
                                          np.array([pos[b]], dtype=np.int32), D ** -0.5)
        mx, mean = attention_errors(out[b:b + 1], ref)
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (b, mx, mean)
        np.testing.assert_allclose(lse[:, b:b + 1].cpu().numpy().T, ref_lse, atol=2e-3, rtol=1e-4)


def test_maximum_batch_of_64_requests():
    """The request table's limit (64 requests in one call) with ragged lengths from 1 token upwards:
    scores, anchors, sets, attention of every row, and the cache update against the oracle."""
    from paper_2609_33503_b200 import binding as B
    rng = np.random.default_rng(64)
    ctx = tuple(int(x) for x in np.concatenate([[1, 2, 127, 128, 129, 700], rng.integers(3, 600, size=58)]))
    q = tuple(int(x) for x in rng.integers(1, 40, size=64))
    w = inputs.scaled_down(inputs.qwen14b_32k("literal"), ctx, q, n_layers=2, chunk=64).replace(ratio=0.2)
    assert w.n_req == 64
    case = Case(w)
    s = case.make_session()
    views = case.cache_views()
    s.score_select(case.q_layers, views)
    anchors = s.anchors.cpu().numpy()
    for l in range(w.n_layers):
        for b in range(w.n_req):
            check_anchor_band(case.raw[(l, b)], case.k[b], anchors[l, case.k_cu[b]:case.k_cu[b + 1]])
    s.build_active_sets(case.anchors_tensor())
    n_u, n_r = s.counts()
    assert n_u == [len(case.sets[b].u_pos) for b in range(64)]
    u_pos, u_cu = s.u_pos.cpu().numpy(), s.u_cu.cpu().numpy()
    for b in range(64):
        assert np.array_equal(u_pos[u_cu[b]:u_cu[b + 1]], case.sets[b].u_pos)
    for l in range(w.n_layers):
        assert n_r[l] == case.max_targets(l)
        f = case.fresh[l]
        out = torch.zeros_like(f.q_new)
        s.attention(l, views[l], f.q_new, f.k_new, f.v_new, out, case.max_targets(l), case.max_ctx())
        st, detail = B.relaxkv_read_device_status()
        assert st == 0, (st, detail)
        for b in range(64):
            ref, _ = case.oracle_attention(l, b)
            mx, mean = attention_errors(out[f.row_cu[b]:f.row_cu[b + 1]], ref)
            assert mx <= MAX_ABS and mean <= MEAN_ABS, (l, b, mx, mean)
        k2, v2 = case.k_cache[l].clone(), case.v_cache[l].clone()
        s.scatter(l, B.CacheView(k2, v2, [int(x) for x in case.ctx_cu[:-1]]), f.k_new, f.v_new, case.max_targets(l))
        for b in range(64):
            pos = torch.from_numpy(case.sets[b].positions(l).astype(np.int64)).to(k2.device) + int(case.ctx_cu[b])
            assert torch.equal(k2[pos], f.k_new[f.row_cu[b]:f.row_cu[b + 1]])
        assert int((k2 != case.k_cache[l]).any(dim=(1, 2)).sum()) <= sum(case.max_targets(l))
    # one request more than the table holds is refused before any launch
    too_many = B.Shape(w.n_q_heads, w.n_kv_heads, w.head_dim, ctx + (5,), q + (1,))
    assert B.relaxkv_workspace_bytes(too_many, 2, case.k + [1]) == 0


def test_ragged_batch_with_a_64k_context_sampled_rows():
    """Two requests of the ragged benchmark batch (65 536 and 8 192 context tokens) in one call, two layers,
    Qwen3-14B head geometry.  The anchors are drawn at random (the oracle's scoring of 64K keys is not needed
    to check what follows): the repair schedule must match the oracle's bit for bit, the attention of
    sampled target rows and the cache update must match the oracle."""
    from paper_2609_33503_b200 import binding as B
    ctx, q = (65536, 8192), (64, 32)
    w = inputs.scaled_down(inputs.qwen14b_32k("calibrated"), ctx, q, n_layers=2, chunk=512)
    rng = np.random.default_rng(7)
    k = [max(1, round(0.15 * t)) for t in ctx]
    override = [[np.sort(rng.choice(t, size=kb, replace=False)).astype(np.int32) for t, kb in zip(ctx, k)] for _ in range(2)]
    case = Case(w, anchors_override=override)
    assert case.k == k
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    n_u, n_r = s.counts()
    u_pos, u_cu = s.u_pos.cpu().numpy(), s.u_cu.cpu().numpy()
    r_rank, r_cu = s.r_rank.cpu().numpy(), s.r_cu.cpu().numpy()
    for b in range(2):
        assert np.array_equal(u_pos[u_cu[b]:u_cu[b + 1]], case.sets[b].u_pos)
    views = case.cache_views()
    for l in range(2):
        for b in range(2):
            i = l * 2 + b
            assert np.array_equal(r_rank[r_cu[i]:r_cu[i + 1]], case.sets[b].ranks(l))
        f = case.fresh[l]
        out = torch.zeros_like(f.q_new)
        s.attention(l, views[l], f.q_new, f.k_new, f.v_new, out, n_r[l], n_u)
        st, detail = B.relaxkv_read_device_status()
        assert st == 0, (st, detail)
        for b in range(2):
            n = f.row_cu[b + 1] - f.row_cu[b]
            rows = sampled_rows(n, 50, 12, seed=10 * l + b)
            ref, _ = case.oracle_attention(l, b, rows=rows)
            got = out[f.row_cu[b]:f.row_cu[b + 1]][torch.from_numpy(rows.astype(np.int64)).to(out.device)]
            mx, mean = attention_errors(got, ref)
            assert mx <= MAX_ABS and mean <= MEAN_ABS, (l, b, mx, mean)
        k2, v2 = case.k_cache[l].clone(), case.v_cache[l].clone()
        s.scatter(l, B.CacheView(k2, v2, [0, ctx[0]]), f.k_new, f.v_new, n_r[l])
        for b in range(2):
            pos = torch.from_numpy(case.sets[b].positions(l).astype(np.int64)).to(k2.device) + (0 if b == 0 else ctx[0])
            assert torch.equal(k2[pos], f.k_new[f.row_cu[b]:f.row_cu[b + 1]]) and torch.equal(v2[pos], f.v_new[f.row_cu[b]:f.row_cu[b + 1]])


def test_whole_ragged_batch_of_eight_in_one_call():
    """All eight requests of the ragged benchmark batch (8K ... 64K context tokens, Qwen3-14B head geometry, the
    benchmark's query lengths) packed into ONE call per step, two layers - the launch configuration the ragged
    benchmark times.  Anchors are drawn at random (the oracle's scoring of 250K keys is not what is checked here):
    the repair schedule must equal the oracle's bit for bit for every request, the attention of sampled target rows
    of every request must match the oracle in both context modes, and the cache update must be bit-exact."""
    from paper_2609_33503_b200 import binding as B
    w = inputs.ragged8(n_layers=2)
    ctx = w.ctx_lens
    rng = np.random.default_rng(88)
    k = [max(1, round(0.15 * t)) for t in ctx]
    override = [[np.sort(rng.choice(t, size=kb, replace=False)).astype(np.int32) for t, kb in zip(ctx, k)] for _ in range(2)]
    case = Case(w, anchors_override=override)
    assert case.k == k and w.n_req == 8
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    n_u, n_r = s.counts()
    u_pos, u_cu = s.u_pos.cpu().numpy(), s.u_cu.cpu().numpy()
    r_rank, r_cu = s.r_rank.cpu().numpy(), s.r_cu.cpu().numpy()
    for b in range(8):
        assert np.array_equal(u_pos[u_cu[b]:u_cu[b + 1]], case.sets[b].u_pos)
    views = case.cache_views()
    offs = [int(x) for x in case.ctx_cu[:-1]]
    for l in range(2):
        for b in range(8):
            i = l * 8 + b
            assert np.array_equal(r_rank[r_cu[i]:r_cu[i + 1]], case.sets[b].ranks(l))
        f = case.fresh[l]
        for mode, full_prefix in ((B.CTX_UNION, False), (B.CTX_FULL_PREFIX, True)):
            out = torch.zeros_like(f.q_new)
            s.attention(l, views[l], f.q_new, f.k_new, f.v_new, out, n_r[l], n_u, mode=mode)
            st, detail = B.relaxkv_read_device_status()
            assert st == 0, (st, detail)
            for b in range(8):
                n = f.row_cu[b + 1] - f.row_cu[b]
                rows = sampled_rows(n, 25, 6, seed=100 * l + b)
                if full_prefix:
                    rows = rows[::5]
                ref, _ = case.oracle_attention(l, b, full_prefix=full_prefix, rows=rows)
                got = out[f.row_cu[b]:f.row_cu[b + 1]][torch.from_numpy(rows.astype(np.int64)).to(out.device)]
                mx, mean = attention_errors(got, ref)
                assert mx <= MAX_ABS and mean <= MEAN_ABS, (l, b, full_prefix, mx, mean)
        k2, v2 = case.k_cache[l].clone(), case.v_cache[l].clone()
        s.scatter(l, B.CacheView(k2, v2, offs), f.k_new, f.v_new, n_r[l])
        touched = torch.zeros(int(case.ctx_cu[-1]), dtype=torch.bool, device=k2.device)
        for b in range(8):
            pos = torch.from_numpy(case.sets[b].positions(l).astype(np.int64)).to(k2.device) + offs[b]
            assert torch.equal(k2[pos], f.k_new[f.row_cu[b]:f.row_cu[b + 1]]) and torch.equal(v2[pos], f.v_new[f.row_cu[b]:f.row_cu[b + 1]])
            touched[pos] = True
        assert torch.equal(k2[~touched], case.k_cache[l][~touched]) and torch.equal(v2[~touched], case.v_cache[l][~touched])


def test_controlled_configurations_at_32k_sampled_rows():
    """The explicit-list entry points at the size the benchmark times them (32K context, Qwen3-14B heads): global
    repair targets that need not lie in U (a top-m of a seeded score vector, context U), and a layer-wise sparse
    context of |U| entries with the method's targets.  Random anchors (what is checked is the list path, not the
    scoring); sampled target rows against the oracle's list attention, the cache update bit-exact."""
    from oracle import relaxkv_oracle as orc
    from paper_2609_33503_b200 import binding as B
    T = 32768
    w = inputs.qwen14b_32k("calibrated", 0.15, n_layers=2)
    rng = np.random.default_rng(321)
    k = [max(1, round(0.15 * T))]
    override = [[np.sort(rng.choice(T, size=k[0], replace=False)).astype(np.int32)] for _ in range(2)]
    case = Case(w, anchors_override=override)
    s = case.make_session()
    sets = case.sets[0]
    n_u = len(sets.u_pos)
    g = rng.random(T).astype(np.float32)
    view = case.cache_views()[0]
    cfgs = {"global_targets": (sets.u_pos.astype(np.int32), orc.topk(g.astype(np.float64), min(int(0.2 * T), n_u)).astype(np.int32)),
            "layerwise_sparse": (orc.topk(rng.random(T), n_u).astype(np.int32), sets.positions(0).astype(np.int32))}
    for name, (ctx, tgt) in cfgs.items():
        q, kn, vn = inputs.fresh_qkv(w, 0, 0, case.k_cache[0], case.v_cache[0], torch.from_numpy(tgt.astype(np.int64)))
        dev = case.device
        ctx_pos, tgt_pos = torch.from_numpy(ctx).to(dev), torch.from_numpy(tgt).to(dev)
        ctx_cu = torch.tensor([0, len(ctx)], dtype=torch.int32, device=dev)
        tgt_cu = torch.tensor([0, len(tgt)], dtype=torch.int32, device=dev)
        out = torch.zeros_like(q)
        B.relaxkv_list_attention(s.shape, view, q, kn, vn, ctx_pos, ctx_cu, tgt_pos, tgt_cu, [len(tgt)], [len(ctx)], out, s.workspace)
        st, detail = B.relaxkv_read_device_status()
        assert st == 0, (name, st, detail)
        rows = sampled_rows(len(tgt), 50, 16, seed=9)
        ref, _ = orc.list_attention(case.req_k(0, 0), case.req_v(0, 0), inputs.bf16_bits(q), inputs.bf16_bits(kn), inputs.bf16_bits(vn),
                                    ctx, tgt, case.scale, rows=rows)
        mx, mean = attention_errors(out[torch.from_numpy(rows.astype(np.int64)).to(dev)], ref)
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (name, mx, mean)
        k2, v2 = case.k_cache[0].clone(), case.v_cache[0].clone()
        B.relaxkv_scatter_kv_lists(s.shape, B.CacheView(k2, v2, [0]), kn, vn, tgt_pos, tgt_cu, [len(tgt)])
        pos = tgt_pos.long()
        assert torch.equal(k2[pos], kn) and torch.equal(v2[pos], vn)
        keep = torch.ones(T, dtype=torch.bool, device=dev)
        keep[pos] = False
        assert torch.equal(k2[keep], case.k_cache[0][keep]) and torch.equal(v2[keep], case.v_cache[0][keep])


def test_query_prefill_attention_at_32k():
    """relaxkv_query_prefill_attention at the benchmark's size: 128 query tokens behind a 32K context, Qwen3-14B heads
    (the launch the time-to-first-token region makes per layer).  Every query row against the oracle's causal attention;
    the emitted context scores against the oracle's supplied-normaliser scores in full."""
    from oracle import relaxkv_oracle as orc
    from paper_2609_33503_b200 import binding as B
    w = inputs.qwen14b_32k("calibrated", 0.15, n_layers=1)
    T, Qn, H, Hkv, D = 32768, 128, w.n_q_heads, w.n_kv_heads, w.head_dim
    scale = D ** -0.5
    q, k, v = inputs.layer_qkv(w, 0, 0, "cuda")
    g = torch.Generator(device="cuda").manual_seed(17)
    k_all = torch.cat([k, torch.randn(Qn + 1, Hkv, D, device="cuda", generator=g).to(torch.bfloat16)]).contiguous()
    v_all = torch.cat([v, torch.randn(Qn + 1, Hkv, D, device="cuda", generator=g).to(torch.bfloat16)]).contiguous()
    shape = B.Shape(H, Hkv, D, [T], [Qn], scale)
    ext = B.Shape(H, Hkv, D, [T + Qn], [Qn], scale)
    ws = torch.empty(B.relaxkv_workspace_bytes(ext, 1) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    out = torch.zeros_like(q)
    lse = torch.zeros(H, Qn, dtype=torch.float32, device="cuda")
    raw = torch.zeros(T, dtype=torch.float32, device="cuda")
    B.relaxkv_query_prefill_attention(shape, B.CacheView(k_all, v_all, [0]), q, out, lse, raw, ws)
    st, detail = B.relaxkv_read_device_status()
    assert st == 0, (st, detail)
    kb, vb, qb = inputs.bf16_bits(k_all[:T + Qn]), inputs.bf16_bits(v_all[:T + Qn]), inputs.bf16_bits(q)
    ref, ref_lse = orc.list_attention(kb, vb, qb, None, None, np.arange(T + Qn), np.arange(T, T + Qn), scale)
    mx, mean = attention_errors(out, ref)
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
    np.testing.assert_allclose(lse.cpu().numpy().T, ref_lse, atol=2e-3, rtol=1e-4)
    ref_raw = orc.raw_scores(qb, kb[:T], scale, lse=ref_lse.T)
    got = raw.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref_raw) <= 1e-3 * ref_raw + 1e-6 / T), np.abs(got / ref_raw - 1).max()
