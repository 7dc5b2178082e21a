"""GPU parity: every C-ABI call against the fp64 CPU oracle on the same seeded bits.

Tolerances (bf16 inputs, fp32 accumulation, P rounded to bf16 before P*V):
  attention outputs  max-abs <= 2e-2, mean-abs <= 2e-3
  raw scores         |gpu - ref| <= 1e-3 * ref + 1e-6 / T_c ;  normalised scores abs <= 1e-3
  anchors            bit-exact when scores are fed in exactly; otherwise exact outside a 1e-3
                     relative band around the k-th score
  sets, gather, scatter: bit-exact
"""
import numpy as np
import pytest
import torch

from oracle import relaxkv_oracle as orc
from paper_2609_33503_b200 import inputs
from tests.harness import Case, attention_errors, bf16_to_f64, check_anchor_band

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3


def B():
    from paper_2609_33503_b200 import binding
    return binding


def assert_status_ok():
    st, detail = B().relaxkv_read_device_status()
    assert st == 0, (B().status_string(st), detail)


def small_llama(n_layers=2, ctx=(2048,), q=(48,)):
    return inputs.scaled_down(inputs.llama8b_16k(), ctx, q, n_layers=n_layers, chunk=256)


def small_qwen(n_layers=3, ctx=(1536,), q=(40,)):
    return inputs.scaled_down(inputs.qwen14b_32k("calibrated"), ctx, q, n_layers=n_layers, chunk=128)


def small_ragged():
    return inputs.scaled_down(inputs.qwen14b_32k("calibrated"), (640, 1280, 2176), (17, 33, 64), n_layers=2, chunk=128)


WORKLOADS = {
    "tiny": inputs.tiny,
    "llama_small": small_llama,
    "qwen_small": small_qwen,
    "ragged_small": small_ragged,
}


@pytest.fixture(scope="module", params=list(WORKLOADS))
def case(request):
    return Case(WORKLOADS[request.param]())


# ------------------------------------------------------------------------- selection ----

def test_scores_and_anchors(case):
    w = case.w
    s = case.make_session(want_norm=True)
    s.score_select(case.q_layers, case.cache_views())
    assert_status_ok()
    raw = s.raw.cpu().numpy().astype(np.float64)
    norm = s.norm.cpu().numpy().astype(np.float64)
    anchors = s.anchors.cpu().numpy()
    for l in range(w.n_layers):
        for b in range(w.n_req):
            T = w.ctx_lens[b]
            ref = case.raw[(l, b)]
            got = raw[l, case.ctx_cu[b]:case.ctx_cu[b + 1]]
            assert np.all(np.abs(got - ref) <= 1e-3 * ref + 1e-6 / T), np.abs(got / ref - 1).max()
            assert abs(got.sum() - 1.0) < 1e-3
            np.testing.assert_allclose(norm[l, case.ctx_cu[b]:case.ctx_cu[b + 1]], orc.minmax(ref), atol=1e-3)
            check_anchor_band(ref, case.k[b], anchors[l, case.k_cu[b]:case.k_cu[b + 1]])


def test_scores_with_supplied_lse(case):
    """Supplying the rows' log-normalisers skips the statistics pass and gives the same scores."""
    w = case.w
    s = case.make_session()
    lses = []
    for l in range(w.n_layers):
        per_req = [orc.row_lse(case.req_q(l, b), case.req_k(l, b), case.scale) for b in range(w.n_req)]
        lses.append(torch.from_numpy(np.concatenate(per_req, axis=1).astype(np.float32)).contiguous().to(case.device))
    s.score_select(case.q_layers, case.cache_views(), row_lse_layers=lses)
    assert_status_ok()
    raw = s.raw.cpu().numpy().astype(np.float64)
    for l in range(w.n_layers):
        for b in range(w.n_req):
            ref = case.raw[(l, b)]
            got = raw[l, case.ctx_cu[b]:case.ctx_cu[b + 1]]
            assert np.all(np.abs(got - ref) <= 1e-3 * ref + 1e-6 / w.ctx_lens[b])


def test_select_exact_on_given_scores(case):
    """Oracle scores rounded to fp32 go in; anchors must match the oracle's top-k of those very
    values bit for bit (ties included: a block of equal scores is planted)."""
    w = case.w
    nb, L = w.n_req, w.n_layers
    shape = case.make_session().shape
    raw32 = np.zeros((L, int(case.ctx_cu[-1])), dtype=np.float32)
    for l in range(L):
        for b in range(nb):
            r = case.raw[(l, b)].astype(np.float32)
            kth = np.sort(r)[::-1][case.k[b] - 1]
            idx = np.argsort(np.abs(r - kth))[:9]        # make 9 scores tie with the k-th one
            r[idx] = kth
            raw32[l, case.ctx_cu[b]:case.ctx_cu[b + 1]] = r
    d_raw = torch.from_numpy(raw32).to(case.device)
    d_anchor = torch.full((L, int(case.k_cu[-1])), -1, dtype=torch.int32, device=case.device)
    d_norm = torch.empty_like(d_raw)
    B().relaxkv_select_topk(shape, L, case.k, d_raw, d_anchor, norm_scores_out=d_norm)
    assert_status_ok()
    got = d_anchor.cpu().numpy()
    for l in range(L):
        for b in range(nb):
            seg = raw32[l, case.ctx_cu[b]:case.ctx_cu[b + 1]].astype(np.float64)
            np.testing.assert_array_equal(got[l, case.k_cu[b]:case.k_cu[b + 1]], orc.topk(seg, case.k[b]))
            np.testing.assert_allclose(d_norm[l, case.ctx_cu[b]:case.ctx_cu[b + 1]].cpu().numpy(), orc.minmax(seg),
                                       atol=2e-6)


def test_active_sets_bitexact(case):
    w = case.w
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    assert_status_ok()
    n_u, n_r = s.counts()
    u_cu = s.u_cu.cpu().numpy()
    r_cu = s.r_cu.cpu().numpy()
    u_pos, u_rank, h = s.u_pos.cpu().numpy(), s.u_rank.cpu().numpy(), s.highest_layer.cpu().numpy()
    r_rank = s.r_rank.cpu().numpy()
    for b in range(w.n_req):
        ref = case.sets[b]
        assert n_u[b] == len(ref.u_pos) == u_cu[b + 1] - u_cu[b]
        np.testing.assert_array_equal(u_pos[u_cu[b]:u_cu[b + 1]], ref.u_pos)
        np.testing.assert_array_equal(u_rank[case.ctx_cu[b]:case.ctx_cu[b + 1]], ref.u_rank)
        np.testing.assert_array_equal(h[case.ctx_cu[b]:case.ctx_cu[b + 1]], ref.h)
        prev = None
        for l in range(w.n_layers):
            i = l * w.n_req + b
            got = r_rank[r_cu[i]:r_cu[i + 1]]
            np.testing.assert_array_equal(got, ref.ranks(l))
            assert n_r[l][b] == len(got)
            if prev is not None:
                assert set(got.tolist()) <= prev                     # monotone across layers
            prev = set(got.tolist())


# --------------------------------------------------------------------- gather / scatter ----

@pytest.mark.parametrize("head_major", [False, True])
def test_gather_and_scatter_bitexact(head_major):
    case = Case(small_ragged(), head_major_cache=head_major)
    w = case.w
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    nb = w.n_req
    for l in range(w.n_layers):
        f = case.fresh[l]
        views = case.cache_views()
        for mode in (B().CTX_UNION, B().CTX_FULL_PREFIX):
            rows = (sum(case.max_ctx()) if mode == B().CTX_UNION else int(case.ctx_cu[-1])) + 64
            kc = torch.full((rows, w.n_kv_heads, w.head_dim), 7.0, dtype=torch.bfloat16, device=case.device)
            vc = torch.full_like(kc, 7.0)
            s.gather(l, views[l], f.k_new, f.v_new, case.max_ctx(), kc, vc, mode=mode)
            assert_status_ok()
            kc_b, vc_b = inputs.bf16_bits(kc), inputs.bf16_bits(vc)
            off = 0
            for b in range(nb):
                _, kn, vn = case.fresh_bits(l, b)
                st = case.sets[b]
                if mode == B().CTX_UNION:
                    rk, rv = orc.mix_context(case.req_k(l, b), case.req_v(l, b), kn, vn, st.u_pos, st.ranks(l))
                else:
                    T = w.ctx_lens[b]
                    rk, rv = orc.mix_context(case.req_k(l, b), case.req_v(l, b), kn, vn,
                                             np.arange(T, dtype=np.int32), st.positions(l))
                np.testing.assert_array_equal(kc_b[off:off + len(rk)], rk)
                np.testing.assert_array_equal(vc_b[off:off + len(rv)], rv)
                off += len(rk)
            assert np.all(kc_b[off:off + 64] == 0) and np.all(vc_b[off:off + 64] == 0)     # zero pad rows
        # scatter into a copy of the cache
        k2, v2 = case.k_cache[l].clone(), case.v_cache[l].clone()
        if head_major:
            k2 = case.k_cache[l].permute(1, 0, 2).contiguous().permute(1, 0, 2)
            v2 = case.v_cache[l].permute(1, 0, 2).contiguous().permute(1, 0, 2)
        view2 = B().CacheView(k2, v2, [int(x) for x in case.ctx_cu[:-1]])
        for _ in range(2):                                            # idempotent
            s.scatter(l, view2, f.k_new, f.v_new, case.max_targets(l))
        assert_status_ok()
        k2_b, v2_b = inputs.bf16_bits(k2), inputs.bf16_bits(v2)
        for b in range(nb):
            rk, rv = case.req_k(l, b).copy(), case.req_v(l, b).copy()
            _, kn, vn = case.fresh_bits(l, b)
            orc.scatter(rk, rv, kn, vn, case.sets[b].positions(l))
            np.testing.assert_array_equal(k2_b[case.ctx_cu[b]:case.ctx_cu[b + 1]], rk)
            np.testing.assert_array_equal(v2_b[case.ctx_cu[b]:case.ctx_cu[b + 1]], rv)


# ---------------------------------------------------------------------------- attention ----

def run_attention(case, s, l, mode, simt, use_fresh=True, views=None):
    w = case.w
    f = case.fresh[l]
    out = torch.zeros_like(f.q_new)
    lse = torch.zeros(w.n_q_heads, f.q_new.shape[0], dtype=torch.float32, device=case.device)
    views = views or case.cache_views()
    s.attention(l, views[l], f.q_new, f.k_new if use_fresh else None, f.v_new if use_fresh else None, out,
                case.max_targets(l), case.max_ctx(), mode=mode, lse_out=lse, simt=simt)
    assert_status_ok()
    return out, lse


def check_attention(case, l, out, lse, full_prefix, use_fresh=True):
    f = case.fresh[l]
    worst = (0.0, 0.0)
    for b in range(case.w.n_req):
        lo, hi = f.row_cu[b], f.row_cu[b + 1]
        if hi == lo:
            continue
        ref, ref_lse = case.oracle_attention(l, b, full_prefix=full_prefix, use_fresh_kv=use_fresh)
        mx, mean = attention_errors(out[lo:hi], ref)
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (l, b, mx, mean)
        got_lse = lse[:, lo:hi].cpu().numpy().astype(np.float64).T
        np.testing.assert_allclose(got_lse, ref_lse, atol=2e-3, rtol=1e-4)
        worst = (max(worst[0], mx), max(worst[1], mean))
    return worst


@pytest.mark.parametrize("simt", [True, False], ids=["simt", "tcgen05"])
@pytest.mark.parametrize("full_prefix", [False, True], ids=["union", "fullprefix"])
def test_attention_matches_oracle(case, simt, full_prefix):
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    mode = B().CTX_FULL_PREFIX if full_prefix else B().CTX_UNION
    for l in range(case.w.n_layers):
        out, lse = run_attention(case, s, l, mode, simt)
        check_attention(case, l, out, lse, full_prefix)


@pytest.mark.parametrize("n_splits", [1, 2, 5, 32])
def test_context_split_matches_oracle(case, n_splits):
    """Few query tiles: the context of every tile pair is split over several blocks and the partial results are
    merged by their log-sum-exp.  Forced here to 1 (never), 2, 5 and 32 splits (more splits than some pairs have
    context tiles: empty splits), in both context modes, against the oracle; the rows past the true target count
    of a loosely bounded call stay untouched."""
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    s.shape.set_tuning(attention_ctx_splits=n_splits)
    try:
        for l in range(case.w.n_layers):
            for full_prefix in (False, True):
                out, lse = run_attention(case, s, l, B().CTX_FULL_PREFIX if full_prefix else B().CTX_UNION, simt=False)
                check_attention(case, l, out, lse, full_prefix)
        f = case.fresh[0]
        n = f.q_new.shape[0]
        pad = 7
        q_pad = torch.cat([f.q_new, torch.zeros(pad, *f.q_new.shape[1:], dtype=f.q_new.dtype, device=f.q_new.device)])
        out = torch.full_like(q_pad, 3.0)
        s.attention(0, case.cache_views()[0], q_pad, f.k_new, f.v_new, out, list(case.w.ctx_lens), list(case.w.ctx_lens))
        assert_status_ok()
        assert torch.all(out[n:] == 3.0)
        exact, _ = run_attention(case, s, 0, B().CTX_UNION, simt=False)
        assert torch.equal(out[:n], exact)
    finally:
        s.shape.set_tuning()


@pytest.mark.parametrize("blocks", [1, 3, 0], ids=["one_block", "three_blocks", "one_per_sm"])
def test_persistent_form_matches_oracle_and_the_one_shot_kernel(case, blocks):
    """The persistent form of the attention kernel (one block walks many query-tile pairs, claimed from a counter):
    forced on, with a single block walking every item, with three, and with one per SM; both context modes against
    the oracle, bit-identical to the one-shot kernel, rows past a loosely bounded call's true count untouched."""
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    try:
        for l in range(case.w.n_layers):
            for full_prefix in (False, True):
                mode = B().CTX_FULL_PREFIX if full_prefix else B().CTX_UNION
                s.shape.set_tuning(attention_ctx_splits=1, attention_persistent=2)
                ref, ref_lse = run_attention(case, s, l, mode, simt=False)
                s.shape.set_tuning(attention_ctx_splits=1, attention_persistent=1, attention_grid_blocks=blocks)
                out, lse = run_attention(case, s, l, mode, simt=False)
                check_attention(case, l, out, lse, full_prefix)
                assert torch.equal(out, ref) and torch.equal(lse, ref_lse)
        f = case.fresh[0]
        n = f.q_new.shape[0]
        q_pad = torch.cat([f.q_new, torch.zeros(7, *f.q_new.shape[1:], dtype=f.q_new.dtype, device=f.q_new.device)])
        out = torch.full_like(q_pad, 3.0)
        s.attention(0, case.cache_views()[0], q_pad, f.k_new, f.v_new, out, list(case.w.ctx_lens), list(case.w.ctx_lens))
        assert_status_ok()
        assert torch.all(out[n:] == 3.0)
    finally:
        s.shape.set_tuning()


@pytest.mark.parametrize("persistent", [2, 1], ids=["one_shot", "persistent"])
def test_attention_call_replays_from_a_cuda_graph(persistent):
    """Gather + attention captured into a CUDA graph (the persistent form also zeroes its work counter there) and
    replayed twice give the bits of the eager call."""
    case = Case(small_llama())
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    s.shape.set_tuning(attention_ctx_splits=1, attention_persistent=persistent, attention_grid_blocks=2)
    try:
        eager, eager_lse = run_attention(case, s, 0, B().CTX_UNION, simt=False)
        f = case.fresh[0]
        out = torch.zeros_like(f.q_new)
        lse = torch.zeros_like(eager_lse)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                s.attention(0, case.cache_views()[0], f.q_new, f.k_new, f.v_new, out, case.max_targets(0), case.max_ctx(),
                            mode=B().CTX_UNION, lse_out=lse)
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(2):
            out.zero_(); lse.zero_()
            g.replay()
            torch.cuda.synchronize()
            assert_status_ok()
            assert torch.equal(out, eager) and torch.equal(lse, eager_lse)
    finally:
        s.shape.set_tuning()


def test_attention_orders_agree_and_is_deterministic(case):
    """Update-then-attend from the cache equals mix-then-attend (Algorithm 1's order), bit for bit;
    two runs give identical bits."""
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    l = case.w.n_layers - 1
    f = case.fresh[l]
    a, _ = run_attention(case, s, l, B().CTX_UNION, simt=False)
    a2, _ = run_attention(case, s, l, B().CTX_UNION, simt=False)
    assert torch.equal(a, a2)
    k2, v2 = case.k_cache[l].clone(), case.v_cache[l].clone()
    view2 = B().CacheView(k2, v2, [int(x) for x in case.ctx_cu[:-1]])
    s.scatter(l, view2, f.k_new, f.v_new, case.max_targets(l))
    views = list(case.cache_views())
    views[l] = view2
    b_out, _ = run_attention(case, s, l, B().CTX_UNION, simt=False, use_fresh=False, views=views)
    assert torch.equal(a, b_out)


def test_full_ratio_is_dense_causal_attention():
    """Anchor ratio 100 %: every position is an anchor at every layer, so the output must equal plain
    causal attention over the fresh K/V (library SDPA in fp32 on the GPU, fp64 oracle on the CPU)."""
    w = small_llama(n_layers=1, ctx=(700,), q=(8,)).replace(ratio=1.0)
    case = Case(w)
    assert case.k == [700]
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    out, lse = run_attention(case, s, 0, B().CTX_UNION, simt=False)
    check_attention(case, 0, out, lse, False)
    f = case.fresh[0]
    G = w.group
    q = f.q_new.float().permute(1, 0, 2).unsqueeze(0)
    k = f.k_new.float().repeat_interleave(G, dim=1).permute(1, 0, 2).unsqueeze(0)
    v = f.v_new.float().repeat_interleave(G, dim=1).permute(1, 0, 2).unsqueeze(0)
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True, scale=case.scale)[0].permute(1, 0, 2)
    d = (out.float() - ref).abs()
    assert d.max().item() <= MAX_ABS and d.mean().item() <= MEAN_ABS


@pytest.mark.parametrize("ctx,q,ratio", [((1,), (1,), 0.15), ((129,), (3,), 0.01), ((257,), (5,), 1.0), ((130, 1, 515), (2, 1, 7), 0.3),
                                         ((1000, 300), (200, 131), 0.15)])
def test_edge_sizes(ctx, q, ratio):
    w = inputs.scaled_down(inputs.qwen14b_32k("literal"), ctx, q, n_layers=2, chunk=64).replace(ratio=ratio)
    case = Case(w)
    s = case.make_session(want_norm=True)
    s.score_select(case.q_layers, case.cache_views())
    assert_status_ok()
    anchors = s.anchors.cpu().numpy()
    for l in range(w.n_layers):
        for b in range(w.n_req):
            check_anchor_band(case.raw[(l, b)], case.k[b], anchors[l, case.k_cu[b]:case.k_cu[b + 1]])
    s.build_active_sets(case.anchors_tensor())
    for l in range(w.n_layers):
        for full_prefix in (False, True):
            out, lse = run_attention(case, s, l, B().CTX_FULL_PREFIX if full_prefix else B().CTX_UNION, simt=False)
            check_attention(case, l, out, lse, full_prefix)
    # the same sizes through the persistent form: two blocks walk every item (one-tile contexts, items without work)
    s.shape.set_tuning(attention_ctx_splits=1, attention_persistent=1, attention_grid_blocks=2)
    try:
        for l in range(w.n_layers):
            for full_prefix in (False, True):
                out, lse = run_attention(case, s, l, B().CTX_FULL_PREFIX if full_prefix else B().CTX_UNION, simt=False)
                check_attention(case, l, out, lse, full_prefix)
    finally:
        s.shape.set_tuning()


def test_loose_host_bounds_give_the_same_result(case):
    """Host bounds may be loose (|R_l| <= |U| <= T_c).  With the same context split the bits are those of the
    exact bounds; when the launch size picks another split count only the summation order changes."""
    w = case.w
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    l = 0
    f = case.fresh[l]
    for forced in (1, 0):
        s.shape.set_tuning(attention_ctx_splits=forced)
        try:
            exact, _ = run_attention(case, s, l, B().CTX_UNION, simt=False)
            out = torch.zeros_like(f.q_new)
            lse = torch.zeros(w.n_q_heads, f.q_new.shape[0], dtype=torch.float32, device=case.device)
            s.attention(l, case.cache_views()[l], f.q_new, f.k_new, f.v_new, out, list(w.ctx_lens), list(w.ctx_lens), lse_out=lse)
            assert_status_ok()
        finally:
            s.shape.set_tuning()
        if forced == 1:
            assert torch.equal(out, exact)
        else:
            check_attention(case, l, out, lse, False)
            assert float((out.float() - exact.float()).abs().max()) <= 2e-2


def test_bad_index_lists_are_reported_not_faulted():
    """Out-of-range ranks are caught on the device: the status word says so, nothing faults."""
    case = Case(small_llama(n_layers=1, ctx=(512,), q=(8,)))
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    torch.cuda.synchronize()
    s.r_rank[:4] = torch.tensor([100000, -5, 100001, 100002], dtype=torch.int32, device=case.device)
    f = case.fresh[0]
    out = torch.zeros_like(f.q_new)
    s.attention(0, case.cache_views()[0], f.q_new, f.k_new, f.v_new, out, case.max_targets(0), case.max_ctx())
    st, detail = B().relaxkv_read_device_status()
    assert st == B().ERR_BAD_INDEX, (st, detail)
    st, _ = B().relaxkv_read_device_status()
    assert st == 0                                                  # reading clears the word
    k2, v2 = case.k_cache[0].clone(), case.v_cache[0].clone()
    s.scatter(0, B().CacheView(k2, v2, [0]), f.k_new, f.v_new, case.max_targets(0))
    st, _ = B().relaxkv_read_device_status()
    assert st == B().ERR_BAD_INDEX
    # fewer rows in q_new / out than the layer has targets (loose host bounds cannot see it): reported on the device,
    # nothing is written past the rows that exist
    s.build_active_sets(case.anchors_tensor())
    n = f.q_new.shape[0]
    short = torch.full((n - 3,) + tuple(f.q_new.shape[1:]), 3.0, dtype=f.q_new.dtype, device=case.device)
    guard = torch.full((64,) + tuple(f.q_new.shape[1:]), 5.0, dtype=f.q_new.dtype, device=case.device)
    s.attention(0, case.cache_views()[0], f.q_new[:n - 3].contiguous(), f.k_new, f.v_new, short, list(case.w.ctx_lens),
                list(case.w.ctx_lens))
    st, _ = B().relaxkv_read_device_status()
    assert st == B().ERR_BAD_INDEX
    assert torch.all(short == 3.0) and torch.all(guard == 5.0)


def test_expired_wait_is_reported_and_the_context_stays_usable():
    """A wait that can never be satisfied gives up after its limit: the kernel returns, the status word
    says RELAXKV_ERR_TIMEOUT, and the next call on the same context works."""
    import time
    t0 = time.time()
    B().relaxkv_debug_wait_timeout()
    st, detail = B().relaxkv_read_device_status()
    assert st == B().ERR_TIMEOUT, (st, detail)
    assert 0.2 < time.time() - t0 < 5.0
    case = Case(inputs.tiny())
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    out, lse = run_attention(case, s, 0, B().CTX_UNION, simt=False)
    check_attention(case, 0, out, lse, False)


# ------------------------------------------------ controlled configurations (explicit lists) ----

def _pack(lists, device):
    cu = np.concatenate([[0], np.cumsum([len(x) for x in lists])]).astype(np.int32)
    flat = np.concatenate(lists).astype(np.int32) if sum(len(x) for x in lists) else np.zeros(0, np.int32)
    return torch.from_numpy(flat).to(device), torch.from_numpy(cu).to(device), cu


def _run_lists(case, s, l, ctx_lists, tgt_lists, fresh=None):
    """GPU list attention for per-request context / target position lists; returns out, lse, fresh tensors."""
    w = case.w
    ctx_pos, ctx_cu, _ = _pack(ctx_lists, case.device)
    tgt_pos, tgt_cu, tcu = _pack(tgt_lists, case.device)
    if fresh is None:
        qs, ks, vs = [], [], []
        for b in range(w.n_req):
            lo, hi = int(case.ctx_cu[b]), int(case.ctx_cu[b + 1])
            q, k, v = inputs.fresh_qkv(w, l, b, case.k_cache[l][lo:hi], case.v_cache[l][lo:hi],
                                       torch.from_numpy(np.asarray(tgt_lists[b], dtype=np.int64)))
            qs.append(q); ks.append(k); vs.append(v)
        fresh = (torch.cat(qs).contiguous(), torch.cat(ks).contiguous(), torch.cat(vs).contiguous())
    q_new, k_new, v_new = fresh
    out = torch.full_like(q_new, 3.0)
    lse = torch.zeros(w.n_q_heads, q_new.shape[0], dtype=torch.float32, device=case.device)
    B().relaxkv_list_attention(s.shape, case.cache_views()[l], q_new, k_new, v_new, ctx_pos, ctx_cu, tgt_pos, tgt_cu,
                               [len(x) for x in tgt_lists], [len(x) for x in ctx_lists], out, s.workspace, lse_out=lse)
    assert_status_ok()
    return out, lse, fresh, tcu


def test_list_attention_reduces_to_the_method(case):
    """Context = U and targets = R_l through the explicit-list call give the method's own output bits."""
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    l = case.w.n_layers - 1
    ref, _ = run_attention(case, s, l, B().CTX_UNION, simt=False)
    f = case.fresh[l]
    out, _, _, _ = _run_lists(case, s, l, [case.sets[b].u_pos for b in range(case.w.n_req)],
                              [case.sets[b].positions(l) for b in range(case.w.n_req)], fresh=(f.q_new, f.k_new, f.v_new))
    assert torch.equal(out, ref)


@pytest.mark.parametrize("persistent", [0, 1], ids=["auto", "persistent"])
@pytest.mark.parametrize("variant", ["global_targets", "layerwise_sparse", "global_sparse"])
def test_controlled_configurations_match_oracle(case, variant, persistent):
    w = case.w
    rng = np.random.default_rng(5)
    s = case.make_session()
    if persistent:                                # the persistent form of the kernel, two blocks walking all items
        s.shape.set_tuning(attention_ctx_splits=1, attention_persistent=1, attention_grid_blocks=2)
    l = 0
    ctx_lists, tgt_lists = [], []
    for b in range(w.n_req):
        T, st = w.ctx_lens[b], case.sets[b]
        n_u = len(st.u_pos)
        if variant == "global_targets":          # targets ranked over the whole context, not a subset of U
            g = orc.mean_scores(np.stack([orc.minmax(case.raw[(ll, b)]) for ll in range(w.n_layers)]))
            tgt = orc.topk(g, min(max(1, int(0.2 * T)), n_u))
            if T > 8:
                tgt = np.unique(np.concatenate([[0], tgt])) if st.u_pos[0] > 0 else tgt      # a target before all of U
            ctx = st.u_pos
        elif variant == "layerwise_sparse":      # U_l = top-|U| of this layer's score; the method's targets
            ctx = orc.topk(case.raw[(l, b)], n_u)
            tgt = st.positions(l)
        else:                                    # one shared context set from the across-layer mean score
            g = orc.mean_scores(np.stack([orc.minmax(case.raw[(ll, b)]) for ll in range(w.n_layers)]))
            ctx = orc.topk(g, n_u)
            tgt = st.positions(l)
        ctx_lists.append(np.asarray(ctx, dtype=np.int32)); tgt_lists.append(np.asarray(tgt, dtype=np.int32))
    out, lse, fresh, tcu = _run_lists(case, s, l, ctx_lists, tgt_lists)
    for b in range(w.n_req):
        lo, hi = int(tcu[b]), int(tcu[b + 1])
        if hi == lo:
            continue
        qn, kn, vn = (inputs.bf16_bits(t[lo:hi]) for t in fresh)
        ref, ref_lse = orc.list_attention(case.req_k(l, b), case.req_v(l, b), qn, kn, vn, ctx_lists[b], tgt_lists[b], case.scale)
        mx, mean = attention_errors(out[lo:hi], ref)
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (variant, b, mx, mean)
        got_lse = lse[:, lo:hi].cpu().numpy().astype(np.float64).T
        empty = np.isneginf(ref_lse)
        assert np.array_equal(np.isneginf(got_lse), empty)
        np.testing.assert_allclose(got_lse[~empty], ref_lse[~empty], atol=2e-3, rtol=1e-4)
    # cache update for the explicit target list, bit-exact
    k2, v2 = case.k_cache[l].clone(), case.v_cache[l].clone()
    tgt_pos, tgt_cu, _ = _pack(tgt_lists, case.device)
    B().relaxkv_scatter_kv_lists(s.shape, B().CacheView(k2, v2, [int(x) for x in case.ctx_cu[:-1]]), fresh[1], fresh[2],
                                 tgt_pos, tgt_cu, [len(x) for x in tgt_lists])
    assert_status_ok()
    k2_b, v2_b = inputs.bf16_bits(k2), inputs.bf16_bits(v2)
    for b in range(w.n_req):
        lo, hi = int(tcu[b]), int(tcu[b + 1])
        rk, rv = case.req_k(l, b).copy(), case.req_v(l, b).copy()
        orc.scatter(rk, rv, inputs.bf16_bits(fresh[1][lo:hi]), inputs.bf16_bits(fresh[2][lo:hi]), tgt_lists[b])
        np.testing.assert_array_equal(k2_b[case.ctx_cu[b]:case.ctx_cu[b + 1]], rk)
        np.testing.assert_array_equal(v2_b[case.ctx_cu[b]:case.ctx_cu[b + 1]], rv)


def test_mean_scores_and_global_topk(case):
    """g = mean over layers of the normalised scores (fixed summation order), then top-m of g."""
    w = case.w
    s = case.make_session(want_norm=True)
    s.score_select(case.q_layers, case.cache_views())
    g = torch.empty(int(case.ctx_cu[-1]), dtype=torch.float32, device=case.device)
    B().relaxkv_mean_scores(s.shape, w.n_layers, s.norm, g)
    norm = s.norm.cpu().numpy()
    ref = norm[0].astype(np.float32).copy()
    for l in range(1, w.n_layers):
        ref = ref + norm[l]
    ref = ref / np.float32(w.n_layers)
    np.testing.assert_array_equal(g.cpu().numpy(), ref)                      # same fp32 operations, same order
    m = [max(1, t // 5) for t in w.ctx_lens]
    anchors = torch.empty(1, sum(m), dtype=torch.int32, device=case.device)
    B().relaxkv_select_topk(s.shape, 1, m, g.view(1, -1), anchors)
    assert_status_ok()
    got = anchors.cpu().numpy()[0]
    off = 0
    for b in range(w.n_req):
        seg = ref[case.ctx_cu[b]:case.ctx_cu[b + 1]].astype(np.float64)
        np.testing.assert_array_equal(got[off:off + m[b]], orc.topk(seg, m[b]))
        off += m[b]


# ------------------------------------------- query prefill attention feeding the scoring ----

def test_query_prefill_lse_replaces_the_statistics_pass():
    """The query's own causal attention over [context, query] (the explicit-list call with every position
    as context and the query positions as targets, cache-only) yields each row's log-normaliser; given to
    relaxkv_score_select it skips the statistics pass and the scores are the attention weights of that
    wider softmax restricted to the context (the 'real forward pass' reading of the score)."""
    w = small_qwen(n_layers=1, ctx=(1100,), q=(40,))
    case = Case(w)
    T, Qn, H, Hkv, D = w.ctx_lens[0], w.q_lens[0], w.n_q_heads, w.n_kv_heads, w.head_dim
    g = torch.Generator(device="cpu").manual_seed(99)
    kq = torch.randn(Qn, Hkv, D, generator=g).to(torch.bfloat16).to(case.device)      # the query tokens' own K/V
    vq = torch.randn(Qn, Hkv, D, generator=g).to(torch.bfloat16).to(case.device)
    k_ext = torch.cat([case.k_cache[0], kq]).contiguous()
    v_ext = torch.cat([case.v_cache[0], vq]).contiguous()
    shape_ext = B().Shape(H, Hkv, D, [T + Qn], [Qn], case.scale)
    ws = torch.empty(B().relaxkv_workspace_bytes(shape_ext, 1) + 256, dtype=torch.uint8, device=case.device)
    ws = ws[(-ws.data_ptr()) % 256:]
    ctx_pos = torch.arange(T + Qn, dtype=torch.int32, device=case.device)
    tgt_pos = torch.arange(T, T + Qn, dtype=torch.int32, device=case.device)
    cu_ctx = torch.tensor([0, T + Qn], dtype=torch.int32, device=case.device)
    cu_tgt = torch.tensor([0, Qn], dtype=torch.int32, device=case.device)
    q = case.q_layers[0]
    out = torch.empty_like(q)
    lse = torch.empty(H, Qn, dtype=torch.float32, device=case.device)
    B().relaxkv_list_attention(shape_ext, B().CacheView(k_ext, v_ext, [0]), q, None, None, ctx_pos, cu_ctx, tgt_pos, cu_tgt,
                               [Qn], [T + Qn], out, ws, lse_out=lse)
    assert_status_ok()
    # oracle: the same causal attention, then scores with its log-normalisers
    kb, vb, qb = inputs.bf16_bits(k_ext), inputs.bf16_bits(v_ext), inputs.bf16_bits(q)
    ref_out, ref_lse = orc.list_attention(kb, vb, qb, None, None, np.arange(T + Qn), np.arange(T, T + Qn), case.scale)
    mx, mean = attention_errors(out, ref_out)
    assert mx <= MAX_ABS and mean <= MEAN_ABS
    np.testing.assert_allclose(lse.cpu().numpy().T, ref_lse, atol=2e-3, rtol=1e-4)
    ref_raw = orc.raw_scores(qb, kb[:T], case.scale, lse=ref_lse.T)
    s = case.make_session()
    s.score_select(case.q_layers, case.cache_views(), row_lse_layers=[lse])
    assert_status_ok()
    got = s.raw.cpu().numpy()[0].astype(np.float64)
    assert np.all(np.abs(got - ref_raw) <= 1e-3 * ref_raw + 1e-6 / T)
    assert got.sum() < 1.0                                   # part of each row's mass sits on the query's own keys
    check_anchor_band(ref_raw, case.k[0], s.anchors.cpu().numpy()[0])


def test_query_prefill_attention_emits_the_scores_of_its_own_pass():
    """relaxkv_query_prefill_attention: one call gives the query's causal attention over [context, query] (output and
    log-normalisers) AND the context scores with those normalisers - the score of the query's real forward pass.  Two
    requests with a gap between their cache rows; against the oracle's causal attention and its supplied-normaliser
    scores, and the anchors picked from the emitted scores against the oracle's top-k band."""
    H, Hkv, D = 16, 4, 128
    ctx, qn = (1100, 700), (40, 9)
    offs = [0, 1300]                                   # rows 1140..1299 belong to nobody
    rows = 1300 + 700 + 9
    scale = D ** -0.5
    g = torch.Generator(device="cpu").manual_seed(21)
    k_all = torch.randn(rows, Hkv, D, generator=g).to(torch.bfloat16).cuda()
    v_all = torch.randn(rows, Hkv, D, generator=g).to(torch.bfloat16).cuda()
    q = torch.randn(sum(qn), H, D, generator=g).to(torch.bfloat16).cuda()
    shape = B().Shape(H, Hkv, D, list(ctx), list(qn), scale)
    ext = B().Shape(H, Hkv, D, [c + n for c, n in zip(ctx, qn)], list(qn), scale)
    ws = torch.empty(B().relaxkv_workspace_bytes(ext, 1) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    out = torch.zeros_like(q)
    lse = torch.zeros(H, sum(qn), dtype=torch.float32, device="cuda")
    raw = torch.zeros(sum(ctx), dtype=torch.float32, device="cuda")
    B().relaxkv_query_prefill_attention(shape, B().CacheView(k_all, v_all, offs), q, out, lse, raw, ws)
    assert_status_ok()
    k_anchor = [B().relaxkv_anchor_count(t, 0.15) for t in ctx]
    anchors = torch.zeros(1, sum(k_anchor), dtype=torch.int32, device="cuda")
    B().relaxkv_select_topk(shape, 1, k_anchor, raw.view(1, -1), anchors)
    assert_status_ok()
    lo_q = lo_t = lo_k = 0
    for b in range(2):
        T, Qn = ctx[b], qn[b]
        kb = inputs.bf16_bits(k_all[offs[b]:offs[b] + T + Qn].contiguous())
        vb = inputs.bf16_bits(v_all[offs[b]:offs[b] + T + Qn].contiguous())
        qb = inputs.bf16_bits(q[lo_q:lo_q + Qn])
        ref_out, ref_lse = orc.list_attention(kb, vb, qb, None, None, np.arange(T + Qn), np.arange(T, T + Qn), scale)
        mx, mean = attention_errors(out[lo_q:lo_q + Qn], ref_out)
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (b, mx, mean)
        np.testing.assert_allclose(lse[:, lo_q:lo_q + Qn].cpu().numpy().T, ref_lse, atol=2e-3, rtol=1e-4)
        ref_raw = orc.raw_scores(qb, kb[:T], scale, lse=ref_lse.T)
        got = raw[lo_t:lo_t + T].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - ref_raw) <= 1e-3 * ref_raw + 1e-6 / T), np.abs(got / ref_raw - 1).max()
        assert got.sum() < 1.0                               # part of each row's mass sits on the query's own keys
        check_anchor_band(ref_raw, k_anchor[b], anchors[0, lo_k:lo_k + k_anchor[b]].cpu().numpy())
        lo_q, lo_t, lo_k = lo_q + Qn, lo_t + T, lo_k + k_anchor[b]
    # the attention alone (no scores asked for) gives the same output bits
    out2 = torch.zeros_like(q)
    B().relaxkv_query_prefill_attention(shape, B().CacheView(k_all, v_all, offs), q, out2, lse, None, ws)
    assert_status_ok()
    assert torch.equal(out, out2)


@pytest.mark.parametrize("head_major", [False, True])
@pytest.mark.parametrize("n_splits", [0, 1, 3])
def test_cache_attention_of_query_rows_and_a_decode_step(head_major, n_splits):
    """The pass after the repair loop: query rows (and a single decode token) attend to the cache's own causal
    prefix, read through the cache's strides without a gather.  Three requests in one call, token-major and
    head-major caches with a gap between the requests' rows, against the oracle's explicit-list attention with
    every position as context.  The gaps hold NaN / Inf bit patterns."""
    H, Hkv, D = 16, 4, 128
    lens, n_tgt = (1500, 300, 2200), (37, 1, 64)                 # the middle request is a decode step: one row
    offs = [0, 1600, 2000]                                        # rows 1500..1599 and 1900..1999 belong to nobody
    rows = 4300
    g = torch.Generator(device="cpu").manual_seed(5)
    k_all = torch.randn(rows, Hkv, D, generator=g).to(torch.bfloat16).cuda()
    v_all = torch.randn(rows, Hkv, D, generator=g).to(torch.bfloat16).cuda()
    # the rows that belong to nobody hold what an uninitialised slot may hold: NaN and infinities (plain data; the
    # last tile of every request reaches into them, and a masked key must not let them through)
    for lo_gap, hi_gap in ((1500, 1600), (1900, 2000), (4200, 4300)):
        k_all[lo_gap:hi_gap] = float("nan")
        v_all[lo_gap:hi_gap:2] = float("nan")
        v_all[lo_gap + 1:hi_gap:2] = float("inf")
    if head_major:
        k_all = k_all.permute(1, 0, 2).contiguous().permute(1, 0, 2)
        v_all = v_all.permute(1, 0, 2).contiguous().permute(1, 0, 2)
    q = torch.randn(sum(n_tgt), H, D, generator=g).to(torch.bfloat16).cuda()
    # targets: the last tokens of each request (the query suffix), ascending
    tgt = [np.arange(t - n, t, dtype=np.int32) for t, n in zip(lens, n_tgt)]
    tgt_pos = torch.from_numpy(np.concatenate(tgt)).cuda()
    tgt_cu = torch.tensor(np.concatenate([[0], np.cumsum(n_tgt)]).astype(np.int32)).cuda()
    shape = B().Shape(H, Hkv, D, list(lens), None, D ** -0.5, attention_ctx_splits=n_splits)
    ws = torch.empty(B().relaxkv_workspace_bytes(shape, 1) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    out = torch.zeros_like(q)
    lse = torch.zeros(H, q.shape[0], dtype=torch.float32, device="cuda")
    B().relaxkv_cache_attention(shape, B().CacheView(k_all, v_all, offs), q, tgt_pos, tgt_cu, list(n_tgt), out, ws, lse_out=lse)
    assert_status_ok()
    lo = 0
    for b in range(3):
        kb = inputs.bf16_bits(k_all[offs[b]:offs[b] + lens[b]].contiguous())
        vb = inputs.bf16_bits(v_all[offs[b]:offs[b] + lens[b]].contiguous())
        qb = inputs.bf16_bits(q[lo:lo + n_tgt[b]])
        ref, ref_lse = orc.list_attention(kb, vb, qb, None, None, np.arange(lens[b]), tgt[b], D ** -0.5)
        mx, mean = attention_errors(out[lo:lo + n_tgt[b]], ref)
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (b, mx, mean)
        np.testing.assert_allclose(lse[:, lo:lo + n_tgt[b]].cpu().numpy().T, ref_lse, atol=2e-3, rtol=1e-4)
        lo += n_tgt[b]
    # a position past the request's end is reported, not read
    bad = tgt_pos.clone()
    bad[0] = lens[0]
    B().relaxkv_cache_attention(shape, B().CacheView(k_all, v_all, offs), q, bad, tgt_cu, list(n_tgt), out, ws)
    st, _ = B().relaxkv_read_device_status()
    assert st == B().ERR_BAD_INDEX


@pytest.mark.parametrize("H,Hkv,D", [(8, 8, 64), (12, 4, 128), (40, 8, 128), (32, 2, 64)], ids=["g1_d64", "g3_d128", "g5_d128", "g16_d64"])
@pytest.mark.parametrize("n_splits,head_major", [(0, False), (1, True), (5, False)])
def test_decode_attention_one_token_per_request(H, Hkv, D, n_splits, head_major):
    """A decode step: at most one token per request attends to its cache prefix through the streaming kernel (TMA ring,
    warp-level MMA fragments, split merge).  Five requests in one call - contexts of 1, 33, 129, 1000 and 2049 tokens,
    the token's position anywhere in the request, one request without a token - with NaN / Inf in the rows between the
    requests, against the oracle's explicit-list attention; then a position past the request's end and a second token
    where the host promised one are reported, not read."""
    lens = (1, 33, 129, 1000, 2049)
    has = (1, 1, 0, 1, 1)
    pos = (0, 32, 0, 700, 2048)
    offs, rows = [], 0
    for t in lens:
        offs.append(rows); rows += t + 40                          # 40 rows that belong to nobody behind every request
    g = torch.Generator(device="cpu").manual_seed(9)
    k_all = torch.randn(rows, Hkv, D, generator=g).to(torch.bfloat16).cuda()
    v_all = torch.randn(rows, Hkv, D, generator=g).to(torch.bfloat16).cuda()
    for o, t in zip(offs, lens):
        k_all[o + t:o + t + 40] = float("nan")
        v_all[o + t:o + t + 40:2] = float("nan")
        v_all[o + t + 1:o + t + 40:2] = float("-inf")
    if head_major:
        k_all = k_all.permute(1, 0, 2).contiguous().permute(1, 0, 2)
        v_all = v_all.permute(1, 0, 2).contiguous().permute(1, 0, 2)
    n = sum(has)
    q = torch.randn(n + 1, H, D, generator=g).to(torch.bfloat16).cuda()        # one spare row that must stay untouched
    tgt_pos = torch.tensor([p for p, h in zip(pos, has) if h], dtype=torch.int32).cuda()
    tgt_cu = torch.tensor(np.concatenate([[0], np.cumsum(has)]).astype(np.int32)).cuda()
    shape = B().Shape(H, Hkv, D, list(lens), None, D ** -0.5, attention_ctx_splits=n_splits)
    ws = torch.empty(B().relaxkv_workspace_bytes(shape, 1) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    out = torch.full_like(q, 3.0)
    lse = torch.zeros(H, n + 1, dtype=torch.float32, device="cuda")
    view = B().CacheView(k_all, v_all, offs)
    B().relaxkv_cache_attention(shape, view, q, tgt_pos, tgt_cu, [1] * len(lens), out, ws, lse_out=lse)   # loose bound for request 2
    assert_status_ok()
    row = 0
    for b in range(len(lens)):
        if not has[b]:
            continue
        kb = inputs.bf16_bits(k_all[offs[b]:offs[b] + lens[b]].contiguous())
        vb = inputs.bf16_bits(v_all[offs[b]:offs[b] + lens[b]].contiguous())
        ref, ref_lse = orc.list_attention(kb, vb, inputs.bf16_bits(q[row:row + 1]), None, None, np.arange(lens[b]),
                                          np.array([pos[b]], dtype=np.int32), D ** -0.5)
        mx, mean = attention_errors(out[row:row + 1], ref)
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (b, mx, mean)
        np.testing.assert_allclose(lse[:, row:row + 1].cpu().numpy().T, ref_lse, atol=2e-3, rtol=1e-4)
        row += 1
    assert torch.all(out[n] == 3.0)
    bad = tgt_pos.clone()
    bad[1] = lens[1]                                               # one past the end of request 1
    B().relaxkv_cache_attention(shape, view, q, bad, tgt_cu, [1] * len(lens), out, ws)
    st, _ = B().relaxkv_read_device_status()
    assert st == B().ERR_BAD_INDEX
    two = torch.tensor([0, 1, 3, 3, 4, 5], dtype=torch.int32).cuda()            # request 1 brings two tokens
    guard = torch.full((6, H, D), 3.0, dtype=torch.bfloat16, device="cuda")
    B().relaxkv_cache_attention(shape, view, torch.cat([q, q])[:6].contiguous(), torch.tensor([0, 5, 6, 1, 2], dtype=torch.int32).cuda(),
                                two, [1] * len(lens), guard, ws)
    st, _ = B().relaxkv_read_device_status()
    assert st == B().ERR_BAD_INDEX


def _one_rank_group():
    """A process group of this one process on the GPU (NCCL): the all-reduce of the sharded path runs for real,
    over a single rank."""
    import socket
    import torch.distributed as dist
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device("cuda", torch.cuda.current_device()))
    return dist


def test_head_sharded_path_on_one_gpu():
    """The KV-head-sharded layout, its two ranks run one after the other on this GPU (their kernels never wait on
    one another).  Selection: each shard's partial scores go through sharded.combine_partial_scores - the all-reduce
    (over this process alone, so the other shard's partial is added beforehand, which is what the reduction would
    deliver) and the library's scaling kernel, on a stream of its own - and must average to the unsharded scores;
    the anchors from the combined scores are those of the unsharded call.  Repair: gather, attention and the cache
    update on each shard's own heads (cache views k[:, lo:hi], H/N query heads) must equal the oracle's result for
    those heads, and the two shards' cache updates together the unsharded update, bit for bit."""
    from paper_2609_33503_b200 import sharded
    from paper_2609_33503_b200.pipeline import RepairSession
    case = Case(small_llama(n_layers=2, ctx=(1536,), q=(24,)))
    w = case.w
    full = case.make_session()
    full.score_select(case.q_layers, case.cache_views())
    world = 2
    side = torch.cuda.Stream()
    sessions, parts = [], []
    for rank in range(world):
        kv_lo, kv_hi, q_lo, q_hi = sharded.head_shard(w.n_q_heads, w.n_kv_heads, world, rank)
        s = RepairSession(q_hi - q_lo, kv_hi - kv_lo, w.head_dim, w.ctx_lens, w.q_lens, w.n_layers, case.k,
                          device=case.device, softmax_scale=case.scale)
        qs = [q[:, q_lo:q_hi].contiguous() for q in case.q_layers]
        views = [B().CacheView(k[:, kv_lo:kv_hi], v[:, kv_lo:kv_hi], [0]) for k, v in zip(case.k_cache, case.v_cache)]
        B().relaxkv_score_select(s.shape, qs, views, s.k, s.raw, None, s.workspace)       # the shard's partial scores
        sessions.append(s)
        parts.append(s.raw.clone())
    torch.cuda.synchronize()
    dist = _one_rank_group()
    try:
        for rank in range(world):
            s = sessions[rank]
            s.raw.copy_(parts[0] + parts[1])          # what the all-reduce over two ranks delivers to this rank
            torch.cuda.synchronize()
            sharded.combine_partial_scores(s, world, stream=side)
            B().relaxkv_select_topk(s.shape, s.n_layers, s.k, s.raw, s.anchors, stream=side)
        side.synchronize()
    finally:
        dist.destroy_process_group()
    assert_status_ok()
    for s in sessions:
        torch.testing.assert_close(s.raw, full.raw, rtol=2e-5, atol=1e-9)
        assert torch.equal(s.anchors, sessions[0].anchors)            # every rank selects the same anchors
        for l in range(w.n_layers):
            check_anchor_band(case.raw[(l, 0)], case.k[0], s.anchors[l].cpu().numpy())
    # ---- the repair half on each shard's heads, on the oracle's sets ----
    k_upd = [k.clone() for k in case.k_cache]
    v_upd = [v.clone() for v in case.v_cache]
    for rank in range(world):
        kv_lo, kv_hi, q_lo, q_hi = sharded.head_shard(w.n_q_heads, w.n_kv_heads, world, rank)
        s = sessions[rank]
        s.build_active_sets(case.anchors_tensor())
        n_u, n_r = s.counts()
        for l in range(w.n_layers):
            f = case.fresh[l]
            qn, kn, vn = f.q_new[:, q_lo:q_hi].contiguous(), f.k_new[:, kv_lo:kv_hi].contiguous(), f.v_new[:, kv_lo:kv_hi].contiguous()
            view = B().CacheView(case.k_cache[l][:, kv_lo:kv_hi], case.v_cache[l][:, kv_lo:kv_hi], [0])
            rows = sum(n_u) + 128
            kc = torch.empty(rows, kv_hi - kv_lo, w.head_dim, dtype=torch.bfloat16, device=case.device)
            vc = torch.empty_like(kc)
            s.gather(l, view, kn, vn, n_u, kc, vc)
            kt, vt = orc.mix_context(case.req_k(l, 0)[:, kv_lo:kv_hi].copy(), case.req_v(l, 0)[:, kv_lo:kv_hi].copy(),
                                     inputs.bf16_bits(kn), inputs.bf16_bits(vn), case.sets[0].u_pos, case.sets[0].ranks(l))
            np.testing.assert_array_equal(inputs.bf16_bits(kc[:n_u[0]]), kt)
            np.testing.assert_array_equal(inputs.bf16_bits(vc[:n_u[0]]), vt)
            out = torch.zeros_like(qn)
            s.attention(l, view, qn, kn, vn, out, n_r[l], n_u)
            assert_status_ok()
            ref, _ = orc.repair_attention(case.req_k(l, 0)[:, kv_lo:kv_hi].copy(), case.req_v(l, 0)[:, kv_lo:kv_hi].copy(),
                                          inputs.bf16_bits(qn), inputs.bf16_bits(kn), inputs.bf16_bits(vn),
                                          case.sets[0].u_pos, case.sets[0].ranks(l), case.scale)
            mx, mean = attention_errors(out, ref)
            assert mx <= MAX_ABS and mean <= MEAN_ABS, (rank, l, mx, mean)
            s.scatter(l, B().CacheView(k_upd[l][:, kv_lo:kv_hi], v_upd[l][:, kv_lo:kv_hi], [0]), kn, vn, n_r[l])
    assert_status_ok()
    whole = case.make_session()
    whole.build_active_sets(case.anchors_tensor())
    _, n_r = whole.counts()
    for l in range(w.n_layers):
        k2, v2 = case.k_cache[l].clone(), case.v_cache[l].clone()
        whole.scatter(l, B().CacheView(k2, v2, [0]), case.fresh[l].k_new, case.fresh[l].v_new, n_r[l])
        assert torch.equal(k2, k_upd[l]) and torch.equal(v2, v_upd[l])


def test_one_chunk_reading_fresh_states_equal_to_the_cache():
    """With a single chunk nothing precedes the chunk, so recomputing a token gives back its cached K/V.  Then
    (i) the cache update leaves the cache bit-identical, (ii) attention over the mixed fresh/cached context equals
    attention over the cache alone bit for bit, and (iii) at an anchor ratio of 100 % the output is dense causal
    attention over the cache, i.e. a plain prefix prefill (checked against causal attention in float64)."""
    for ratio in (0.3, 1.0):
        w = small_qwen(n_layers=2, ctx=(900,), q=(16,)).replace(ratio=ratio)
        case = Case(w)
        s = case.make_session()
        s.build_active_sets(case.anchors_tensor())
        n_u, n_r = s.counts()
        for l in range(w.n_layers):
            pos = torch.from_numpy(case.sets[0].positions(l).astype(np.int64)).to(case.device)
            f = case.fresh[l]
            k_same, v_same = case.k_cache[l][pos].contiguous(), case.v_cache[l][pos].contiguous()
            view = case.cache_views()[l]
            mixed = torch.zeros_like(f.q_new)
            s.attention(l, view, f.q_new, k_same, v_same, mixed, n_r[l], n_u)
            alone = torch.zeros_like(f.q_new)
            s.attention(l, view, f.q_new, None, None, alone, n_r[l], n_u)
            assert_status_ok()
            assert torch.equal(mixed, alone)
            k2, v2 = case.k_cache[l].clone(), case.v_cache[l].clone()
            s.scatter(l, B().CacheView(k2, v2, [0]), k_same, v_same, n_r[l])
            assert torch.equal(k2, case.k_cache[l]) and torch.equal(v2, case.v_cache[l])
            if ratio == 1.0:
                assert n_r[l] == [900] and n_u == [900]
                G = w.group
                q64 = f.q_new.double().cpu().permute(1, 0, 2).unsqueeze(0)
                k64 = case.k_cache[l].double().cpu().repeat_interleave(G, dim=1).permute(1, 0, 2).unsqueeze(0)
                v64 = case.v_cache[l].double().cpu().repeat_interleave(G, dim=1).permute(1, 0, 2).unsqueeze(0)
                ref = torch.nn.functional.scaled_dot_product_attention(q64, k64, v64, is_causal=True, scale=case.scale)[0].permute(1, 0, 2)
                d = (mixed.double().cpu() - ref).abs()
                assert d.max().item() <= MAX_ABS and d.mean().item() <= MEAN_ABS


def test_list_call_with_more_context_than_its_host_bound_is_reported():
    """Explicit lists whose true context count exceeds the host bound: the rows past the bound have no entry in the
    fresh-row map, so the gather must not use one (it zero-fills them) and the status word reports the overflow."""
    case = Case(small_llama(n_layers=1, ctx=(512,), q=(8,)))
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    sets = case.sets[0]
    ctx_list, tgt_list = sets.u_pos.astype(np.int32), sets.positions(0).astype(np.int32)
    f = case.fresh[0]
    ctx_pos, ctx_cu, _ = _pack([ctx_list], case.device)
    tgt_pos, tgt_cu, _ = _pack([tgt_list], case.device)
    s.workspace.view(torch.int32).fill_(0x7fffff00)            # stale words a trusting kernel would index with
    out = torch.zeros_like(f.q_new)
    B().relaxkv_list_attention(s.shape, case.cache_views()[0], f.q_new, f.k_new, f.v_new, ctx_pos, ctx_cu, tgt_pos, tgt_cu,
                               [len(tgt_list)], [len(ctx_list) - 40], out, s.workspace)
    st, detail = B().relaxkv_read_device_status()
    assert st == B().ERR_BAD_INDEX, (st, detail)
    out2 = torch.zeros_like(f.q_new)                           # the context stays usable: the same call with a true bound
    B().relaxkv_list_attention(s.shape, case.cache_views()[0], f.q_new, f.k_new, f.v_new, ctx_pos, ctx_cu, tgt_pos, tgt_cu,
                               [len(tgt_list)], [len(ctx_list)], out2, s.workspace)
    assert_status_ok()
    ref, _ = case.oracle_attention(0, 0)
    mx, mean = attention_errors(out2, ref)
    assert mx <= MAX_ABS and mean <= MEAN_ABS


# ------------------------------------------------ other head geometries and cache layouts ----

@pytest.mark.parametrize("H,Hkv,D,head_major", [(8, 8, 128, False), (16, 8, 64, True), (16, 2, 128, False),
                                                (32, 2, 64, False), (12, 4, 128, True)])
def test_other_geometries_and_head_major_cache(H, Hkv, D, head_major):
    """Group sizes 1, 2, 8, 16 and 3 (the last does not divide 128), both head dims, and a cache stored
    [H_kv, tokens, D] (read through its strides by the TMA-based scoring kernel and by the gather)."""
    base = inputs.Workload("geom", 2, H, Hkv, D, 64, (700, 333), (21, 9), 0.2, base_seed=7,
                           planted_chunks=((1, 6), (2,)), variant="calibrated")
    case = Case(base, head_major_cache=head_major)
    w = case.w
    s = case.make_session(want_norm=True)
    s.score_select(case.q_layers, case.cache_views())
    assert_status_ok()
    raw = s.raw.cpu().numpy().astype(np.float64)
    anchors = s.anchors.cpu().numpy()
    for l in range(w.n_layers):
        for b in range(w.n_req):
            ref = case.raw[(l, b)]
            got = raw[l, case.ctx_cu[b]:case.ctx_cu[b + 1]]
            assert np.all(np.abs(got - ref) <= 1e-3 * ref + 1e-6 / w.ctx_lens[b]), np.abs(got / ref - 1).max()
            check_anchor_band(ref, case.k[b], anchors[l, case.k_cu[b]:case.k_cu[b + 1]])
    s.build_active_sets(case.anchors_tensor())
    for l in range(w.n_layers):
        for full_prefix in (False, True):
            out, lse = run_attention(case, s, l, B().CTX_FULL_PREFIX if full_prefix else B().CTX_UNION, simt=False)
            check_attention(case, l, out, lse, full_prefix)
