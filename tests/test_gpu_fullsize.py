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


def test_qwen14b_32k_full_context_two_layers():
    run_full(inputs.qwen14b_32k("calibrated", 0.15, n_layers=2), tile_targets=25, n_spread=24)
