"""The workspace-free variant of the repair-schedule call.

Some callers of this library own no device memory beyond their inputs and outputs (a plug-in inside
an inference server, a runtime with a sealed memory pool) and cannot hand over a workspace.
relaxkv_build_active_sets_static keeps its scratch inside the library instead.  This test calls it
through the C ABI twice in a row and checks every output against relaxkv_build_active_sets: integer
work, so the results must be identical bit for bit.  It is collected last so that a failure here
cannot hide the result of any other test.
"""
import numpy as np
import pytest
import torch

from paper_2609_33503_b200 import inputs

pytestmark = pytest.mark.gpu


def _random_anchors(rng, n_layers, ctx_lens, k):
    rows = []
    for _ in range(n_layers):
        rows.append(np.concatenate([np.sort(rng.choice(t, size=kb, replace=False)) for t, kb in zip(ctx_lens, k)]))
    return torch.from_numpy(np.stack(rows).astype(np.int32)).cuda()


def test_static_scratch_variant_matches_workspace_variant():
    from paper_2609_33503_b200 import binding as B
    from paper_2609_33503_b200.pipeline import RepairSession
    rng = np.random.default_rng(11)
    ctx_lens, q_lens, n_layers = (700, 1300, 257), (4, 4, 4), 5
    k = [B.relaxkv_anchor_count(t, 0.15) for t in ctx_lens]
    for call in range(2):                      # two calls in a row share the library's scratch array
        anchors = _random_anchors(rng, n_layers, ctx_lens, k)
        ref = RepairSession(40, 8, 128, ctx_lens, q_lens, n_layers, k)
        got = RepairSession(40, 8, 128, ctx_lens, q_lens, n_layers, k)
        for t in (got.highest_layer, got.u_pos, got.u_cu, got.u_rank, got.r_rank, got.r_cu):
            t.fill_(-7)
        got.counts_pinned.fill_(-7)
        ref.build_active_sets(anchors)
        B.relaxkv_build_active_sets_static(got.shape, n_layers, k, anchors, got.highest_layer, got.u_pos, got.u_cu,
                                           got.u_rank, got.r_rank, got.r_cu, counts_pinned=got.counts_pinned)
        torch.cuda.synchronize()
        st, detail = B.relaxkv_read_device_status()
        assert st == 0, (st, detail)
        n_u = int(ref.u_cu[-1].item())
        n_r = int(ref.r_cu[-1].item())
        assert torch.equal(got.u_cu, ref.u_cu) and torch.equal(got.r_cu, ref.r_cu)
        assert torch.equal(got.highest_layer, ref.highest_layer) and torch.equal(got.u_rank, ref.u_rank)
        assert torch.equal(got.u_pos[:n_u], ref.u_pos[:n_u])
        assert torch.equal(got.r_rank[:n_r], ref.r_rank[:n_r])
        assert torch.equal(got.counts_pinned, ref.counts_pinned)
        assert n_u > 0 and n_r >= n_u


def test_static_scratch_variant_rejects_oversized_problems():
    from paper_2609_33503_b200 import binding as B
    shape = B.Shape(8, 2, 128, [64] * 64, [1] * 64)
    dummy = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(B.RelaxKVError) as e:      # 64 requests x (1 + 200 layers) counts > 8192
        B.relaxkv_build_active_sets_static(shape, 200, [1] * 64, dummy, dummy, dummy, dummy, dummy, dummy, dummy)
    assert e.value.status == B.ERR_UNSUPPORTED_SHAPE
