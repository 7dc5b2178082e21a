"""GPU parity of the dense block work of the active targets (Algorithm 1, steps 14/16/20) against the fp64
block oracle, operation by operation on identical bf16 inputs, then one whole layer of the repair loop.

Tolerances: every kernel rounds its output to bf16 once (relative 2^-9) after fp32 arithmetic, so
|gpu - ref| <= 2^-8 * |ref| + abs_floor, with abs_floor scaled to the magnitude of the sum being rounded."""
import numpy as np
import pytest
import torch

from oracle import relaxkv_block_oracle as blk
from oracle import relaxkv_oracle as orc
from paper_2609_33503_b200 import inputs

pytestmark = pytest.mark.gpu


def B():
    from paper_2609_33503_b200 import binding
    return binding


def bits(t):
    return inputs.bf16_bits(t)


def rnd(*shape, scale=1.0, seed=0):
    g = torch.Generator(device="cpu").manual_seed(seed)
    return (torch.randn(*shape, generator=g) * scale).to(torch.bfloat16).cuda()


def close(got: torch.Tensor, ref: np.ndarray, abs_floor: float):
    g = got.float().cpu().numpy().astype(np.float64)
    err = np.abs(g - ref)
    assert np.all(err <= 2.0 ** -8 * np.abs(ref) + abs_floor), float((err - 2.0 ** -8 * np.abs(ref)).max())


@pytest.mark.parametrize("M,N,K,res", [(300, 512, 320, False), (129, 264, 72, True), (1000, 1024, 2048, True), (1, 8, 8, False),
                                       (257, 1280, 640, False)])
def test_linear(M, N, K, res):
    x, w = rnd(M, K, seed=1), rnd(N, K, scale=K ** -0.5, seed=2)
    r = rnd(M, N, seed=3) if res else None
    y = torch.full((M, N), 7.0, dtype=torch.bfloat16, device="cuda")
    B().relaxkv_linear(x, w, y, residual=r)
    st, detail = B().relaxkv_read_device_status()
    assert st == 0, (st, detail)
    ref = blk.linear(blk.f64(bits(x)), blk.f64(bits(w)), blk.f64(bits(r)) if res else None)
    close(y, ref, abs_floor=2e-3)
    torch.testing.assert_close(y.float(), (x.float() @ w.float().T + (r.float() if res else 0)), rtol=2e-2, atol=2e-2)


def test_rmsnorm_rope_swiglu():
    x, w = rnd(77, 640, seed=4, scale=3.0), rnd(640, seed=5)
    y = torch.empty_like(x)
    B().relaxkv_rmsnorm(x, w, y, 1e-6)
    close(y, blk.rmsnorm(blk.f64(bits(x)), blk.f64(bits(w)), 1e-6), abs_floor=1e-3)
    for D in (64, 128):
        q = rnd(53, 5, D, seed=6)
        pos = torch.tensor(np.random.default_rng(0).integers(0, 66000, size=53).astype(np.int32)).cuda()
        ref = blk.rope(blk.f64(bits(q)), pos.cpu().numpy(), 1e6)
        B().relaxkv_rope(q, pos, 1e6)
        close(q, ref, abs_floor=2e-3)
    gu = rnd(41, 2 * 264, seed=7, scale=2.0)
    out = torch.empty(41, 264, dtype=torch.bfloat16, device="cuda")
    B().relaxkv_swiglu(gu, out)
    close(out, blk.swiglu(blk.f64(bits(gu))), abs_floor=1e-3)


def test_target_positions_and_row_carry():
    from tests.harness import Case
    w = inputs.scaled_down(inputs.qwen14b_32k("calibrated"), (640, 900), (9, 17), n_layers=3, chunk=128)
    case = Case(w)
    s = case.make_session()
    s.build_active_sets(case.anchors_tensor())
    n_u, n_r = s.counts()
    C = 72
    for l in range(w.n_layers):
        total = sum(n_r[l])
        pos = torch.full((total,), -1, dtype=torch.int32, device="cuda")
        B().relaxkv_target_positions(s.shape, s.u_pos, s.u_cu, s.r_rank, s.r_cu_layer(l), n_r[l], pos)
        ref = np.concatenate([case.sets[b].positions(l) for b in range(w.n_req)])
        np.testing.assert_array_equal(pos.cpu().numpy(), ref)
        if l + 1 < w.n_layers:
            h = rnd(total, C, seed=10 + l)
            nxt = sum(n_r[l + 1])
            out = torch.zeros(nxt, C, dtype=torch.bfloat16, device="cuda")
            B().relaxkv_carry_rows(s.shape, h, out, s.r_rank, s.r_cu_layer(l), s.r_cu_layer(l + 1), n_r[l + 1])
            off = 0
            refs = []
            for b in range(w.n_req):
                hb = blk.f64(bits(h[off:off + n_r[l][b]]))
                refs.append(blk.compact_rows(hb, case.sets[b].ranks(l), case.sets[b].ranks(l + 1)))
                off += n_r[l][b]
            np.testing.assert_array_equal(out.float().cpu().numpy().astype(np.float64), np.concatenate(refs))
    st, detail = B().relaxkv_read_device_status()
    assert st == 0, (st, detail)
