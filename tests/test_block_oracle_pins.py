"""Pins of the dense-block oracle against library routines and closed forms."""
import numpy as np
import torch

from oracle import relaxkv_block_oracle as blk


def test_rmsnorm_linear_swiglu_match_library_routines():
    rng = np.random.default_rng(0)
    x, w = rng.standard_normal((7, 48)), rng.standard_normal(48)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (48,), torch.from_numpy(w), eps=1e-6).numpy()
    np.testing.assert_allclose(blk.rmsnorm(x, w, 1e-6), ref, rtol=1e-12)
    W, res = rng.standard_normal((20, 48)), rng.standard_normal((7, 20))
    np.testing.assert_allclose(blk.linear(x, W, res), (torch.nn.functional.linear(torch.from_numpy(x), torch.from_numpy(W)) + torch.from_numpy(res)).numpy(), rtol=1e-12)
    gu = rng.standard_normal((5, 32))
    ref = (torch.nn.functional.silu(torch.from_numpy(gu[:, :16])) * torch.from_numpy(gu[:, 16:])).numpy()
    np.testing.assert_allclose(blk.swiglu(gu), ref, rtol=1e-12)


def test_rope_closed_forms():
    rng = np.random.default_rng(1)
    rows, heads, D, theta = 9, 3, 16, 10000.0
    x = rng.standard_normal((rows, heads, D))
    pos = rng.integers(0, 40000, size=rows)
    y = blk.rope(x, pos, theta)
    # complex formulation: (x1 + i x2) * exp(i * pos * freq)
    z = (x[..., :D // 2] + 1j * x[..., D // 2:]) * np.exp(1j * pos[:, None, None] * theta ** (-np.arange(D // 2) * 2.0 / D))
    np.testing.assert_allclose(y, np.concatenate([z.real, z.imag], axis=-1), rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)      # a rotation
    np.testing.assert_array_equal(blk.rope(x, np.zeros(rows, dtype=np.int64), theta), x)                # position 0: identity
    # relative property: <rope(q, m), rope(k, n)> depends on m - n only
    q, k = rng.standard_normal((1, 1, D)), rng.standard_normal((1, 1, D))
    a = (blk.rope(q, np.array([1234]), theta) * blk.rope(k, np.array([1200]), theta)).sum()
    b = (blk.rope(q, np.array([20034]), theta) * blk.rope(k, np.array([20000]), theta)).sum()
    assert abs(a - b) < 1e-9


def test_compact_rows():
    h = np.arange(12.0).reshape(6, 2)
    out = blk.compact_rows(h, np.array([0, 2, 3, 5, 8, 9]), np.array([2, 5, 9]))
    np.testing.assert_array_equal(out, h[[1, 3, 5]])
