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


def test_decoder_block_matches_a_library_built_block():
    """The block chain against the same block assembled from torch's own routines in float64 (rms_norm, linear, silu,
    scaled_dot_product_attention with a causal mask), with and without the per-head Q/K norm; a dropped residual, a
    swapped norm gain or the wrong half of the gate/up matrix would each fail it.  A second check: one row at a time
    (a decode token over the keys before it) equals the rows of the whole-sequence block."""
    import torch.nn.functional as F
    rng = np.random.default_rng(3)
    n, C, H, Hkv, D, I, eps, theta = 11, 48, 4, 2, 16, 40, 1e-5, 1.0e4
    for qk_norm in (False, True):
        W = {"w_in_norm": 1 + 0.1 * rng.standard_normal(C), "wq": rng.standard_normal((H * D, C)) / 7, "wk": rng.standard_normal((Hkv * D, C)) / 7,
             "wv": rng.standard_normal((Hkv * D, C)) / 7, "wo": rng.standard_normal((C, H * D)) / 8, "w_post_norm": 1 + 0.1 * rng.standard_normal(C),
             "w_gate_up": rng.standard_normal((2 * I, C)) / 7, "w_down": rng.standard_normal((C, I)) / 6}
        if qk_norm:
            W["w_q_norm"], W["w_k_norm"] = 1 + 0.1 * rng.standard_normal(D), 1 + 0.1 * rng.standard_normal(D)
        h = rng.standard_normal((n, C))
        pos = np.arange(100, 100 + n)
        G = H // Hkv

        def causal(q, k, v):
            tq = torch.from_numpy(q).permute(1, 0, 2)[None]
            tk = torch.from_numpy(np.repeat(k, G, axis=1)).permute(1, 0, 2)[None]
            tv = torch.from_numpy(np.repeat(v, G, axis=1)).permute(1, 0, 2)[None]
            return F.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2).numpy()

        got = blk.decoder_block(h, W, H, Hkv, D, pos, eps, theta, causal)
        # the same block from library routines
        t = {k_: torch.from_numpy(v_) for k_, v_ in W.items()}
        th = torch.from_numpy(h)
        x = F.rms_norm(th, (C,), t["w_in_norm"], eps=eps)
        q, k, v = F.linear(x, t["wq"]).view(n, H, D), F.linear(x, t["wk"]).view(n, Hkv, D), F.linear(x, t["wv"]).view(n, Hkv, D)
        if qk_norm:
            q, k = F.rms_norm(q, (D,), t["w_q_norm"], eps=eps), F.rms_norm(k, (D,), t["w_k_norm"], eps=eps)
        inv = theta ** (-torch.arange(D // 2, dtype=torch.float64) * 2.0 / D)
        ang = torch.from_numpy(pos).double()[:, None] * inv[None]
        cos, sin = torch.cat([ang.cos(), ang.cos()], -1)[:, None], torch.cat([ang.sin(), ang.sin()], -1)[:, None]
        rot = lambda u: torch.cat([-u[..., D // 2:], u[..., :D // 2]], -1)
        q, k = q * cos + rot(q) * sin, k * cos + rot(k) * sin
        o = torch.from_numpy(causal(q.numpy(), k.numpy(), v.numpy())).reshape(n, H * D)
        a = th + F.linear(o, t["wo"])
        x2 = F.rms_norm(a, (C,), t["w_post_norm"], eps=eps)
        gate, up = F.linear(x2, t["w_gate_up"][:I]), F.linear(x2, t["w_gate_up"][I:])
        ref = a + F.linear(F.silu(gate) * up, t["w_down"])
        np.testing.assert_allclose(got, ref.numpy(), rtol=1e-9, atol=1e-11)

        # row by row (decode): the last row alone, attending to the keys/values of all rows so far
        kv = {}
        blk.decoder_block(h, W, H, Hkv, D, pos, eps, theta, lambda q_, k_, v_: (kv.update(k=k_, v=v_), causal(q_, k_, v_))[1])

        def last_row(q1, k1, v1):
            kk, vv = np.concatenate([kv["k"][:-1], k1]), np.concatenate([kv["v"][:-1], v1])
            s = np.einsum("hd,thd->ht", q1[0], np.repeat(kk, G, axis=1)) / np.sqrt(D)
            p = np.exp(s - s.max(-1, keepdims=True)); p /= p.sum(-1, keepdims=True)
            return np.einsum("ht,thd->hd", p, np.repeat(vv, G, axis=1))[None]

        one = blk.decoder_block(h[-1:], W, H, Hkv, D, pos[-1:], eps, theta, last_row)
        np.testing.assert_allclose(one, got[-1:], rtol=1e-9, atol=1e-11)
        logits = blk.output_head(got[-1:], W["w_in_norm"], W["wo"].T[:5], eps)
        np.testing.assert_allclose(logits, F.linear(F.rms_norm(torch.from_numpy(got[-1:]), (C,), t["w_in_norm"], eps=eps), t["wo"].T[:5]).numpy(), rtol=1e-12)
