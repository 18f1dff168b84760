"""Pins for the oracle's block arithmetic (CPU only).

Every check compares the oracle with something other than itself: a brute-force
loop, a closed form, an invariant, a special weight setting with a known answer,
or torch's float64 library routines.
"""
import math

import numpy as np
import pytest

from oracle import block as ob
from xema_inputs import bits_to_f64, make_activations, make_block_weights, template


def _f64_weights(t, seed=0):
    return {k: bits_to_f64(v) for k, v in make_block_weights(t, seed).items()}


@pytest.fixture(scope="module")
def tiny():
    t = template("tiny")
    W = _f64_weights(t)
    x, temb = make_activations(t)
    return t, W, bits_to_f64(x), bits_to_f64(temb)


@pytest.fixture(scope="module")
def tiny_out(tiny):
    t, W, x, temb = tiny
    return ob.block_forward(t, W, x, temb, keep=True)


def test_attention_vs_brute_force():
    rng = np.random.default_rng(3)
    q, k, v = rng.standard_normal((5, 8)), rng.standard_normal((11, 8)), rng.standard_normal((11, 8))
    o, lse = ob.attention_head(q, k, v, 0.3)
    for i in range(5):
        w = [math.exp(0.3 * sum(q[i, d] * k[j, d] for d in range(8))) for j in range(11)]
        z = sum(w)
        for d in range(8):
            assert abs(o[i, d] - sum(w[j] * v[j, d] for j in range(11)) / z) < 1e-12
        assert abs(lse[i] - math.log(z)) < 1e-12


def test_attention_block_vs_materialised_scores(tiny, tiny_out):
    """Whole-block o against a materialised S x S probability matrix per head."""
    t, W, x, temb = tiny
    S, H, dh = t.seq, t.heads, t.head_dim
    q = tiny_out["q"][0].reshape(S, H, dh)
    k = tiny_out["k"][0].reshape(S, H, dh)
    v = tiny_out["v"][0].reshape(S, H, dh)
    for hd in range(H):
        P = np.exp(q[:, hd] @ k[:, hd].T / math.sqrt(dh))
        rowsum = P.sum(1)
        P /= rowsum[:, None]
        assert np.abs(P.sum(1) - 1).max() < 1e-12
        assert np.abs(P @ v[:, hd] - tiny_out["o"][0].reshape(S, H, dh)[:, hd]).max() < 1e-12
        assert np.abs(np.exp(tiny_out["lse"][0, hd]) - rowsum).max() < 1e-9 * rowsum.max()


def test_linear_vs_triple_loop():
    rng = np.random.default_rng(5)
    x, w, b = rng.standard_normal((3, 4)), rng.standard_normal((5, 4)), rng.standard_normal(5)
    y = ob.linear(x, w, b)
    for i in range(3):
        for o in range(5):
            assert abs(y[i, o] - (sum(x[i, k] * w[o, k] for k in range(4)) + b[o])) < 1e-13


def test_layer_norm_and_rms_norm_invariants():
    rng = np.random.default_rng(6)
    v = rng.standard_normal((7, 64)) * 3 + 2
    y = ob.layer_norm(v, 1e-6)
    assert np.abs(y.mean(1)).max() < 1e-13
    var = v.var(1)                                   # biased
    assert np.abs((y * y).mean(1) - var / (var + 1e-6)).max() < 1e-12
    # unbiased variance would differ at the 1/64 level; make sure it is the biased one
    assert np.abs(y[0] - (v[0] - v[0].mean()) / math.sqrt(((v[0] - v[0].mean()) ** 2).sum() / 64 + 1e-6)).max() < 1e-13
    r = ob.rms_norm(v, np.ones(64), 0.0)
    assert np.abs((r * r).mean(1) - 1).max() < 1e-13
    g = rng.standard_normal(64)
    assert np.abs(ob.rms_norm(v, g, 1e-6) - v / np.sqrt((v * v).mean(1, keepdims=True) + 1e-6) * g).max() < 1e-13


def test_gelu_tanh_values():
    assert ob.gelu_tanh(np.array(0.0)) == 0.0
    # tanh form at 1: 0.841192; the erf form would give 0.841345
    assert abs(float(ob.gelu_tanh(np.array(1.0))) - 0.8411919906) < 1e-9
    assert abs(float(ob.gelu_tanh(np.array(30.0))) - 30.0) < 1e-12
    assert abs(float(ob.gelu_tanh(np.array(-30.0)))) < 1e-12
    z = np.linspace(-4, 4, 33)
    assert np.abs(ob.gelu_tanh(z) - z - ob.gelu_tanh(-z)).max() < 1e-13      # g(z) - g(-z) = z


def test_silu_values():
    assert ob.silu(np.array(0.0)) == 0.0
    assert abs(float(ob.silu(np.array(1.0))) - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15
    assert abs(float(ob.silu(np.array(-2.0))) + 2.0 / (1.0 + math.exp(2.0))) < 1e-15


def test_token_positions_and_angles():
    t = template("tiny")                              # 32 text + 4 x 8 x 8
    pos = ob.token_positions(t)
    assert (pos[:32] == 0).all()
    assert tuple(pos[32]) == (0, 0, 0) and tuple(pos[32 + 7]) == (0, 0, 7)
    assert tuple(pos[32 + 8]) == (0, 1, 0) and tuple(pos[32 + 64]) == (1, 0, 0)
    assert tuple(pos[-1]) == (3, 7, 7)
    ang = ob.rope_angles(t)                           # sections 16, 24, 24 -> 8 + 12 + 12 pairs
    assert ang.shape == (288, 32)
    row = 32 + 2 * 64 + 3 * 8 + 5                     # (t, h, w) = (2, 3, 5)
    assert ang[row, 0] == 2.0 and ang[row, 8] == 3.0 and ang[row, 20] == 5.0
    assert abs(ang[row, 1] - 2.0 * 10000.0 ** (-2.0 / 16)) < 1e-15
    assert abs(ang[row, 9] - 3.0 * 10000.0 ** (-2.0 / 24)) < 1e-15
    assert abs(ang[row, 31] - 5.0 * 10000.0 ** (-22.0 / 24)) < 1e-15


def test_rope_properties():
    rng = np.random.default_rng(8)
    v = rng.standard_normal((4, 2, 8))
    ang = rng.standard_normal((4, 4))
    r = ob.apply_rope(v, ang)
    # pair norms preserved
    assert np.abs(r[..., 0::2] ** 2 + r[..., 1::2] ** 2 - v[..., 0::2] ** 2 - v[..., 1::2] ** 2).max() < 1e-13
    # angle 0 is the identity
    assert np.array_equal(ob.apply_rope(v, np.zeros((4, 4))), v)
    # one pair, one radian: (1, 0) -> (cos 1, sin 1)
    e = np.zeros((1, 1, 2)); e[0, 0, 0] = 1.0
    out = ob.apply_rope(e, np.ones((1, 1)))
    assert abs(out[0, 0, 0] - math.cos(1.0)) < 1e-15 and abs(out[0, 0, 1] - math.sin(1.0)) < 1e-15


def test_rope_relative_position_property():
    """Shifting every video token's (t, h, w) by a constant leaves q.k between video tokens
    unchanged, so with no text tokens the attention output is unchanged."""
    t = template("tiny", s_text=0, grid_t=2, grid_h=3, grid_w=4, hidden=128, heads=2, ffn=256)
    rng = np.random.default_rng(9)
    S, H, dh = t.seq, t.heads, t.head_dim
    q, k, v = (rng.standard_normal((S, H, dh)) for _ in range(3))
    pos = ob.token_positions(t)
    outs = []
    for shift in ((0, 0, 0), (5, 2, 9)):
        ang = ob.rope_angles(t, pos + np.array(shift))
        qr, kr = ob.apply_rope(q, ang), ob.apply_rope(k, ang)
        outs.append(np.stack([ob.attention_head(qr[:, h], kr[:, h], v[:, h], 0.125)[0] for h in range(H)]))
    assert np.abs(outs[0] - outs[1]).max() < 1e-12


def test_zero_gates_give_identity(tiny):
    t, W, x, temb = tiny
    D = t.hidden
    W0 = dict(W)
    W0["w_mod"] = W["w_mod"].copy(); W0["b_mod"] = W["b_mod"].copy()
    for gate in (2, 5):
        W0["w_mod"][gate * D:(gate + 1) * D] = 0
        W0["b_mod"][gate * D:(gate + 1) * D] = 0
    assert np.array_equal(ob.block_forward(t, W0, x, temb)["y"], x)


def test_constant_v_and_zero_k(tiny):
    t, W, x, temb = tiny
    D = t.hidden
    Wc = {k: v.copy() for k, v in W.items()}
    Wc["w_qkv"][2 * D:] = 0
    Wc["b_qkv"][2 * D:] = np.linspace(-1, 1, D)
    out = ob.block_forward(t, Wc, x, temb, keep=True)
    assert np.abs(out["o"][0] - np.linspace(-1, 1, D)).max() < 1e-13
    Wk = {k: v.copy() for k, v in W.items()}
    Wk["w_qkv"][D:2 * D] = 0
    Wk["b_qkv"][D:2 * D] = 0
    out = ob.block_forward(t, Wk, x, temb, keep=True)
    assert np.abs(out["o"][0] - out["v"][0].mean(0)).max() < 1e-12
    assert np.abs(out["lse"] - math.log(t.seq)).max() < 1e-12


def test_chunked_equals_unchunked(tiny, tiny_out):
    t, W, x, temb = tiny
    for C in (1, 2, 3, 5, (1, 1, 2), (2, 1, 3), (3, 2, 1)):
        out = ob.block_forward_chunked(t, W, x, temb, C)
        assert np.abs(out["y"] - tiny_out["y"]).max() < 1e-12
        assert np.abs(out["lse"] - tiny_out["lse"]).max() < 1e-12


def test_row_subset_equals_full(tiny, tiny_out):
    t, W, x, temb = tiny
    rows = np.array([0, 31, 32, 100, 143, 144, 287])
    sub = ob.block_forward(t, W, x, temb, rows=rows, row_block=3)
    assert np.abs(sub["y"] - tiny_out["y"][:, rows]).max() < 1e-12
    assert np.abs(sub["lse"] - tiny_out["lse"][:, :, rows]).max() < 1e-12


def test_batch_elements_are_independent():
    t = template("tiny", batch=2, grid_t=1, hidden=128, heads=2, ffn=256)
    W = _f64_weights(t, 2)
    x, temb = make_activations(t)
    x, temb = bits_to_f64(x), bits_to_f64(temb)
    both = ob.block_forward(t, W, x, temb)["y"]
    t1 = t.with_(batch=1)
    for b in range(2):
        one = ob.block_forward(t1, W, x[b:b + 1], temb[b:b + 1])["y"]
        assert np.abs(one[0] - both[b]).max() < 1e-12


def test_block_vs_torch_float64(tiny, tiny_out):
    """A second statement of the block from torch's own float64 routines."""
    torch = pytest.importorskip("torch")
    F = torch.nn.functional
    t, W, x, temb = tiny
    tw = {k: torch.from_numpy(v) for k, v in W.items()}
    X, Te = torch.from_numpy(x), torch.from_numpy(temb)
    B, S, D = X.shape
    H, dh = t.heads, t.head_dim
    m = F.linear(F.silu(Te), tw["w_mod"], tw["b_mod"]).view(B, 1, 6, D)
    sh1, sc1, g1, sh2, sc2, g2 = (m[:, :, i] for i in range(6))
    h = F.layer_norm(X, (D,), eps=t.ln_eps) * (1 + sc1) + sh1
    q, k, v = F.linear(h, tw["w_qkv"], tw["b_qkv"]).view(B, S, 3, H, dh).unbind(2)
    q = F.rms_norm(q, (dh,), tw["g_q"], eps=t.rms_eps)
    k = F.rms_norm(k, (dh,), tw["g_k"], eps=t.rms_eps)
    # RoPE through complex multiplication, frequencies built here independently
    n = torch.arange(S - t.s_text)
    pos = torch.zeros(S, 3, dtype=torch.float64)
    pos[t.s_text:, 0] = (n // (t.grid_h * t.grid_w)).double()
    pos[t.s_text:, 1] = ((n // t.grid_w) % t.grid_h).double()
    pos[t.s_text:, 2] = (n % t.grid_w).double()
    ang = torch.cat([pos[:, a:a + 1] * t.rope_base ** (-torch.arange(0, d, 2, dtype=torch.float64) / d)
                     for a, d in enumerate((t.rope_dim_t, t.rope_dim_h, t.rope_dim_w))], dim=1)
    rot = torch.polar(torch.ones_like(ang), ang)[None, :, None, :]

    def rope(z):
        zc = torch.view_as_complex(z.reshape(B, S, H, dh // 2, 2).contiguous())
        return torch.view_as_real(zc * rot).reshape(B, S, H, dh)

    o = F.scaled_dot_product_attention(rope(q).transpose(1, 2), rope(k).transpose(1, 2), v.transpose(1, 2))
    o = o.transpose(1, 2).reshape(B, S, D)
    res = X + g1 * F.linear(o, tw["w_o"], tw["b_o"])
    h2 = F.layer_norm(res, (D,), eps=t.ln_eps) * (1 + sc2) + sh2
    y = res + g2 * F.linear(F.gelu(F.linear(h2, tw["w_1"], tw["b_1"]), approximate="tanh"), tw["w_2"], tw["b_2"])
    assert np.abs(y.numpy() - tiny_out["y"]).max() < 1e-10
    assert np.abs(o.numpy() - tiny_out["o"]).max() < 1e-10
    assert np.abs(res.numpy() - tiny_out["res"]).max() < 1e-10


def test_step_is_block_composition():
    t = template("tiny", grid_t=1, hidden=128, heads=2, ffn=256, n_blocks=3)
    Ws = [_f64_weights(t, s) for s in range(3)]
    x, temb = make_activations(t)
    x, temb = bits_to_f64(x), bits_to_f64(temb)
    y = x
    for W in Ws:
        y = ob.block_forward(t, W, y, temb)["y"]
    assert np.array_equal(ob.step_forward(t, Ws, x, temb), y)


def test_branches_are_not_negligible(tiny_out):
    """The residual dominates y; the parity statistics are only meaningful if the two
    branches carry signal of the expected size."""
    y = tiny_out["y"]
    rms = lambda a: float(np.sqrt((a * a).mean()))
    assert 0.9 < rms(y) < 1.4
    assert rms(tiny_out["attn_branch"]) > 0.005
    assert rms(tiny_out["ffn_branch"]) > 0.02


def test_sub_batch_split_equals_unchunked():
    t = template("tiny", batch=3)
    W = {k: bits_to_f64(v) for k, v in make_block_weights(t, 0).items()}
    x, temb = make_activations(t)
    x, temb = bits_to_f64(x), bits_to_f64(temb)
    ref = ob.block_forward(t, W, x, temb)
    for chunks, axes in [((1, 1, 3), (0, 0, 1)), ((2, 3, 2), (1, 1, 1)), ((2, 2, 3), (0, 1, 0))]:
        out = ob.block_forward_chunked(t, W, x, temb, chunks, axes)
        assert np.abs(out["y"] - ref["y"]).max() < 1e-12 and np.abs(out["lse"] - ref["lse"]).max() < 1e-12
