"""Float64 definition of one DiT denoising block (test infrastructure only).

The paper describes the denoiser only as repeated attention + feed-forward
blocks whose activations scale with H*W*T; the operator definitions below are
the standard ones and are this repository's reading:

  1. adaLN-Zero modulation: m = silu(temb) W_mod^T + b_mod, split into
     shift1, scale1, gate1, shift2, scale2, gate2 (each of width D).
  2. h = LN(x) (1 + scale1) + shift1; LN has no affine, biased variance.
  3. [q | k | v] = h W_qkv^T + b_qkv, viewed as H heads of width dh.
  4. per-head RMSNorm of q and k with learned gains g_q, g_k.
  5. multi-axis RoPE on q and k: the head features are split into three
     consecutive sections (t, h, w); adjacent pairs inside a section of width d
     rotate by position * base^(-2j/d).  Text tokens sit at position (0,0,0).
  6. full bidirectional softmax attention over all S tokens, scale dh^-1/2.
  7. res = x + gate1 * (o W_o^T + b_o)
  8. h2 = LN(res) (1 + scale2) + shift2
  9. g = gelu_tanh(h2 W_1^T + b_1)
 10. y = res + gate2 * (g W_2^T + b_2)

Nothing is rounded between the steps.  Every step is row-local except the
attention, where a query row needs its own q and every row's k and v; that is
why `rows=` can select a subset of output rows without changing their values.
"""
from __future__ import annotations

import math
import numpy as np

F64 = np.float64


def silu(z):
    return z / (1.0 + np.exp(-z))


def gelu_tanh(z):
    """0.5 z (1 + tanh(sqrt(2/pi) (z + 0.044715 z^3)))"""
    return 0.5 * z * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (z + 0.044715 * z ** 3)))


def linear(x, w, b):
    """y = x W^T + b with W stored [out, in]."""
    return x @ w.T + b


def modulation(t, W, temb):
    """Step 1: six [B, D] modulation vectors from the timestep embedding."""
    m = linear(silu(np.asarray(temb, F64)), W["w_mod"], W["b_mod"])
    D = t.hidden
    return tuple(m[:, i * D:(i + 1) * D] for i in range(6))


def layer_norm(v, eps):
    mu = v.mean(axis=-1, keepdims=True)
    c = v - mu
    var = (c * c).mean(axis=-1, keepdims=True)
    return c / np.sqrt(var + eps)


def rms_norm(v, g, eps):
    """Per-head RMSNorm over the last axis (width dh) with gain g."""
    ms = (v * v).mean(axis=-1, keepdims=True)
    return v / np.sqrt(ms + eps) * g


def token_positions(t):
    """[S, 3] integer (t, h, w) position of every token; text tokens at the origin."""
    S, St = t.seq, t.s_text
    pos = np.zeros((S, 3), dtype=np.int64)
    n = np.arange(S - St)
    pos[St:, 0] = n // (t.grid_h * t.grid_w)
    pos[St:, 1] = (n // t.grid_w) % t.grid_h
    pos[St:, 2] = n % t.grid_w
    return pos


def rope_angles(t, pos=None):
    """[S, dh/2] rotation angle of every adjacent feature pair of a head."""
    pos = token_positions(t) if pos is None else pos
    cols = []
    for axis, d in enumerate((t.rope_dim_t, t.rope_dim_h, t.rope_dim_w)):
        j = np.arange(d // 2, dtype=F64)
        freq = float(t.rope_base) ** (-2.0 * j / d) if d > 0 else j
        cols.append(pos[:, axis:axis + 1].astype(F64) * freq[None, :])
    return np.concatenate(cols, axis=1)


def apply_rope(v, ang):
    """Rotate adjacent pairs (2j, 2j+1) of the last axis of v [R, H, dh] by ang [R, dh/2]."""
    a, b = v[..., 0::2], v[..., 1::2]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    out = np.empty_like(v)
    out[..., 0::2] = a * c - b * s
    out[..., 1::2] = a * s + b * c
    return out


def attention_head(q, k, v, scale):
    """softmax(q k^T * scale) v for one head.  q [R, dh]; k, v [S, dh].
    Returns (o [R, dh], lse [R]) with lse the natural log of the row sum of exp."""
    s = (q @ k.T) * scale
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    z = e.sum(axis=1, keepdims=True)
    return (e / z) @ v, (m + np.log(z))[:, 0]


def qkv_heads(t, W, h, ang, which):
    """Steps 3-5 for the rows in h: projection slice `which` in {"q","k","v"},
    head view, and (q, k only) RMSNorm + RoPE."""
    D, H, dh = t.hidden, t.heads, t.head_dim
    i = "qkv".index(which)
    z = linear(h, W["w_qkv"][i * D:(i + 1) * D], W["b_qkv"][i * D:(i + 1) * D])
    z = z.reshape(-1, H, dh)
    if which == "v":
        return z
    z = rms_norm(z, W["g_q"] if which == "q" else W["g_k"], t.rms_eps)
    return apply_rope(z, ang)


def block_forward(t, W, x, temb, rows=None, row_block=2048, keep=False):
    """One block, float64.  x [B,S,D], temb [B,Dt]; W maps names to float64 arrays.

    rows: optional sorted array of token rows; the result then holds only those
    rows (k and v are still computed for every row).  row_block only bounds the
    size of the score matrix held at once; every row's arithmetic is unchanged.
    Returns {"y": [B,R,D], "lse": [B,H,R]} plus intermediates when keep=True.
    """
    x = np.asarray(x, F64)
    B, S, D = x.shape
    H, dh = t.heads, t.head_dim
    rows = np.arange(S) if rows is None else np.asarray(rows)
    R = len(rows)
    shift1, scale1, gate1, shift2, scale2, gate2 = modulation(t, W, temb)
    ang = rope_angles(t)
    scale = 1.0 / math.sqrt(dh)
    out = {"y": np.empty((B, R, D)), "lse": np.empty((B, H, R))}
    if keep:
        for name in ("h1", "q", "o", "res", "h2"):
            out[name] = np.empty((B, R, D))
        out["attn_branch"] = np.empty((B, R, D))
        out["ffn_branch"] = np.empty((B, R, D))
        out["k"] = np.empty((B, S, D))
        out["v"] = np.empty((B, S, D))
    for b in range(B):
        h_all = layer_norm(x[b], t.ln_eps) * (1.0 + scale1[b]) + shift1[b]
        k = qkv_heads(t, W, h_all, ang, "k")                    # [S,H,dh]
        v = qkv_heads(t, W, h_all, ang, "v")
        h_r = h_all[rows]
        q = qkv_heads(t, W, h_r, ang[rows], "q")                # [R,H,dh]
        o = np.empty((R, H, dh))
        for hd in range(H):
            kh, vh = np.ascontiguousarray(k[:, hd]), np.ascontiguousarray(v[:, hd])
            for r0 in range(0, R, row_block):
                r1 = min(r0 + row_block, R)
                o[r0:r1, hd], out["lse"][b, hd, r0:r1] = attention_head(q[r0:r1, hd], kh, vh, scale)
        o = o.reshape(R, D)
        attn_branch = gate1[b] * linear(o, W["w_o"], W["b_o"])
        res = x[b, rows] + attn_branch
        h2 = layer_norm(res, t.ln_eps) * (1.0 + scale2[b]) + shift2[b]
        g = gelu_tanh(linear(h2, W["w_1"], W["b_1"]))
        ffn_branch = gate2[b] * linear(g, W["w_2"], W["b_2"])
        out["y"][b] = res + ffn_branch
        if keep:
            out["h1"][b], out["q"][b], out["o"][b] = h_r, q.reshape(R, D), o
            out["res"][b], out["h2"][b] = res, h2
            out["attn_branch"][b], out["ffn_branch"][b] = attn_branch, ffn_branch
            out["k"][b], out["v"][b] = k.reshape(S, D), v.reshape(S, D)
    return out


def block_forward_chunked(t, W, x, temb, chunks, axes=(0, 0, 0)):
    """The same block evaluated in the chunked three-phase order the library uses
    (all KV chunks; then Q/attention/projection per chunk; then the FFN per chunk),
    chunk c covering rows [floor(c S / C), floor((c+1) S / C)); `chunks` is one count or
    a per-phase triple.  A phase whose axis is 1 is split into sub-batches instead (piece c =
    batch elements [floor(c B / C), floor((c+1) B / C)), all rows).  Used to show that either
    split is lossless; not a second definition."""
    x = np.asarray(x, F64)
    B, S, D = x.shape
    H, dh = t.heads, t.head_dim
    ca, cb, cc = (chunks, chunks, chunks) if isinstance(chunks, int) else chunks
    if any(axes):
        # a sub-batch piece holds whole batch elements: evaluate every element of the piece with
        # that phase unchunked along the rows
        y = np.empty((B, S, D))
        lse = np.empty((B, H, S))
        cuts = [[c * B // C for c in range(C + 1)] if ax else None for C, ax in zip((ca, cb, cc), axes)]
        for b in range(B):
            counts = tuple(1 if ax else C for C, ax in zip((ca, cb, cc), axes))
            assert all(cut is None or any(cut[i] <= b < cut[i + 1] for i in range(len(cut) - 1)) for cut in cuts)
            tb = t.with_(batch=1)
            out = block_forward_chunked(tb, W, x[b:b + 1], np.asarray(temb)[b:b + 1], counts)
            y[b], lse[b] = out["y"][0], out["lse"][0]
        return {"y": y, "lse": lse}
    rows_of = lambda C: [c * S // C for c in range(C + 1)]
    shift1, scale1, gate1, shift2, scale2, gate2 = modulation(t, W, temb)
    ang = rope_angles(t)
    scale = 1.0 / math.sqrt(dh)
    y = np.empty((B, S, D))
    lse = np.empty((B, H, S))
    for b in range(B):
        k = np.empty((S, H, dh))
        v = np.empty((S, H, dh))
        r = rows_of(ca)
        for c in range(ca):
            sl = slice(r[c], r[c + 1])
            h = layer_norm(x[b, sl], t.ln_eps) * (1.0 + scale1[b]) + shift1[b]
            k[sl] = qkv_heads(t, W, h, ang[sl], "k")
            v[sl] = qkv_heads(t, W, h, ang[sl], "v")
        res = np.empty((S, D))
        r = rows_of(cb)
        for c in range(cb):
            sl = slice(r[c], r[c + 1])
            h = layer_norm(x[b, sl], t.ln_eps) * (1.0 + scale1[b]) + shift1[b]
            q = qkv_heads(t, W, h, ang[sl], "q")
            o = np.empty_like(q)
            for hd in range(H):
                o[:, hd], lse[b, hd, sl] = attention_head(q[:, hd], k[:, hd], v[:, hd], scale)
            res[sl] = x[b, sl] + gate1[b] * linear(o.reshape(-1, D), W["w_o"], W["b_o"])
        r = rows_of(cc)
        for c in range(cc):
            sl = slice(r[c], r[c + 1])
            h2 = layer_norm(res[sl], t.ln_eps) * (1.0 + scale2[b]) + shift2[b]
            g = gelu_tanh(linear(h2, W["w_1"], W["b_1"]))
            y[b, sl] = res[sl] + gate2[b] * linear(g, W["w_2"], W["b_2"])
    return {"y": y, "lse": lse}


def step_forward(t, weights_per_block, x, temb):
    """n_blocks stacked blocks: the output of block l is the input of block l+1;
    the same timestep embedding feeds every block."""
    x = np.asarray(x, F64)
    for W in weights_per_block:
        x = block_forward(t, W, x, temb)["y"]
    return x
