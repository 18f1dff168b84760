"""Per-kernel parity against the oracle's operator definitions, through the C ABI (GPU)."""
import math

import numpy as np
import pytest
import torch

from oracle import block as ob
from paper_2607_11136_b200 import binding as xb
from xema_inputs import bf16_bits, bits_to_f64, template

from gpu_util import DEV, assert_bf16_close, assert_close, from_dev_bf16, rand_bf16, to_dev

pytestmark = pytest.mark.gpu


def _sync_status(status):
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device status 0x%08x" % (int(status.item()) & 0xFFFFFFFF)


def test_mod_gemv():
    rng = np.random.default_rng(0)
    for B, Dt, n_out in ((1, 512, 3072), (4, 512, 6 * 3072), (3, 64, 40)):
        tb, tf = rand_bf16(rng, (B, Dt))
        wb, wf = rand_bf16(rng, (n_out, Dt), 0.02)
        bb, bf = rand_bf16(rng, (n_out,), 0.02)
        out = torch.empty(B, n_out, dtype=torch.float32, device=DEV)
        t_dev, w_dev, b_dev = to_dev(tb), to_dev(wb), to_dev(bb)
        xb.xema_op_mod(t_dev.data_ptr(), w_dev.data_ptr(), b_dev.data_ptr(), out.data_ptr(), B, Dt, n_out)
        torch.cuda.synchronize()
        ref = ob.linear(ob.silu(tf), wf, bf)
        assert_close(out.cpu().numpy(), ref, "mod", rel=1e-4, cos=0.999999)


@pytest.mark.parametrize("D,in_f32", [(512, 0), (512, 1), (3072, 0), (3072, 1), (768, 0), (1280, 1)])
def test_ln_modulate(D, in_f32):
    rng = np.random.default_rng(1)
    B, S, rows, row0 = 2, 70, 37, 11
    if in_f32:
        xf32 = (rng.standard_normal((B, S, D), dtype=np.float32) * 1.5 + 0.3).astype(np.float32)
        x_dev, xf = torch.from_numpy(xf32).to(DEV), xf32.astype(np.float64)
        base = x_dev.data_ptr() + row0 * D * 4
    else:
        xbits, xf = rand_bf16(rng, (B, S, D), 1.5)
        x_dev = to_dev(xbits)
        base = x_dev.data_ptr() + row0 * D * 2
    mod = rng.standard_normal((B, 6 * D), dtype=np.float32) * 0.3
    mod_dev = torch.from_numpy(mod).to(DEV)
    out = torch.empty(B, rows, D, dtype=torch.int16, device=DEV)
    xb.xema_op_ln_modulate(base, in_f32, S, out.data_ptr(), mod_dev.data_ptr(), mod_dev.data_ptr() + D * 4, 6 * D, B,
                           rows, D, 1e-6)
    torch.cuda.synchronize()
    m64 = mod.astype(np.float64)
    ref = ob.layer_norm(xf[:, row0:row0 + rows], 1e-6) * (1 + m64[:, None, D:2 * D]) + m64[:, None, :D]
    assert_bf16_close(from_dev_bf16(out), ref, "ln", atol_rms=1e-4)


@pytest.mark.parametrize("name", ["tiny", "flux"])
def test_rmsnorm_rope(name):
    t = template(name)
    rng = np.random.default_rng(2)
    B, H, dh = 2, 6, t.head_dim
    S = t.seq
    rows, pos0 = 45, t.s_text - 7                     # spans the text / video boundary
    ld = 2 * H * dh + 8 * 3                           # strided rows, like the K half of kv
    xbits, xf = rand_bf16(rng, (B, S, ld), 2.0)
    gb, gf = rand_bf16(rng, (dh,), 1.0)
    x_dev, g_dev = to_dev(xbits), to_dev(gb)
    rope = torch.from_numpy(xb.xema_rope_table(xb.make_config(t))).to(DEV)
    xb.xema_op_rmsnorm_rope(x_dev.data_ptr() + pos0 * ld * 2, ld, S, g_dev.data_ptr(), rope.data_ptr(), pos0, B,
                            rows, H, dh, 1e-6)
    torch.cuda.synchronize()
    got = from_dev_bf16(x_dev)
    ang = ob.rope_angles(t)[pos0:pos0 + rows]
    ref = xf.copy()
    for b in range(B):
        v = xf[b, pos0:pos0 + rows, :H * dh].reshape(rows, H, dh)
        ref[b, pos0:pos0 + rows, :H * dh] = ob.apply_rope(ob.rms_norm(v, gf, 1e-6), ang).reshape(rows, H * dh)
    # untouched: other rows, and the features beyond heads*dh of the touched rows
    mask = np.ones_like(ref, bool)
    mask[:, pos0:pos0 + rows, :H * dh] = False
    assert np.array_equal(got[mask], xf[mask])
    assert_bf16_close(got[~mask], ref[~mask], "rmsnorm_rope", atol_rms=1e-4)


def _gemm_case(rng, B, rows, N, K, epi, a_extra_rows=5):
    ab, af = rand_bf16(rng, (B, rows + a_extra_rows, K))
    wb, wf = rand_bf16(rng, (N, K), 0.05)
    bb, bf = rand_bf16(rng, (N,), 0.5)
    a_dev, w_dev, b_dev = to_dev(ab), to_dev(wb), to_dev(bb)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out_rows = rows + 3                                 # output lives inside a larger tensor
    acc = af[:, :rows] @ wf.T + bf
    kw = dict(a=a_dev.data_ptr(), lda=K, a_batch_rows=rows + a_extra_rows, w=w_dev.data_ptr(), ldw=K,
              bias=b_dev.data_ptr(), ldo=N, out_batch_rows=out_rows, batch=B, rows=rows, N=N, K=K, epilogue=epi)
    keep = [a_dev, w_dev, b_dev]
    if epi in (xb.EPI_BIAS, xb.EPI_BIAS_GELU):
        out = torch.full((B, out_rows, N), 0x7FC0, dtype=torch.int16, device=DEV)
        ref = acc if epi == xb.EPI_BIAS else ob.gelu_tanh(acc)
    else:
        gate = rng.standard_normal((B, N), dtype=np.float32) * 0.3
        g_dev = torch.from_numpy(gate).to(DEV)
        keep.append(g_dev)
        kw.update(gate=g_dev.data_ptr(), gate_stride=N, ldr=N, resid_batch_rows=rows)
        if epi == xb.EPI_GATE_RES_F32:
            rb, rf = rand_bf16(rng, (B, rows, N))
            r_dev = to_dev(rb)
            out = torch.full((B, out_rows, N), float("nan"), dtype=torch.float32, device=DEV)
        else:
            r32 = rng.standard_normal((B, rows, N), dtype=np.float32)
            rf, r_dev = r32.astype(np.float64), torch.from_numpy(r32).to(DEV)
            out = torch.full((B, out_rows, N), 0x7FC0, dtype=torch.int16, device=DEV)
        keep.append(r_dev)
        kw.update(resid=r_dev.data_ptr())
        ref = rf + gate.astype(np.float64)[:, None, :] * acc
    kw.update(out=out.data_ptr())
    xb.xema_op_gemm(status=status.data_ptr(), **kw)
    _sync_status(status)
    got = out.cpu().numpy().astype(np.float64) if out.dtype == torch.float32 else from_dev_bf16(out)
    # rows past `rows` of every batch element must be untouched
    tail = out[:, rows:].cpu().numpy()
    if out.dtype == torch.float32:
        assert np.isnan(tail).all()
    else:
        assert (tail.view(np.uint16) == 0x7FC0).all()
    return got[:, :rows], ref


@pytest.mark.parametrize("epi", [0, 1, 2, 3])
@pytest.mark.parametrize("B,rows,N,K", [(1, 128, 256, 64), (1, 300, 512, 512), (2, 77, 384, 192),
                                        (1, 1000, 3072, 3072), (1, 129, 1024, 2048), (3, 257, 256, 128),
                                        (1, 5000, 768, 320)])
def test_gemm_epilogues(epi, B, rows, N, K):
    rng = np.random.default_rng(100 + epi)
    got, ref = _gemm_case(rng, B, rows, N, K, epi)
    if epi == xb.EPI_GATE_RES_F32:
        assert_close(got, ref, ("gemm", epi, B, rows, N, K), rel=1e-4, cos=0.9999999)      # fp32 output
    else:
        assert_bf16_close(got, ref, ("gemm", epi, B, rows, N, K), atol_rms=2e-3 if epi == xb.EPI_BIAS_GELU else 2e-4)


def test_gemm_many_tiles_persistent():
    """More tiles than SMs so every CTA runs several tiles through both TMEM accumulators."""
    rng = np.random.default_rng(7)
    got, ref = _gemm_case(rng, 1, 2222, 6144, 512, xb.EPI_BIAS)
    assert_bf16_close(got, ref, "gemm persistent", atol_rms=2e-4)


def test_gemm_rows_are_chunk_invariant():
    """The same rows computed as part of a large and of a small, offset problem: identical bits."""
    rng = np.random.default_rng(8)
    rows, N, K = 700, 512, 1024
    ab, _ = rand_bf16(rng, (1, rows, K))
    wb, _ = rand_bf16(rng, (N, K), 0.05)
    bb, _ = rand_bf16(rng, (N,), 0.5)
    a_dev, w_dev, b_dev = to_dev(ab), to_dev(wb), to_dev(bb)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    full = torch.zeros(1, rows, N, dtype=torch.int16, device=DEV)
    common = dict(lda=K, w=w_dev.data_ptr(), ldw=K, bias=b_dev.data_ptr(), ldo=N, batch=1, N=N, K=K,
                  epilogue=xb.EPI_BIAS_GELU)
    xb.xema_op_gemm(status=status.data_ptr(), a=a_dev.data_ptr(), a_batch_rows=rows, out=full.data_ptr(),
                    out_batch_rows=rows, rows=rows, **common)
    r0, n = 233, 301
    part = torch.zeros(1, n, N, dtype=torch.int16, device=DEV)
    xb.xema_op_gemm(status=status.data_ptr(), a=a_dev.data_ptr() + r0 * K * 2, a_batch_rows=n, out=part.data_ptr(),
                    out_batch_rows=n, rows=n, **common)
    _sync_status(status)
    assert torch.equal(full[:, r0:r0 + n], part)


def _exponent_units(q_f32, dh):
    """What the Q projection's fused epilogue hands the attention: q multiplied by
    log2(e) / sqrt(dh) in float32 and rounded to bf16 once.  Returns (bits, the exact float64 q
    those bits stand for)."""
    c = np.float32(xb.exponent_scale(dh))
    bits = bf16_bits(q_f32.astype(np.float32) * c)
    return bits, bits_to_f64(bits) / np.float64(c)


def _attention_case(rng, B, rows, keys, H, dh, q_scale=1.0):
    D = H * dh
    qb, qf = _exponent_units(rng.standard_normal((B, rows, D), dtype=np.float32) * np.float32(q_scale), dh)
    kvb, kvf = rand_bf16(rng, (B, keys, 2 * D))
    q_dev, kv_dev = to_dev(qb), to_dev(kvb)
    o = torch.full((B, rows, D), 0x7FC0, dtype=torch.int16, device=DEV)
    lse = torch.full((B, H, rows), float("nan"), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    xb.xema_op_attention(q_dev.data_ptr(), D, rows, kv_dev.data_ptr(), kv_dev.data_ptr() + D * 2, 2 * D, keys,
                         o.data_ptr(), lse.data_ptr(), B, rows, keys, H, dh, status=status.data_ptr(), q_scale=1.0)
    _sync_status(status)
    ref_o = np.empty((B, rows, H, dh))
    ref_l = np.empty((B, H, rows))
    for b in range(B):
        for h in range(H):
            ref_o[b, :, h], ref_l[b, h] = ob.attention_head(qf[b, :, h * dh:(h + 1) * dh],
                                                            kvf[b, :, h * dh:(h + 1) * dh],
                                                            kvf[b, :, D + h * dh:D + (h + 1) * dh], 1 / math.sqrt(dh))
    return from_dev_bf16(o), ref_o.reshape(B, rows, D), lse.cpu().numpy(), ref_l


@pytest.mark.parametrize("B,rows,keys,H,dh", [(1, 128, 128, 1, 64), (1, 128, 256, 2, 64), (1, 200, 500, 3, 64),
                                              (2, 77, 1000, 2, 64), (1, 144, 288, 8, 64), (1, 300, 2222, 2, 64),
                                              (1, 128, 128, 1, 128), (2, 150, 700, 2, 128)])
def test_attention(B, rows, keys, H, dh):
    rng = np.random.default_rng(200 + rows + keys)
    got_o, ref_o, got_l, ref_l = _attention_case(rng, B, rows, keys, H, dh)
    assert_bf16_close(got_o, ref_o, ("attention o", B, rows, keys, H, dh), atol_rms=1.5e-2, cos=0.9999)
    assert np.abs(got_l - ref_l).max() < 2e-3


def test_attention_peaked_scores():
    """Large |q| makes the softmax peaked and moves the running max by more than the lazy
    threshold between key blocks, so the O rescale path runs."""
    rng = np.random.default_rng(9)
    got_o, ref_o, got_l, ref_l = _attention_case(rng, 1, 256, 1500, 2, 64, q_scale=6.0)
    assert_bf16_close(got_o, ref_o, "attention peaked", atol_rms=1.5e-2, cos=0.9999)
    assert np.abs(got_l - ref_l).max() < 5e-3 * max(1.0, np.abs(ref_l).max())


@pytest.mark.parametrize("dh", [64, 128])
def test_attention_with_a_plain_q(dh):
    """A q that was not multiplied beforehand: the library is told the scale.  The head_dim 64
    kernel then multiplies its copy of the q tiles itself, which rounds q a second time (relative
    2^-9 per element), so the bound is the element-wise bf16 bound with twice the slack."""
    rng = np.random.default_rng(44 + dh)
    B, rows, keys, H = 1, 200, 700, 2
    D = H * dh
    qb, qf = rand_bf16(rng, (B, rows, D))
    kvb, kvf = rand_bf16(rng, (B, keys, 2 * D))
    q_dev, kv_dev = to_dev(qb), to_dev(kvb)
    o = torch.full((B, rows, D), 0x7FC0, dtype=torch.int16, device=DEV)
    lse = torch.full((B, H, rows), float("nan"), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    xb.xema_op_attention(q_dev.data_ptr(), D, rows, kv_dev.data_ptr(), kv_dev.data_ptr() + D * 2, 2 * D, keys,
                         o.data_ptr(), lse.data_ptr(), B, rows, keys, H, dh, status=status.data_ptr())
    _sync_status(status)
    got = from_dev_bf16(o)
    for h in range(H):
        ref_o, ref_l = ob.attention_head(qf[0, :, h * dh:(h + 1) * dh], kvf[0, :, h * dh:(h + 1) * dh],
                                         kvf[0, :, D + h * dh:D + (h + 1) * dh], 1 / math.sqrt(dh))
        assert_bf16_close(got[0, :, h * dh:(h + 1) * dh], ref_o, ("plain q", dh, h), atol_rms=3e-2, cos=0.9999)
        assert np.abs(lse.cpu().numpy()[0, h] - ref_l).max() < 4e-3


def test_attention_rows_are_chunk_invariant():
    rng = np.random.default_rng(10)
    B, rows, keys, H, dh = 1, 500, 900, 2, 64
    D = H * dh
    qb, _ = rand_bf16(rng, (B, rows, D), 2.0)
    kvb, _ = rand_bf16(rng, (B, keys, 2 * D))
    q_dev, kv_dev = to_dev(qb), to_dev(kvb)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)

    def run(r0, n):
        o = torch.zeros(B, n, D, dtype=torch.int16, device=DEV)
        lse = torch.zeros(B, H, n, dtype=torch.float32, device=DEV)
        xb.xema_op_attention(q_dev.data_ptr() + r0 * D * 2, D, n, kv_dev.data_ptr(), kv_dev.data_ptr() + D * 2, 2 * D,
                             keys, o.data_ptr(), lse.data_ptr(), B, n, keys, H, dh, status=status.data_ptr())
        return o, lse

    o_all, l_all = run(0, rows)
    o_part, l_part = run(167, 211)
    _sync_status(status)
    assert torch.equal(o_all[:, 167:167 + 211], o_part)
    assert torch.equal(l_all[:, :, 167:167 + 211], l_part)


@pytest.mark.parametrize("name,norm_all", [("tiny", True), ("tiny", False), ("flux", True), ("flux", False)])
def test_gemm_epilogue_rmsnorm_rope(name, norm_all):
    """Linear + per-head RMSNorm * gain + RoPE fused in the GEMM epilogue: the Q product
    (every head) and the K|V product (heads of the first half only)."""
    t = template(name)
    dh = t.head_dim
    rng = np.random.default_rng(31 + dh + norm_all)
    H, K, rows, pos0, B = 4, 192, 200, t.s_text - 20, 2         # rows span the text / video boundary
    Dh = H * dh
    N = Dh if norm_all else 2 * Dh
    ab, af = rand_bf16(rng, (B, rows, K))
    wb, wf = rand_bf16(rng, (N, K), 0.08)
    bb, bf = rand_bf16(rng, (N,), 0.3)
    gb, gf = rand_bf16(rng, (dh,), 1.0)
    a_dev, w_dev, b_dev, g_dev = to_dev(ab), to_dev(wb), to_dev(bb), to_dev(gb)
    rope = torch.from_numpy(xb.xema_rope_table(xb.make_config(t))).to(DEV)
    out = torch.full((B, rows, N), 0x7FC0, dtype=torch.int16, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    xb.xema_op_gemm(status=status.data_ptr(), a=a_dev.data_ptr(), lda=K, a_batch_rows=rows, w=w_dev.data_ptr(), ldw=K,
                    bias=b_dev.data_ptr(), out=out.data_ptr(), ldo=N, out_batch_rows=rows, batch=B, rows=rows, N=N,
                    K=K, epilogue=xb.EPI_BIAS_NORM_ROPE, head_dim=dh, norm_cols=Dh, rope_pos0=pos0, rms_eps=1e-6,
                    norm_gain=g_dev.data_ptr(), rope=rope.data_ptr())
    _sync_status(status)
    acc = af @ wf.T + bf
    ang = ob.rope_angles(t)[pos0:pos0 + rows]
    ref = acc.copy()
    for b in range(B):
        v = acc[b, :, :Dh].reshape(rows, H, dh)
        ref[b, :, :Dh] = ob.apply_rope(ob.rms_norm(v, gf, 1e-6), ang).reshape(rows, Dh)
    assert_bf16_close(from_dev_bf16(out), ref, ("gemm norm+rope", name, norm_all), atol_rms=3e-4)


@pytest.mark.parametrize("offset", [-260.0, -100.0, 100.0, 260.0])
def test_attention_dh64_scores_far_from_zero(offset):
    """Every score of a row lies near `offset` (in exponents to base 2), with a spread of a few
    units: far below zero the unnormalised probabilities underflow, far above they overflow, and
    in between (|offset| = 100) the sums leave the range the kernel trusts.  The head_dim-64
    kernel forms 2^score without a reference in its first pass, so all of these must be caught
    by its range check and repeated against the row's true maximum; rows of an ordinary head in
    the same launch are unaffected."""
    rng = np.random.default_rng(91)
    B, rows, keys, H, dh = 1, 300, 700, 2, 64
    D = H * dh
    u = rng.standard_normal(dh)
    u /= np.linalg.norm(u)
    q = rng.standard_normal((B, rows, D))
    kv = rng.standard_normal((B, keys, 2 * D))
    # head 0: q = a u + noise, k = b u + noise with a * b / 8 * log2(e) = offset
    a = 30.0
    b = offset * 8.0 / 1.4426950408889634 / a
    q[0, :, :dh] = a * u + 0.3 * rng.standard_normal((rows, dh))
    kv[0, :, :dh] = b * u + 0.3 * rng.standard_normal((keys, dh))
    (qb, qf), kvb = _exponent_units(q, dh), bf16_bits(kv.astype(np.float32))
    kvf = bits_to_f64(kvb)
    q_dev, kv_dev = to_dev(qb), to_dev(kvb)
    o = torch.zeros(B, rows, D, dtype=torch.int16, device=DEV)
    lse = torch.zeros(B, H, rows, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    xb.xema_op_attention(q_dev.data_ptr(), D, rows, kv_dev.data_ptr(), kv_dev.data_ptr() + D * 2, 2 * D, keys,
                         o.data_ptr(), lse.data_ptr(), B, rows, keys, H, dh, status=status.data_ptr(), q_scale=1.0)
    _sync_status(status)
    got = from_dev_bf16(o)
    expo = (qf[0, :, :dh] @ kvf[0, :, :dh].T) / math.sqrt(dh) * 1.4426950408889634
    assert abs(np.median(expo) - offset) < 0.1 * abs(offset) and expo.max() - expo.min() > 10
    for h in range(H):
        ref_o, ref_l = ob.attention_head(qf[0, :, h * dh:(h + 1) * dh], kvf[0, :, h * dh:(h + 1) * dh],
                                         kvf[0, :, D + h * dh:D + (h + 1) * dh], 1 / math.sqrt(dh))
        assert_bf16_close(got[0, :, h * dh:(h + 1) * dh], ref_o, ("scores far from zero", offset, h), atol_rms=2e-2, cos=0.9999)
        assert np.abs(lse.cpu().numpy()[0, h] - ref_l).max() < 1e-3 * max(np.abs(ref_l).max(), 1.0)


def test_attention_dh64_rows_keep_their_bits_when_neighbours_repeat():
    """Rows 128..255 of a CTA get scores in the hundreds and make the whole CTA repeat its pass;
    rows 0..127 of the same CTA (and the rows of the next CTA) must come out with exactly the
    bits they have when nothing repeats."""
    rng = np.random.default_rng(17)
    B, rows, keys, H, dh = 1, 384, 900, 1, 64
    q = rng.standard_normal((B, rows, dh))
    kv = rng.standard_normal((B, keys, 2 * dh))
    loud = q.copy()
    loud[0, 128:256] *= 60.0                                   # exponents of +-300 and more
    kvb = bf16_bits(kv.astype(np.float32))
    kv_dev = to_dev(kvb)
    outs = []
    for qq in (q, loud):
        qb, _ = _exponent_units(qq, dh)
        q_dev = to_dev(qb)
        o = torch.zeros(B, rows, dh, dtype=torch.int16, device=DEV)
        lse = torch.zeros(B, H, rows, dtype=torch.float32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        xb.xema_op_attention(q_dev.data_ptr(), dh, rows, kv_dev.data_ptr(), kv_dev.data_ptr() + dh * 2, 2 * dh, keys,
                             o.data_ptr(), lse.data_ptr(), B, rows, keys, H, dh, status=status.data_ptr(), q_scale=1.0)
        _sync_status(status)
        outs.append((o.cpu().numpy(), lse.cpu().numpy()))
    (o0, l0), (o1, l1) = outs
    quiet = np.r_[0:128, 256:rows]
    assert np.array_equal(o0[:, quiet], o1[:, quiet]) and np.array_equal(l0[:, :, quiet], l1[:, :, quiet])
    assert not np.array_equal(o0[:, 128:256], o1[:, 128:256])
    assert np.isfinite(l1).all()


@pytest.mark.parametrize("dh", [64, 128])
def test_attention_scores_growing_along_the_keys(dh):
    """Keys whose scores rise steadily with the key index: the running max moves by more than
    the lazy threshold again and again (every few blocks), the worst case for the rescale path;
    and scores so far below the max that the exponentials underflow (the polynomial's clamp)."""
    rng = np.random.default_rng(77)
    B, rows, keys, H = 1, 200, 1100, 2
    D = H * dh
    u = rng.standard_normal((H, dh))
    u /= np.linalg.norm(u, axis=1, keepdims=True)
    ramp = np.linspace(-1.0, 1.0, keys)[:, None]
    q = np.empty((B, rows, D)); kv = rng.standard_normal((B, keys, 2 * D))
    for h in range(H):
        q[0, :, h * dh:(h + 1) * dh] = u[h] * 40.0 + 0.3 * rng.standard_normal((rows, dh))
        kv[0, :, h * dh:(h + 1) * dh] = u[h] * ramp * 60.0 + 0.3 * rng.standard_normal((keys, dh))
    (qb, qf), kvb = _exponent_units(q, dh), bf16_bits(kv.astype(np.float32))
    kvf = bits_to_f64(kvb)
    q_dev, kv_dev = to_dev(qb), to_dev(kvb)
    o = torch.zeros(B, rows, D, dtype=torch.int16, device=DEV)
    lse = torch.zeros(B, H, rows, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    xb.xema_op_attention(q_dev.data_ptr(), D, rows, kv_dev.data_ptr(), kv_dev.data_ptr() + D * 2, 2 * D, keys,
                         o.data_ptr(), lse.data_ptr(), B, rows, keys, H, dh, status=status.data_ptr(), q_scale=1.0)
    _sync_status(status)
    got = from_dev_bf16(o)
    for h in range(H):
        ref_o, ref_l = ob.attention_head(qf[0, :, h * dh:(h + 1) * dh], kvf[0, :, h * dh:(h + 1) * dh],
                                         kvf[0, :, D + h * dh:D + (h + 1) * dh], 1 / math.sqrt(dh))
        # the scores span several hundred in the exp2 domain
        span = (qf[0, :, h * dh:(h + 1) * dh] @ kvf[0, :, h * dh:(h + 1) * dh].T) / math.sqrt(dh) * 1.4427
        assert span.max() - span.min() > 300
        assert_bf16_close(got[0, :, h * dh:(h + 1) * dh], ref_o, ("growing scores", dh, h), atol_rms=2e-2, cos=0.9999)
        assert np.abs(lse.cpu().numpy()[0, h] - ref_l).max() < 1e-3 * np.abs(ref_l).max()
