"""Single-kernel micro-benchmark through the C ABI (also the small case used for ncu captures).

  python -m paper_2607_11136_b200.opbench attention --rows 2222 --keys 17776 --heads 48 --head-dim 64
  python -m paper_2607_11136_b200.opbench gemm --rows 8888 --n 12288 --k 3072 --epilogue 1
  python -m paper_2607_11136_b200.opbench ln --rows 17776 --d 3072 [--f32]
  python -m paper_2607_11136_b200.opbench rope --rows 17776 --heads 48 --head-dim 64

Inputs are seeded N(0,1) bf16 (weights N(0, 0.02^2)); timing uses CUDA events on the launching
stream after warm-up; every repetition touches more than the L2 capacity or an L2 flush buffer
is written in between (--flush).  Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as xb


def _randn_bf16(shape, scale, gen):
    return (torch.randn(shape, device="cuda", generator=gen, dtype=torch.float32) * scale).to(torch.bfloat16)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["attention", "gemm", "ln", "rope"])
    ap.add_argument("--rows", type=int, default=2222)
    ap.add_argument("--keys", type=int, default=17776)
    ap.add_argument("--heads", type=int, default=48)
    ap.add_argument("--head-dim", type=int, default=64)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--n", type=int, default=3072)
    ap.add_argument("--k", type=int, default=3072)
    ap.add_argument("--d", type=int, default=3072)
    ap.add_argument("--epilogue", type=int, default=0)
    ap.add_argument("--f32", action="store_true")
    ap.add_argument("--reps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--flush", action="store_true", help="write a 256 MB buffer between repetitions")
    a = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    torch.cuda.set_device(0)
    gen = torch.Generator(device="cuda").manual_seed(0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    B = a.batch
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if a.flush else None

    if a.op == "attention":
        D = a.heads * a.head_dim
        # q in exponent units (as the block's Q projection delivers it): N(0,1) times log2(e) / sqrt(head_dim)
        q = _randn_bf16((B, a.rows, D), xb.exponent_scale(a.head_dim), gen)
        kv = _randn_bf16((B, a.keys, 2 * D), 1.0, gen)
        o = torch.empty_like(q)
        lse = torch.empty(B, a.heads, a.rows, dtype=torch.float32, device="cuda")

        def run():
            xb.xema_op_attention(q.data_ptr(), D, a.rows, kv.data_ptr(), kv.data_ptr() + 2 * D, 2 * D, a.keys,
                                 o.data_ptr(), lse.data_ptr(), B, a.rows, a.keys, a.heads, a.head_dim,
                                 status=status.data_ptr(), stream=stream, q_scale=1.0)
        flops = 4.0 * B * a.rows * a.keys * D
        nbytes = 4.0 * B * a.rows * D + 4.0 * B * a.keys * D + 4.0 * B * a.heads * a.rows
    elif a.op == "gemm":
        x = _randn_bf16((B, a.rows, a.k), 1.0, gen)
        w = _randn_bf16((a.n, a.k), 0.02, gen)
        bias = _randn_bf16((a.n,), 0.02, gen)
        f32_out = a.epilogue == xb.EPI_GATE_RES_F32
        out = torch.empty(B, a.rows, a.n, dtype=torch.float32 if f32_out else torch.bfloat16, device="cuda")
        gate = torch.randn(B, a.n, device="cuda", generator=gen) * 0.3
        if a.epilogue == xb.EPI_GATE_RES_F32:
            resid = _randn_bf16((B, a.rows, a.n), 1.0, gen)
        elif a.epilogue == xb.EPI_GATE_RES_BF16:
            resid = torch.randn(B, a.rows, a.n, device="cuda", generator=gen)
        else:
            resid = None

        def run():
            xb.xema_op_gemm(status=status.data_ptr(), stream=stream, a=x.data_ptr(), lda=a.k, a_batch_rows=a.rows,
                            w=w.data_ptr(), ldw=a.k, bias=bias.data_ptr(), out=out.data_ptr(), ldo=a.n,
                            out_batch_rows=a.rows, resid=resid.data_ptr() if resid is not None else None, ldr=a.n,
                            resid_batch_rows=a.rows, gate=gate.data_ptr(), gate_stride=a.n, batch=B, rows=a.rows,
                            N=a.n, K=a.k, epilogue=a.epilogue)
        flops = 2.0 * B * a.rows * a.n * a.k
        nbytes = 2.0 * B * a.rows * a.k + 2.0 * a.n * a.k + out.numel() * out.element_size() + \
            (resid.numel() * resid.element_size() if resid is not None else 0)
    elif a.op == "ln":
        x = torch.randn(B, a.rows, a.d, device="cuda", generator=gen)
        if not a.f32:
            x = x.to(torch.bfloat16)
        mod = torch.randn(B, 6 * a.d, device="cuda", generator=gen) * 0.3
        out = torch.empty(B, a.rows, a.d, dtype=torch.bfloat16, device="cuda")

        def run():
            xb.xema_op_ln_modulate(x.data_ptr(), int(a.f32), a.rows, out.data_ptr(), mod.data_ptr(),
                                   mod.data_ptr() + 4 * a.d, 6 * a.d, B, a.rows, a.d, 1e-6, stream=stream)
        flops = 8.0 * B * a.rows * a.d
        nbytes = B * a.rows * a.d * (6.0 if a.f32 else 4.0)
    else:
        D = a.heads * a.head_dim
        x = _randn_bf16((B, a.rows, D), 1.0, gen)
        g = _randn_bf16((a.head_dim,), 1.0, gen)
        rope = torch.randn(a.rows, a.head_dim // 2, 2, device="cuda", generator=gen)

        def run():
            xb.xema_op_rmsnorm_rope(x.data_ptr(), D, a.rows, g.data_ptr(), rope.data_ptr(), 0, B, a.rows, a.heads,
                                    a.head_dim, 1e-6, stream=stream)
        flops = 12.0 * B * a.rows * D
        nbytes = 4.0 * B * a.rows * D + 4.0 * a.rows * a.head_dim

    for _ in range(a.warmup):
        run()
    torch.cuda.synchronize()
    times = []
    for _ in range(a.reps):
        if flush_buf is not None:
            flush_buf.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        run()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    if int(status.item()) != 0:
        raise SystemExit("device status 0x%08x" % (int(status.item()) & 0xFFFFFFFF))
    ms = sum(times) / len(times)
    print(json.dumps({"op": a.op, "args": {k: v for k, v in vars(a).items() if k != "op"}, "ms": ms,
                      "ms_min": min(times), "tflops": flops / ms / 1e9, "gbs": nbytes / ms / 1e6,
                      "flops": flops, "bytes": nbytes}))


if __name__ == "__main__":
    main()
