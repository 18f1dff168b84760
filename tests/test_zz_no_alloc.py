"""xema_block_forward_static: the block forward for callers that cannot allocate device memory
(no cudaMalloc, no framework allocator -- e.g. a plug-in that only ever receives its input and
output buffers).  Its intermediates live in a fixed array inside the library, so the test
checks that it computes exactly what xema_block_forward computes with a caller-owned arena,
on two calls in a row that reuse the same array, and that it allocates nothing."""
import numpy as np
import pytest
import torch

from paper_2607_11136_b200 import binding as xb
from paper_2607_11136_b200.session import BlockSession
from xema_inputs import bits_to_f64, make_activations, make_block_weights, template

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(DEV)


def test_static_arena_block_matches_arena_block_twice_in_a_row():
    t = template("tiny")
    cfg = xb.make_config(t)
    w = make_block_weights(t, 0)
    cases = []
    for seed, chunks in ((1_000_000, 2), (1_000_001, 1)):
        x, temb = make_activations(t, seed)
        s = BlockSession(t, [w], chunks=chunks)
        s.set_inputs(x, temb)
        s.forward()
        cases.append((chunks, x, temb, s.output_bits()))
    # everything the new entry point needs is allocated here, before the calls
    w_dev = {k: _dev(v) for k, v in w.items()}
    ptrs = {k: v.data_ptr() for k, v in w_dev.items()}
    rope = torch.from_numpy(xb.xema_rope_table(cfg)).to(DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    x_devs = [(_dev(x), _dev(temb)) for _, x, temb, _ in cases]
    outs = [torch.zeros(t.batch, t.seq, t.hidden, dtype=torch.int16, device=DEV) for _ in cases]
    stream = torch.cuda.current_stream().cuda_stream
    # a first call before measuring: the device address of the scratch array is looked up once
    xb.xema_block_forward_static(cfg, 1, ptrs, rope.data_ptr(), x_devs[0][0].data_ptr(), x_devs[0][1].data_ptr(),
                                 outs[0].data_ptr(), status.data_ptr(), stream)
    torch.cuda.synchronize()
    outs[0].zero_()
    free0, _ = torch.cuda.mem_get_info()
    for (chunks, _, _, _), (xd, td), out in zip(cases, x_devs, outs):          # two calls in a row
        xb.xema_block_forward_static(cfg, chunks, ptrs, rope.data_ptr(), xd.data_ptr(), td.data_ptr(),
                                     out.data_ptr(), status.data_ptr(), stream)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, "the entry point must not allocate device memory"
    assert int(status.item()) == 0
    for (chunks, _, _, want), out in zip(cases, outs):
        got = out.cpu().numpy().view(np.uint16)
        ref = bits_to_f64(want)
        rms = float(np.sqrt((ref * ref).mean()))
        assert np.abs(bits_to_f64(got) - ref).max() <= 2e-2 * rms       # the tolerance of the block tests
        assert np.array_equal(got, want), chunks                         # in fact the same bits


def test_static_arena_rejects_templates_beyond_its_maximum():
    t = template("cogvideox")
    cfg = xb.make_config(t)
    dummy = torch.zeros(64, dtype=torch.int16, device=DEV)
    ptrs = {k: dummy.data_ptr() for k in xb._WEIGHT_FIELDS}
    with pytest.raises(xb.XemaError) as e:
        xb.xema_block_forward_static(cfg, 8, ptrs, dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(),
                                     dummy.data_ptr())
    assert e.value.status == xb.XEMA_ENOSPC
    assert xb.Plan(cfg, 8).peak_bytes > xb.STATIC_ARENA_BYTES
