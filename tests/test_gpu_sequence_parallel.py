"""Sequence-parallel shards of the block on ONE GPU: the P shards run one after the other in one
process, each in its own arena; the exchange of keys and values is a device-to-device copy of
every shard's rows into every other shard's kv tensor (what an all-gather into the ranks' own
arenas leaves behind).  The concatenated outputs must be the bits of the unsharded block: a row's
arithmetic does not depend on which rows share its tile, its chunk or its GPU."""
import numpy as np
import pytest
import torch

from paper_2607_11136_b200.session import BlockSession
from xema_inputs import make_activations, make_block_weights, template

pytestmark = pytest.mark.gpu


def _run_sharded(t, dev_w, x, temb, P, chunks, axes=None):
    shards = [BlockSession(t, dev_w, chunks=chunks, axes=axes, shard=(p, P)) for p in range(P)]
    for s in shards:
        assert s.arena.numel() == s.plan.peak_bytes and (s.plan.row0, s.plan.rows) == (s.plan.row0, s.seq)
        s.set_inputs(x[:, s.plan.row0:s.plan.row0 + s.plan.rows], temb)
    stream = torch.cuda.current_stream().cuda_stream
    at = 0
    for l in range(t.n_blocks):
        op = shards[0].plan.gather_point(l)[0]
        for s in shards:
            assert s.plan.gather_point(l)[0] == op
            s.plan.forward_range(at, op, stream)
        # the exchange: every shard's own rows of kv<l> go to all the others
        for src in shards:
            r0, n = src.plan.row0, src.plan.rows
            for dst in shards:
                if dst is not src:
                    dst.kv(l)[:, r0:r0 + n].copy_(src.kv(l)[:, r0:r0 + n])
        at = op
    for s in shards:
        s.plan.forward_range(at, s.plan.n_ops, stream)
    outs = [s.output_bits() for s in shards]
    peaks = [s.plan.peak_bytes for s in shards]
    return np.concatenate(outs, axis=1), peaks


@pytest.mark.parametrize("P,chunks,axes", [(2, (1, 1, 1), None), (3, (2, 1, 3), None), (4, (1, 2, 1), None)])
def test_tiny_block_shards_equal_the_unsharded_block(P, chunks, axes):
    t = template("tiny")
    w = make_block_weights(t, 0)
    x, temb = make_activations(t)
    s = BlockSession(t, [w], chunks=1)
    s.set_inputs(x, temb)
    s.forward()
    want = s.output_bits().copy()
    y, _ = _run_sharded(t, s.weights, x, temb, P, chunks, axes)
    assert y.shape == want.shape and np.array_equal(y, want)


def test_batched_two_block_step_shards_with_sub_batches():
    """Two blocks, batch 2, the feed-forward phase split into sub-batches: one exchange per block."""
    t = template("tiny", batch=2).with_(n_blocks=2)
    ws = [make_block_weights(t, l) for l in range(2)]
    x, temb = make_activations(t)
    s = BlockSession(t, ws, chunks=1)
    s.set_inputs(x, temb)
    s.forward()
    want = s.output_bits().copy()
    y, _ = _run_sharded(t, s.weights, x, temb, 2, (1, 2, 2), (0, 0, 1))
    assert np.array_equal(y, want)


def test_cogvideox_block_in_four_shards():
    """CogVideoX-shaped block, 4 shards of 4444 rows, feed-forward in two chunks: every shard's
    arena is 301 270 272 bytes (the unsharded plan needs 600 760 320), outputs bit-identical."""
    t = template("cogvideox")
    w = make_block_weights(t, 0)
    x, temb = make_activations(t)
    s = BlockSession(t, [w], chunks=(1, 1, 2))
    s.set_inputs(x, temb)
    s.forward()
    want = s.output_bits().copy()
    dev_w = s.weights
    del s
    y, peaks = _run_sharded(t, dev_w, x, temb, 4, (1, 1, 2))
    assert peaks == [301270272] * 4
    assert np.array_equal(y, want)
