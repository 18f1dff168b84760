"""Whole-block / whole-step parity with the oracle through xema_block_forward / xema_step_forward."""
import numpy as np
import pytest
import torch

from oracle import block as ob
from paper_2607_11136_b200 import binding as xb
from paper_2607_11136_b200.session import BlockSession
from xema_inputs import bits_to_f64, make_activations, make_block_weights, sample_rows, template

from gpu_util import DEV, assert_bf16_close, assert_close, check_block_parity, expect_raw_bound

pytestmark = pytest.mark.gpu


def _f64(w):
    return {k: bits_to_f64(v) for k, v in w.items()}


@pytest.fixture(scope="module")
def tiny_case():
    t = template("tiny")
    w = make_block_weights(t, 0)
    x, temb = make_activations(t)
    ref = ob.block_forward(t, _f64(w), bits_to_f64(x), bits_to_f64(temb), keep=True)
    return t, w, x, temb, ref


def _run(t, weights, x, temb, chunks):
    s = BlockSession(t, weights, chunks=chunks)
    s.set_inputs(x, temb)
    s.forward()
    return s, s.output_bits()


def test_tiny_block_matches_oracle_and_chunks_are_bit_identical(tiny_case):
    t, w, x, temb, ref = tiny_case
    outs = {}
    for C in (1, 2, 3):
        s, y = _run(t, [w], x, temb, C)
        outs[C] = y
        st = assert_close(bits_to_f64(y), ref["y"], ("tiny block", C))
        # the residual dominates y; check the two branches on their own as well
        res = s.view("res0", torch.float32, (1, t.seq, t.hidden)).cpu().numpy().astype(np.float64)
        x64 = bits_to_f64(x)
        assert_close(res - x64, ref["attn_branch"], ("attention branch", C), rel=6e-2, cos=0.999)
        # y is rounded to bf16, so y - res carries half an ulp of y on top of the branch error
        ffn = bits_to_f64(y) - res
        bound = 1.15 * 2.0 ** -8 * np.abs(ref["y"]) + 6e-2 * np.sqrt((ref["ffn_branch"] ** 2).mean())
        assert (np.abs(ffn - ref["ffn_branch"]) <= bound).all(), ("ffn branch", C)
        assert st["rel"] < 2e-2
    assert np.array_equal(outs[1], outs[2]) and np.array_equal(outs[1], outs[3])


def test_tiny_lse_and_intermediates(tiny_case):
    t, w, x, temb, ref = tiny_case
    # intermediates share arena addresses with later tensors: stop after ATTN_0 (op 7 of 12)
    s = BlockSession(t, [w], chunks=1)
    s.set_inputs(x, temb)
    s.plan.forward_prefix(8, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    s.check_status()
    lse = s.view("lse0_0", torch.float32, (1, t.heads, t.seq)).cpu().numpy()
    assert np.abs(lse - ref["lse"]).max() < 2e-2
    # q leaves its projection multiplied by log2(e) / sqrt(head_dim) (exponent units for the attention)
    q = bits_to_f64(s.view("q0_0", torch.int16, (1, t.seq, t.hidden)).cpu().numpy().view(np.uint16))
    assert_close(q / xb.exponent_scale(t.head_dim), ref["q"], "q after RMSNorm+RoPE", rel=3e-2, cos=0.9999)
    kv = bits_to_f64(s.view("kv0", torch.int16, (1, t.seq, 2 * t.hidden)).cpu().numpy().view(np.uint16))
    assert_close(kv[..., :t.hidden], ref["k"], "k", rel=3e-2, cos=0.9999)
    assert_close(kv[..., t.hidden:], ref["v"], "v", rel=3e-2, cos=0.9999)
    o = bits_to_f64(s.view("o0_0", torch.int16, (1, t.seq, t.hidden)).cpu().numpy().view(np.uint16))
    assert_close(o, ref["o"], "attention output", rel=4e-2, cos=0.9995)


def test_zero_gates_return_the_input_bits(tiny_case):
    t, w, x, temb, _ = tiny_case
    D = t.hidden
    w0 = {k: v.copy() for k, v in w.items()}
    for gate in (2, 5):
        w0["w_mod"][gate * D:(gate + 1) * D] = 0
        w0["b_mod"][gate * D:(gate + 1) * D] = 0
    _, y = _run(t, [w0], x, temb, 2)
    assert np.array_equal(y, x)


def test_constant_v_gives_constant_attention_output(tiny_case):
    t, w, x, temb, _ = tiny_case
    D = t.hidden
    wc = {k: v.copy() for k, v in w.items()}
    wc["w_qkv"][2 * D:] = 0
    from xema_inputs import bf16_bits
    const = bf16_bits(np.linspace(-1, 1, D).astype(np.float32))
    wc["b_qkv"][2 * D:] = const
    s = BlockSession(t, [wc], chunks=1)
    s.set_inputs(x, temb)
    s.plan.forward_prefix(8, torch.cuda.current_stream().cuda_stream)      # up to and including ATTN_0
    torch.cuda.synchronize()
    o = s.view("o0_0", torch.int16, (t.seq, D)).cpu().numpy().view(np.uint16)
    # softmax weights sum to one: every row reproduces the constant to bf16 accuracy
    assert np.abs(bits_to_f64(o) - bits_to_f64(const)).max() < 1e-2


def test_forward_stays_inside_the_planned_arena(tiny_case):
    t, w, x, temb, _ = tiny_case
    cfg = xb.make_config(t)
    plan = xb.Plan(cfg, 2)
    guard = 1 << 20
    arena = torch.full((plan.peak_bytes + guard,), 0x5A, dtype=torch.uint8, device=DEV)
    free0, _ = torch.cuda.mem_get_info()
    s = BlockSession(t, [w], chunks=2, arena=arena)
    s.set_inputs(x, temb)
    s.forward()
    torch.cuda.synchronize()
    assert bool((arena[plan.peak_bytes:] == 0x5A).all())
    assert s.plan.n_ops == 23 and s.plan.launch_count() == 23 - 2 * 2      # KROPE, QROPE run inside the GEMMs
    # the forward call itself allocated nothing on the device
    free1, _ = torch.cuda.mem_get_info()
    s.forward()
    torch.cuda.synchronize()
    free2, _ = torch.cuda.mem_get_info()
    assert free2 == free1


def test_budget_selects_chunks_and_fits(tiny_case):
    t, w, x, temb, ref = tiny_case
    for budget, want in ((2076672, 1), (2076671, 2), (1786368, 2), (1700000, 3)):
        s = BlockSession(t, [w], budget_bytes=budget, per_phase=False)
        assert s.chunks == want and s.plan.peak_bytes <= budget and s.arena.numel() == s.plan.peak_bytes
    s.set_inputs(x, temb)
    s.forward()
    assert_close(bits_to_f64(s.output_bits()), ref["y"], "budgeted tiny block")


def test_per_phase_chunks_are_bit_identical_and_fit(tiny_case):
    """Chunking only the phases that need it: any triple of per-phase counts gives the bits of
    the unchunked block; the budget search picks (1, 1, C) and its plan fits the budget."""
    t, w, x, temb, ref = tiny_case
    _, base = _run(t, [w], x, temb, 1)
    for counts in [(1, 1, 2), (1, 1, 3), (2, 1, 3), (3, 2, 1), (1, 4, 2), (5, 3, 7)]:
        s, y = _run(t, [w], x, temb, counts)
        assert s.phase_chunks == counts and s.plan.n_ops == 1 + 3 * counts[0] + 5 * counts[1] + 3 * counts[2]
        assert np.array_equal(y, base), counts
    for budget, want in ((2076672, (1, 1, 1)), (2076671, (1, 1, 2)), (1634304, (1, 1, 2)), (1634303, (1, 1, 3)),
                         (1496064, (1, 1, 3))):
        s = BlockSession(t, [w], budget_bytes=budget)
        assert s.chunks == want and s.plan.peak_bytes <= budget and s.arena.numel() == s.plan.peak_bytes
        s.set_inputs(x, temb)
        s.forward()
        assert np.array_equal(s.output_bits(), base), budget
    assert_close(bits_to_f64(base), ref["y"], "per-phase tiny block")
    with pytest.raises(xb.XemaError) as e:
        BlockSession(t, [w], budget_bytes=1496063)
    assert e.value.status == xb.XEMA_EBUDGET


def test_batch_two_small_block():
    t = template("tiny", batch=2, grid_t=2)
    w = make_block_weights(t, 3)
    x, temb = make_activations(t)
    ref = ob.block_forward(t, _f64(w), bits_to_f64(x), bits_to_f64(temb))
    outs = []
    for C in (1, 2):
        _, y = _run(t, [w], x, temb, C)
        assert_close(bits_to_f64(y), ref["y"], ("batch 2", C))
        outs.append(y)
    assert np.array_equal(outs[0], outs[1])


def test_head_dim_128_small_block():
    t = template("flux", s_text=40, grid_h=12, grid_w=10, hidden=512, heads=4, ffn=1024)
    w = make_block_weights(t, 5)
    x, temb = make_activations(t)
    ref = ob.block_forward(t, _f64(w), bits_to_f64(x), bits_to_f64(temb))
    outs = []
    for C in (1, 3):
        _, y = _run(t, [w], x, temb, C)
        assert_close(bits_to_f64(y), ref["y"], ("head_dim 128", C))
        outs.append(y)
    assert np.array_equal(outs[0], outs[1])


def test_small_step_teacher_forced_and_free_running():
    """Three stacked blocks: each block is compared with the oracle applied to the GPU's own
    bf16 input of that block; the free-running end-to-end error is checked more loosely."""
    t = template("tiny", n_blocks=3)
    ws = [make_block_weights(t, l) for l in range(3)]
    x, temb = make_activations(t)
    s = BlockSession(t, ws, chunks=2)
    s.set_inputs(x, temb)
    s.forward()
    y = s.output_bits()
    temb64 = bits_to_f64(temb)
    free = ob.step_forward(t, [_f64(w) for w in ws], bits_to_f64(x), temb64)
    assert_close(bits_to_f64(y), free, "free-running step", rel=6e-2, cos=0.999)
    # hidden states of successive blocks may share arena addresses, so run prefixes instead
    t1 = t.with_(n_blocks=1)
    cur = x
    for l in range(3):
        _, nxt = _run(t1, [ws[l]], cur, temb, 2)
        ref = ob.block_forward(t1, _f64(ws[l]), bits_to_f64(cur), temb64)["y"]
        assert_close(bits_to_f64(nxt), ref, ("teacher-forced block", l))
        cur = nxt
    assert np.array_equal(cur, y)


@pytest.mark.parametrize("name", ["cogvideox"])
def test_full_size_block_sampled_rows(name):
    """CogVideoX-shaped block at full size: budgets equal to the planned peaks select
    C = 1, 2, 4, 8; outputs are bit-identical across C; sampled rows match the oracle."""
    t = template(name)
    cfg = xb.make_config(t)
    w = make_block_weights(t, 0)
    x, temb = make_activations(t)
    # chunk starts of every count tried, plus both sides of the 128- and 256-row tile edges at the
    # start and next to the ragged tail (17776 = 69 * 256 + 112: last full tile ends at row 17664)
    bounds = [c * t.seq // C for C in (2, 4, 8) for c in range(1, C)] + [128, 256, t.seq // 256 * 256,
                                                                         t.seq // 128 * 128]
    rows = sample_rows(t, boundaries=bounds, n_random=1100)
    assert len(rows) >= 1024 and {t.seq // 256 * 256 - 1, t.seq // 256 * 256, t.seq - 1} <= set(rows.tolist())
    ref = ob.block_forward(t, _f64(w), bits_to_f64(x), bits_to_f64(temb), rows=rows)["y"]
    dev_w = None
    first = None
    parity = None
    for C in (1, 2, 4, 8):
        peak = xb.Plan(cfg, C).peak_bytes
        s = BlockSession(t, [dev_w or w], budget_bytes=peak, per_phase=False)
        dev_w = s.weights[0]
        assert s.chunks == C and s.arena.numel() == peak
        s.set_inputs(x, temb)
        s.forward()
        y = s.output_bits()
        if first is None:
            first = y
            parity = check_block_parity("full-size %s" % name, y[:, rows], ref)
        else:
            assert np.array_equal(first, y), C
        del s
        torch.cuda.empty_cache()
    # per-phase search at the budgets the uniform search needs C = 2 and C >= 6 for
    for budget, want, peak in ((640 << 20, (1, 1, 2), 600760320), (560 << 20, (1, 1, 3), 549565440)):
        s = BlockSession(t, [dev_w], budget_bytes=budget)
        assert s.chunks == want and s.arena.numel() == peak
        s.set_inputs(x, temb)
        s.forward()
        assert np.array_equal(first, s.output_bits()), want
        del s
        torch.cuda.empty_cache()
    expect_raw_bound(parity)


def test_bounded_wait_gives_up_and_reports():
    """A wait on a barrier nothing completes runs out after its limit, sets the status word and
    leaves the context usable (the next forward call still matches the oracle)."""
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    waited = torch.zeros(1, dtype=torch.int64, device=DEV)
    limit = 2_000_000                                   # about a millisecond of SM cycles
    xb.xema_selftest_wait_timeout(status.data_ptr(), limit, waited.data_ptr())
    torch.cuda.synchronize()
    assert (int(status.item()) & 0xFFFFFFFF) == xb.DEVICE_STATUS_TIMEOUT
    assert limit <= int(waited.item()) < 50 * limit
    # the session turns a non-zero status word into an error ...
    t = template("tiny")
    w = make_block_weights(t, 0)
    x, temb = make_activations(t)
    s = BlockSession(t, [w], chunks=1)
    s.status.copy_(status)
    with pytest.raises(xb.XemaError) as e:
        s.check_status()
    assert e.value.status == xb.XEMA_ETIMEOUT
    # ... and the context is still good for real work
    s.status.zero_()
    s.set_inputs(x, temb)
    s.forward()
    ref = ob.block_forward(t, _f64(w), bits_to_f64(x), bits_to_f64(temb))["y"]
    assert_close(bits_to_f64(s.output_bits()), ref, "block after a timed-out wait")


def test_forward_host_two_batched_blocks_in_pieces():
    """Two blocks, batch 2: row pieces (each piece = the same rows of both batch elements, a
    strided copy) and sub-batches in the first and the last phase; bits of the arena forward."""
    t = template("tiny", batch=2).with_(n_blocks=2)
    ws = [make_block_weights(t, l) for l in range(2)]
    x, temb = make_activations(t)
    stream = torch.cuda.current_stream().cuda_stream
    want = None
    for chunks, axes in (((1, 1, 1), None), ((3, 1, 2), None), ((2, 2, 2), (1, 0, 1)), ((2, 1, 3), (0, 0, 0))):
        s = BlockSession(t, ws, chunks=chunks, axes=axes)
        s.set_inputs(x, temb)
        s.forward()
        got = s.output_bits().copy()
        if want is None:
            want = got
        assert np.array_equal(got, want)
        x_h = torch.from_numpy(x.view(np.int16)).pin_memory()
        t_h = torch.from_numpy(temb.view(np.int16)).pin_memory()
        y_h = torch.zeros_like(x_h).pin_memory()
        for _ in range(2):
            y_h.zero_()
            s.arena.fill_(0x7F)
            s.plan.forward_host(x_h.data_ptr(), t_h.data_ptr(), y_h.data_ptr(), stream)
            torch.cuda.synchronize()
            assert np.array_equal(y_h.numpy().view(np.uint16), want), (chunks, axes)
        s.check_status()


@pytest.mark.parametrize("chunks", [(1, 1, 2), (3, 2, 3), (1, 1, 1)])
def test_forward_host_equals_arena_forward(tiny_case, chunks):
    """xema_forward_host (pinned host buffers in and out; with several pieces in the first or the
    last phase their copies overlap the neighbouring pieces' launches through the plan's own
    copy stream) returns the bits of set_inputs / forward / output_bits, three times in a row,
    and allocates no device memory after its first call."""
    t, w, x, temb, ref = tiny_case
    s = BlockSession(t, [w], chunks=chunks)
    s.set_inputs(x, temb)
    s.forward()
    want = s.output_bits().copy()
    x_h = torch.from_numpy(x.view(np.int16)).pin_memory()
    t_h = torch.from_numpy(temb.view(np.int16)).pin_memory()
    y_h = torch.zeros_like(x_h).pin_memory()
    stream = torch.cuda.current_stream().cuda_stream
    free0 = None
    for _ in range(3):
        y_h.zero_()
        # scribble over the arena: every input byte the forward reads must come from the host copy
        s.arena.fill_(0x7F)
        s.plan.forward_host(x_h.data_ptr(), t_h.data_ptr(), y_h.data_ptr(), stream)
        torch.cuda.synchronize()
        assert np.array_equal(y_h.numpy().view(np.uint16), want)
        if free0 is None:
            free0, _ = torch.cuda.mem_get_info()     # the first call may create the copy stream
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    s.check_status()
    # an unbound plan is refused
    with pytest.raises(xb.XemaError) as e:
        xb.Plan(xb.make_config(t), 1).forward_host(x_h.data_ptr(), t_h.data_ptr(), y_h.data_ptr(), stream)
    assert e.value.status == xb.XEMA_ESTATE


def test_pipelined_host_to_host_equals_serial(tiny_case):
    """run_pipelined (copies of neighbouring steps overlapped with compute) returns, for every
    step, the bits of a plain set_inputs / forward / output_bits round trip."""
    t, w, x, temb, ref = tiny_case
    s = BlockSession(t, [w], chunks=(1, 1, 2))
    rng = np.random.default_rng(5)
    xs = [x] + [(x.astype(np.uint32) ^ (rng.integers(0, 2, x.shape, dtype=np.uint32) << 15)).astype(np.uint16)
                for _ in range(4)]               # sign flips: still finite bf16 values
    want = []
    for xi in xs:
        s.set_inputs(xi, temb)
        s.forward()
        want.append(s.output_bits().copy())
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).pin_memory()
    x_h = [pin(xi) for xi in xs]
    t_h = [pin(temb) for _ in xs]
    y_h = [torch.empty_like(x_h[0]).pin_memory() for _ in xs]
    for _ in range(2):                           # a second call reuses the staging buffers
        done = s.run_pipelined(x_h, t_h, y_h)
        done.synchronize()
        torch.cuda.synchronize()
        s.check_status()
        for got, exp in zip(y_h, want):
            assert np.array_equal(got.numpy().view(np.uint16).reshape(exp.shape), exp)
    assert np.array_equal(want[0], _run(t, [w], x, temb, 1)[1])
    assert s.staging_bytes == 2 * x.size * 2 + temb.size * 2


def test_sub_batch_pieces_are_bit_identical_to_row_chunks():
    """Temporary serialization: phases split into sub-batches (whole batch elements, all rows)
    give the bits of the unsplit block, match the oracle, and the budget search picks them."""
    t = template("tiny", batch=3, grid_t=2)
    w = make_block_weights(t, 4)
    x, temb = make_activations(t)
    ref = ob.block_forward(t, _f64(w), bits_to_f64(x), bits_to_f64(temb))
    _, base = _run(t, [w], x, temb, 1)
    assert_close(bits_to_f64(base), ref["y"], "batch 3 unsplit")
    for chunks, axes in [((1, 1, 3), (0, 0, 1)), ((2, 3, 2), (1, 1, 1)), ((2, 2, 3), (0, 1, 0)), ((3, 1, 2), (1, 0, 0))]:
        s = BlockSession(t, [w], chunks=chunks, axes=axes)
        assert s.axes == axes and s.phase_chunks == chunks
        s.set_inputs(x, temb)
        s.forward()
        assert np.array_equal(s.output_bits(), base), (chunks, axes)
    cfg = xb.make_config(t)
    p1 = xb.Plan(cfg, 1).peak_bytes
    s = BlockSession(t, [w], budget_bytes=int(0.9 * p1), serialize=True)
    # two sub-batches of three requests would still hold two of them in one piece
    assert s.phase_chunks == (1, 1, 3) and s.axes == (0, 0, 1) and s.plan.peak_bytes <= int(0.9 * p1)
    s.set_inputs(x, temb)
    s.forward()
    assert np.array_equal(s.output_bits(), base)


def test_flux_batch_four_serialized_ffn():
    """Flux-style block, batch 4, budget at 0.9 of the unsplit peak: the feed-forward phase runs as
    two sub-batches of two requests; same bits as the unsplit block at sampled rows and overall."""
    t = template("flux", batch=4)
    w = make_block_weights(t, 0)
    x, temb = make_activations(t)
    cfg = xb.make_config(t)
    p1 = xb.Plan(cfg, 1).peak_bytes
    s1 = BlockSession(t, [w], chunks=1)
    s1.set_inputs(x, temb)
    s1.forward()
    y1 = s1.output_bits()
    dev_w = s1.weights
    del s1
    s = BlockSession(t, dev_w, budget_bytes=int(0.9 * p1), serialize=True)
    assert s.phase_chunks == (1, 1, 2) and s.axes == (0, 0, 1) and s.plan.peak_bytes == s.arena.numel() <= int(0.9 * p1)
    s.set_inputs(x, temb)
    s.forward()
    assert np.array_equal(s.output_bits(), y1)


def test_redundant_layer_norm_launch_is_elided_only_when_in_place(tiny_case):
    """With one piece in the key/value and attention phases LN1B would rewrite what LN1A left at
    the same arena address; the executor skips that launch (12 logical ops, 9 launches) and the
    output bits do not change; with two pieces nothing is skipped."""
    t, w, x, temb, ref = tiny_case
    s2, y2 = _run(t, [w], x, temb, 2)
    s1, y1 = _run(t, [w], x, temb, (1, 1, 2))
    assert np.array_equal(y1, y2)
    names = [s1.plan.op(i)["name"] for i in range(s1.plan.n_ops)]
    assert names == ["MOD", "LN1A", "KV", "KROPE", "LN1B", "Q", "QROPE", "ATTN", "PROJ", "LN2", "FFN1", "FFN2", "LN2",
                     "FFN1", "FFN2"]
    assert s1.plan.tensor("h1a0_0") == s1.plan.tensor("h1b0_0")
    assert s1.plan.launch_count() == 15 - 3                 # KROPE, QROPE and LN1B launch nothing
    assert s2.plan.launch_count() == 23 - 4
    # the intermediate the elided launch would have written is what the Q projection reads
    s1.set_inputs(x, temb)
    s1.plan.forward_prefix(5, torch.cuda.current_stream().cuda_stream)      # up to and including LN1B
    torch.cuda.synchronize()
    h1 = s1.view("h1b0_0", torch.int16, (1, t.seq, t.hidden)).cpu().numpy().view(np.uint16)
    assert_bf16_close(bits_to_f64(h1), ref["h1"], "h1 left in place by LN1A")


def test_forward_replayed_from_a_cuda_graph(tiny_case):
    """A captured forward pass replays to the same bits as the eager one (every address is static)."""
    t, w, x, temb, ref = tiny_case
    s, want = _run(t, [w], x, temb, (1, 1, 2))
    g = s.capture()
    for _ in range(3):
        s.set_inputs(x, temb)
        s.hid_out().zero_()
        g.replay()
        assert np.array_equal(s.output_bits(), want)
    import time
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(200):
        g.replay()
    torch.cuda.synchronize()
    t_graph = (time.perf_counter() - t0) / 200
    t0 = time.perf_counter()
    for _ in range(200):
        s.forward()
    torch.cuda.synchronize()
    t_eager = (time.perf_counter() - t0) / 200
    print("tiny block: %.1f us per replayed graph, %.1f us eager" % (t_graph * 1e6, t_eager * 1e6))
    s.check_status()


@pytest.mark.parametrize("name,chunks", [("tiny", (1, 2, 3)), ("cogvideox", (1, 1, 2))])
def test_guard_bands_between_arena_neighbours_stay_intact(name, chunks):
    """Debug layout with 4 KiB kept free after every tensor (the stand-in for a memory checker):
    run op by op, the band after every live tensor keeps its pattern after every op; the output
    has the bits of the ordinary layout.  The checker itself is shown to see a damaged band."""
    t = template(name)
    w = make_block_weights(t, 0)
    x, temb = make_activations(t)
    s = BlockSession(t, [w], chunks=chunks)
    s.set_inputs(x, temb)
    s.forward()
    want = s.output_bits().copy()
    G = 4096
    g = BlockSession(t, s.weights, chunks=chunks, guard_bytes=G)
    tensors = g.plan.tensors()
    assert g.plan.guard_bytes == G and g.plan.max_live_bytes == s.plan.max_live_bytes
    assert s.plan.peak_bytes < g.plan.peak_bytes <= s.plan.peak_bytes + G * len(tensors)
    # no two tensors that live together come closer than the guard
    for i, a in enumerate(tensors):
        for b in tensors[i + 1:]:
            if a["birth"] < b["death"] and b["birth"] < a["death"]:
                lo, hi = (a, b) if a["offset"] < b["offset"] else (b, a)
                assert lo["offset"] + lo["bytes"] + G <= hi["offset"], (lo["name"], hi["name"])
    g.set_inputs(x, temb)
    assert g.forward_guarded() == []
    assert np.array_equal(g.output_bits(), want)
    g.check_status()
    # negative control: a byte written into the band behind the block input is reported by the
    # first op (the input is live from op 0) and by every op up to the input's last use
    g.set_inputs(x, temb)
    hid0 = next(d for d in tensors if d["name"] == "hid0")
    real_fill = torch.Tensor.fill_
    damaged = {"done": False}

    def fill_then_damage(self_, value):
        out = real_fill(self_, value)
        if not damaged["done"] and self_.data_ptr() == g.arena.data_ptr() + hid0["offset"] + hid0["bytes"]:
            self_[7] = 0
            damaged["done"] = True
        return out

    torch.Tensor.fill_ = fill_then_damage
    try:
        bad = g.forward_guarded()
    finally:
        torch.Tensor.fill_ = real_fill
    assert damaged["done"] and bad and bad[0][:1] == (0,) and all(b[2] == "hid0" and b[3] == 1 for b in bad)
    assert len(bad) == hid0["death"]
