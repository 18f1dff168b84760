"""The allocator plug-in (static-memory runtime for ordinary PyTorch code).  PyTorch lets a
process replace its allocator only before the first CUDA allocation, so the GPU part runs the
demo module in a child process."""
import json
import os
import subprocess
import sys

import pytest

from paper_2607_11136_b200 import binding as xb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_plugin_state_machine_without_a_gpu():
    xb.xema_pluggable_mode(xb.ALLOC_PASSTHROUGH)
    with pytest.raises(xb.XemaError) as e:
        xb.xema_pluggable_mode(7)
    assert e.value.status == xb.XEMA_EINVAL
    xb.xema_pluggable_mode(xb.ALLOC_RECORD)             # clears any plan
    with pytest.raises(xb.XemaError) as e:
        xb.xema_pluggable_recorded()                    # still recording
    assert e.value.status == xb.XEMA_ESTATE
    with pytest.raises(xb.XemaError) as e:
        xb.xema_pluggable_set_plan(256, 1 << 20, [])    # only in pass-through mode
    assert e.value.status == xb.XEMA_ESTATE
    xb.xema_pluggable_mode(xb.ALLOC_PASSTHROUGH)
    assert xb.xema_pluggable_recorded() == ([], 0)
    with pytest.raises(xb.XemaError) as e:
        xb.xema_pluggable_mode(xb.ALLOC_REPLAY)         # no plan
    assert e.value.status == xb.XEMA_ESTATE
    with pytest.raises(xb.XemaError) as e:
        xb.xema_pluggable_step_begin()                  # not replaying
    assert e.value.status == xb.XEMA_ESTATE
    with pytest.raises(xb.XemaError) as e:
        xb.xema_pluggable_set_plan(256, 1 << 20, [0])   # one offset for an empty recording
    assert e.value.status == xb.XEMA_EINVAL
    served, fallback, nxt = xb.xema_pluggable_stats()
    assert nxt == 0 and served >= 0 and fallback >= 0


def _demo(*args):
    r = subprocess.run([sys.executable, "-m", "paper_2607_11136_b200.pluggable_demo", *args], cwd=ROOT,
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    return json.loads(r.stdout.strip().splitlines()[-1])


@pytest.mark.gpu
def test_eager_pytorch_block_on_the_planned_arena():
    args = ["--tokens", "4096", "--hidden", "1024", "--heads", "16", "--chunks", "2"]
    d = _demo(*args)
    assert d["replay_identical_to_record"] and d["finite"] and d["first_request_at_planned_offset"]
    assert d["fallback"] == 0 and d["served"] == 3 * d["requests_per_step"] > 0
    assert d["next_index_after_step"] == d["requests_per_step"] == d["events"]
    # reuse: the arena is smaller than the sum of the requests, never smaller than the largest
    # simultaneous set, and Algorithm 1 stays close to that bound on this trace
    assert d["largest_request_bytes"] <= d["max_live_bytes"] <= d["arena_peak_bytes"] < d["sum_of_request_bytes"]
    assert d["arena_peak_bytes"] <= 1.1 * d["max_live_bytes"]
    c = _demo(*args, "--caching")
    # the same step under torch's caching allocator reserves at least its own active peak
    assert c["reserved_peak_bytes"] - c["parameter_bytes"] >= 0
    print("plug-in arena %d B (max-live %d) for %d requests/step; torch caching allocator: step active peak %d B, "
          "reserved %d B incl. %d B of parameters" % (d["arena_peak_bytes"], d["max_live_bytes"], d["requests_per_step"],
                                                     c["step_allocated_peak_bytes"], c["reserved_peak_bytes"],
                                                     c["parameter_bytes"]))
