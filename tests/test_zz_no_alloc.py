"""ps_eval_compact_noalloc: the filter-and-compact call for programs that may
not allocate device memory -- their GPU memory belongs to another allocator (a
framework's caching pool, a serving cache), or they cannot take the device-wide
stall of cudaMalloc/cudaFree inside their loop.  It keeps its scratch tables in
a fixed array of the library instead of the context's growable buffer.

Checked here through the C interface: its output equals that of the allocating
entry point (ps_eval_batch with a filter) and that of the CPU oracle bit for
bit, on two calls in a row that share the fixed array -- the second smaller
than the first, so leftovers of the first would show; the device's free memory
is the same before and after a call on a larger window than any before it (the
property the entry point exists for); and a window beyond the array's capacity
is refused.  This file sorts last so that a failure here cannot hide another
test's result.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2601_02311_b200 import synth

pytestmark = pytest.mark.gpu

FIELDS = ("mem", "comm_paper", "comm_ext", "host", "flags")


def run_noalloc(gs, first, count, filt):
    dev = gs.ctx.torch_device
    out = gs.alloc_outputs(count)                       # the caller's own outputs
    idx = torch.empty(max(count, 1), dtype=torch.int64, device=dev)
    n = torch.full((1,), -1, dtype=torch.int64, device=dev)
    gs.compact_noalloc_into(first, count, out, filt, idx, n)
    gs.ctx.check_status()
    k = int(n.item())
    res = {name: out[name][:k].cpu().numpy().view(np.uint32 if name == "flags" else np.uint64)
           for name in FIELDS}
    res["idx"] = idx[:k].cpu().numpy().view(np.uint64)
    return res


def test_noalloc_compaction_equals_allocating_entry_point_twice():
    import paper_2601_02311_b200.ps as ps
    ctx = ps.Context(0)
    space = synth.config("C3", n_models=3)
    gs, os_ = ctx.space(space), O.Space(space)
    calls = [
        (777, 1_500_001, dict(require_flags=ps.F_VALID, cap_bytes=192 * synth.GB)),
        (725_000 + 300_003, 90_000, dict(require_flags=ps.F_GI | ps.F_SC, cap_bytes=80 * synth.GB,
                                    host_cap=8 * synth.GB)),
    ]
    for first, count, filt in calls:
        got = run_noalloc(gs, first, count, filt)
        want = gs.compact(first, count, filt)
        oracle = os_.compact_range(first, count, filt)
        assert len(want["idx"]) > 0
        for name in FIELDS + ("idx",):
            assert np.array_equal(got[name], want[name]), name
            assert np.array_equal(got[name], oracle[name]), name
    # nothing is allocated: with the caller's buffers in place, a call on a window larger than
    # any before it leaves the device's free memory where it was
    first, count, filt = 0, 2_000_003, calls[0][2]
    dev = ctx.torch_device
    out = gs.alloc_outputs(count)
    idx = torch.empty(count, dtype=torch.int64, device=dev)
    n = torch.zeros(1, dtype=torch.int64, device=dev)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info(dev)[0]
    gs.compact_noalloc_into(first, count, out, filt, idx, n)
    ctx.check_status()
    assert torch.cuda.mem_get_info(dev)[0] == free_before
    assert int(n.item()) == len(os_.compact_range(first, count, filt)["idx"])
    # an empty window writes a zero count
    n = torch.full((1,), -1, dtype=torch.int64, device=ctx.torch_device)
    gs.compact_noalloc_into(5, 0, {}, calls[0][2], None, n)
    assert int(n.item()) == 0
    gs.close()
    ctx.close()


def test_noalloc_refuses_windows_beyond_its_fixed_array():
    import paper_2601_02311_b200.ps as ps
    ctx = ps.Context(0)
    space = synth.config("C2", n_models=160)            # 256 points per group
    gs = ctx.space(space)
    too_many = (ps.NOALLOC_MAX_GROUPS + 1) * 256
    assert gs.size >= too_many
    n = torch.zeros(1, dtype=torch.int64, device=ctx.torch_device)
    with pytest.raises(ps.PsError) as e:
        gs.compact_noalloc_into(0, too_many, {}, dict(cap_bytes=1), None, n)
    assert e.value.code == ps.E_NOALLOC_LIMIT
    assert "fixed array" in str(e.value)
    # the largest window that fits is accepted
    gs.compact_noalloc_into(0, ps.NOALLOC_MAX_GROUPS * 256, {}, dict(cap_bytes=1), None, n)
    ctx.check_status()
    gs.close()
    ctx.close()
