"""Nothing is written outside the caller's buffers.  Every output is a view into
a larger buffer filled with a pattern; after a call the pattern before and after
the view must be intact and the view must equal the oracle.  The views start at
every alignment the interface allows (8-byte for the 64-bit arrays, 4-byte for
the flags) and windows start and end inside groups.  A compaction may use up to
`count` slots of each output, so its guard sits after `count`; the slots
between the last survivor and `count` are checked to be left alone as well."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2601_02311_b200 import synth

pytestmark = pytest.mark.gpu

GUARD = 96                     # elements on either side
PATTERN64 = 0x5A5A5A5A5A5A5A5A
PATTERN32 = 0x5A5A5A5A
FIELDS = ("mem", "comm_paper", "comm_ext", "host", "flags")


@pytest.fixture(scope="module")
def ps():
    import paper_2601_02311_b200.ps as ps_mod
    return ps_mod


@pytest.fixture(scope="module")
def ctx(ps):
    c = ps.Context(0)
    yield c
    c.close()


def guarded(count, dtype, shift, dev):
    """A buffer of GUARD + shift + count + GUARD elements filled with the pattern,
    and the view [GUARD + shift, GUARD + shift + count) into it."""
    pat = PATTERN32 if dtype == torch.int32 else PATTERN64
    whole = torch.full((2 * GUARD + shift + count,), pat, dtype=dtype, device=dev)
    return whole, whole[GUARD + shift:GUARD + shift + count]


def guards_intact(whole, shift, count):
    pat = PATTERN32 if whole.dtype == torch.int32 else PATTERN64
    lo, hi = GUARD + shift, GUARD + shift + count
    return bool((whole[:lo] == pat).all()) and bool((whole[hi:] == pat).all())


def unsigned(t):
    a = t.cpu().numpy()
    return a.view(np.uint32 if a.dtype == np.int32 else np.uint64)


@pytest.mark.parametrize("shift", [0, 1, 2, 3])
@pytest.mark.parametrize("name,nm", [("C3", 1), ("C2", 1)])
def test_materialise_stays_inside(ctx, name, nm, shift):
    space = synth.config(name, n_models=nm)
    gs, os_ = ctx.space(space), O.Space(space)
    dev = ctx.torch_device
    n_codes = 625 if name == "C3" else 256
    for first, count in ((0, 7 * n_codes), (3 * n_codes + 17, 40 * n_codes + 5), (n_codes - 1, 2),
                         (5 * n_codes, n_codes), (11, 3 * n_codes - 11)):
        bufs, out = {}, {}
        for k in FIELDS:
            dt = torch.int32 if k == "flags" else torch.int64
            bufs[k], out[k] = guarded(count, dt, shift, dev)
        gs.eval_batch_into(first, count, out)
        ctx.check_status()
        want = os_.eval_range(first, count)
        for k in FIELDS:
            assert guards_intact(bufs[k], shift, count), (k, first, count, shift)
            assert np.array_equal(unsigned(out[k]), want[k]), (k, first, count, shift)


@pytest.mark.parametrize("shift", [0, 1, 3])
def test_compaction_stays_inside(ctx, shift):
    space = synth.config("C3", n_models=1)
    gs, os_ = ctx.space(space), O.Space(space)
    dev = ctx.torch_device
    for filt in (dict(require_flags=O.F_GI | O.F_SC | O.F_CV, cap_bytes=80 * synth.GB),
                 dict(require_flags=0)):
        first, count = 625 * 9 + 123, 625 * 70 + 77
        bufs, out = {}, {}
        for k in FIELDS:
            dt = torch.int32 if k == "flags" else torch.int64
            bufs[k], out[k] = guarded(count, dt, shift, dev)
        idx_whole, idx = guarded(count, torch.int64, shift, dev)
        n_whole, n = guarded(1, torch.int64, 0, dev)
        gs.eval_batch_into(first, count, out, filt, idx, n)
        ctx.check_status()
        want = os_.compact_range(first, count, filt)
        k_surv = int(n.item())
        assert k_surv == len(want["idx"])
        assert guards_intact(idx_whole, shift, count) and guards_intact(n_whole, 0, 1)
        assert np.array_equal(unsigned(idx[:k_surv]), want["idx"])
        for k in FIELDS:
            assert guards_intact(bufs[k], shift, count), (k, shift)
            assert np.array_equal(unsigned(out[k][:k_surv]), want[k]), (k, shift)
            # slots past the survivors are left alone
            pat = PATTERN32 if k == "flags" else PATTERN64
            assert bool((out[k][k_surv:] == pat).all()), (k, shift)


def test_sweep_outputs_stay_inside(ctx, ps):
    space = synth.config("C3", n_models=3)
    gs = ctx.space(space)
    dev = ctx.torch_device
    caps = [80 * synth.GB, 192 * synth.GB]
    for kind, filt, n_caps in ((ps.REDUCE_PARETO, dict(require_flags=7, host_cap=64 * synth.GB), 2),
                               (ps.REDUCE_TOPK, dict(require_flags=7), 1)):
        n_bytes = 3 * n_caps * 64 * 40
        whole = torch.full((n_bytes + 2 * 1024,), 0x5A, dtype=torch.uint8, device=dev)
        cnt_whole = torch.full((3 * n_caps + 64,), PATTERN32, dtype=torch.int32, device=dev)
        gs.sweep_into(filt, caps[:n_caps] if kind == ps.REDUCE_PARETO else caps[1:], kind, 64,
                      whole[1024:1024 + n_bytes], cnt_whole[32:32 + 3 * n_caps])
        ctx.check_status()
        assert bool((whole[:1024] == 0x5A).all()) and bool((whole[1024 + n_bytes:] == 0x5A).all())
        assert bool((cnt_whole[:32] == PATTERN32).all()) and bool((cnt_whole[32 + 3 * n_caps:] == PATTERN32).all())
