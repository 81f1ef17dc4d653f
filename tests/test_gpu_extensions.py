"""Bit-exact parity of the CUDA library with the oracle when a gathered state
holds two unit buffers (proof of Theorem 1, case S*) and a step runs several
micro-batches (gradient accumulation, "Limitations"): materialise, compaction,
both sweeps, and the range checks of the two fields."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2601_02311_b200 import synth

pytestmark = pytest.mark.gpu

VALID = O.F_GI | O.F_SC | O.F_CV


@pytest.fixture(scope="module")
def ps():
    import paper_2601_02311_b200.ps as ps_mod
    return ps_mod


@pytest.fixture(scope="module")
def ctx(ps):
    c = ps.Context(0)
    yield c
    c.close()


def ext(space, sstar_units, g):
    s = dict(space)
    s["sstar_units"], s["grad_accum_steps"] = sstar_units, g
    return s


def same(got, want):
    for k in want:
        assert np.array_equal(np.asarray(got[k]), np.asarray(want[k])), k


@pytest.mark.parametrize("sstar_units,g", [(2, 1), (1, 4), (2, 64), (0, 0)])
def test_materialise_and_compaction(ctx, sstar_units, g):
    for name, nm in (("C0b", None), ("C1", 3), ("C3", 1)):
        space = ext(synth.config(name, n_models=nm), sstar_units, g)
        gs, os_ = ctx.space(space), O.Space(space)
        n = min(gs.size, 400_000)
        first = (gs.size - n) // 3
        same(gs.eval_batch(first, n), os_.eval_range(first, n))
        filt = dict(require_flags=O.F_GI | O.F_SC, cap_bytes=80 * synth.GB, host_cap=500 * synth.GB)
        same(gs.compact(first, n, filt), os_.compact_range(first, n, filt))
    ctx.check_status()


def test_values_differ_from_the_plain_space(ctx):
    """The fields reach the kernels: ZeRO-3 at N = 8 in the worked example with
    a unit, two buffers, four micro-batches."""
    gs = ctx.space(ext(synth.config("C0b"), 2, 4))
    r = gs.eval_batch(3 * 625 + 32, 1)
    assert int(r["mem"][0]) == 140_000_000_000 + 2 * 1_610_612_736
    assert int(r["comm_paper"][0]) == 122_500_000_000 + 4 * 245_000_000_000


@pytest.mark.parametrize("sstar_units,g", [(2, 3), (1, 16)])
def test_sweeps(ctx, ps, sstar_units, g):
    space = ext(synth.config("C3", n_models=4), sstar_units, g)
    gs, os_ = ctx.space(space), O.Space(space)
    for comm_kind in (O.COMM_PAPER, O.COMM_PAPER_PLUS_EXT):
        filt = dict(require_flags=VALID, comm_kind=comm_kind, host_cap=64 * synth.GB)
        caps = [80 * synth.GB, 192 * synth.GB]
        ge, gc = gs.sweep(filt, caps, ps.REDUCE_PARETO, 64)
        oe, oc = os_.sweep(filt, caps, O.KIND_PARETO, 64, n_threads=8)
        assert ge.tobytes() == oe.tobytes() and gc.tolist() == oc.tolist()
        filt = dict(require_flags=VALID, comm_kind=comm_kind)
        ge, gc = gs.sweep(filt, caps[1:], ps.REDUCE_TOPK, 64)
        oe, oc = os_.sweep(filt, caps[1:], O.KIND_TOPK, 64, n_threads=8)
        assert ge.tobytes() == oe.tobytes() and gc.tolist() == oc.tolist()
    ctx.check_status()


def test_field_ranges(ctx, ps):
    for bad in (dict(sstar_units=3), dict(grad_accum_steps=65)):
        space = dict(synth.config("C0"))
        space.update(bad)
        with pytest.raises(ps.PsError) as e:
            ctx.space(space)
        assert e.value.code == ps.E_RANGE
