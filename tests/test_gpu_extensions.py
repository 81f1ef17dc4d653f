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


# ------------------------------------------------------------ k-way replication
@pytest.mark.parametrize("k,sstar_units,g", [(2, 1, 1), (4, 2, 3), (1 << 12, 1, 1), (6, 1, 2)])
def test_k_way_replication_materialise_and_compaction(ctx, k, sstar_units, g):
    """Every shard held k times (Section 1's "k-way replication"): all five outputs of every
    point, and the compaction, on power-of-two spaces and on ragged device counts (where k
    need not divide D)."""
    spaces = [synth.config("C0b"), synth.config("C1", n_models=3), synth.config("C3", n_models=1),
              synth.ragged_space(4, n_models=2)]
    for base in spaces:
        space = dict(ext(base, sstar_units, g), replication_k=k)
        gs, os_ = ctx.space(space), O.Space(space)
        n = min(gs.size, 400_000)
        first = (gs.size - n) // 3
        same(gs.eval_batch(first, n), os_.eval_range(first, n))
        for filt in (dict(require_flags=O.F_GI | O.F_SC, cap_bytes=80 * synth.GB, host_cap=500 * synth.GB),
                     dict(require_flags=O.F_PAPER_PRICED | O.F_GI, cap_bytes=192 * synth.GB)):
            same(gs.compact(first, n, filt), os_.compact_range(first, n, filt))
    ctx.check_status()


@pytest.mark.parametrize("k", [2, 8, 3])
def test_k_way_replication_sweeps(ctx, ps, k):
    for base in (synth.config("C3", n_models=4), synth.ragged_space(9, n_models=2)):
        space = dict(base, replication_k=k)
        gs, os_ = ctx.space(space), O.Space(space)
        for comm_kind in (O.COMM_PAPER, O.COMM_PAPER_PLUS_EXT):
            filt = dict(require_flags=O.F_GI | O.F_SC, comm_kind=comm_kind, host_cap=64 * synth.GB)
            caps = [80 * synth.GB, 192 * synth.GB]
            ge, gc = gs.sweep(filt, caps, ps.REDUCE_PARETO, 64)
            oe, oc = os_.sweep(filt, caps, O.KIND_PARETO, 64, n_threads=8)
            assert ge.tobytes() == oe.tobytes() and gc.tolist() == oc.tolist()
            filt = dict(require_flags=VALID, comm_kind=comm_kind)
            ge, gc = gs.sweep(filt, caps[1:], ps.REDUCE_TOPK, 64)
            oe, oc = os_.sweep(filt, caps[1:], O.KIND_TOPK, 64, n_threads=8)
            assert ge.tobytes() == oe.tobytes() and gc.tolist() == oc.tolist()
    ctx.check_status()


def test_k_way_replication_reaches_the_kernels(ctx):
    """ZeRO-3 at N = 8 in the worked example with two copies of every shard: 16P/4 bytes."""
    gs = ctx.space(dict(synth.config("C0"), replication_k=2))
    r = gs.eval_batch(3 * 625 + 32, 1)
    P = 70_000_000_000
    assert int(r["mem"][0]) == 16 * P // 4
    assert int(r["comm_paper"][0]) == (3 * 2 * P // 4 + 2 * (2 * P // 4) // 2) + 2 * (3 * 2 * P // 4)
