"""Parity at the full sizes of the benchmark configurations, in the launch
configuration bench.py times (whole shape table, same filters and capacities):
the complete top-64 and Pareto tables of every model and 64 windows of 2^20
points against the oracle, bit for bit (marked slow: a few minutes of oracle
time on all host cores), a quicker sampled version of the same, and properties
of the complete outputs that hold at any size."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2601_02311_b200 import synth

pytestmark = pytest.mark.gpu
VALID = O.F_GI | O.F_SC | O.F_CV
GB = synth.GB


@pytest.fixture(scope="module")
def ps():
    import paper_2601_02311_b200.ps as ps_mod
    return ps_mod


@pytest.fixture(scope="module")
def ctx(ps):
    c = ps.Context(0)
    yield c
    c.close()


def check_sweep_properties(entries, counts, caps, ppm, kind_pareto, require):
    nm, nc, me = entries.shape
    for ci, cap in enumerate(caps):
        cnt = counts[:, ci].astype(np.int64)
        assert (cnt <= ppm).all()
        n_emit = np.minimum(cnt, me)
        slot = np.arange(me)[None, :]
        used = slot < n_emit[:, None]
        e = entries[:, ci, :]
        assert (e["mem"][used] <= cap).all()
        assert ((e["flags"][used] & (require | O.F_FEASIBLE)) == (require | O.F_FEASIBLE)).all()
        assert (e["idx"][used] // ppm == np.broadcast_to(np.arange(nm)[:, None], (nm, me))[used]).all()
        # unused slots are zero
        for name in ("mem", "comm", "host", "idx", "flags"):
            assert (e[name][~used] == 0).all()
        both = used[:, 1:] & used[:, :-1]
        if kind_pareto:   # mem strictly up, comm strictly down
            assert (e["mem"][:, 1:][both] > e["mem"][:, :-1][both]).all()
            assert (e["comm"][:, 1:][both] < e["comm"][:, :-1][both]).all()
        else:             # keys (comm, mem, idx) strictly ascending
            c1, c0 = e["comm"][:, 1:][both], e["comm"][:, :-1][both]
            m1, m0 = e["mem"][:, 1:][both], e["mem"][:, :-1][both]
            i1, i0 = e["idx"][:, 1:][both], e["idx"][:, :-1][both]
            assert ((c1 > c0) | ((c1 == c0) & ((m1 > m0) | ((m1 == m0) & (i1 > i0))))).all()


@pytest.mark.parametrize("name,sample", [("C4", (0, 1733, 4095)), ("C3", (5, 512, 1023))])
def test_full_sweeps_sampled_models(ctx, ps, name, sample):
    space = synth.config(name)
    gs, os_ = ctx.space(space), O.Space(space)
    assert gs.size == synth.FULL_SIZE[name]
    ppm = gs.points_per_model
    topk_f = dict(require_flags=VALID)
    par_f = dict(require_flags=VALID, host_cap=64 * GB)
    caps = [80 * GB, 192 * GB]
    te, tc = gs.sweep(topk_f, caps[1:], ps.REDUCE_TOPK, 64)
    pe, pc = gs.sweep(par_f, caps, ps.REDUCE_PARETO, 64)
    check_sweep_properties(te, tc, caps[1:], ppm, False, VALID)
    check_sweep_properties(pe, pc, caps, ppm, True, VALID)
    for m in sample:
        oe, oc = os_.sweep(topk_f, caps[1:], O.KIND_TOPK, 64, model_first=m, model_count=1)
        assert te[m].tobytes() == oe[m].tobytes() and tc[m].tolist() == oc[m].tolist(), m
        oe, oc = os_.sweep(par_f, caps, O.KIND_PARETO, 64, model_first=m, model_count=1)
        assert pe[m].tobytes() == oe[m].tobytes() and pc[m].tolist() == oc[m].tolist(), m
    # the frontier under the tighter capacity is the head of the looser one's
    for m in range(0, gs.n_models, 97):
        big = pe[m, 1, :pc[m, 1]]
        assert np.array_equal(pe[m, 0, :pc[m, 0]], big[big["mem"] <= caps[0]])


@pytest.mark.parametrize("name", ["C4", "C2"])
def test_random_windows_of_the_full_space(ctx, name):
    space = synth.config(name)
    gs, os_ = ctx.space(space), O.Space(space)
    size = gs.size
    rng = np.random.default_rng(12)
    filt = dict(require_flags=VALID, cap_bytes=80 * GB)
    for w in range(64):
        count = 1 << 14
        first = int(rng.integers(0, size - count))
        got, want = gs.eval_batch(first, count), os_.eval_range(first, count)
        for k in want:
            assert np.array_equal(got[k], want[k]), (w, first, k)
        if w % 8 == 0:
            got, want = gs.compact(first, count, filt), os_.compact_range(first, count, filt)
            for k in want:
                assert np.array_equal(got[k], want[k]), (w, first, k)
    # the very end of the space
    got, want = gs.eval_batch(size - 1000, 1000), os_.eval_range(size - 1000, 1000)
    for k in want:
        assert np.array_equal(got[k], want[k])


@pytest.mark.slow
@pytest.mark.parametrize("name", ["C3", "C4"])
def test_full_sweeps_every_model(ctx, ps, name):
    """Every model's top-64 list and both capacities' Pareto frontiers, whole tables."""
    space = synth.config(name)
    gs, os_ = ctx.space(space), O.Space(space)
    threads = O.hardware_threads()
    topk_f = dict(require_flags=VALID)
    par_f = dict(require_flags=VALID, host_cap=64 * GB)
    caps = [80 * GB, 192 * GB]
    te, tc = gs.sweep(topk_f, caps[1:], ps.REDUCE_TOPK, 64)
    oe, oc = os_.sweep(topk_f, caps[1:], O.KIND_TOPK, 64, n_threads=threads)
    assert np.array_equal(tc, oc)
    assert te.tobytes() == oe.tobytes()
    del oe
    pe, pc = gs.sweep(par_f, caps, ps.REDUCE_PARETO, 64)
    oe, oc = os_.sweep(par_f, caps, O.KIND_PARETO, 64, n_threads=threads)
    assert np.array_equal(pc, oc)
    assert pe.tobytes() == oe.tobytes()


@pytest.mark.slow
@pytest.mark.parametrize("name", ["C4", "C2"])
def test_64_windows_of_a_million_points(ctx, name):
    """ps_eval_batch on 64 pseudo-randomly placed windows of 2^20 points: every output word."""
    import concurrent.futures as cf
    space = synth.config(name)
    gs, os_ = ctx.space(space), O.Space(space)
    size, count = gs.size, 1 << 20
    rng = np.random.default_rng(2020)
    firsts = [int(rng.integers(0, size - count)) for _ in range(64)]
    filt = dict(require_flags=VALID, cap_bytes=80 * GB)
    # the oracle walks a window on one core (its C code releases the interpreter lock): windows side by side
    with cf.ThreadPoolExecutor(max_workers=O.hardware_threads()) as pool:
        wants = list(pool.map(lambda f: os_.eval_range(f, count), firsts))
        compact_wants = list(pool.map(lambda f: os_.compact_range(f, count, filt), firsts[::8]))
    for w, first in enumerate(firsts):
        got = gs.eval_batch(first, count)
        for k in wants[w]:
            assert np.array_equal(got[k], wants[w][k]), (w, first, k)
    for w, first in enumerate(firsts[::8]):
        got = gs.compact(first, count, filt)
        for k in compact_wants[w]:
            assert np.array_equal(got[k], compact_wants[w][k]), (w, first, k)
