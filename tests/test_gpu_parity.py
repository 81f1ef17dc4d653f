"""Bit-exact parity of the CUDA library (through its C interface) with the CPU
oracle on the same seeded inputs.  Everything is an integer or a boolean, so
the tolerance is zero."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2601_02311_b200 import synth

pytestmark = pytest.mark.gpu

FIELDS = ("mem", "comm_paper", "comm_ext", "host", "flags")
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


def both(ctx, space):
    return ctx.space(space), O.Space(space)


def assert_same_arrays(got, want, what=""):
    for k in want:
        if k not in got:
            continue
        g, w = np.asarray(got[k]), np.asarray(want[k])
        assert g.shape == w.shape, (what, k, g.shape, w.shape)
        if not np.array_equal(g, w):
            bad = np.nonzero(g != w)[0]
            raise AssertionError(f"{what} {k}: {len(bad)} mismatches, first at {bad[0]}: "
                                 f"gpu {g[bad[0]]} oracle {w[bad[0]]}")


def assert_same_sweep(got, want, model_slice=slice(None)):
    ge, gc = got
    we, wc = want
    assert np.array_equal(gc[model_slice], wc[model_slice]), (gc[model_slice], wc[model_slice])
    g, w = ge[model_slice], we[model_slice]
    for name in ("mem", "comm", "host", "idx", "flags"):
        if not np.array_equal(g[name], w[name]):
            bad = np.argwhere(g[name] != w[name])[0]
            raise AssertionError(f"{name} differs at {tuple(bad)}: gpu {g[name][tuple(bad)]} "
                                 f"oracle {w[name][tuple(bad)]}")


# ------------------------------------------------------------------ worked example
def test_worked_example_all_outputs(ctx):
    for name in ("C0", "C0b"):
        gs, os_ = both(ctx, synth.config(name))
        assert gs.size == os_.size == 4375
        assert_same_arrays(gs.eval_batch(0, 4375), os_.eval_range(0, 4375), name)


def test_worked_example_printed_values(ctx):
    """The numbers the paper prints, straight from the kernels."""
    gs = ctx.space(synth.config("C0"))
    r = gs.eval_batch(0, 4375)
    n8 = 3 * 625
    assert int(r["mem"][n8 + 0]) == 1_120_000_000_000        # Example 3, data parallel
    assert int(r["mem"][n8 + 32]) == 140_000_000_000         # Example 3, ZeRO-3 at N = 8
    assert int(r["comm_paper"][n8 + 0]) == 245_000_000_000   # Example 4
    assert int(r["comm_paper"][n8 + 32]) == 367_500_000_000  # Example 4
    for ni in range(1, 7):
        b = ni * 625
        assert 2 * int(r["comm_paper"][b + 32]) == 3 * int(r["comm_paper"][b + 0])


# ------------------------------------------------------------------ materialise
@pytest.mark.parametrize("name,n_models", [("C1", 6), ("C2", 2), ("C3", 1)])
def test_materialise_whole_small_space(ctx, name, n_models):
    gs, os_ = both(ctx, synth.config(name, n_models=n_models))
    n = gs.size
    assert n == os_.size
    assert_same_arrays(gs.eval_batch(0, n), os_.eval_range(0, n), name)


def test_materialise_ragged_windows(ctx):
    """Windows that start and end inside groups, one shorter than a group, one
    of a single point, one empty, one ending at the last point of the space."""
    gs, os_ = both(ctx, synth.config("C2", n_models=3))
    n = gs.size
    for first, count in [(1, 77), (255, 2), (256 * 5 + 13, 256 * 9 + 200), (n - 1000, 1000),
                         (n - 1, 1), (12345, 0), (n, 0), (100_000, 300_001)]:
        got = gs.eval_batch(first, count)
        want = os_.eval_range(first, count)
        assert_same_arrays(got, want, f"window {first}+{count}")


def test_materialise_subset_of_outputs(ctx):
    gs, os_ = both(ctx, synth.config("C1", n_models=2))
    got = gs.eval_batch(500, 20000, fields=("mem", "flags"))
    want = os_.eval_range(500, 20000)
    assert set(got) == {"mem", "flags"}
    assert_same_arrays(got, want)


def test_awkward_device_counts_and_mode_mask(ctx):
    """N that are primes or have repeated factors, T and K not powers of two,
    three allowed modes (27 + 54 = 81 codes per group)."""
    space = synth.ragged_space(21)
    gs, os_ = both(ctx, space)
    n = gs.size
    assert n == os_.size
    assert_same_arrays(gs.eval_batch(0, n), os_.eval_range(0, n), "ragged")
    for idx in list(range(0, n, 997)) + [n - 1]:
        assert gs.decode(idx) == os_.decode(idx)


def test_single_mode_space(ctx):
    """mode_mask with one bit: one point per group."""
    space = synth.ragged_space(5, n_models=2)
    space["mode_mask"] = 0b00100
    gs, os_ = both(ctx, space)
    n = gs.size
    assert_same_arrays(gs.eval_batch(0, n), os_.eval_range(0, n), "single mode")


# ------------------------------------------------------------------ compaction
@pytest.mark.parametrize("cap_gb,require,host_cap", [(80, VALID, O.NO_LIMIT), (192, O.F_GI | O.F_SC, 10 ** 10),
                                                     (10 ** 6, 0, O.NO_LIMIT), (0, 0, O.NO_LIMIT)])
def test_compaction_in_index_order(ctx, cap_gb, require, host_cap):
    gs, os_ = both(ctx, synth.config("C3", n_models=2))
    first, count = 4321, 700_001
    filt = dict(cap_bytes=cap_gb * synth.GB, require_flags=require, host_cap=host_cap)
    got = gs.compact(first, count, filt)
    want = os_.compact_range(first, count, filt)
    assert len(got["idx"]) == len(want["idx"])
    assert_same_arrays(got, want, "compaction")


def test_compaction_c2_under_80gb(ctx):
    gs, os_ = both(ctx, synth.config("C2", n_models=4))
    n = gs.size
    filt = dict(cap_bytes=80 * synth.GB, require_flags=VALID)
    got = gs.compact(0, n, filt)
    want = os_.compact_range(0, n, filt)
    assert_same_arrays(got, want, "C2 compaction")
    assert np.all(got["flags"] & O.F_FEASIBLE)


# ------------------------------------------------------------------ sweeps
@pytest.mark.parametrize("comm_kind", [O.COMM_PAPER, O.COMM_PAPER_PLUS_EXT])
@pytest.mark.parametrize("host_cap", [0, 16 * synth.GB, O.NO_LIMIT])
def test_pareto_c3_sample(ctx, ps, comm_kind, host_cap):
    space = synth.config("C3", n_models=5)
    gs, os_ = both(ctx, space)
    filt = dict(require_flags=VALID, comm_kind=comm_kind, host_cap=host_cap)
    caps = [80 * synth.GB, 192 * synth.GB]
    got = gs.sweep(filt, caps, ps.REDUCE_PARETO, 64)
    want = os_.sweep(filt, caps, O.KIND_PARETO, 64, n_threads=8)
    assert_same_sweep(got, want)


@pytest.mark.parametrize("k,host_cap", [(64, O.NO_LIMIT), (7, 16 * synth.GB)])
def test_topk_over_a_table_of_many_models(ctx, ps, k, host_cap):
    """Enough models for two waves of the small top-k blocks (2 x 148 x 9 = 2664): the sweep then
    runs in blocks of two warps.  Also with a budget that the same table does not take that
    path with (skipping allowed), and with a capacity beyond 2^53 (the general kernels)."""
    space = synth.config("C1", n_models=2700)
    gs, os_ = both(ctx, space)
    caps = [40 * synth.GB, 192 * synth.GB]
    for filt in (dict(require_flags=VALID, host_cap=host_cap),
                 dict(require_flags=VALID, host_cap=host_cap, skip_rejected=1)):
        got = gs.sweep(filt, caps, ps.REDUCE_TOPK, k)
        want = os_.sweep({f: v for f, v in filt.items() if f != "skip_rejected"}, caps, O.KIND_TOPK, k, n_threads=8)
        assert_same_sweep(got, want)
    big = [1 << 60]
    filt = dict(require_flags=VALID, host_cap=host_cap)
    assert_same_sweep(gs.sweep(filt, big, ps.REDUCE_TOPK, k), os_.sweep(filt, big, O.KIND_TOPK, k, n_threads=8))


def test_sweeps_after_the_model_table_is_replaced(ctx, ps):
    """ps_space_set_models: the records, and the order in which the sweeps' blocks take the
    models, follow the new table (the old table's models reversed, then shapes of another
    seed: another order of expected work each time)."""
    space = synth.config("C3", n_models=24)
    gs = ctx.space(space)
    filt = dict(require_flags=VALID, host_cap=64 * synth.GB)
    caps = [80 * synth.GB, 192 * synth.GB]
    other = synth.config("C4", n_models=24)["models"]
    for models in (space["models"][::-1].copy(), other, space["models"]):
        gs.set_models(models)
        os_ = O.Space(dict(space, models=models))
        assert_same_sweep(gs.sweep(filt, caps, ps.REDUCE_PARETO, 64), os_.sweep(filt, caps, O.KIND_PARETO, 64, n_threads=8))
        assert_same_sweep(gs.sweep(dict(require_flags=VALID), caps[1:], ps.REDUCE_TOPK, 64),
                          os_.sweep(dict(require_flags=VALID), caps[1:], O.KIND_TOPK, 64, n_threads=8))
        first = 5 * gs.points_per_model + 777
        assert_same_arrays(gs.eval_batch(first, 30_000), os_.eval_range(first, 30_000), "window")


def test_pareto_many_caps_unsorted_and_truncated(ctx, ps):
    """Capacities in arbitrary order; an output shorter than the frontier still
    gets the true length in counts."""
    space = synth.config("C3", n_models=3)
    gs, os_ = both(ctx, space)
    filt = dict(require_flags=VALID, host_cap=0)
    caps = [192 * synth.GB, 8 * synth.GB, 10 ** 15, 1, 40 * synth.GB]
    got = gs.sweep(filt, caps, ps.REDUCE_PARETO, 3)
    want = os_.sweep(filt, caps, O.KIND_PARETO, 3, n_threads=8)
    assert want[1].max() > 3
    assert_same_sweep(got, want)
    assert gs.last_sweep_status == ps.E_TRUNCATED          # the notice; the next call is not blocked
    got = gs.sweep(filt, caps, ps.REDUCE_PARETO, 64)
    assert gs.last_sweep_status == ps.OK
    assert_same_sweep(got, os_.sweep(filt, caps, O.KIND_PARETO, 64, n_threads=8))


def test_pareto_without_requirements(ctx, ps):
    """No required flags: invalid compositions compete too, ties are everywhere."""
    space = synth.config("C2", n_models=2)
    gs, os_ = both(ctx, space)
    filt = dict(require_flags=0, comm_kind=O.COMM_PAPER)
    caps = [192 * synth.GB]
    assert_same_sweep(gs.sweep(filt, caps, ps.REDUCE_PARETO, 128),
                      os_.sweep(filt, caps, O.KIND_PARETO, 128, n_threads=8))


def test_pareto_worked_example_ties(ctx, ps):
    """Activations excluded: the 625 codes collapse to 125 results, so the
    smallest-index rule decides every entry."""
    gs, os_ = both(ctx, synth.config("C0"))
    for comm_kind in (0, 1):
        filt = dict(require_flags=O.F_GI | O.F_SC, comm_kind=comm_kind, host_cap=0)
        caps = [80 * synth.GB, 2000 * synth.GB]
        assert_same_sweep(gs.sweep(filt, caps, ps.REDUCE_PARETO, 64),
                          os_.sweep(filt, caps, O.KIND_PARETO, 64))


def test_pareto_ragged_space(ctx, ps):
    space = synth.ragged_space(33, n_models=4)
    gs, os_ = both(ctx, space)
    rec = O.model_record(space["models"][0:1])
    caps = [16 * rec["P"] // 7, 16 * rec["P"]]
    for require in (VALID, O.F_GI | O.F_SC, 0):
        filt = dict(require_flags=require, host_cap=rec["P"])
        assert_same_sweep(gs.sweep(filt, caps, ps.REDUCE_PARETO, 96),
                          os_.sweep(filt, caps, O.KIND_PARETO, 96, n_threads=4))


@pytest.mark.parametrize("k", [64, 7, 33])
def test_topk_c4_sample(ctx, ps, k):
    space = synth.config("C4", n_models=3)
    gs, os_ = both(ctx, space)
    filt = dict(require_flags=VALID)
    caps = [192 * synth.GB]
    assert_same_sweep(gs.sweep(filt, caps, ps.REDUCE_TOPK, k),
                      os_.sweep(filt, caps, O.KIND_TOPK, k, n_threads=8))


def test_topk_two_caps_host_cap_and_few_survivors(ctx, ps):
    space = synth.ragged_space(8, n_models=3)
    gs, os_ = both(ctx, space)
    rec = O.model_record(space["models"][0:1])
    filt = dict(require_flags=VALID, host_cap=0, comm_kind=O.COMM_PAPER)
    caps = [rec["P"], 20 * rec["P"]]
    got = gs.sweep(filt, caps, ps.REDUCE_TOPK, 64)
    want = os_.sweep(filt, caps, O.KIND_TOPK, 64, n_threads=4)
    assert want[1].min() < 64        # some (model, cap) has fewer survivors than slots
    assert_same_sweep(got, want)


def test_sweeps_are_deterministic(ctx, ps):
    space = synth.config("C3", n_models=4)
    gs = ctx.space(space)
    filt = dict(require_flags=VALID, host_cap=16 * synth.GB)
    a = gs.sweep(filt, [80 * synth.GB, 192 * synth.GB], ps.REDUCE_PARETO, 64)
    b = gs.sweep(filt, [80 * synth.GB, 192 * synth.GB], ps.REDUCE_PARETO, 64)
    assert a[0].tobytes() == b[0].tobytes() and a[1].tobytes() == b[1].tobytes()


# ------------------------------------------------------------------ single compositions
def test_check_composition_matches_oracle(ctx):
    rng = np.random.default_rng(0)
    shapes = synth.zoo(6, 77)
    for trial in range(200):
        shape = shapes[trial % 6:trial % 6 + 1]
        T = int(rng.choice([1, 2, 3, 4, 8, 16]))
        K = int(rng.choice([1, 2, 3, 5, 8]))
        D = int(rng.choice([1, 2, 7, 64]))
        N = T * K * D if trial % 5 else T * K * D + 1
        code_tp = int(rng.choice([156, 31, 0, 32, 624]))
        code_pp = int(rng.choice([31, 31, 156, 5]))
        code_dp = int(rng.integers(0, 625))
        args = (N, T, K, D, code_tp, code_pp, code_dp)
        kw = dict(act_variant=trial % 2, cap_bytes=80 * synth.GB, comm_kind=trial % 2)
        assert ctx.check_composition(shape, *args, **kw) == O.check_composition(shape, *args, **kw)


def test_decode_matches_oracle(ctx):
    space = synth.config("C4", n_models=3)
    gs, os_ = both(ctx, space)
    rng = np.random.default_rng(1)
    for idx in rng.integers(0, gs.size, 300):
        assert gs.decode(int(idx)) == os_.decode(int(idx))


# ------------------------------------------------------------------ errors
def test_argument_errors(ctx, ps):
    space = synth.config("C1", n_models=1)
    gs = ctx.space(space)
    with pytest.raises(ps.PsError) as e:
        gs.eval_batch(gs.size - 5, 6)
    assert e.value.code == ps.E_BADINDEX
    bad = dict(space)
    bad["mode_mask"] = 0
    with pytest.raises(ps.PsError) as e:
        ctx.space(bad)
    assert e.value.code == ps.E_RANGE
    huge = synth.zoo(1, 3)
    huge["hidden"] = 1 << 20
    bad = dict(space, models=huge)
    with pytest.raises(ps.PsError) as e:
        ctx.space(bad)
    assert e.value.code == ps.E_RANGE
    with pytest.raises(ps.PsError) as e:
        gs.sweep(dict(), [1], ps.REDUCE_TOPK, ps.TOPK_MAX + 1)
    assert e.value.code == ps.E_RANGE
    assert ctx.status() == ps.OK


# ------------------------------------------------------------------ Algorithm 1
def to_query_records(ps, q):
    rec = np.zeros(len(q), dtype=ps.SELECT_QUERY_DTYPE)
    rec["param_elems"], rec["layer_elems"], rec["device_bytes"] = q[:, 0], q[:, 1], q[:, 2]
    rec["n_devices"] = q[:, 3]
    rec["w_param"], rec["w_grad"], rec["w_opt"], rec["fast_interconnect"] = q[:, 4], q[:, 5], q[:, 6], q[:, 7]
    return rec


@pytest.mark.parametrize("n,tp_degree,headroom", [(100_003, 8, (7, 10)), (1, 4, (1, 2)), (0, 8, (7, 10)),
                                                   (4097, 6, (9, 10))])
def test_select_matches_oracle(ctx, ps, n, tp_degree, headroom):
    q = synth.select_queries(n, seed=n + tp_degree)
    got = ctx.select(to_query_records(ps, q), headroom=headroom, tp_degree=tp_degree)
    want = O.select(q, headroom=headroom, tp_degree=tp_degree)
    assert len(got) == n
    for j, name in enumerate(("mem", "comm", "branch", "T", "code_dp", "flags")):
        assert np.array_equal(got[name].astype(np.uint64), want[:, j]), name
    if n > 1000:
        assert set(np.unique(want[:, 2]).tolist()) == {0, 1, 2, 3}     # every branch is exercised


# ------------------------------------------------------------------ extremes
def extreme_space():
    """Shapes at the edges of the supported ranges (2^46 parameters, 16-byte
    widths, the largest boundary tensor, the largest stored activations) and
    device counts up to 2^24 with non-trivial T and K."""
    m = synth.zoo(4, 99)
    m["param_elems_override"][0] = 1 << 46
    m["w_param"][0], m["w_grad"][0], m["w_opt"][0], m["w_act"][0] = 16, 16, 16, 16
    m["layers"][1], m["hidden"][1], m["heads"][1] = 1024, 1 << 16, 1 << 16
    m["param_elems_override"][1] = (1 << 46) - 12345
    m["seq"][1], m["micro_batch"][1], m["vocab"][1] = 1 << 10, 1 << 4, 1 << 24      # S b H = 2^30
    m["seq"][2], m["micro_batch"][2], m["hidden"][2], m["heads"][2] = 1 << 17, 8, 1 << 16, 1 << 13
    m["layers"][2] = 32                                     # stored activations 2^57.3 bytes, S b H = 2^36
    m["layers"][3], m["hidden"][3], m["heads"][3], m["vocab"][3] = 1, 1, 1, 1
    m["seq"][3], m["micro_batch"][3] = 1, 1
    return dict(models=m, n_values=np.asarray([1, 1 << 24, 3 * (1 << 20), 16777213], dtype=np.uint32),
                t_enum_max=64, k_enum_max=1 << 24, tp_max_valid=8, n_act_variants=2, n_tpa_variants=2,
                mode_mask=0x1F, tp_coll_per_layer=64)


def test_extreme_shapes_and_device_counts(ctx, ps):
    space = extreme_space()
    gs, os_ = both(ctx, space)
    n = gs.size
    assert n == os_.size and n < 6_000_000
    got, want = gs.eval_batch(0, n), os_.eval_range(0, n)
    assert_same_arrays(got, want, "extreme")
    assert int(want["mem"].max()) < 1 << 62 and int((want["comm_paper"] + want["comm_ext"]).max()) < 1 << 63
    filt = dict(require_flags=O.F_GI | O.F_SC, host_cap=1 << 40)
    caps = [1 << 30, 1 << 45]
    assert_same_sweep(gs.sweep(filt, caps, ps.REDUCE_PARETO, 128), os_.sweep(filt, caps, O.KIND_PARETO, 128, n_threads=4))
    assert_same_sweep(gs.sweep(filt, caps, ps.REDUCE_TOPK, 64), os_.sweep(filt, caps, O.KIND_TOPK, 64, n_threads=4))


def test_smallest_possible_space(ctx, ps):
    """One model, one device, one mode, no variants: a single point."""
    m = synth.zoo(1, 1)
    space = dict(models=m, n_values=np.asarray([1], dtype=np.uint32), t_enum_max=1, k_enum_max=1,
                 tp_max_valid=8, n_act_variants=1, n_tpa_variants=1, mode_mask=0b00001, tp_coll_per_layer=4)
    gs, os_ = both(ctx, space)
    assert gs.size == os_.size == 1
    assert_same_arrays(gs.eval_batch(0, 1), os_.eval_range(0, 1))
    filt = dict(require_flags=VALID)
    for kind_g, kind_o in ((ps.REDUCE_PARETO, O.KIND_PARETO), (ps.REDUCE_TOPK, O.KIND_TOPK)):
        assert_same_sweep(gs.sweep(filt, [O.NO_LIMIT], kind_g, 4), os_.sweep(filt, [O.NO_LIMIT], kind_o, 4))


@pytest.mark.parametrize("cap", [(1 << 53) - 2, (1 << 53) - 1, 1 << 60])
def test_sweeps_around_the_exact_double_limit(ctx, ps, cap):
    """A power-of-two space runs kernels compiled for byte counts below 2^53 when
    the capacity allows it and the general ones otherwise: same results."""
    space = synth.config("C3", n_models=2)
    gs, os_ = both(ctx, space)
    caps = [192 * synth.GB, cap]
    filt = dict(require_flags=VALID, host_cap=64 * synth.GB)
    assert_same_sweep(gs.sweep(filt, caps, ps.REDUCE_PARETO, 64),
                      os_.sweep(filt, caps, O.KIND_PARETO, 64, n_threads=8))
    filt = dict(require_flags=VALID)
    assert_same_sweep(gs.sweep(filt, [cap], ps.REDUCE_TOPK, 64),
                      os_.sweep(filt, [cap], O.KIND_TOPK, 64, n_threads=8))



@pytest.mark.gpu
@pytest.mark.parametrize("tp_degree", [1, 2, 63, 64, 65, 100, 4096])
def test_select_divisor_search_paths(ctx, ps, tp_degree):
    """The largest divisor of N not above tp_degree: degrees up to 64 go through the host's
    tables, larger ones and device counts above 2^24 through the plain search; the extremes of
    the documented ranges (P = 2^46, N = 2^24, a layer as large as the model) go through the
    reciprocal divisions."""
    q = synth.select_queries(3000, seed=900 + tp_degree)
    q[:, 7] = 1                                   # fast interconnect: the tensor-parallel branch is open
    q[::3, 2] = 1 << 30                           # small devices: many queries reach that branch
    q[::3, 1] = q[::3, 0] // 3                    # with a layer too large for a device
    odd = np.arange(len(q)) % 5 == 0
    q[odd, 3] = (np.arange(odd.sum()) * 7919 + 1) % ((1 << 24) - 1) + 1     # any count up to 2^24
    q[1, 3] = 1 << 24
    q[2, 3] = (1 << 24) - 1
    q[4, 0], q[4, 1], q[4, 3] = 1 << 46, 1 << 46, 1 << 24
    q[5, 0], q[5, 1], q[5, 3] = 1 << 46, (1 << 46) - 1, 3 * 5 * 7 * 11 * 13 * 17
    got = ctx.select(to_query_records(ps, q), tp_degree=tp_degree)
    want = O.select(q, tp_degree=tp_degree)
    for j, name in enumerate(("mem", "comm", "branch", "T", "code_dp", "flags")):
        assert np.array_equal(got[name].astype(np.uint64), want[:, j]), name
    assert (want[:, 2] == 2).sum() > 100          # the branch is exercised
    if tp_degree > 2:
        assert len(np.unique(want[want[:, 2] == 2, 3])) > 2      # with several degrees

@pytest.mark.parametrize("host_cap", [0, 8 * synth.GB, 200 * synth.GB])
def test_topk_with_a_host_budget_on_a_power_of_two_space(ctx, ps, host_cap):
    """The top-k kernels compiled for a host budget, in the power-of-two case."""
    space = synth.config("C4", n_models=2)
    gs, os_ = both(ctx, space)
    for comm_kind in (O.COMM_PAPER, O.COMM_PAPER_PLUS_EXT):
        filt = dict(require_flags=VALID, host_cap=host_cap, comm_kind=comm_kind)
        caps = [80 * synth.GB]
        assert_same_sweep(gs.sweep(filt, caps, ps.REDUCE_TOPK, 64),
                          os_.sweep(filt, caps, O.KIND_TOPK, 64, n_threads=8))


def long_frontier_space():
    """One model, 64 neighbouring device counts, no model axes: every device count
    contributes two entries to the frontier and the single-device point one more --
    129 entries, one more than the sweep's fast lists hold."""
    models = synth.zoo(1, 5, max_layers=160, max_hidden_mult=256)
    models["w_param"], models["w_grad"], models["w_opt"] = 2, 1, 2
    return synth._space(models, list(range(100, 164)), t_enum_max=1, k_enum_max=1, n_act=1, n_tpa=1,
                        mode_mask=0b1111)


def test_pareto_frontier_longer_than_the_fast_lists(ctx, ps):
    """A frontier beyond 128 entries takes the slow exact path and is still the oracle's."""
    space = long_frontier_space()
    gs, os_ = both(ctx, space)
    filt = dict(require_flags=O.F_GI | O.F_SC, host_cap=0)
    caps = [1 << 62, 30 * synth.GB]
    want = os_.sweep(filt, caps, O.KIND_PARETO, 192, n_threads=8)
    assert want[1][0, 0] > 128
    assert_same_sweep(gs.sweep(filt, caps, ps.REDUCE_PARETO, 192), want)
    assert gs.last_sweep_status == ps.OK
    # rows shorter than the frontier: its head, the true count, and the notice
    assert_same_sweep(gs.sweep(filt, caps, ps.REDUCE_PARETO, 16), os_.sweep(filt, caps, O.KIND_PARETO, 16, n_threads=8))
    assert gs.last_sweep_status == ps.E_TRUNCATED
    # the same model among ordinary ones: only it takes the slow path
    mixed = dict(space)
    mixed["models"] = np.concatenate([synth.zoo(2, 6), space["models"], synth.zoo(2, 7)])
    gs, os_ = both(ctx, mixed)
    assert_same_sweep(gs.sweep(filt, caps, ps.REDUCE_PARETO, 192), os_.sweep(filt, caps, O.KIND_PARETO, 192, n_threads=8))


def test_select_compare_matches_oracle(ctx, ps):
    """Algorithm 1's choice beside the frontier, for every model of a single-N composition space."""
    import torch
    for n_value, mask in ((64, 0x1F), (512, 0b10111)):
        space = synth.config("C3", n_models=40)
        space["n_values"] = np.array([n_value], dtype=np.uint32)
        space["mode_mask"] = mask
        gs, os_ = both(ctx, space)
        filt = dict(require_flags=VALID, host_cap=64 * synth.GB)
        caps = [40 * synth.GB, 80 * synth.GB]
        d_out, d_counts = gs.alloc_sweep(len(caps), 24)
        gs.sweep_into(filt, caps, ps.REDUCE_PARETO, 24, d_out, d_counts)
        oe, oc = os_.sweep(filt, caps, O.KIND_PARETO, 24, n_threads=8)
        for cap_index in (0, 1):
            got = gs.select_compare(0, caps[cap_index], filt, d_out, d_counts, len(caps), cap_index, 24)
            want = O.select_compare(os_, 0, caps[cap_index], filt, oe, oc, cap_index)
            names = ("alg_mem", "alg_comm", "alg_idx", "best_mem", "best_comm", "best_idx", "branch", "T",
                     "code_dp", "alg_flags", "status")
            for k, name in enumerate(names):
                assert np.array_equal(got[name].astype(np.uint64), want[:, k]), (n_value, cap_index, name)
        assert len(set(got["status"].tolist())) > 1            # more than one outcome occurs
    ctx.check_status()


def test_sweeps_that_skip_rejected_factorisations_give_the_same_tables(ctx, ps):
    """skip_rejected leaves out the factorisations the required composition flags reject at sight:
    less work, identical results (and identical survivor counts)."""
    for space in (synth.config("C3", n_models=5), synth.ragged_space(3, n_models=2)):
        gs, os_ = both(ctx, space)
        caps = [80 * synth.GB, 192 * synth.GB]
        for req in (VALID, O.F_GI | O.F_SC | O.F_T_HEADS):
            filt = dict(require_flags=req, host_cap=64 * synth.GB)
            want = os_.sweep(filt, caps, O.KIND_PARETO, 64, n_threads=8)
            assert_same_sweep(gs.sweep(dict(filt, skip_rejected=1), caps, ps.REDUCE_PARETO, 64), want)
            filt = dict(require_flags=req)
            want = os_.sweep(filt, caps[1:], O.KIND_TOPK, 64, n_threads=8)
            assert_same_sweep(gs.sweep(dict(filt, skip_rejected=1), caps[1:], ps.REDUCE_TOPK, 64), want)
