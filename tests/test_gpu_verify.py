"""ps_verify_batch (the verification protocol of Section 7.1 as a batched GPU
run) against its oracle, the CPU simulator oracle/sim/placement_sim.py, on the
same problems: the match bit and the three byte counts of all 625 placements on
1-4 logical devices must be equal, the trajectories equal to 1e-12 -- and both
must agree with the closed-form rules (Theorems 1-4) as the library evaluates
them."""
import numpy as np
import pytest

from oracle import oracle as O
from oracle.sim import placement_sim as sim

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ps():
    import paper_2601_02311_b200.ps as ps_mod
    return ps_mod


@pytest.fixture(scope="module")
def ctx(ps):
    c = ps.Context(0)
    yield c
    c.close()


def problems(units, h, b, accum, seed):
    """One problem per device count; returns (data, offsets[D], per-D (theta0, xs, ys))."""
    chunks, offsets, parts, at = [], {}, {}, 0
    for D in (1, 2, 3, 4):
        theta0, xs, ys = sim.make_problem(units, h, b, D, seed + D, accum)
        flat = np.concatenate([theta0] + [x.reshape(-1) for xj in xs for x in xj] +
                              [y.reshape(-1) for yj in ys for y in yj])
        offsets[D], parts[D] = at, (theta0, xs, ys)
        chunks.append(flat)
        at += len(flat)
    return np.concatenate(chunks), offsets, parts


@pytest.mark.parametrize("units,h,b,accum,nbuf", [(3, 5, 2, 1, 1), (2, 7, 3, 1, 1), (3, 5, 2, 3, 2)])
def test_verifier_equals_simulator_and_rules(ctx, ps, units, h, b, accum, nbuf):
    data, offsets, parts = problems(units, h, b, accum, seed=100 * units + h)
    cases = np.zeros(625 * 4, dtype=ps.VERIFY_CASE_DTYPE)
    k = 0
    for D in (1, 2, 3, 4):
        for code in range(625):
            cases[k] = (code, D, offsets[D])
            k += 1
    shape = dict(units=units, h=h, b=b, accum=accum, steps=3, gather_buffers=nbuf)
    got, theta = ctx.verify_batch(shape, cases, data, want_theta=True)
    rec = dict(P=units * h, unit=h, A0=units * b * h, A1=units * b * h, UA0=b * h, UA1=b * h, Sbh=b * h,
               L=units, heads=1, w_theta=sim.W_THETA, w_omega=sim.W_OMEGA, w_grad=sim.W_GRAD, w_act=2)
    n_match = 0
    for k, c in enumerate(cases):
        D, code = int(c["D"]), int(c["code"])
        theta0, xs, ys = parts[D]
        want = sim.simulate_problem(units, h, b, D, code, theta0, xs, ys, steps=3, gather_buffers=nbuf)
        g = got[k]
        assert bool(g["match"]) == want["match"], (code, D)
        assert (int(g["mem"]), int(g["comm"]), int(g["host"])) == (want["mem"], want["comm"], want["host"]), (code, D)
        if want["theta"] is not None:
            assert np.allclose(theta[k], want["theta"], rtol=1e-12, atol=1e-14), (code, D)
        # the rules, evaluated by the oracle: valid exactly when the run matched, and then the same bytes
        r = O.eval_record(rec, D, 1, 1, D, 0, 0, code, sstar_units=nbuf if units >= 2 else 1,
                          grad_accum_steps=accum)
        valid = (r["flags"] & (O.F_GI | O.F_SC)) == (O.F_GI | O.F_SC)
        assert valid == bool(g["match"]), (code, D)
        if valid:
            n_match += 1
            assert int(g["mem"]) == r["mem"] and int(g["comm"]) == r["comm_paper"] + r["comm_ext"], (code, D)
            assert int(g["host"]) == r["host"], (code, D)
    assert n_match == 475 + 3 * 171


def test_verifier_reports_bad_cases_without_touching_memory(ctx, ps):
    data, offsets, _ = problems(2, 4, 2, 1, seed=3)
    cases = np.zeros(4, dtype=ps.VERIFY_CASE_DTYPE)
    cases[0] = (32, 2, offsets[2])
    cases[1] = (32, 5, 0)                      # too many devices
    cases[2] = (700, 2, offsets[2])            # no such placement
    cases[3] = (32, 4, len(data) - 3)          # data runs past the end
    shape = dict(units=2, h=4, b=2)
    with pytest.raises(ps.PsError) as e:
        ctx.verify_batch(shape, cases, data)
    assert e.value.code == ps.E_DEVICE
    good = ctx.verify_batch(shape, cases[:1], data)          # the status was cleared: the next call works
    assert good[0]["match"] == 1
    with pytest.raises(ps.PsError) as e:
        ctx.verify_batch(dict(units=9, h=4, b=2), cases[:1], data)
    assert e.value.code == ps.E_RANGE
