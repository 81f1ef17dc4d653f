"""The closed-form rules against the brute-force training simulator: for every
one of the 625 placements on 1-4 logical devices, (a) the gradient-integrity
and state-consistency predicates hold exactly when the placed run reproduces
the single-device trajectory, and (b) on valid placements the bytes held, sent
and moved over the host link equal the formulas.  Tensor sizes are chosen not
to be divisible by the device counts."""
import pytest

from oracle import oracle as O
from oracle.sim import placement_sim as sim


def toy_record(units, h, b):
    return dict(P=units * h, unit=h, A0=units * b * h, A1=units * b * h, UA0=b * h, UA1=b * h,
                Sbh=b * h, L=units, heads=1, w_theta=sim.W_THETA, w_omega=sim.W_OMEGA,
                w_grad=sim.W_GRAD, w_act=2)


@pytest.mark.parametrize("units,h,b", [(3, 5, 2), (2, 7, 3)])
@pytest.mark.parametrize("D", [1, 2, 3, 4])
def test_all_placements(units, h, b, D):
    rec = toy_record(units, h, b)
    n_valid = 0
    for code in range(625):
        r = O.eval_record(rec, D, 1, 1, D, 0, 0, code)
        valid = (r["flags"] & (O.F_GI | O.F_SC)) == (O.F_GI | O.F_SC)
        s = sim.simulate(units, h, b, D, code, steps=3, seed=code % 7)
        assert valid == s["match"], (code, D)
        if valid:
            n_valid += 1
            assert s["mem"] == r["mem"], (code, D)
            # T = K = 1: comm_ext is the data-axis part alone
            assert s["comm"] == r["comm_paper"] + r["comm_ext"], (code, D)
            assert s["host"] == r["host"], (code, D)
    assert n_valid == (475 if D == 1 else 171)


def test_ring_volumes_match_section_2_3():
    """Explicit rings: the busiest device sends E - floor(E/D) elements in a
    reduce-scatter and in an all-gather."""
    import numpy as np
    for E in (7, 15, 16, 101):
        for D in (2, 3, 4, 5):
            cuts = sim.bounds(E, D)
            books = sim.Books(D)
            full = [np.arange(E, dtype=float) + i for i in range(D)]
            red = sim.ring_reduce_scatter(full, cuts, 1, books, "rs")
            for i in range(D):
                assert np.allclose(red[i], sum(full)[cuts[i]:cuts[i + 1]])
            got = sim.ring_all_gather(red, 1, books, "ag")
            for i in range(D):
                assert np.allclose(got[i], sum(full))
            assert [int(s.max()) for _, s in books.phases] == [E - E // D, E - E // D]
