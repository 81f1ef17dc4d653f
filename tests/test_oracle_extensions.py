"""Pins of the two extensions the paper names without working them out: the
second unit buffer of an overlapped gather (proof of Theorem 1, case S*) and
gradient accumulation ("Limitations").  Closed forms, invariants, and the
brute-force simulator running several micro-batches per step with a prefetched
unit buffer."""
import numpy as np
import pytest

from oracle import oracle as O
from oracle.sim import placement_sim as sim
from paper_2601_02311_b200 import synth

MODES = ("R", "S", "SG", "M", "O")


def digits(code):
    return code % 5, (code // 5) % 5, (code // 25) % 5, code // 125


def with_ext(space, sstar_units=1, grad_accum_steps=1):
    s = dict(space)
    s["sstar_units"] = sstar_units
    s["grad_accum_steps"] = grad_accum_steps
    return s


def test_overlapped_gather_adds_one_unit_per_gathered_state():
    """C0b (L=80, H=8192, P=70e9): the unit is 12 H^2 = 805 306 368 elements.
    mem(2 buffers) - mem(1 buffer) = unit bytes of every state in mode S*, and
    nothing else changes.  ZeRO-3 at N=8: 140 GB + 2 x 1 610 612 736 B."""
    base = synth.config("C0b")
    one = O.Space(with_ext(base)).eval_range(0, 4375)
    two = O.Space(with_ext(base, sstar_units=2)).eval_range(0, 4375)
    unit = 12 * 8192 * 8192
    widths = (2, 12, 2)
    for idx in range(4375):
        th, om, gr, ac = digits(idx % 625)
        extra = sum(w * unit for w, m in zip(widths, (th, om, gr)) if m == 2)
        assert int(two["mem"][idx]) - int(one["mem"][idx]) == extra     # activations excluded in C0b
    for k in ("comm_paper", "comm_ext", "host", "flags"):
        assert np.array_equal(one[k], two[k])
    z3 = 3 * 625 + 32
    assert int(one["mem"][z3]) == 140_000_000_000 + 1_610_612_736
    assert int(two["mem"][z3]) == 140_000_000_000 + 2 * 1_610_612_736


def test_overlapped_gather_of_activations():
    """pi_A = S*: the slice plus one or two layers' activations."""
    space = synth.config("C1", n_models=2)
    one = O.Space(with_ext(space)).eval_range(0, 625 * 8)
    two = O.Space(with_ext(space, sstar_units=2)).eval_range(0, 625 * 8)
    rec = O.model_record(space["models"][0:1])
    for idx in range(625 * 8):
        th, om, gr, ac = digits(idx % 625)
        v = (idx // 625) % 2
        extra = sum(w * rec["unit"] for w, m in zip((2, 12, 2), (th, om, gr)) if m == 2)
        extra += rec["UA0" if v == 0 else "UA1"] if ac == 2 else 0
        assert int(two["mem"][idx]) - int(one["mem"][idx]) == extra, idx


@pytest.mark.parametrize("g", [2, 3, 8, 64])
def test_accumulation_leaves_gradient_synchronisation_alone(g):
    """Data parallel, ZeRO-1 and ZeRO-2 move gradients only: per step the bytes
    are those of g = 1 while g times the samples are processed -- the paper's
    "reduced by a factor equal to the number of accumulation steps".  ZeRO-3
    also gathers the parameters for every micro-batch: x w_G + g 2 x w_Theta."""
    base = synth.config("C0")
    one = O.Space(with_ext(base)).eval_range(0, 4375)
    acc = O.Space(with_ext(base, grad_accum_steps=g)).eval_range(0, 4375)
    assert np.array_equal(one["mem"], acc["mem"])
    assert np.array_equal(one["flags"], acc["flags"])
    P = 70_000_000_000
    for ni, N in enumerate((1, 2, 4, 8, 16, 32, 64)):
        x = P - P // N
        for code in (0, 5, 30):
            i = ni * 625 + code
            assert int(acc["comm_paper"][i]) == int(one["comm_paper"][i])
            assert int(acc["comm_ext"][i]) == int(one["comm_ext"][i])
        i = ni * 625 + 32
        assert int(acc["comm_paper"][i]) == x * 2 + g * 2 * x * 2
        # ZeRO-Offload (O,O,S,R): Theta loaded twice per micro-batch and stored once,
        # Omega loaded and stored once; the gathers after each load are per micro-batch
        i = ni * 625 + 49
        sh = -(-P // N)
        assert int(acc["host"][i]) == (2 * g + 1) * sh * 2 + 2 * sh * 12
        assert int(acc["comm_ext"][i]) == g * 2 * x * 2
        assert int(acc["comm_paper"][i]) == x * 2


def test_accumulation_in_a_composition_space():
    """Random windows of a composition space, g = 5 against g = 1: memory and flags
    do not change; Theorem 2's volume grows by (g - 1) x 2 x w_Theta exactly where
    the parameters are gathered; with a single replica (D = 1) the only traffic is
    the model axes', which is paid per micro-batch; offloaded activations cross the
    host link per micro-batch."""
    space = synth.config("C3", n_models=1)
    g = 5
    osp1, ospg = O.Space(with_ext(space)), O.Space(with_ext(space, grad_accum_steps=g))
    n = osp1.points_per_model
    rec = O.model_record(space["models"][0:1])
    rng = np.random.default_rng(5)
    for first in rng.integers(0, n - 2500, 12):
        a, b = osp1.eval_range(int(first), 2500), ospg.eval_range(int(first), 2500)
        assert np.array_equal(a["mem"], b["mem"]) and np.array_equal(a["flags"], b["flags"])
        for j in range(0, 2500, 7):
            p = osp1.decode(int(first) + j)
            th = p["code_dp"] % 5
            E2 = -(-(-(-rec["P"] // p["T"])) // p["K"])
            x = E2 - E2 // p["D"]
            grown = (g - 1) * 2 * x * rec["w_theta"] if th == 2 else 0
            assert int(b["comm_paper"][j]) - int(a["comm_paper"][j]) == grown
    idx = next(i for i in range(0, n, 625) if (lambda p: p["D"] == 1 and p["T"] > 1 and p["K"] > 1)(osp1.decode(i)))
    a, b = osp1.eval_range(idx, 625), ospg.eval_range(idx, 625)
    assert np.array_equal(b["comm_ext"], g * a["comm_ext"]) and int(a["comm_ext"][0]) > 0
    assert int(a["comm_paper"].max()) == 0 and int(b["comm_paper"].max()) == 0
    assert int(b["host"][4 * 125]) == g * int(a["host"][4 * 125]) > 0        # code (R,R,R,O)


@pytest.mark.parametrize("D", [2, 3])
def test_simulator_with_micro_batches_and_prefetch(D):
    """All 625 placements with three micro-batches per step and a prefetched unit
    buffer: validity is unchanged, and on valid placements the bytes held, sent
    and moved over the host link equal the formulas."""
    units, h, b, g = 3, 5, 2, 3
    rec = dict(P=units * h, unit=h, A0=units * b * h, A1=units * b * h, UA0=b * h, UA1=b * h,
               Sbh=b * h, L=units, heads=1, w_theta=sim.W_THETA, w_omega=sim.W_OMEGA,
               w_grad=sim.W_GRAD, w_act=2)
    n_valid = 0
    for code in range(625):
        r = O.eval_record(rec, D, 1, 1, D, 0, 0, code, sstar_units=2, grad_accum_steps=g)
        valid = (r["flags"] & (O.F_GI | O.F_SC)) == (O.F_GI | O.F_SC)
        s = sim.simulate(units, h, b, D, code, steps=3, seed=code % 5, accum=g, gather_buffers=2)
        assert valid == s["match"], (code, D)
        if valid:
            n_valid += 1
            assert s["mem"] == r["mem"], (code, D)
            assert s["comm"] == r["comm_paper"] + r["comm_ext"], (code, D)
            assert s["host"] == r["host"], (code, D)
    assert n_valid == 171


# ------------------------------------------------------------ k-way replication
# Section 1 names "k-way replication for 1 < k < N" as a straightforward extension of
# the replicated / sharded pair.  Reading: the sharded modes cut a state into D / k
# shards and every shard is held by k devices; gathers stay inside a group of D / k
# devices, a gradient is reduced to shards inside each group and then all-reduced
# across the k copies of each shard.
def test_k_way_replication_interpolates_between_sharded_and_replicated():
    space = synth.config("C1", n_models=2)
    n_values = space["n_values"].tolist()
    plain = O.Space(space).eval_range(0, 625 * 2 * len(n_values))
    for k in (2, 8, 1 << 10):
        repl = O.Space(dict(space, replication_k=k)).eval_range(0, 625 * 2 * len(n_values))
        for ni, N in enumerate(n_values):
            base = ni * 2 * 625
            if N == 1:
                # one device: nothing to replicate
                for name in plain:
                    assert np.array_equal(plain[name][base:base + 1250], repl[name][base:base + 1250])
            if k >= N:
                # as many copies as devices: a "shard" is the whole tensor, so S costs what R costs
                # (all three states sharded vs replicated: ZeRO-2-like code 30 + Theta S vs DP, code 0)
                s_all = base + 1 + 5 + 25          # (S, S, S, R)
                assert repl["mem"][s_all] == repl["mem"][base]
                assert repl["comm_paper"][s_all] == repl["comm_paper"][base]
                assert repl["flags"][s_all] & O.F_GI       # every device has all of Theta
    # k = 1 is the plain space
    same = O.Space(dict(space, replication_k=1)).eval_range(0, 1250)
    for name in plain:
        assert np.array_equal(plain[name][:1250], same[name])


def test_k_way_replication_on_the_worked_example():
    """70B parameters, N = 8, two copies of every shard (four shards): ZeRO-3 holds
    16P/4 = 280 GB; its gradients cost a reduce-scatter over 4 devices, (3/4) 2P, plus
    an all-reduce of the 2P/4 shard over 2 copies, 2 (1/2) 2P/4; its parameters two
    gathers over 4 devices, 2 (3/4) 2P."""
    space = dict(synth.config("C0"), replication_k=2)
    res = O.Space(space).eval_range(0, 4375)
    P = 70_000_000_000
    z3 = 3 * 625 + 32                                      # N = 8
    assert int(res["mem"][z3]) == 16 * P // 4
    assert int(res["comm_paper"][z3]) == (3 * 2 * P // 4 + 2 * (2 * P // 4) // 2) + 2 * (3 * 2 * P // 4)
    # data parallelism does not shard anything: unchanged
    assert int(res["mem"][3 * 625]) == 16 * P and int(res["comm_paper"][3 * 625]) == 245_000_000_000
    # N = 2 with two copies: ZeRO-3 is data parallelism in all but name
    z3_2 = 1 * 625 + 32
    assert int(res["mem"][z3_2]) == 16 * P and int(res["comm_paper"][z3_2]) == 2 * (2 * P // 2)


@pytest.mark.parametrize("D,k", [(4, 2), (6, 3), (3, 3), (4, 3)])
def test_k_way_replication_against_the_simulator(D, k):
    """All 625 placements with every shard held k times (gcd(k, D) times where k does not
    divide D): valid exactly when the run reproduces the single-device trajectory, and
    then the bytes held, sent and moved over the host link are the simulator's."""
    units, h, b = 3, 5, 2
    rec = dict(P=units * h, unit=h, A0=units * b * h, A1=units * b * h, UA0=b * h, UA1=b * h, Sbh=b * h,
               L=units, heads=1, w_theta=sim.W_THETA, w_omega=sim.W_OMEGA, w_grad=sim.W_GRAD, w_act=2)
    for code in range(625):
        r = O.eval_record(rec, D, 1, 1, D, 0, 0, code, replication_k=k)
        valid = (r["flags"] & (O.F_GI | O.F_SC)) == (O.F_GI | O.F_SC)
        s = sim.simulate(units, h, b, D, code, steps=3, seed=code % 5, copies=k)
        assert valid == s["match"], (code, D, k)
        if valid:
            assert (s["mem"], s["comm"], s["host"]) == (r["mem"], r["comm_paper"] + r["comm_ext"], r["host"]), code
