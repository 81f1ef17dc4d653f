"""Pins of the CPU oracle to what the paper and the mathematics fix: the
numbers the paper prints, closed forms, invariants, Table 2, brute-force
enumeration, brute-force dominance.  No GPU involved."""
import itertools

import numpy as np
import pytest

from conftest import read_golden_table2, read_golden_values
from oracle import oracle as O
from paper_2601_02311_b200 import synth

R, S, SG, M, Oo = 0, 1, 2, 3, 4
GOLD = read_golden_values("paper_worked_example.txt")
TABLE2 = read_golden_table2()
VALID = O.F_GI | O.F_SC | O.F_CV


def code_of(t, o, g, a):
    return t + 5 * o + 25 * g + 125 * a


@pytest.fixture(scope="module")
def c0():
    sp = O.Space(synth.config("C0"))
    return sp, sp.eval_range(0, sp.size)


def at(res, n_index, code):
    i = n_index * 625 + code
    return {k: int(v[i]) for k, v in res.items()}


# ------------------------------------------------------------ printed values
def test_table1_state_sizes():
    """Table 1 / Remark 1: 2P, 4P + 8P, 2P bytes; total 16 P."""
    rec = O.model_record(synth.worked_example())
    P = rec["P"]
    assert P == GOLD["P"]
    assert rec["w_theta"] * P == GOLD["table1_params_fp16"]
    assert rec["w_grad"] * P == GOLD["table1_grads_fp16"]
    assert rec["w_omega"] * P == GOLD["table1_master_fp32"] + GOLD["table1_adam_fp32"]
    assert (rec["w_theta"] + rec["w_grad"] + rec["w_omega"]) * P == GOLD["table1_total"]


def test_example3_memory(c0):
    """Example 3: 1120 GB under DP for every N; 140 GB under ZeRO-3 at N = 8; 8x."""
    sp, res = c0
    dp, z3 = TABLE2["data_parallel"][0], TABLE2["zero_stage_3_fsdp"][0]
    for ni in range(7):
        assert at(res, ni, dp)["mem"] == GOLD["dp_mem_per_device"]
    n8 = 3
    assert sp.decode(n8 * 625)["N"] == 8
    assert at(res, n8, z3)["mem"] == GOLD["zero3_mem_n8"]
    assert at(res, n8, dp)["mem"] == GOLD["mem_reduction_n8"] * at(res, n8, z3)["mem"]


def test_example4_communication(c0):
    """Example 4: 3.5 P and 5.25 P bytes at N = 8; ratio 1.5 for every N >= 2."""
    sp, res = c0
    dp, z3 = TABLE2["data_parallel"][0], TABLE2["zero_stage_3_fsdp"][0]
    assert at(res, 3, dp)["comm_paper"] == GOLD["dp_comm_n8"]
    assert at(res, 3, z3)["comm_paper"] == GOLD["zero3_comm_n8"]
    for ni in range(1, 7):
        assert 2 * at(res, ni, z3)["comm_paper"] == GOLD["comm_ratio_times_2"] * at(res, ni, dp)["comm_paper"]
    # both strategies move nothing beyond what Theorem 2 prices
    assert at(res, 3, dp)["comm_ext"] == 0 and at(res, 3, z3)["comm_ext"] == 0
    assert at(res, 3, dp)["flags"] & O.F_PAPER_PRICED
    assert at(res, 3, z3)["flags"] & O.F_PAPER_PRICED


def test_unit_term_of_theorem1():
    """Theorem 1: mu(S*, s) = s/N + s_unit; for L = 80, H = 8192 the unit is
    12 H^2 x 2 B = 1 610 612 736 B on top of Example 3's 140 GB."""
    sp = O.Space(synth.config("C0b"))
    r = sp.eval_range(3 * 625 + TABLE2["zero_stage_3_fsdp"][0], 1)
    assert int(r["mem"][0]) == GOLD["zero3_mem_n8"] + 12 * 8192 * 8192 * 2
    assert 12 * 8192 * 8192 * 2 == 1_610_612_736


# ------------------------------------------------------------ closed forms
def test_zero_stage_closed_forms(c0):
    """From Theorem 1 and Table 2: ZeRO-1 4P + 12P/N, ZeRO-2 2P + 14P/N, ZeRO-3 16P/N
    (the last is printed in Section 7.1)."""
    sp, res = c0
    P = GOLD["P"]
    for ni in range(7):
        N = 1 << ni
        assert P % N == 0
        assert at(res, ni, TABLE2["zero_stage_1"][0])["mem"] == 4 * P + 12 * P // N
        assert at(res, ni, TABLE2["zero_stage_2"][0])["mem"] == 2 * P + 14 * P // N
        assert at(res, ni, TABLE2["zero_stage_3_fsdp"][0])["mem"] == 16 * P // N


def test_mu_table_each_state(c0):
    """Theorem 1's five cases, state by state, against Python integers."""
    sp, res = c0
    P = GOLD["P"]
    w = (2, 12, 2)
    for ni in range(7):
        N = 1 << ni
        for state in range(3):
            for mode, expect in ((R, w[state] * P), (S, w[state] * P // N),
                                 (SG, w[state] * P // N), (M, 0), (Oo, 0)):
                # all other states offloaded => they contribute nothing
                pis = [Oo, Oo, Oo, Oo]
                pis[state] = mode
                assert at(res, ni, code_of(*pis))["mem"] == expect


def test_replicated_memory_independent_of_n(c0):
    sp, res = c0
    for code in (0, code_of(R, R, R, M), code_of(R, R, R, Oo)):
        vals = {at(res, ni, code)["mem"] for ni in range(7)}
        assert len(vals) == 1


def test_corollary1_transitions():
    """Corollary 1 on a model whose sizes are not divisible by N."""
    space = synth.config("C1", n_models=3)
    sp = O.Space(space)
    per_n = 2 * 625
    for m in range(3):
        rec = O.model_record(space["models"][m:m + 1])
        for ni, N in enumerate(space["n_values"]):
            base = m * sp.points_per_model + ni * per_n
            r = sp.eval_range(base, 625)
            x = rec["P"] - rec["P"] // int(N)       # ring volume, elements
            c = lambda code: int(r["comm_paper"][code])
            assert c(5) == c(0)                       # (1) sharding Omega: no change
            assert c(0) - c(30) == x * 2              # (2) gradient term halves
            assert c(0) == 2 * x * 2
            assert c(32) - c(30) == 2 * x * 2         # (3) + two all-gathers of Theta
            mem = lambda code: int(r["mem"][code])
            assert mem(5) <= mem(0) and mem(30) <= mem(5)


def test_single_device_has_no_communication(c0):
    sp, res = c0
    for code in range(625):
        a = at(res, 0, code)
        assert a["comm_paper"] == 0 and a["comm_ext"] == 0
    assert at(res, 0, 1)["mem"] == at(res, 0, 0)["mem"]   # a shard of one is the tensor


def test_shards_of_eq2_sum_to_tensor_and_max_is_ceil():
    """eq. (2) boundaries floor(i E / N): the shards tile the tensor and the
    largest has ceil(E/N) elements -- the figure mu(S, .) must charge."""
    rec = dict(P=0, unit=0, A0=0, A1=0, UA0=0, UA1=0, Sbh=1, L=1, heads=1,
               w_theta=1, w_omega=1, w_grad=1, w_act=1)
    for E in (1, 2, 7, 15, 16, 1000003):
        for N in (1, 2, 3, 4, 7, 8, 64, 1000):
            cuts = [(i * E) // N for i in range(N + 1)]
            sizes = [cuts[i + 1] - cuts[i] for i in range(N)]
            assert sum(sizes) == E
            rec["P"] = E
            r = O.eval_record(rec, N, 1, 1, N, 0, 0, code_of(S, Oo, Oo, Oo))
            assert r["mem"] == max(sizes) == -(-E // N)
            # ring volume: everything except the smallest shard (Section 2.3)
            r = O.eval_record(rec, N, 1, 1, N, 0, 0, code_of(R, R, S, R))
            assert r["comm_paper"] == E - min(sizes)


def test_collective_cost_relations():
    """Section 2.3: all-reduce = 2 x reduce-scatter = 2 x all-gather."""
    rec = dict(P=999, unit=0, A0=0, A1=0, UA0=0, UA1=0, Sbh=1, L=1, heads=1,
               w_theta=2, w_omega=12, w_grad=2, w_act=2)
    for N in (2, 3, 8, 10):
        ar = O.eval_record(rec, N, 1, 1, N, 0, 0, code_of(R, R, R, R))["comm_paper"]
        rs = O.eval_record(rec, N, 1, 1, N, 0, 0, code_of(R, S, S, R))["comm_paper"]
        ag2 = O.eval_record(rec, N, 1, 1, N, 0, 0, code_of(SG, S, S, R))["comm_paper"] - rs
        assert ar == 2 * rs == ag2


# ------------------------------------------------------------ Table 2, predicates
def test_table2_rows_are_valid(c0):
    sp, res = c0
    for name, (code, role) in TABLE2.items():
        if role != "data":
            continue
        for ni in range(7):
            assert at(res, ni, code)["flags"] & VALID == VALID, name
    assert TABLE2["tensor_parallel"][0] == 156 and TABLE2["pipeline_parallel"][0] == 31
    shape = synth.zoo(1, 5)
    shape["heads"], shape["layers"] = 8, 24
    ok = O.check_composition(shape, 64, 4, 2, 8, 156, 31, 32)
    assert ok["flags"] & VALID == VALID and ok["flags"] & O.F_AXIS_FORM
    for bad_tp in (0, 32, 157):
        r = O.check_composition(shape, 64, 4, 2, 8, bad_tp, 31, 32)
        assert not r["flags"] & O.F_AXIS_FORM and not r["flags"] & O.F_CV
    r = O.check_composition(shape, 64, 4, 2, 8, 156, 156, 32)
    assert not r["flags"] & O.F_CV
    # an absent axis (degree 1) is not looked at
    r = O.check_composition(shape, 8, 1, 1, 8, 0, 0, 32)
    assert r["flags"] & VALID == VALID


def test_predicate_counts(c0):
    """171 of the 625 data-axis codes are valid with several replicas (57
    (Theta, Omega, G) triples x 3 activation modes), 475 with one."""
    sp, res = c0
    for ni in range(7):
        fl = res["flags"][ni * 625:(ni + 1) * 625]
        n_valid = int(((fl & 3) == 3).sum())
        assert n_valid == (475 if ni == 0 else 171)


def test_composition_validity_bits():
    shape = synth.zoo(1, 9)
    shape["heads"], shape["layers"] = 12, 30
    f = lambda N, T, K, D: O.check_composition(shape, N, T, K, D, 156, 31, 0)["flags"]
    assert f(24, 4, 3, 2) & O.F_CV
    assert not f(24, 4, 3, 3) & O.F_CV                     # T K D != N
    fl = f(40, 8, 5, 1)                                    # 8 does not divide 12 heads
    assert not fl & O.F_T_HEADS and fl & O.F_K_LAYERS and not fl & O.F_CV
    fl = f(16, 4, 4, 1)                                    # 4 does not divide 30 layers
    assert fl & O.F_T_HEADS and not fl & O.F_K_LAYERS and not fl & O.F_CV
    fl = f(12, 12, 1, 1)                                   # Proposition 1: TP beyond a node
    assert fl & O.F_T_HEADS and not fl & O.F_TP_LE_MAX and not fl & O.F_CV


def test_nesting_order_tp_then_pp_then_data():
    """Remark 4: split by T, then K, then shard over D, with ceilings at each level."""
    rec = dict(P=1000003, unit=1001, A0=777777, A1=5555, UA0=7777, UA1=55, Sbh=4099, L=10,
               heads=6, w_theta=2, w_omega=12, w_grad=2, w_act=2)
    cd = lambda a, b: -(-a // b)
    for (T, K, D) in ((1, 1, 1), (3, 1, 1), (1, 5, 1), (3, 5, 7), (6, 2, 4)):
        E2 = cd(cd(rec["P"], T), K)
        u = cd(rec["unit"], T)
        N = T * K * D
        r = O.eval_record(rec, N, T, K, D, 0, 0, code_of(R, S, SG, M))
        assert r["mem"] == 2 * E2 + 12 * cd(E2, D) + 2 * (cd(E2, D) + u) + cd(7777, T)
        r = O.eval_record(rec, N, T, K, D, 1, 1, code_of(M, Oo, Oo, S))
        assert r["mem"] == 2 * u + cd(5555, D)             # tau = 1: activations not split by T
        r = O.eval_record(rec, N, T, K, D, 0, 0, code_of(R, R, R, R))
        x = E2 - E2 // D
        assert r["comm_paper"] == 2 * x * 2
        # all replicated on the data axis: whatever is left in comm_ext is model-axis traffic,
        # whose volume tests/test_oracle_vs_composition_sim.py pins with byte counters
        assert (r["comm_ext"] == 0) == (T == 1 and K == 1)


def test_host_bytes_and_offload_row(c0):
    """ZeRO-Offload (O, O, S, R) at N = 8: only the gradient shard stays on the GPU."""
    sp, res = c0
    P = GOLD["P"]
    a = at(res, 3, TABLE2["zero_offload"][0])
    assert a["mem"] == 2 * P // 8
    assert a["host"] == 3 * (2 * P // 8) + 2 * (12 * P // 8)
    assert a["flags"] & O.F_USES_HOST and not a["flags"] & O.F_PAPER_PRICED


def test_activation_formula_closed_form():
    """Reading (the paper prints no activation size): per layer 34 S b H + 5 a S^2 b
    bytes, 2 S b H with full checkpointing."""
    shape = synth.zoo(1, 11)
    L, H, a = int(shape["layers"][0]), int(shape["hidden"][0]), int(shape["heads"][0])
    Sq, b, V = int(shape["seq"][0]), int(shape["micro_batch"][0]), int(shape["vocab"][0])
    rec = O.model_record(shape)
    assert rec["P"] == 12 * L * H * H + V * H
    assert rec["unit"] == 12 * H * H
    assert rec["A0"] == L * (34 * Sq * b * H + 5 * a * Sq * Sq * b)
    assert rec["A1"] == L * 2 * Sq * b * H
    assert rec["A0"] == L * rec["UA0"] and rec["A1"] == L * rec["UA1"]


# ------------------------------------------------------------ enumeration
def py_factorisations(N, t_max, k_max):
    return [(T, K, N // (T * K)) for T in range(1, N + 1) if N % T == 0 and T <= t_max
            for K in range(1, N // T + 1) if (N // T) % K == 0 and K <= k_max]


def test_space_sizes_and_factorisation_counts():
    for name, n in synth.FULL_SIZE.items():
        assert O.Space(synth.config(name)).size == n
    assert sum(O.num_factorisations(1 << j, 8, 1 << 14) for j in range(13)) == 290
    assert sum(O.num_factorisations(1 << j, 1 << 14, 1 << 14) for j in range(15)) == 680
    for N in (1, 6, 12, 30, 97, 360):
        assert O.num_factorisations(N, 12, 36) == len(py_factorisations(N, 12, 36))


def test_decode_is_the_canonical_order():
    """Model-major, N in the given order, (T asc, K asc), activation variant,
    tensor-axis variant, data-axis code fastest with the Theta digit fastest."""
    space = synth.ragged_space(4, n_models=2)
    sp = O.Space(space)
    modes = [m for m in range(5) if space["mode_mask"] >> m & 1]
    expect = []
    for model in range(2):
        for N in space["n_values"]:
            for (T, K, D) in py_factorisations(int(N), space["t_enum_max"], space["k_enum_max"]):
                for v in range(2):
                    for tau in range(2):
                        for a, g, o, t in itertools.product(modes, repeat=4):
                            expect.append((model, int(N), T, K, D, v, tau, code_of(t, o, g, a)))
    assert sp.size == len(expect)
    step = 37
    for idx in list(range(0, sp.size, step)) + [sp.size - 1]:
        p = sp.decode(idx)
        got = (p["model"], p["N"], p["T"], p["K"], p["D"], p["act_variant"], p["tpa_variant"],
               p["code_dp"])
        assert got == expect[idx]
        assert p["code_tp"] == (156 if p["tpa_variant"] == 0 else 31) and p["code_pp"] == 31


def test_fig2_rank_layout():
    """Figure 2 / Theorem 6(1): TP(4) x DP(2) on 8 devices -- tensor groups are
    {0..3} and {4..7}; data-parallel partners are i and i+4.  With
    rank = (d K + k) T + t the same groups come out."""
    T, K, D = 4, 1, 2
    rank = lambda d, k, t: (d * K + k) * T + t
    groups = [[rank(d, 0, t) for t in range(T)] for d in range(D)]
    assert groups == [[0, 1, 2, 3], [4, 5, 6, 7]]
    assert [[rank(d, 0, t) for d in range(D)] for t in range(T)] == [[0, 4], [1, 5], [2, 6], [3, 7]]


# ------------------------------------------------------------ filter, reductions
def brute_frontier(mem, comm, idx):
    keep = []
    n = len(mem)
    for i in range(n):
        dominated = False
        for j in range(n):
            if j == i:
                continue
            if mem[j] <= mem[i] and comm[j] <= comm[i]:
                if mem[j] < mem[i] or comm[j] < comm[i] or idx[j] < idx[i]:
                    dominated = True
                    break
        if not dominated:
            keep.append(i)
    keep.sort(key=lambda i: mem[i])
    return keep


@pytest.mark.parametrize("comm_kind", [O.COMM_PAPER, O.COMM_PAPER_PLUS_EXT])
def test_pareto_against_quadratic_dominance(comm_kind):
    space = synth.ragged_space(7, n_models=2)
    space["n_values"] = np.asarray([1, 2, 6, 12], dtype=np.uint32)
    sp = O.Space(space)
    ppm = sp.points_per_model
    filt = dict(require_flags=VALID, comm_kind=comm_kind)
    rec = [O.model_record(space["models"][m:m + 1]) for m in range(2)]
    caps = [16 * rec[0]["P"] // 5, 16 * rec[0]["P"] * 2]
    entries, counts = sp.sweep(filt, caps, O.KIND_PARETO, 64)
    for m in range(2):
        r = sp.eval_range(m * ppm, ppm)
        comm = r["comm_paper"] if comm_kind == O.COMM_PAPER else r["comm_paper"] + r["comm_ext"]
        for ci, cap in enumerate(caps):
            ok = np.nonzero(((r["flags"] & VALID) == VALID) & (r["mem"] <= cap))[0]
            assert len(ok) < 12000
            keep = brute_frontier(r["mem"][ok].tolist(), comm[ok].tolist(), ok.tolist())
            n = int(counts[m, ci])
            assert n == len(keep) and n <= 64
            got = entries[m, ci, :n]
            assert got["idx"].tolist() == [m * ppm + int(ok[i]) for i in keep]
            assert got["mem"].tolist() == [int(r["mem"][ok[i]]) for i in keep]
            assert got["comm"].tolist() == [int(comm[ok[i]]) for i in keep]
            assert all(f & O.F_FEASIBLE for f in got["flags"])


def test_frontier_under_smaller_cap_is_a_prefix():
    """Dominance only looks at points with smaller-or-equal memory, so the
    frontier under a tighter capacity is the head of the looser one's."""
    space = synth.config("C3", n_models=2)
    space["n_values"] = np.asarray([8, 64, 512], dtype=np.uint32)
    sp = O.Space(space)
    caps = [20 * synth.GB, 80 * synth.GB, 192 * synth.GB]
    entries, counts = sp.sweep(dict(require_flags=VALID), caps, O.KIND_PARETO, 256)
    for m in range(2):
        big = entries[m, 2, :counts[m, 2]]
        for ci in (0, 1):
            head = big[big["mem"] <= caps[ci]]
            got = entries[m, ci, :counts[m, ci]]
            assert np.array_equal(got, head)


def test_topk_against_full_sort():
    space = synth.ragged_space(3, n_models=2)
    sp = O.Space(space)
    ppm = sp.points_per_model
    rec = O.model_record(space["models"][0:1])
    cap = 16 * rec["P"]
    filt = dict(require_flags=O.F_GI | O.F_SC, host_cap=40 * rec["P"])
    entries, counts = sp.sweep(filt, [cap], O.KIND_TOPK, 16)
    for m in range(2):
        r = sp.eval_range(m * ppm, ppm)
        comm = r["comm_paper"] + r["comm_ext"]
        ok = np.nonzero(((r["flags"] & 3) == 3) & (r["mem"] <= cap) & (r["host"] <= 40 * rec["P"]))[0]
        order = sorted(ok.tolist(), key=lambda i: (int(comm[i]), int(r["mem"][i]), i))
        assert counts[m, 0] == len(ok)
        n = min(16, len(ok))
        assert entries[m, 0, :n]["idx"].tolist() == [m * ppm + i for i in order[:n]]


def test_compaction_is_filter_in_index_order():
    space = synth.config("C2", n_models=1)
    sp = O.Space(space)
    first, count = 12345, 30000
    filt = dict(require_flags=VALID, cap_bytes=80 * synth.GB)
    full = sp.eval_range(first, count, filt)
    keep = ((full["flags"] & VALID) == VALID) & (full["mem"] <= 80 * synth.GB)
    got = sp.compact_range(first, count, filt)
    assert got["idx"].tolist() == (first + np.nonzero(keep)[0]).tolist()
    assert np.array_equal(got["mem"], full["mem"][keep])
    assert np.array_equal(got["flags"], full["flags"][keep])
    assert np.all((full["flags"] & O.F_FEASIBLE != 0) == (full["mem"] <= 80 * synth.GB))


def test_generator_is_deterministic_and_in_range():
    a, b = synth.zoo(64, 2, max_layers=160, max_hidden_mult=256), synth.zoo(64, 2, max_layers=160, max_hidden_mult=256)
    assert a.tobytes() == b.tobytes()
    assert a["layers"].min() >= 12 and a["layers"].max() <= 160
    assert (a["hidden"] % 128 == 0).all() and a["hidden"].max() <= 32768
    assert (a["heads"] * 128 == a["hidden"]).all()
    assert synth.table_checksum(a) != synth.table_checksum(synth.zoo(64, 3))


# ------------------------------------------------------------ Algorithm 1
def _q(P, layer, Md, N, fast=1):
    return [P, layer, Md, N, 2, 2, 12, fast]


def test_algorithm1_on_the_papers_example():
    """Section 1 / Example 3: a 70B model needs 1120 GB, far more than an 80 GB GPU;
    ZeRO-3 needs 16P/N.  With the 0.7 headroom of Algorithm 1: not data parallel;
    ZeRO-3 once 1120/N < 56 GB, i.e. from N = 32 (35 GB); below that the last branch."""
    P, Md = 70_000_000_000, 80 * synth.GB
    layer = 12 * 8192 * 8192
    r = O.select(np.array([_q(P, layer, Md, N) for N in (1, 8, 16, 32, 64)], dtype=np.uint64))
    assert r[:, 2].tolist() == [3, 3, 3, 1, 1]          # layer state 12.9 GB < 0.3 * 80 GB: no TP
    assert r[3, 0] == 16 * P // 32 + layer * 2            # Theorem 1: 16P/N plus the gathered unit
    assert r[4, 4] == 32 and r[4, 3] == 1
    # a 1B model fits one device with headroom: data parallel, 16 P bytes, all-reduce of 2P
    r = O.select(np.array([_q(10 ** 9, 0, Md, 8)], dtype=np.uint64))
    assert r[0].tolist()[:5] == [16 * 10 ** 9, 2 * (10 ** 9 - 10 ** 9 // 8) * 2, 0, 1, 0]
    assert r[0, 5] == O.F_FEASIBLE


def test_algorithm1_thresholds_are_strict_and_exact():
    Md = 10 ** 10
    # M_model = 16 P; boundary 16 P = 0.7 M_d  <=>  P = 437 500 000
    r = O.select(np.array([_q(437_499_999, 0, Md, 4), _q(437_500_000, 0, Md, 4)], dtype=np.uint64))
    assert r[:, 2].tolist() == [0, 1]
    # ZeRO-3 boundary 16 P / N = 0.7 M_d at N = 4  <=>  P = 1 750 000 000
    r = O.select(np.array([_q(1_749_999_999, 0, Md, 4), _q(1_750_000_000, 0, Md, 4)], dtype=np.uint64))
    assert r[:, 2].tolist() == [1, 3]
    # layer boundary 16 * layer > 0.3 M_d  <=>  layer > 187 500 000; needs a fast interconnect
    big = 10 ** 12
    r = O.select(np.array([_q(big, 187_500_000, Md, 8), _q(big, 187_500_001, Md, 8),
                           _q(big, 187_500_001, Md, 8, fast=0), _q(big, 187_500_001, Md, 12)],
                          dtype=np.uint64))
    assert r[:, 2].tolist() == [3, 2, 3, 2]
    assert r[1, 3] == 8 and r[3, 3] == 6                  # largest divisor of N not above 8
    # tensor parallelism divides the state before the data axis shards it (Remark 4)
    E2 = -(-big // 8)
    assert r[1, 0] == 16 * E2 + 2 * (-(-187_500_001 // 8))


def test_algorithm1_beside_the_frontier_on_the_papers_example():
    """70B parameters on 80 GB devices, data axis only.  Among the placements built
    from R, S and S* Algorithm 1's ZeRO-3 is the whole frontier from N = 32 on:
    16P/N bytes and 3 (N-1)/N |G| of traffic, 1.5x data parallelism's.  With all
    five modes it is off the frontier: consuming gradients as they are produced
    (S*, S, M, R) moves the same bytes and holds 2P/N less.  At N = 8 nothing fits."""
    P, Md = GOLD["P"], 80 * synth.GB
    filt = dict(require_flags=O.F_GI | O.F_SC, host_cap=0, comm_kind=O.COMM_PAPER_PLUS_EXT)
    for N in (32, 64):
        x = 2 * (P - P // N)                                   # ring volume of |G| = |Theta| = 2P bytes
        for mask, on in ((0b00111, True), (0x1F, False)):
            space = synth._space(synth.worked_example(False), [N], t_enum_max=1, k_enum_max=1, n_act=1, n_tpa=1,
                                 mode_mask=mask)
            sp = O.Space(space)
            e, c = sp.sweep(filt, [Md], O.KIND_PARETO, 16)
            r = O.select_compare(sp, 0, Md, filt, e, c, 0)[0]
            assert (r[6], r[7], r[8]) == (1, 1, 32)            # branch 1: ZeRO-3
            assert r[0] == 16 * P // N and r[1] == 3 * x and 2 * r[1] == 3 * (2 * x)
            assert r[10] == (1 | 2 | 4 if on else 1 | 2 | 8)
            if on:
                assert c[0, 0] == 1 and (r[3], r[4], r[5]) == (r[0], r[1], r[2])
            else:
                assert (r[3], r[4]) == (14 * P // N, 3 * x)    # no gradient shard is kept
                assert sp.decode(int(r[5]))["code_dp"] == code_of(SG, S, M, R)
    space = synth._space(synth.worked_example(False), [8], t_enum_max=1, k_enum_max=1, n_act=1, n_tpa=1,
                         mode_mask=0x1F)
    sp = O.Space(space)
    e, c = sp.sweep(filt, [Md], O.KIND_PARETO, 16)
    r = O.select_compare(sp, 0, Md, filt, e, c, 0)[0]
    assert r[6] == 3 and r[10] == (1 | 16) and r[0] == 16 * P // 8
