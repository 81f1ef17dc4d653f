"""The composition rules (Theorems 6-7, Remark 4) and the nesting of the shard
formulas against a brute-force TP x PP x DP run of a two-layer network."""
import numpy as np
import pytest

from oracle import oracle as O
from oracle.sim import composition_sim as sim


@pytest.mark.parametrize("T,K,D", [(1, 1, 3), (2, 1, 2), (4, 1, 3), (1, 2, 2), (2, 2, 3), (4, 2, 2)])
def test_grid_matches_single_device_and_formulas(T, K, D):
    n, h, b = 6, 8, 3
    W1, W2, xs, ys = sim.make(n, h, b, D, seed=T * 100 + K * 10 + D)
    ref1, ref2 = sim.run_single(W1, W2, xs, ys, steps=4)
    g1, g2, held, sent, consistent = sim.run_grid(W1, W2, xs, ys, T, K, D, steps=4)
    assert consistent
    assert np.allclose(g1, ref1, rtol=1e-12, atol=1e-14) and np.allclose(g2, ref2, rtol=1e-12, atol=1e-14)
    # nesting: P elements -> ceil(P/T) -> ceil(./K) per position; data axis replicated (code 0)
    P = 2 * h * n
    rec = dict(P=P, unit=0, A0=0, A1=0, UA0=0, UA1=0, Sbh=1, L=2, heads=4, w_theta=1, w_omega=1,
               w_grad=1, w_act=1)
    r = O.eval_record(rec, T * K * D, T, K, D, 0, 0, 0)
    assert r["flags"] & O.F_CV
    assert r["mem"] == 3 * held                     # Theta, Omega, G replicated over the data axis
    E2 = -(-(-(-P // T)) // K)
    assert held == E2
    # data-parallel all-reduce of G over D replicas: 2 ring phases of E2 - floor(E2/D) elements.
    # The simulator reduces layer by layer, so compare with the per-layer sum when a device holds two.
    layers_here = 2 // K
    e_layer = E2 // layers_here
    assert sent == layers_here * 2 * (e_layer - e_layer // D)
    if layers_here == 1 or (e_layer % D == 0):
        assert r["comm_paper"] == sent


def test_summing_weight_gradients_inside_a_tensor_group_diverges():
    """Theorem 6(3): the data-parallel sync aggregates across tensor groups, not within."""
    n, h, b, T, D = 6, 8, 3, 2, 2
    W1, W2, xs, ys = sim.make(n, h, b, D, seed=5)
    ref1, ref2 = sim.run_single(W1, W2, xs, ys, steps=3)
    g1, g2, *_ = sim.run_grid(W1, W2, xs, ys, T, 1, D, steps=3, sum_inside_tensor_group=True)
    assert not np.allclose(g1, ref1, rtol=1e-6)


def test_composition_validity_needs_divisibility():
    """T must divide the heads and K the layers (what the grid run needs to split evenly)."""
    rec = dict(P=96, unit=0, A0=0, A1=0, UA0=0, UA1=0, Sbh=1, L=2, heads=4, w_theta=1, w_omega=1,
               w_grad=1, w_act=1)
    assert O.eval_record(rec, 8, 4, 2, 1, 0, 0, 0)["flags"] & O.F_CV
    assert not O.eval_record(rec, 9, 3, 1, 3, 0, 0, 0)["flags"] & O.F_CV      # 3 does not divide 4 heads
    assert not O.eval_record(rec, 6, 1, 3, 2, 0, 0, 0)["flags"] & O.F_CV      # 3 does not divide 2 layers


# ------------------------------------------------------------ model-axis traffic
# The oracle's tensor- and pipeline-axis volume against bytes counted by explicit
# rings inside every tensor group and by the transfers between pipeline stages
# of a six-block network (Section 2.3 ring costs; Theorem 6 "All-Reduce on
# activations"; Proposition 1 "at least one collective per layer").  The
# harness's block needs one all-reduce forward and one backward, so it is
# compared with the oracle at two all-reduces per layer (a transformer layer is
# two such blocks, attention and MLP: the default of four).
DEEP = dict(blocks=6, n=7, h=12, b=5)          # boundary tensor of 35 elements: not divisible by 2, 3, 4
WIDTH = 2


def deep_record(blocks, E, T):
    return dict(P=1000, unit=0, A0=0, A1=0, UA0=0, UA1=0, Sbh=E, L=blocks, heads=12, w_theta=1,
                w_omega=1, w_grad=1, w_act=WIDTH)


@pytest.mark.parametrize("T", [1, 2, 3, 4])
@pytest.mark.parametrize("K", [1, 2, 3])
@pytest.mark.parametrize("shard_activations", [False, True])
def test_model_axis_traffic_from_byte_counters(T, K, shard_activations):
    blocks, n, h, b = DEEP["blocks"], DEEP["n"], DEEP["h"], DEEP["b"]
    D, steps = 2, 3
    W1, W2, xs, ys = sim.make_deep(blocks, n, h, b, D, seed=10 * T + K)
    ref1, ref2, ref_din = sim.run_deep_single(W1, W2, xs, ys, steps)
    got = sim.run_deep_grid(W1, W2, xs, ys, T, K, D, shard_activations, steps, width=WIDTH)
    # the grid really trains the same network: every counted transfer was needed
    scale = max(np.abs(w).max() for w in ref1 + ref2)
    for a, c in zip(got["W1"] + got["W2"], ref1 + ref2):
        assert np.abs(a - c).max() <= 1e-9 * scale
    assert np.abs(np.concatenate(got["d_in"]) - ref_din).max() <= 1e-9 * np.abs(ref_din).max()

    E = b * n
    tau = 0 if shard_activations else 1
    r = O.eval_record(deep_record(blocks, E, T), T * K * D, T, K, D, 0, tau, 0, tp_coll_per_layer=2)
    # data axis fully replicated (code 0): comm_ext is the model-axis traffic alone
    assert r["comm_ext"] == got["tensor_bytes"] + got["pipeline_bytes"]
    # and each part by itself, against the oracle with the other part switched off
    r_tp = O.eval_record(deep_record(blocks, E, T), T * D, T, 1, D, 0, tau, 0, tp_coll_per_layer=2)
    assert r_tp["comm_ext"] * (blocks // K) == got["tensor_bytes"] * blocks     # layers per stage scale it
    r_pp = O.eval_record(deep_record(blocks, E, T), T * K * D, T, K, D, 0, tau, 0, tp_coll_per_layer=0)
    assert r_pp["comm_ext"] == got["pipeline_bytes"]
    if T == 1:
        assert got["tensor_bytes"] == 0
    if K == 1:
        assert got["pipeline_bytes"] == 0


def test_model_axis_traffic_with_uneven_stages():
    """Five blocks over three stages: 2, 2 and 1 -- the fullest stage has ceil(5/3) blocks."""
    blocks, n, h, b, T, K, D = 5, 7, 12, 5, 3, 3, 1
    W1, W2, xs, ys = sim.make_deep(blocks, n, h, b, D, seed=3)
    got = sim.run_deep_grid(W1, W2, xs, ys, T, K, D, False, 1, width=WIDTH)
    r = O.eval_record(deep_record(blocks, b * n, T), T * K * D, T, K, D, 0, 1, 0, tp_coll_per_layer=2)
    assert r["comm_ext"] == got["tensor_bytes"] + got["pipeline_bytes"]


def test_model_axis_traffic_scales_with_micro_batches():
    """Gradient accumulation: the model axes move their traffic once per micro-batch."""
    rec = deep_record(6, 35, 3)
    one = O.eval_record(rec, 18, 3, 3, 2, 0, 0, 0, tp_coll_per_layer=2)
    four = O.eval_record(rec, 18, 3, 3, 2, 0, 0, 0, tp_coll_per_layer=2, grad_accum_steps=4)
    assert four["comm_ext"] == 4 * one["comm_ext"]
