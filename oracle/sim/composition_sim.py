"""TEST INFRASTRUCTURE -- brute-force check of the composition rules on a
two-layer network y = W2 tanh(W1 x), trained with plain SGD in fp64 on a grid
of logical devices rank = (d*K + k)*T + t (Remark 4: tensor axis innermost,
pipeline axis in the middle, data axis outermost).

  tensor axis (Table 2: Theta, Omega, G sharded): W1 is split by rows and W2
      by columns over the T devices of a group; every device of the group sees
      the same samples; the partial outputs are summed over the group
      (Theorem 6: "All-Reduce on activations").  A device's weight gradient is
      complete for its shard: nothing is summed inside the group (Theorem 6(3)).
  pipeline axis: stage 0 holds W1, stage 1 holds W2 (Theorem 7); the boundary
      tensor goes forward and its gradient comes back.
  data axis: D replicas with different samples; gradients are averaged over
      the replicas that hold the same shard (Theorem 6(3), Theorem 7(2)).

The simulator keeps books of the parameter elements each device holds and of
the elements it sends in the data-axis all-reduce (explicit ring).  Only tests
import this module.
"""
from __future__ import annotations

import numpy as np

from .placement_sim import Books, bounds, ring_all_gather, ring_reduce_scatter


def make(n, h, b, D, seed):
    rng = np.random.default_rng(seed)
    W1 = rng.normal(scale=0.5, size=(h, n))
    W2 = rng.normal(scale=0.5, size=(n, h))
    xs = [rng.normal(size=(b, n)) for _ in range(D)]
    ys = [rng.uniform(-0.5, 0.5, size=(b, n)) for _ in range(D)]
    return W1, W2, xs, ys


def grads(W1, W2, x, y):
    """Mean-over-samples gradients of 0.5 ||W2 tanh(W1 x) - y||^2."""
    hid = np.tanh(x @ W1.T)
    out = hid @ W2.T
    d_out = (out - y) / x.shape[0]
    g2 = d_out.T @ hid
    d_hid = (d_out @ W2) * (1 - hid * hid)
    g1 = d_hid.T @ x
    return g1, g2


def run_single(W1, W2, xs, ys, steps, lr=0.1):
    x, y = np.concatenate(xs), np.concatenate(ys)
    W1, W2 = W1.copy(), W2.copy()
    for _ in range(steps):
        g1, g2 = grads(W1, W2, x, y)
        W1 -= lr * g1
        W2 -= lr * g2
    return W1, W2


def run_grid(W1, W2, xs, ys, T, K, D, steps, lr=0.1, sum_inside_tensor_group=False):
    """Returns (W1, W2 reassembled, params held per device (max), data-axis
    elements sent by the busiest device per step)."""
    h, n = W1.shape
    assert h % T == 0 and K in (1, 2)
    hs = h // T
    # device (d, k, t) holds its slices; with K = 1 a device holds both layers
    w1 = {(d, t): W1[t * hs:(t + 1) * hs].copy() for d in range(D) for t in range(T)}
    w2 = {(d, t): W2[:, t * hs:(t + 1) * hs].copy() for d in range(D) for t in range(T)}
    held = (hs * n) * (2 if K == 1 else 1)
    sent_max = 0
    for _ in range(steps):
        g1, g2 = {}, {}
        for d in range(D):
            x, y = xs[d], ys[d]
            # forward: every tensor rank computes its slice of the hidden layer and
            # its partial output; the partial outputs are summed over the group
            hid = {t: np.tanh(x @ w1[(d, t)].T) for t in range(T)}
            out = sum(hid[t] @ w2[(d, t)].T for t in range(T))          # all-reduce on activations
            d_out = (out - y) / x.shape[0]
            for t in range(T):
                g2[(d, t)] = d_out.T @ hid[t]
                d_hid = (d_out @ w2[(d, t)]) * (1 - hid[t] * hid[t])
                g1[(d, t)] = d_hid.T @ x
            if sum_inside_tensor_group:
                # the mistake Theorem 6(3) rules out: also reducing weight gradients inside the group
                total = sum(g1[(d, t)] for t in range(T))
                for t in range(T):
                    g1[(d, t)] = total.copy()
        # data axis: ring all-reduce among the replicas that hold the same shard
        sent_step = 0
        for t in range(T):
            for which, g in ((1, g1), (2, g2)):
                flat = [g[(d, t)].reshape(-1) for d in range(D)]
                E = flat[0].size
                books = Books(D)
                red = ring_reduce_scatter(flat, bounds(E, D), 1, books, "rs")
                full = ring_all_gather(red, 1, books, "ag")
                per_layer = sum(int(s.max()) for _, s in books.phases)
                if K == 2:
                    sent_step = max(sent_step, per_layer)               # a device holds one layer
                elif which == 1:
                    first = per_layer
                else:
                    sent_step = max(sent_step, first + per_layer)       # a device holds both
                for d in range(D):
                    g[(d, t)] = (full[d] / D).reshape(g[(d, t)].shape)
        sent_max = max(sent_max, sent_step)
        for key in w1:
            w1[key] -= lr * g1[key]
            w2[key] -= lr * g2[key]
    W1n = np.concatenate([w1[(0, t)] for t in range(T)], axis=0)
    W2n = np.concatenate([w2[(0, t)] for t in range(T)], axis=1)
    consistent = all(np.array_equal(w1[(d, t)], w1[(0, t)]) and np.array_equal(w2[(d, t)], w2[(0, t)])
                     for d in range(D) for t in range(T))
    return W1n, W2n, held, sent_max, consistent
