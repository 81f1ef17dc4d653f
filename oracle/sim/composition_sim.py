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


# ---------------------------------------------------------------------------
# Traffic on the model axes, counted on a deeper network.
#
# `blocks` blocks a -> W2 tanh(W1 a) on a (b x n) boundary tensor of E = b*n
# elements; block l is split over the T devices of a tensor group as above
# (W1 by rows, W2 by columns) and the blocks are dealt to K pipeline stages,
# ceil(blocks / K) to a stage.  Every collective inside a tensor group is an
# explicit ring over the flattened boundary tensor with the shard boundaries of
# eq. (2) and counts the bytes each rank sends; every transfer between stages
# counts the bytes its sender sends.
#
#   tensor axis replicates activations (Table 2's (S,S,S,R)): a block's partial
#       outputs are all-reduced in the forward pass (Theorem 6: "All-Reduce on
#       activations"), the partial gradients with respect to its input in the
#       backward pass -- two all-reduces per block and micro-batch;
#   tensor axis shards activations ((S,S,S,S), sequence parallelism): a rank
#       holds an element shard of the boundary tensor between blocks; a block
#       all-gathers its input and reduce-scatters its output (and the same for
#       the gradients on the way back) -- the two halves of a ring all-reduce,
#       so the volume is the same (Section 2.3).  The gathered input of a block
#       is kept for its backward pass;
#   pipeline axis: rank t of a stage sends what it holds of the boundary tensor
#       (all of it, or its shard) to rank t of the next stage, and the gradient
#       comes back the same way.
#
# The gradient with respect to the network's input is part of the result (it
# is what an embedding in front of the first block would need), so the first
# block's backward collective is as necessary as every other.
def make_deep(blocks, n, h, b, D, seed):
    rng = np.random.default_rng(seed)
    W1 = [rng.normal(scale=0.6, size=(h, n)) for _ in range(blocks)]
    W2 = [rng.normal(scale=0.6, size=(n, h)) for _ in range(blocks)]
    xs = [rng.normal(size=(b, n)) for _ in range(D)]
    ys = [rng.uniform(-0.5, 0.5, size=(b, n)) for _ in range(D)]
    return W1, W2, xs, ys


def deep_grads(W1, W2, x, y, scale):
    """Gradients of scale * 0.5 ||net(x) - y||^2 summed over the samples; also
    the gradient with respect to x."""
    blocks = len(W1)
    a, hid = [x], []
    for l in range(blocks):
        hid.append(np.tanh(a[l] @ W1[l].T))
        a.append(hid[l] @ W2[l].T)
    d = (a[blocks] - y) * scale
    g1, g2 = [None] * blocks, [None] * blocks
    for l in reversed(range(blocks)):
        g2[l] = d.T @ hid[l]
        dh = (d @ W2[l]) * (1 - hid[l] * hid[l])
        g1[l] = dh.T @ a[l]
        d = dh @ W1[l]
    return g1, g2, d


def run_deep_single(W1, W2, xs, ys, steps, lr=0.05):
    x, y = np.concatenate(xs), np.concatenate(ys)
    W1, W2 = [w.copy() for w in W1], [w.copy() for w in W2]
    d_in = None
    for _ in range(steps):
        g1, g2, d_in = deep_grads(W1, W2, x, y, 1.0 / x.shape[0])
        for l in range(len(W1)):
            W1[l] -= lr * g1[l]
            W2[l] -= lr * g2[l]
    return W1, W2, d_in


class _Ranks:
    """The T ranks of one tensor group and the bytes they send, one record per
    collective (a ring phase is charged to its busiest rank, as in Section 2.3)."""

    def __init__(self, T, E, width):
        self.T, self.E, self.width = T, E, width
        self.cut = bounds(E, T)
        self.phases = []          # per ring phase: bytes sent by each rank

    def all_gather(self, shards):
        sent = np.zeros(self.T, dtype=np.int64)
        out = ring_all_gather(shards, self.width, None, None, sent)
        self.phases.append(sent)
        return out

    def reduce_scatter(self, fulls):
        sent = np.zeros(self.T, dtype=np.int64)
        out = ring_reduce_scatter(fulls, self.cut, self.width, None, None, sent)
        self.phases.append(sent)
        return out

    def busiest(self):
        return sum(int(s.max()) for s in self.phases)


def run_deep_grid(W1, W2, xs, ys, T, K, D, shard_activations, steps, width=2, lr=0.05):
    """Returns dict(W1, W2, d_in (last step, per replica), tensor_bytes, pipeline_bytes):
    tensor_bytes  = bytes a device sends inside its tensor group per step, for the
                    stage that sends most (each ring phase charged to its busiest rank);
    pipeline_bytes = bytes the busiest device sends to neighbouring stages per step."""
    blocks = len(W1)
    h, n = W1[0].shape
    b = xs[0].shape[0]
    E = b * n
    assert h % T == 0
    hs = h // T
    per_stage = -(-blocks // K)
    stage_of = [l // per_stage for l in range(blocks)]
    w1 = [[W1[l][t * hs:(t + 1) * hs].copy() for t in range(T)] for l in range(blocks)]
    w2 = [[W2[l][:, t * hs:(t + 1) * hs].copy() for t in range(T)] for l in range(blocks)]
    cut = bounds(E, T)
    tensor_bytes = pipeline_bytes = 0
    d_in_last = None
    for _ in range(steps):
        G1 = [[np.zeros_like(w1[l][t]) for t in range(T)] for l in range(blocks)]
        G2 = [[np.zeros_like(w2[l][t]) for t in range(T)] for l in range(blocks)]
        d_in_last = []
        step_tensor = np.zeros(K, dtype=np.int64)             # per stage (any replica: they do the same)
        step_pipe = np.zeros((K, T), dtype=np.int64)
        for d in range(D):
            groups = [_Ranks(T, E, width) for _ in range(K)]  # this replica's tensor group of every stage
            pipe = np.zeros((K, T), dtype=np.int64)
            scale = 1.0 / (b * D)

            def hand_over(held, src, dst):
                # rank t of stage src sends what it holds to rank t of stage dst
                for t in range(T):
                    pipe[src, t] += held[t].size * width
                return [p.copy() for p in held]

            # ---- forward
            if shard_activations:
                held = [xs[d].reshape(-1)[cut[t]:cut[t + 1]].copy() for t in range(T)]
            else:
                held = [xs[d].reshape(-1).copy() for _ in range(T)]
            a_in, hid = [None] * blocks, [None] * blocks
            for l in range(blocks):
                k = stage_of[l]
                if l > 0 and stage_of[l - 1] != k:
                    held = hand_over(held, stage_of[l - 1], k)
                full = groups[k].all_gather(held) if shard_activations else held
                a_in[l] = [f.reshape(b, n) for f in full]
                hid[l] = [np.tanh(a_in[l][t] @ w1[l][t].T) for t in range(T)]
                partial = [(hid[l][t] @ w2[l][t].T).reshape(-1) for t in range(T)]
                summed = groups[k].reduce_scatter(partial)
                held = summed if shard_activations else groups[k].all_gather(summed)
            # ---- loss gradient on what each rank holds of the output
            y_flat = ys[d].reshape(-1)
            if shard_activations:
                held = [(held[t] - y_flat[cut[t]:cut[t + 1]]) * scale for t in range(T)]
            else:
                held = [(held[t] - y_flat) * scale for t in range(T)]
            # ---- backward
            for l in reversed(range(blocks)):
                k = stage_of[l]
                if l < blocks - 1 and stage_of[l + 1] != k:
                    held = hand_over(held, stage_of[l + 1], k)
                full = groups[k].all_gather(held) if shard_activations else held
                partial = []
                for t in range(T):
                    dout = full[t].reshape(b, n)
                    G2[l][t] += dout.T @ hid[l][t]
                    dh = (dout @ w2[l][t]) * (1 - hid[l][t] * hid[l][t])
                    G1[l][t] += dh.T @ a_in[l][t]            # complete for the rank's rows: no sum in the group
                    partial.append((dh @ w1[l][t]).reshape(-1))
                summed = groups[k].reduce_scatter(partial)
                held = summed if shard_activations else groups[k].all_gather(summed)
            if shard_activations:
                d_in_last.append(np.concatenate(held).reshape(b, n))
            else:
                d_in_last.append(held[0].reshape(b, n))
            for k in range(K):
                step_tensor[k] = max(step_tensor[k], groups[k].busiest())
            step_pipe = np.maximum(step_pipe, pipe)
        tensor_bytes = max(tensor_bytes, int(step_tensor.max()))
        pipeline_bytes = max(pipeline_bytes, int(step_pipe.max()))
        # data axis: the replicas' gradient contributions add up (the ring that does it is
        # counted by run_grid above and by the placement simulator)
        for l in range(blocks):
            for t in range(T):
                w1[l][t] -= lr * G1[l][t]
                w2[l][t] -= lr * G2[l][t]
    W1n = [np.concatenate(w1[l], axis=0) for l in range(blocks)]
    W2n = [np.concatenate(w2[l], axis=1) for l in range(blocks)]
    return dict(W1=W1n, W2=W2n, d_in=d_in_last, tensor_bytes=tensor_bytes, pipeline_bytes=pipeline_bytes)
