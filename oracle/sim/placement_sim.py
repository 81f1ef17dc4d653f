"""TEST INFRASTRUCTURE -- brute-force simulator of one data-parallel axis.

A few logical devices inside one process train a tiny layered network with
Adam in fp64.  Every state (parameters Theta, optimizer state Omega with the
master copy inside it, gradients G, activations A) is held exactly as its
placement mode says (Definition 1): full copies, contiguous element shards with
the boundaries of eq. (2), nothing, or shards in a separate "host" arena.
Collectives are explicit rings that move chunks from neighbour to neighbour
and count the elements each device sends (Section 2.3).  Whatever a placement
leaves unavailable when it is needed is read as zeros, so a placement that
breaks gradient integrity (Theorem 3) or state consistency (Theorem 4) really
diverges from the single-device run (Definition 4, Theorem 5).

The simulator knows nothing of the closed-form rules; it only executes the
mechanism and keeps books:

  * per state, the high-water mark of bytes a device holds persistently and of
    the unit-sized transient buffer it reconstructs into (Theorem 1's two parts);
  * per logical collective, the bytes the busiest device sends;
  * bytes that cross the host link of a device.

The execution order per step: (1) make Theta available, forward; (2) keep or
drop activations; (3) make Theta available again, backward; (4) synchronise
and deliver gradients; (5) update on the range whose update this device
commits (the whole tensor if Omega is replicated, its shard if Omega's home is
a shard); (6) put Theta back into its home.

Only tests import this module.
"""
from __future__ import annotations

import numpy as np

R, S, SG, M, O = 0, 1, 2, 3, 4   # SG is the paper's S*

W_THETA, W_OMEGA, W_GRAD = 2, 12, 2   # bytes per element (Remark 1); activations count 1 B each


def bounds(E: int, D: int):
    """eq. (2): shard i is [floor(i E / D), floor((i+1) E / D))."""
    return [(i * E) // D for i in range(D + 1)]


class Books:
    def __init__(self, D):
        self.D = D
        self.persist = {}      # state -> per-device high-water bytes
        self.transient = {}    # state -> high-water bytes of the unit buffer
        self.phases = []       # (name, per-device bytes sent)
        self.host = np.zeros(D, dtype=np.int64)

    def hold(self, state, dev, nbytes):
        a = self.persist.setdefault(state, np.zeros(self.D, dtype=np.int64))
        a[dev] = max(a[dev], nbytes)

    def unit_buffer(self, state, nbytes):
        self.transient[state] = max(self.transient.get(state, 0), nbytes)

    def memory(self):
        total = 0
        for st in ("theta", "omega", "grad", "act"):
            p = self.persist.get(st)
            total += (int(p.max()) if p is not None else 0) + self.transient.get(st, 0)
        return total

    def comm(self):
        return sum(int(sent.max()) for _, sent in self.phases)

    def host_bytes(self):
        return int(self.host.max())


def ring_all_gather(chunks, width, books, name, sent=None):
    """chunks[i] is device i's piece; every device ends with all pieces.  Step s:
    device i passes the piece that originated at (i - s) mod D to device i+1."""
    D = len(chunks)
    have = [{i: chunks[i]} for i in range(D)]
    own_sent = np.zeros(D, dtype=np.int64) if sent is None else sent
    for s in range(D - 1):
        moving = []
        for i in range(D):
            c = (i - s) % D
            moving.append((c, have[i][c]))
            own_sent[i] += len(have[i][c]) * width
        for i in range(D):
            c, data = moving[i]
            have[(i + 1) % D][c] = data.copy()
    if sent is None:
        books.phases.append((name, own_sent))
    return [np.concatenate([have[i][c] for c in range(D)]) for i in range(D)]


def ring_reduce_scatter(full, cuts, width, books, name, sent=None):
    """full[i] is device i's whole vector; device i ends with the sum of chunk i
    (chunk c = [cuts[c], cuts[c+1])).  Step s: device i adds its part to the
    travelling partial sum of chunk (i - 1 - s) mod D and passes it on."""
    D = len(full)
    partial = [{c: full[i][cuts[c]:cuts[c + 1]].copy() for c in range(D)} for i in range(D)]
    own_sent = np.zeros(D, dtype=np.int64) if sent is None else sent
    for s in range(D - 1):
        moving = []
        for i in range(D):
            c = (i - 1 - s) % D
            moving.append((c, partial[i][c]))
            own_sent[i] += len(partial[i][c]) * width
        for i in range(D):
            c, data = moving[i]
            j = (i + 1) % D
            partial[j][c] = partial[j][c] + data
    if sent is None:
        books.phases.append((name, own_sent))
    return [partial[i][i] for i in range(D)]


class ToyModel:
    """`units` layers; layer l scales its input elementwise by h parameters and
    applies tanh.  The stored activation of a layer is its input (b x h)."""

    def __init__(self, units, h):
        self.units, self.h = units, h
        self.P = units * h

    def forward(self, theta, x):
        acts = np.zeros((self.units, x.shape[0], self.h))
        cur = x
        for l in range(self.units):
            acts[l] = cur
            cur = np.tanh(theta[l * self.h:(l + 1) * self.h] * cur)
        return acts, cur

    def backward(self, theta, acts, y):
        """Mean-over-samples gradient of 0.5*||out - y||^2, using the given
        parameters and the given stored activations."""
        b = y.shape[0]
        last = np.tanh(theta[(self.units - 1) * self.h:] * acts[self.units - 1])
        dh = (last - y) / b
        g = np.zeros(self.P)
        for l in reversed(range(self.units)):
            th = theta[l * self.h:(l + 1) * self.h]
            out = np.tanh(th * acts[l])
            dz = dh * (1.0 - out * out)
            g[l * self.h:(l + 1) * self.h] = (dz * acts[l]).sum(axis=0)
            dh = dz * th
        return g


def adam(omega, grad, t, lr=0.05, b1=0.9, b2=0.999, eps=1e-8):
    """omega rows: master copy, first moment, second moment.  Returns new omega."""
    master, m, v = omega
    m = b1 * m + (1 - b1) * grad
    v = b2 * v + (1 - b2) * grad * grad
    mh = m / (1 - b1 ** t)
    vh = v / (1 - b2 ** t)
    master = master - lr * mh / (np.sqrt(vh) + eps)
    return np.stack([master, m, v])


def make_problem(units, h, b, D, seed, accum=1):
    """xs[j][i], ys[j][i]: micro-batch j of device i (accum micro-batches per step)."""
    rng = np.random.default_rng(seed)
    theta0 = rng.uniform(0.5, 1.5, units * h)
    xs = [[rng.normal(size=(b, h)) for _ in range(D)] for _ in range(accum)]
    ys = [[rng.uniform(-0.8, 0.8, size=(b, h)) for _ in range(D)] for _ in range(accum)]
    return theta0, xs, ys


def run_single(units, h, xs, ys, theta0, steps):
    """The single-device run on the global batch (Definition 4's yardstick):
    all micro-batches of all devices in one batch."""
    model = ToyModel(units, h)
    x = np.concatenate([xi for xj in xs for xi in xj])
    y = np.concatenate([yi for yj in ys for yi in yj])
    omega = np.stack([theta0.copy(), np.zeros_like(theta0), np.zeros_like(theta0)])
    theta = theta0.copy()
    traj = []
    for t in range(1, steps + 1):
        acts, _ = model.forward(theta, x)
        g = model.backward(theta, acts, y)
        omega = adam(omega, g, t)
        theta = omega[0].copy()
        traj.append((theta.copy(), omega.copy()))
    return traj


class Placed:
    """D devices executing one placement (pi_theta, pi_omega, pi_grad, pi_act).

    `copies` = k-way replication of the sharded modes: the D devices form k shard
    groups of G = D / k devices each (k = gcd(copies, D)); device i sits at shard
    position i mod G of group i div G.  A sharded state is cut into G shards
    (eq. (2)) and shard p is held by the k devices at position p.  Gathers run
    inside a shard group; a gradient is reduced to shards by a reduce-scatter
    inside every shard group followed by an all-reduce of each shard across its
    k copies.  copies = 1 is plain sharding over all D devices."""

    def __init__(self, units, h, b, D, code, theta0, gather_buffers=1, copies=1):
        self.model = ToyModel(units, h)
        # unit buffers a gathered state holds: 2 when the next unit is fetched while
        # the current one is in use (only possible with at least two units)
        self.nbuf = min(gather_buffers, units)
        self.units, self.h, self.b, self.D = units, h, b, D
        self.k = int(np.gcd(copies, D))
        self.G = D // self.k
        self.pT, self.pO, self.pG, self.pA = code % 5, (code // 5) % 5, (code // 25) % 5, code // 125
        self.P = units * h
        self.cut = bounds(self.P, self.G)          # shard positions
        self.cutD = bounds(self.P, D)              # chunks of a ring over all D devices
        self.EA = units * b * h
        self.cutA = bounds(self.EA, self.G)
        omega0 = np.stack([theta0.copy(), np.zeros_like(theta0), np.zeros_like(theta0)])
        # persistent homes; None = not held.  "host" is a separate arena.
        self.theta_gpu = [None] * D
        self.theta_host = [None] * D
        self.omega_gpu = [None] * D
        self.omega_host = [None] * D
        for i in range(D):
            lo, hi = self.shard(i)
            if self.pT == R: self.theta_gpu[i] = theta0.copy()
            elif self.pT in (S, SG): self.theta_gpu[i] = theta0[lo:hi].copy()
            elif self.pT == O: self.theta_host[i] = theta0[lo:hi].copy()
            if self.pO == R: self.omega_gpu[i] = omega0.copy()
            elif self.pO in (S, SG): self.omega_gpu[i] = omega0[:, lo:hi].copy()
            elif self.pO == O: self.omega_host[i] = omega0[:, lo:hi].copy()
        self.update_on_shard = self.pO in (S, SG, O)

    def shard(self, i):
        p = i % self.G
        return self.cut[p], self.cut[p + 1]

    def group_gather(self, pieces, width, sent):
        """All-gather inside every shard group: pieces[i] is device i's piece; returns
        per device the concatenation of its group's pieces (position order)."""
        G, out = self.G, [None] * self.D
        for c in range(self.k):
            tmp = np.zeros(G, dtype=np.int64)
            got = ring_all_gather([pieces[c * G + p] for p in range(G)], width, None, None, tmp)
            for p in range(G):
                out[c * G + p] = got[p]
                sent[c * G + p] += tmp[p]
        return out

    def reduce_to_shards(self, vectors, lo, hi, width, sent_group, sent_rs, sent_ag):
        """Sum over all D devices of vectors[i][lo:hi], delivered as shards: device i
        ends with the part of [lo, hi) inside its shard.  A reduce-scatter inside
        every shard group, then an all-reduce of each shard across its k copies
        whose pieces follow the eq.-(2) cuts of the whole shard."""
        G, k, D = self.G, self.k, self.D
        ucut = [min(max(c, lo), hi) - lo for c in self.cut]
        part = [None] * D
        for c in range(k):
            tmp = np.zeros(G, dtype=np.int64)
            red = ring_reduce_scatter([vectors[c * G + p][lo:hi] for p in range(G)], ucut, width, None, None, tmp)
            for p in range(G):
                part[c * G + p] = red[p]
                sent_group[c * G + p] += tmp[p]
        if k > 1:
            for p in range(G):
                s_lo, s_hi = self.cut[p], self.cut[p + 1]
                sub = [s_lo + (q * (s_hi - s_lo)) // k for q in range(k + 1)]      # cuts of the whole shard
                a0 = min(max(s_lo, lo), hi)                                          # start of this part of it
                rel = [min(max(x, lo), hi) - a0 for x in sub]
                t1, t2 = np.zeros(k, dtype=np.int64), np.zeros(k, dtype=np.int64)
                pieces = ring_reduce_scatter([part[c * G + p] for c in range(k)], rel, width, None, None, t1)
                full = ring_all_gather(pieces, width, None, None, t2)
                for c in range(k):
                    part[c * G + p] = full[c]
                    sent_rs[c * G + p] += t1[c]
                    sent_ag[c * G + p] += t2[c]
        return part

    # ---- Theta as seen by forward / backward on every device
    def theta_for_compute(self, books, tag):
        D, P, h = self.D, self.P, self.h
        out = []
        if self.pT == R:
            for i in range(D):
                books.hold("theta", i, P * W_THETA)
                out.append(self.theta_gpu[i].copy())
        elif self.pT == S:
            for i in range(D):
                lo, hi = self.shard(i)
                books.hold("theta", i, (hi - lo) * W_THETA)
                full = np.zeros(P)
                full[lo:hi] = self.theta_gpu[i]
                out.append(full)
        elif self.pT in (SG, O):
            shards = []
            for i in range(D):
                lo, hi = self.shard(i)
                if self.pT == SG:
                    books.hold("theta", i, (hi - lo) * W_THETA)
                    shards.append(self.theta_gpu[i])
                else:
                    books.host[i] += (hi - lo) * W_THETA          # host -> device
                    shards.append(self.theta_host[i])
            # gathered one reconstruction unit (layer) at a time into a unit buffer
            sent = np.zeros(D, dtype=np.int64)
            fulls = [np.zeros(P) for _ in range(D)]
            for l in range(self.units):
                a, b_ = l * h, (l + 1) * h
                pieces = []
                for i in range(D):
                    lo, hi = self.shard(i)
                    s0, s1 = max(a, lo), min(b_, hi)
                    pieces.append(shards[i][s0 - lo:s1 - lo] if s1 > s0 else np.zeros(0))
                got = self.group_gather(pieces, W_THETA, sent)
                if self.pT == SG:
                    books.unit_buffer("theta", self.nbuf * h * W_THETA)
                for i in range(D):
                    fulls[i][a:b_] = got[i]
            books.phases.append(("gather theta " + tag, sent))
            out = fulls
        else:  # M: cast from the master copy, where Omega is resident
            for i in range(D):
                full = np.zeros(P)
                if self.omega_gpu[i] is not None:
                    if self.pO == R:
                        full[:] = self.omega_gpu[i][0]
                    else:
                        lo, hi = self.shard(i)
                        full[lo:hi] = self.omega_gpu[i][0]
                books.unit_buffer("theta", h * W_THETA)
                out.append(full)
        return out

    def step(self, t, xs, ys, books):
        """One optimizer step over len(xs) micro-batches per device: forward and
        backward run per micro-batch, the local gradients add up (that buffer is
        not a placed state), everything from (4) on happens once."""
        D, P = self.D, self.P
        accum = len(xs)
        local = [np.zeros(P) for _ in range(D)]
        for j in range(accum):
            mb = self.micro_batch(xs[j], ys[j], books)
            for i in range(D):
                local[i] += mb[i] / accum
        self.finish_step(t, local, books)

    def micro_batch(self, xs, ys, books):
        D, P, h, b = self.D, self.P, self.h, self.b
        model = self.model
        # (1) forward
        th_f = self.theta_for_compute(books, "fwd")
        acts = [model.forward(th_f[i], xs[i])[0] for i in range(D)]
        # (2) activations between forward and backward
        kept = []
        if self.pA == R:
            for i in range(D):
                books.hold("act", i, self.EA)
                kept.append(acts[i])
        elif self.pA == O:
            for i in range(D):
                books.host[i] += 2 * self.EA                     # device -> host, host -> device
                kept.append(acts[i])
        elif self.pA in (S, SG):
            slices = []
            for i in range(D):
                p = i % self.G
                lo, hi = self.cutA[p], self.cutA[p + 1]
                books.hold("act", i, hi - lo)
                slices.append(acts[i].reshape(-1)[lo:hi].copy())
            if self.pA == S:
                for i in range(D):
                    p = i % self.G
                    flat = np.zeros(self.EA)
                    flat[self.cutA[p]:self.cutA[p + 1]] = slices[i]
                    kept.append(flat.reshape(acts[i].shape))
            else:
                # gather from the peers of the shard group: their slices belong to other samples
                sent = np.zeros(D, dtype=np.int64)
                got = self.group_gather(slices, 1, sent)
                books.unit_buffer("act", self.nbuf * b * h)
                kept = [g.reshape(acts[0].shape) for g in got]
        # (3) Theta again for backward
        th_b = self.theta_for_compute(books, "bwd")
        if self.pA == M:
            books.unit_buffer("act", b * h)
            kept = [model.forward(th_b[i], xs[i])[0] for i in range(D)]   # recomputed
        return [model.backward(th_b[i], kept[i], ys[i]) for i in range(D)]

    def finish_step(self, t, local, books):
        D, P, h, b = self.D, self.P, self.h, self.b
        # (4) synchronise / deliver gradients (mean over the D replicas)
        grad = [np.zeros(P) for _ in range(D)]     # what the update will read
        zeros = lambda: np.zeros(D, dtype=np.int64)
        if self.pG == R:
            red = ring_reduce_scatter(local, self.cutD, W_GRAD, books, "grad reduce-scatter")
            full = ring_all_gather(red, W_GRAD, books, "grad all-gather")
            for i in range(D):
                books.hold("grad", i, P * W_GRAD)
                grad[i] = full[i] / D
        elif self.pG in (S, O, SG):
            s1, s2, s3 = zeros(), zeros(), zeros()
            red = self.reduce_to_shards(local, 0, P, W_GRAD, s1, s2, s3)
            books.phases += [("grad reduce-scatter in the shard group", s1), ("shard reduce-scatter across copies", s2),
                             ("shard all-gather across copies", s3)]
            if self.pG in (S, O):
                for i in range(D):
                    lo, hi = self.shard(i)
                    if self.pG == S:
                        books.hold("grad", i, (hi - lo) * W_GRAD)
                    else:
                        books.host[i] += 2 * (hi - lo) * W_GRAD      # offload, reload at the update
                    grad[i][lo:hi] = red[i] / D
            else:
                for i in range(D):
                    lo, hi = self.shard(i)
                    books.hold("grad", i, (hi - lo) * W_GRAD)
                sent = zeros()
                for l in range(self.units):
                    a, b_ = l * h, (l + 1) * h
                    pieces = []
                    for i in range(D):
                        lo, hi = self.shard(i)
                        s0, s1_ = max(a, lo), min(b_, hi)
                        pieces.append(red[i][s0 - lo:s1_ - lo] if s1_ > s0 else np.zeros(0))
                    got = self.group_gather(pieces, W_GRAD, sent)
                    books.unit_buffer("grad", self.nbuf * h * W_GRAD)
                    for i in range(D):
                        grad[i][a:b_] = got[i] / D
                books.phases.append(("grad all-gather before use", sent))
        else:  # M: reduced unit by unit as produced, consumed at once
            s1, s2, s3, sent_ag = zeros(), zeros(), zeros(), zeros()
            for l in range(self.units):
                a, b_ = l * h, (l + 1) * h
                books.unit_buffer("grad", h * W_GRAD)
                if self.update_on_shard:
                    red = self.reduce_to_shards(local, a, b_, W_GRAD, s1, s2, s3)
                    for i in range(D):
                        lo, hi = self.shard(i)
                        s0, s1_ = min(max(lo, a), b_), min(max(hi, a), b_)
                        grad[i][s0:s1_] = red[i] / D
                else:
                    ucut = [min(max(c, a), b_) - a for c in self.cutD]
                    red = ring_reduce_scatter([g[a:b_] for g in local], ucut, W_GRAD, books, None, s1)
                    got = ring_all_gather(red, W_GRAD, books, None, sent_ag)
                    for i in range(D):
                        grad[i][a:b_] = got[i] / D
            books.phases.append(("grad reduce per unit", s1))
            if self.update_on_shard:
                books.phases += [("unit shard reduce-scatter across copies", s2), ("unit shard all-gather across copies", s3)]
            else:
                books.phases.append(("grad gather per unit", sent_ag))
        # (5) update
        new_theta = [np.zeros(P) for _ in range(D)]   # valid on the committed range
        for i in range(D):
            lo, hi = self.shard(i)
            if self.pO == R:
                books.hold("omega", i, P * W_OMEGA)
                self.omega_gpu[i] = adam(self.omega_gpu[i], grad[i], t)
                new_theta[i] = self.omega_gpu[i][0].copy()
            elif self.pO == S:
                books.hold("omega", i, (hi - lo) * W_OMEGA)
                self.omega_gpu[i] = adam(self.omega_gpu[i], grad[i][lo:hi], t)
                new_theta[i][lo:hi] = self.omega_gpu[i][0]
            elif self.pO == O:
                books.host[i] += 2 * (hi - lo) * W_OMEGA          # load, store
                self.omega_host[i] = adam(self.omega_host[i], grad[i][lo:hi], t)
                new_theta[i][lo:hi] = self.omega_host[i][0]
            elif self.pO == M:
                lost = adam(np.zeros((3, P)), grad[i], t)         # nothing was kept
                new_theta[i] = lost[0]
        if self.pO == SG:
            # gather all of Omega unit by unit, use it, keep only the own shard's update
            sent = zeros()
            for l in range(self.units):
                a, b_ = l * h, (l + 1) * h
                pieces = []
                for i in range(D):
                    lo, hi = self.shard(i)
                    s0, s1_ = max(a, lo), min(b_, hi)
                    pieces.append(self.omega_gpu[i][0, s0 - lo:s1_ - lo] if s1_ > s0 else np.zeros(0))
                for _row in range(3):          # master, m, v: 3 x 4 bytes per element
                    self.group_gather(pieces, W_OMEGA // 3, sent)
                books.unit_buffer("omega", self.nbuf * h * W_OMEGA)
            books.phases.append(("gather omega", sent))
            for i in range(D):
                lo, hi = self.shard(i)
                books.hold("omega", i, (hi - lo) * W_OMEGA)
                self.omega_gpu[i] = adam(self.omega_gpu[i], grad[i][lo:hi], t)
                new_theta[i][lo:hi] = self.omega_gpu[i][0]
        # (6) Theta back to its home
        if self.pT == R:
            if self.update_on_shard:
                pieces = [new_theta[i][slice(*self.shard(i))] for i in range(D)]
                sent = zeros()
                got = self.group_gather(pieces, W_THETA, sent)
                books.phases.append(("re-replicate theta", sent))
                for i in range(D):
                    self.theta_gpu[i] = got[i]
            else:
                for i in range(D):
                    self.theta_gpu[i] = new_theta[i].copy()
        elif self.pT in (S, SG):
            for i in range(D):
                self.theta_gpu[i] = new_theta[i][slice(*self.shard(i))].copy()
        elif self.pT == O:
            for i in range(D):
                lo, hi = self.shard(i)
                books.host[i] += (hi - lo) * W_THETA   # device -> host
                self.theta_host[i] = new_theta[i][lo:hi].copy()

    # ---- what the job as a whole holds after a step
    def reassemble(self):
        """Returns (list of Theta views, list of Omega views): one per holder (one per
        shard group for a sharded state); a placement is consistent only if every
        view equals the single-device state.  An empty list means the state is
        held nowhere."""
        D, G, k = self.D, self.G, self.k
        groups = [range(c * G, (c + 1) * G) for c in range(k)]
        if self.pO == R:
            omegas = [self.omega_gpu[i] for i in range(D)]
        elif self.pO in (S, SG):
            omegas = [np.concatenate([self.omega_gpu[i] for i in g], axis=1) for g in groups]
        elif self.pO == O:
            omegas = [np.concatenate([self.omega_host[i] for i in g], axis=1) for g in groups]
        else:
            omegas = []
        if self.pT == R:
            thetas = [self.theta_gpu[i] for i in range(D)]
        elif self.pT in (S, SG):
            thetas = [np.concatenate([self.theta_gpu[i] for i in g]) for g in groups]
        elif self.pT == O:
            thetas = [np.concatenate([self.theta_host[i] for i in g]) for g in groups]
        else:
            thetas = [om[0] for om in omegas]   # Theta exists only as the master copy
        return thetas, omegas


def simulate_problem(units, h, b, D, code, theta0, xs, ys, steps=3, gather_buffers=1, copies=1):
    """As simulate(), on a given problem (theta0[P]; xs[j][i], ys[j][i] = micro-batch j of
    device i); also returns the parameters the job holds after the last step (first
    holder's view, None if they are held nowhere)."""
    ref = run_single(units, h, xs, ys, theta0, steps)
    job = Placed(units, h, b, D, code, theta0, gather_buffers, copies)
    match = True
    books = None
    thetas = []
    for t in range(1, steps + 1):
        books = Books(D)
        job.step(t, xs, ys, books)
        thetas, omegas = job.reassemble()
        rt, ro = ref[t - 1]
        if not thetas or not omegas:
            match = False
        for th in thetas:
            if not np.allclose(th, rt, rtol=1e-12, atol=1e-14):
                match = False
        for om in omegas:
            if not np.allclose(om, ro, rtol=1e-12, atol=1e-14):
                match = False
    return dict(match=match, mem=books.memory(), comm=books.comm(), host=books.host_bytes(),
                theta=thetas[0] if thetas else None, ref_theta=ref[-1][0])


def simulate(units, h, b, D, code, steps=3, seed=0, accum=1, gather_buffers=1, copies=1):
    """Run `steps` steps of `accum` micro-batches each; returns dict(match, mem,
    comm, host) where match says whether every step's reassembled Theta and Omega
    equal the single-device run to 1e-12 relative, and the byte figures are those
    of the last step.  gather_buffers = 2: a gathered state prefetches the next
    unit while the current one is in use."""
    theta0, xs, ys = make_problem(units, h, b, D, seed, accum)
    ref = run_single(units, h, xs, ys, theta0, steps)
    job = Placed(units, h, b, D, code, theta0, gather_buffers, copies)
    match = True
    books = None
    for t in range(1, steps + 1):
        books = Books(D)
        job.step(t, xs, ys, books)
        thetas, omegas = job.reassemble()
        rt, ro = ref[t - 1]
        if not thetas or not omegas:
            match = False
        for th in thetas:
            if not np.allclose(th, rt, rtol=1e-12, atol=1e-14):
                match = False
        for om in omegas:
            if not np.allclose(om, ro, rtol=1e-12, atol=1e-14):
                match = False
    return dict(match=match, mem=books.memory(), comm=books.comm(), host=books.host_bytes())
