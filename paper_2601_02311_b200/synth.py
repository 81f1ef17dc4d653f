"""Seeded synthetic inputs for the placement-semantics sweep.

This module only *draws inputs*: transformer shapes and the parameters of the
design space to sweep (device counts, enumeration limits, mode mask).  It holds
none of the method's arithmetic (no parameter counts, no memory or
communication formulas), so both the CUDA library and the independent CPU
oracle can be fed from it without sharing any logic.

Shapes are produced as a numpy structured array whose 48-byte records have the
byte layout of the C struct ``ps_model_shape``; a space is a plain dict.

The paper evaluates no dataset; these workloads follow the value distributions
of the five synthetic configurations the benchmark is quoted on (worked
example, shape zoo, composition sweep, Pareto sweep, stress sweep).
"""
from __future__ import annotations

import numpy as np

# Byte layout of one model shape (48 bytes, little endian, no implicit padding).
SHAPE_DTYPE = np.dtype(
    [
        ("param_elems_override", "<u8"),
        ("layers", "<u4"),
        ("hidden", "<u4"),
        ("heads", "<u4"),
        ("vocab", "<u4"),
        ("seq", "<u4"),
        ("micro_batch", "<u4"),
        ("w_param", "u1"),
        ("w_grad", "u1"),
        ("w_opt", "u1"),
        ("w_act", "u1"),
        ("unit_from_shape", "u1"),
        ("act_enabled", "u1"),
        ("pad", "u1", (10,)),
    ]
)
assert SHAPE_DTYPE.itemsize == 48

_MASK64 = (1 << 64) - 1


class SplitMix64:
    """The SplitMix64 generator (Steele, Lea, Flood 2014): a 64-bit counter
    advanced by the golden-ratio increment and finalised by two xor-shift
    multiplies.  "Uniform in [lo, hi]" below means ``lo + next() % (hi-lo+1)``.
    """

    def __init__(self, seed: int):
        self.state = seed & _MASK64

    def next(self) -> int:
        self.state = (self.state + 0x9E3779B97F4A7C15) & _MASK64
        z = self.state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
        return z ^ (z >> 31)

    def uniform(self, lo: int, hi: int) -> int:
        return lo + self.next() % (hi - lo + 1)

    def choice(self, values):
        return values[self.next() % len(values)]


def zoo(n_models: int, seed: int, *, max_layers: int = 128, max_hidden_mult: int = 128,
        seqs=(2048, 4096, 8192), max_micro_batch: int = 16) -> np.ndarray:
    """Decoder-only transformer shapes.

    Draw order per model: layers, hidden multiple k, vocab, sequence choice,
    micro-batch.  hidden = 128*k, heads = k (head dimension 128), FFN = 4*hidden
    is implied by the paper's 12*H^2 per-layer count.  Mixed-precision Adam
    accounting: 2 B parameters, 2 B gradients, 12 B optimizer+master, 2 B
    activations elements.
    """
    rng = SplitMix64(seed)
    out = np.zeros(n_models, dtype=SHAPE_DTYPE)
    for i in range(n_models):
        layers = rng.uniform(12, max_layers)
        k = rng.uniform(6, max_hidden_mult)
        vocab = rng.uniform(32000, 256000)
        seq = rng.choice(list(seqs))
        mb = rng.uniform(1, max_micro_batch)
        r = out[i]
        r["param_elems_override"] = 0
        r["layers"] = layers
        r["hidden"] = 128 * k
        r["heads"] = k
        r["vocab"] = vocab
        r["seq"] = seq
        r["micro_batch"] = mb
        r["w_param"], r["w_grad"], r["w_opt"], r["w_act"] = 2, 2, 12, 2
        r["unit_from_shape"] = 1
        r["act_enabled"] = 1
    return out


def worked_example(with_unit: bool = False) -> np.ndarray:
    """The paper's 70-billion-parameter example (Table 1, Examples 3 and 4):
    the parameter count is given directly, activations are excluded.  With
    ``with_unit`` the shape of an 80-layer, H = 8192 model is attached so the
    reconstruction-unit term of Theorem 1 becomes visible."""
    out = np.zeros(1, dtype=SHAPE_DTYPE)
    r = out[0]
    r["param_elems_override"] = 70_000_000_000
    r["w_param"], r["w_grad"], r["w_opt"], r["w_act"] = 2, 2, 12, 2
    if with_unit:
        r["layers"], r["hidden"], r["heads"] = 80, 8192, 64
        r["vocab"], r["seq"], r["micro_batch"] = 32000, 4096, 1
        r["unit_from_shape"] = 1
    else:
        # a shape is still needed for the divisibility predicates; one layer,
        # one head keeps every T=K=1 point composition-valid
        r["layers"], r["hidden"], r["heads"] = 1, 1, 1
        r["vocab"], r["seq"], r["micro_batch"] = 1, 1, 1
        r["unit_from_shape"] = 0
    r["act_enabled"] = 0
    return out


def _space(models, n_values, *, t_enum_max, k_enum_max, n_act, n_tpa, mode_mask,
           tp_max_valid=8, tp_coll_per_layer=4):
    return dict(
        models=models,
        n_values=np.asarray(n_values, dtype=np.uint32),
        t_enum_max=t_enum_max,
        k_enum_max=k_enum_max,
        tp_max_valid=tp_max_valid,
        n_act_variants=n_act,
        n_tpa_variants=n_tpa,
        mode_mask=mode_mask,
        tp_coll_per_layer=tp_coll_per_layer,
    )


GB = 10 ** 9  # the paper's "GB" is decimal: 16 B x 70e9 = "1120 GB"

ALL_MODES = 0x1F
NO_OFFLOAD = 0x0F


def config(name: str, *, n_models: int | None = None) -> dict:
    """The five benchmark configurations (and the unit-term variant of the
    first).  ``n_models`` shrinks the zoo for tests; the distributions stay."""
    pow2 = lambda top: [1 << j for j in range(top + 1)]
    if name == "C0":
        return _space(worked_example(False), pow2(6), t_enum_max=1, k_enum_max=1,
                      n_act=1, n_tpa=1, mode_mask=ALL_MODES)
    if name == "C0b":
        return _space(worked_example(True), pow2(6), t_enum_max=1, k_enum_max=1,
                      n_act=1, n_tpa=1, mode_mask=ALL_MODES)
    if name == "C1":
        return _space(zoo(n_models or 256, 0), pow2(10), t_enum_max=1, k_enum_max=1,
                      n_act=2, n_tpa=1, mode_mask=ALL_MODES)
    if name == "C2":
        return _space(zoo(n_models or 256, 1), pow2(12), t_enum_max=8, k_enum_max=1 << 14,
                      n_act=2, n_tpa=2, mode_mask=NO_OFFLOAD)
    if name == "C3":
        return _space(zoo(n_models or 1024, 2, max_layers=160, max_hidden_mult=256),
                      pow2(12), t_enum_max=8, k_enum_max=1 << 14,
                      n_act=2, n_tpa=2, mode_mask=ALL_MODES)
    if name == "C4":
        return _space(zoo(n_models or 4096, 3, max_layers=160, max_hidden_mult=256,
                          seqs=(2048, 4096, 8192, 16384, 32768), max_micro_batch=64),
                      pow2(14), t_enum_max=1 << 14, k_enum_max=1 << 14,
                      n_act=2, n_tpa=2, mode_mask=ALL_MODES)
    raise KeyError(name)


# exact number of points of each full-size configuration
FULL_SIZE = {"C0": 4375, "C0b": 4375, "C1": 3_520_000, "C2": 76_021_760,
             "C3": 742_400_000, "C4": 6_963_200_000}


def ragged_space(seed: int, n_models: int = 3) -> dict:
    """A small space with awkward device counts (not powers of two, primes,
    repeated factors) and a 3-mode mask, for edge-case parity tests."""
    models = zoo(n_models, seed, max_layers=48, max_hidden_mult=24)
    return _space(models, [1, 2, 3, 6, 7, 12, 30, 36, 97, 360], t_enum_max=12,
                  k_enum_max=36, n_act=2, n_tpa=2, mode_mask=0b10110)


def select_queries(n: int, seed: int) -> np.ndarray:
    """Queries for the batched Algorithm 1 as an (n, 8) uint64 array: parameter
    count P (a mantissa in [1, 10) times a power of ten between 1e8 and 1e12),
    elements of one layer (a fraction of P between 1/160 and 1/12, or 0 now and
    then), device bytes in {16, 24, 40, 80, 141, 192} GB, N a power of two up to
    2^14 (or an odd count now and then), byte widths 2/2/12, fast interconnect or
    not.  Both sizes are drawn, not derived from a shape."""
    rng = SplitMix64(seed)
    out = np.zeros((n, 8), dtype=np.uint64)
    for i in range(n):
        params = rng.uniform(1000, 9999) * 10 ** rng.uniform(5, 9)
        layers = rng.uniform(12, 160)
        out[i, 0] = params
        out[i, 1] = params // layers if rng.next() % 8 else 0
        out[i, 2] = rng.choice([16, 24, 40, 80, 141, 192]) * GB
        out[i, 3] = (1 << rng.uniform(0, 14)) if rng.next() % 6 else rng.uniform(1, 3000)
        out[i, 4], out[i, 5], out[i, 6] = 2, 2, 12
        out[i, 7] = rng.next() % 2
    return out


def table_checksum(models: np.ndarray) -> int:
    """Order-dependent 64-bit checksum of a shape table (printed by the bench so
    that two runs can be seen to use the same inputs)."""
    h = 0xCBF29CE484222325
    for b in models.tobytes():
        h = ((h ^ b) * 0x100000001B3) & _MASK64
    return h
