"""TEST INFRASTRUCTURE -- loader for the CPU oracle (``ps_oracle.cpp``).

Compiles the oracle with g++ on first use and exposes its C functions through
ctypes with numpy buffers.  Only tests, the smoke check and the benchmark's
CPU-baseline leg may import this module; it imports nothing from the CUDA
package (inputs arrive as plain numpy arrays and dicts).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ps_oracle.cpp")
_LIB = os.path.join(_HERE, "libps_oracle.so")
_lock = threading.Lock()
_lib = None

ENTRY_DTYPE = np.dtype([("mem", "<u8"), ("comm", "<u8"), ("host", "<u8"), ("idx", "<u8"),
                        ("flags", "<u4"), ("pad", "<u4")])
assert ENTRY_DTYPE.itemsize == 40

KIND_PARETO, KIND_TOPK = 0, 1
COMM_PAPER, COMM_PAPER_PLUS_EXT = 0, 1
NO_LIMIT = (1 << 64) - 1

# flag bits (same meaning as the library's, stated independently)
F_GI, F_SC, F_CV, F_FEASIBLE = 1, 2, 4, 8
F_T_HEADS, F_K_LAYERS, F_TP_LE_MAX, F_AXIS_FORM = 16, 32, 64, 128
F_THETA_AVAIL, F_ACT_AVAIL, F_GRAD_COVER = 256, 512, 1024
F_USES_HOST, F_PAPER_PRICED = 2048, 4096


class _Desc(C.Structure):
    _fields_ = [("models", C.c_void_p), ("n_models", C.c_uint32),
                ("n_values", C.c_void_p), ("n_n", C.c_uint32),
                ("t_enum_max", C.c_uint32), ("k_enum_max", C.c_uint32),
                ("tp_max_valid", C.c_uint32), ("n_act_variants", C.c_uint32),
                ("n_tpa_variants", C.c_uint32), ("mode_mask", C.c_uint32),
                ("tp_coll_per_layer", C.c_uint32), ("sstar_units", C.c_uint32),
                ("grad_accum_steps", C.c_uint32), ("replication_k", C.c_uint32)]


class _Filter(C.Structure):
    _fields_ = [("host_cap", C.c_uint64), ("require_flags", C.c_uint32),
                ("comm_kind", C.c_uint32), ("cap_bytes", C.c_uint64)]


class _Point(C.Structure):
    _fields_ = [("model", C.c_uint32), ("N", C.c_uint32), ("T", C.c_uint32), ("K", C.c_uint32),
                ("D", C.c_uint32), ("act_variant", C.c_uint32), ("tpa_variant", C.c_uint32),
                ("code_dp", C.c_uint16), ("code_tp", C.c_uint16), ("code_pp", C.c_uint16),
                ("pad", C.c_uint16)]


def build(force: bool = False) -> str:
    """Compile the oracle (g++ -O2).  Returns the library path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread",
                                   "-o", tmp, _SRC])
            os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_space_size.restype = C.c_uint64
        L.orc_points_per_model.restype = C.c_uint64
        L.orc_num_factorisations.restype = C.c_uint32
        L.orc_compact_range.restype = C.c_uint64
        L.orc_hardware_threads.restype = C.c_uint32
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else C.c_void_p(a.ctypes.data)


class Space:
    """A design space as the oracle sees it (keeps the input arrays alive)."""

    def __init__(self, space: dict):
        self.models = np.ascontiguousarray(space["models"])
        assert self.models.dtype.itemsize == 48
        self.n_values = np.ascontiguousarray(space["n_values"], dtype=np.uint32)
        self.desc = _Desc(self.models.ctypes.data, len(self.models), self.n_values.ctypes.data,
                          len(self.n_values), space["t_enum_max"], space["k_enum_max"],
                          space["tp_max_valid"], space["n_act_variants"],
                          space["n_tpa_variants"], space["mode_mask"],
                          space["tp_coll_per_layer"], space.get("sstar_units", 1),
                          space.get("grad_accum_steps", 1), space.get("replication_k", 1))
        self.params = {k: v for k, v in space.items() if k not in ("models", "n_values")}

    @property
    def size(self) -> int:
        return lib().orc_space_size(C.byref(self.desc))

    @property
    def points_per_model(self) -> int:
        return lib().orc_points_per_model(C.byref(self.desc))

    def decode(self, idx: int) -> dict:
        p = _Point()
        lib().orc_decode(C.byref(self.desc), C.c_uint64(idx), C.byref(p))
        return {f: getattr(p, f) for f, _ in _Point._fields_ if f != "pad"}

    def eval_range(self, first: int, count: int, filt: dict | None = None) -> dict:
        out = {k: np.empty(count, dtype=np.uint64) for k in ("mem", "comm_paper", "comm_ext", "host")}
        out["flags"] = np.empty(count, dtype=np.uint32)
        f = _mk_filter(filt) if filt is not None else None
        lib().orc_eval_range(C.byref(self.desc), C.c_uint64(first), C.c_uint64(count),
                             C.byref(f) if f is not None else None, _ptr(out["mem"]),
                             _ptr(out["comm_paper"]), _ptr(out["comm_ext"]), _ptr(out["host"]),
                             _ptr(out["flags"]))
        return out

    def compact_range(self, first: int, count: int, filt: dict) -> dict:
        out = {k: np.empty(count, dtype=np.uint64)
               for k in ("idx", "mem", "comm_paper", "comm_ext", "host")}
        out["flags"] = np.empty(count, dtype=np.uint32)
        f = _mk_filter(filt)
        n = lib().orc_compact_range(C.byref(self.desc), C.c_uint64(first), C.c_uint64(count),
                                    C.byref(f), _ptr(out["idx"]), _ptr(out["mem"]),
                                    _ptr(out["comm_paper"]), _ptr(out["comm_ext"]),
                                    _ptr(out["host"]), _ptr(out["flags"]))
        return {k: v[:n].copy() for k, v in out.items()}

    def sweep(self, filt: dict, caps, kind: int, max_entries: int, *, model_first: int = 0,
              model_count: int | None = None, n_threads: int = 1):
        """Returns (entries[n_models, n_caps, max_entries], counts[n_models, n_caps]);
        rows of models outside the requested range stay zero."""
        caps = np.ascontiguousarray(caps, dtype=np.uint64)
        nm = len(self.models)
        if model_count is None:
            model_count = nm - model_first
        entries = np.zeros((nm, len(caps), max_entries), dtype=ENTRY_DTYPE)
        counts = np.zeros((nm, len(caps)), dtype=np.uint32)
        f = _mk_filter(filt)
        lib().orc_sweep(C.byref(self.desc), C.byref(f), _ptr(caps), C.c_uint32(len(caps)),
                        C.c_uint32(kind), C.c_uint32(max_entries), _ptr(entries), _ptr(counts),
                        C.c_uint32(model_first), C.c_uint32(model_count), C.c_uint32(n_threads))
        return entries, counts


def select_compare(space: "Space", n_index: int, device_bytes: int, filt: dict, entries: np.ndarray,
                   counts: np.ndarray, cap_index: int, fast: int = 1, headroom=(7, 10), layer=(3, 10),
                   tp_degree: int = 8) -> np.ndarray:
    """Algorithm 1's choice for every model, as a point of the space, against the frontier
    (entries[n_models, n_caps, max_entries], counts[n_models, n_caps]).  Returns (n_models, 12)
    uint64: alg mem, comm, idx; best mem, comm, idx; branch, T, code, flags, status, 0."""
    entries = np.ascontiguousarray(entries)
    counts = np.ascontiguousarray(counts, dtype=np.uint32)
    nm, n_caps, max_entries = entries.shape
    out = np.zeros((nm, 12), dtype=np.uint64)
    f = _mk_filter(filt)
    lib().orc_select_compare(C.byref(space.desc), C.c_uint32(n_index), C.c_uint64(device_bytes), C.c_uint32(fast),
                             headroom[0], headroom[1], layer[0], layer[1], tp_degree, C.byref(f), _ptr(entries),
                             _ptr(counts), C.c_uint32(n_caps), C.c_uint32(cap_index), C.c_uint32(max_entries),
                             _ptr(out))
    return out


def _mk_filter(filt: dict) -> _Filter:
    return _Filter(filt.get("host_cap", NO_LIMIT), filt.get("require_flags", 0),
                   filt.get("comm_kind", COMM_PAPER_PLUS_EXT), filt.get("cap_bytes", NO_LIMIT))


def num_factorisations(N: int, t_max: int, k_max: int) -> int:
    return lib().orc_num_factorisations(N, t_max, k_max)


def check_composition(shape: np.ndarray, N, T, K, D, code_tp, code_pp, code_dp, act_variant=0,
                      cap_bytes=NO_LIMIT, tp_max_valid=8, tp_coll_per_layer=4,
                      comm_kind=COMM_PAPER_PLUS_EXT) -> dict:
    shape = np.ascontiguousarray(shape)
    out = np.zeros(1, dtype=ENTRY_DTYPE)
    lib().orc_check_composition(_ptr(shape), N, T, K, D, code_tp, code_pp, code_dp, act_variant,
                                C.c_uint64(cap_bytes), tp_max_valid, tp_coll_per_layer, comm_kind,
                                _ptr(out))
    return {k: int(out[0][k]) for k in ("mem", "comm", "host", "flags")}


RECORD_FIELDS = ("P", "unit", "A0", "A1", "UA0", "UA1", "Sbh", "L", "heads",
                 "w_theta", "w_omega", "w_grad", "w_act")


def model_record(shape: np.ndarray) -> dict:
    rec = np.zeros(13, dtype=np.uint64)
    shape = np.ascontiguousarray(shape)
    lib().orc_model_record(_ptr(shape), _ptr(rec))
    return dict(zip(RECORD_FIELDS, (int(x) for x in rec)))


def eval_record(rec: dict, N, T, K, D, v, tau, code, tp_max_valid=8, tp_coll_per_layer=4,
                sstar_units=1, grad_accum_steps=1, replication_k=1) -> dict:
    r = np.array([rec[k] for k in RECORD_FIELDS], dtype=np.uint64)
    out = np.zeros(5, dtype=np.uint64)
    lib().orc_eval_record(_ptr(r), N, T, K, D, v, tau, code, tp_max_valid, tp_coll_per_layer,
                          sstar_units, grad_accum_steps, replication_k, _ptr(out))
    return dict(mem=int(out[0]), comm_paper=int(out[1]), comm_ext=int(out[2]), host=int(out[3]),
                flags=int(out[4]))


def select(queries: np.ndarray, headroom=(7, 10), layer=(3, 10), tp_degree=8) -> np.ndarray:
    """Algorithm 1 on an (n, 8) uint64 array of queries (P, layer elements, device bytes, N,
    w_param, w_grad, w_opt, fast); returns (n, 6): mem, comm, branch, T, code, flags."""
    q = np.ascontiguousarray(queries, dtype=np.uint64)
    out = np.zeros((len(q), 6), dtype=np.uint64)
    lib().orc_select(_ptr(q), C.c_uint64(len(q)), headroom[0], headroom[1], layer[0], layer[1], tp_degree,
                     _ptr(out))
    return out


def hardware_threads() -> int:
    return lib().orc_hardware_threads()
