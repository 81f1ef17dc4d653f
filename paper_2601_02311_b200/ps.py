"""Python binding of the CUDA library (``libps_b200.so``): argument marshalling
only.  Every step of the evaluation runs in the library's kernels; torch is
used for device memory and streams.  Importing this module fails if the library
has not been built (``python -m paper_2601_02311_b200.build``) -- there is no
CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libps_b200.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build the CUDA library first "
        "(python -m paper_2601_02311_b200.build); there is no CPU fallback")
_lib = C.CDLL(LIB_PATH)

# ---- constants of ps.h
OK = 0
E_NULLPTR, E_ALIGN, E_RANGE, E_BADINDEX, E_TRUNCATED, E_CUDA, E_UNIMPLEMENTED, E_DEVICE = \
    -1, -2, -3, -4, -5, -6, -7, -8
E_NOALLOC_LIMIT = -10
NOALLOC_MAX_GROUPS = 131072
F_GI, F_SC, F_CV, F_FEASIBLE = 1, 2, 4, 8
F_T_DIV_HEADS, F_K_DIV_LAYERS, F_TP_LE_MAX, F_AXIS_FORM = 16, 32, 64, 128
F_THETA_AVAIL, F_ACT_AVAIL, F_GRAD_COVER, F_USES_HOST, F_PAPER_PRICED = 256, 512, 1024, 2048, 4096
F_VALID = F_GI | F_SC | F_CV
COMM_PAPER, COMM_PAPER_PLUS_EXT = 0, 1
REDUCE_PARETO, REDUCE_TOPK = 0, 1
NO_LIMIT = (1 << 64) - 1
TOPK_MAX = 64

SELECT_QUERY_DTYPE = np.dtype([("param_elems", "<u8"), ("layer_elems", "<u8"), ("device_bytes", "<u8"),
                               ("n_devices", "<u4"), ("w_param", "u1"), ("w_grad", "u1"), ("w_opt", "u1"),
                               ("fast_interconnect", "u1")])
SELECT_RESULT_DTYPE = np.dtype([("mem", "<u8"), ("comm", "<u8"), ("branch", "<u4"), ("T", "<u4"),
                                ("code_dp", "<u4"), ("flags", "<u4")])
ENTRY_DTYPE = np.dtype([("mem", "<u8"), ("comm", "<u8"), ("host", "<u8"), ("idx", "<u8"),
                        ("flags", "<u4"), ("pad", "<u4")])

EXPORTS = ("ps_create", "ps_destroy", "ps_status", "ps_strerror", "ps_space_create",
           "ps_space_destroy", "ps_space_set_models", "ps_space_rederive", "ps_space_size",
           "ps_space_points_per_model", "ps_space_decode", "ps_eval_batch", "ps_sweep_pareto",
           "ps_check_composition", "ps_int_peak", "ps_eval_compact_noalloc", "ps_select",
           "ps_verify_batch", "ps_select_compare")


class _SpaceDesc(C.Structure):
    _fields_ = [("models", C.c_void_p), ("n_models", C.c_uint32),
                ("n_values", C.c_void_p), ("n_n", C.c_uint32),
                ("t_enum_max", C.c_uint32), ("k_enum_max", C.c_uint32),
                ("tp_max_valid", C.c_uint32), ("n_act_variants", C.c_uint32),
                ("n_tpa_variants", C.c_uint32), ("mode_mask", C.c_uint32),
                ("tp_coll_per_layer", C.c_uint32), ("sstar_units", C.c_uint32),
                ("grad_accum_steps", C.c_uint32), ("replication_k", C.c_uint32)]


class _Filter(C.Structure):
    _fields_ = [("host_cap", C.c_uint64), ("require_flags", C.c_uint32),
                ("comm_kind", C.c_uint32), ("cap_bytes", C.c_uint64),
                ("skip_rejected", C.c_uint32), ("pad", C.c_uint32)]


class _OutSoa(C.Structure):
    _fields_ = [("mem", C.c_void_p), ("comm_paper", C.c_void_p), ("comm_ext", C.c_void_p),
                ("host", C.c_void_p), ("flags", C.c_void_p)]


class _VerifyShape(C.Structure):
    _fields_ = [("units", C.c_uint32), ("h", C.c_uint32), ("b", C.c_uint32), ("accum", C.c_uint32),
                ("steps", C.c_uint32), ("gather_buffers", C.c_uint32), ("w_theta", C.c_uint32),
                ("w_omega", C.c_uint32), ("w_grad", C.c_uint32), ("pad", C.c_uint32),
                ("lr", C.c_double), ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double),
                ("rtol", C.c_double), ("atol", C.c_double)]


SELECT_COMPARE_DTYPE = np.dtype([("alg_mem", "<u8"), ("alg_comm", "<u8"), ("alg_idx", "<u8"), ("best_mem", "<u8"),
                                 ("best_comm", "<u8"), ("best_idx", "<u8"), ("branch", "<u4"), ("T", "<u4"),
                                 ("code_dp", "<u4"), ("alg_flags", "<u4"), ("status", "<u4"), ("pad", "<u4")])
SEL_IN_SPACE, SEL_SURVIVOR, SEL_ON_FRONTIER, SEL_DOMINATED, SEL_FRONTIER_EMPTY, SEL_FRONTIER_TRUNCATED = \
    1, 2, 4, 8, 16, 32
VERIFY_CASE_DTYPE = np.dtype([("code", "<u4"), ("D", "<u4"), ("data_offset", "<u8")])
VERIFY_RESULT_DTYPE = np.dtype([("mem", "<u8"), ("comm", "<u8"), ("host", "<u8"), ("match", "<u4"),
                                ("pad", "<u4"), ("max_rel_err", "<f8")])


class _Point(C.Structure):
    _fields_ = [("model", C.c_uint32), ("N", C.c_uint32), ("T", C.c_uint32), ("K", C.c_uint32),
                ("D", C.c_uint32), ("act_variant", C.c_uint32), ("tpa_variant", C.c_uint32),
                ("code_dp", C.c_uint16), ("code_tp", C.c_uint16), ("code_pp", C.c_uint16),
                ("pad", C.c_uint16)]


_lib.ps_strerror.restype = C.c_char_p
_lib.ps_strerror.argtypes = [C.c_int]
_lib.ps_create.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_void_p]
_lib.ps_destroy.argtypes = [C.c_void_p]
_lib.ps_destroy.restype = None
_lib.ps_status.argtypes = [C.c_void_p]
_lib.ps_space_create.argtypes = [C.c_void_p, C.POINTER(_SpaceDesc), C.POINTER(C.c_void_p)]
_lib.ps_space_destroy.argtypes = [C.c_void_p]
_lib.ps_space_destroy.restype = None
_lib.ps_space_set_models.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32]
_lib.ps_space_rederive.argtypes = [C.c_void_p]
_lib.ps_space_size.argtypes = [C.c_void_p]
_lib.ps_space_size.restype = C.c_uint64
_lib.ps_space_points_per_model.argtypes = [C.c_void_p]
_lib.ps_space_points_per_model.restype = C.c_uint64
_lib.ps_space_decode.argtypes = [C.c_void_p, C.c_uint64, C.POINTER(_Point)]
_lib.ps_eval_batch.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.POINTER(_Filter),
                               _OutSoa, C.c_void_p, C.c_void_p]
_lib.ps_eval_compact_noalloc.argtypes = _lib.ps_eval_batch.argtypes
_lib.ps_sweep_pareto.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(_Filter), C.c_void_p,
                                 C.c_uint32, C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p]
_lib.ps_check_composition.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32,
                                      C.c_uint32, C.c_uint16, C.c_uint16, C.c_uint16, C.c_uint32,
                                      C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_void_p]
_lib.ps_select.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32,
                           C.c_uint32, C.c_uint32, C.c_void_p]
_lib.ps_select_compare.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint64, C.c_uint32, C.c_uint32,
                                   C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32, C.POINTER(_Filter), C.c_void_p,
                                   C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32, C.c_void_p]
_lib.ps_verify_batch.argtypes = [C.c_void_p, C.POINTER(_VerifyShape), C.c_void_p, C.c_uint64, C.c_void_p,
                                 C.c_uint64, C.c_void_p, C.c_void_p]
_lib.ps_int_peak.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_void_p,
                             C.POINTER(C.c_uint64)]


class PsError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {_lib.ps_strerror(code).decode()} ({code})")


def _check(code: int, where: str):
    if code != OK:
        raise PsError(code, where)


def strerror(code: int) -> str:
    return _lib.ps_strerror(code).decode()


def _mk_filter(filt: dict) -> _Filter:
    return _Filter(filt.get("host_cap", NO_LIMIT), filt.get("require_flags", 0),
                   filt.get("comm_kind", COMM_PAPER_PLUS_EXT), filt.get("cap_bytes", NO_LIMIT),
                   1 if filt.get("skip_rejected") else 0, 0)


def _dptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


class Context:
    """ps_ctx: one per (device, stream)."""

    def __init__(self, device: int = 0, stream: torch.cuda.Stream | None = None):
        if not torch.cuda.is_available():
            raise RuntimeError("the placement-semantics library needs a CUDA device")
        self.device = device
        self.torch_device = torch.device("cuda", device)
        self.stream = stream
        handle = C.c_void_p()
        sptr = C.c_void_p(stream.cuda_stream) if stream is not None else None
        _check(_lib.ps_create(C.byref(handle), device, sptr), "ps_create")
        self._h = handle

    def close(self):
        # at interpreter shutdown the module's globals may be gone before the last
        # handle: the process is ending, the driver releases the device memory
        if getattr(self, "_h", None) and _lib is not None:
            _lib.ps_destroy(self._h)
        self._h = None

    __del__ = close

    def status(self) -> int:
        return _lib.ps_status(self._h)

    def check_status(self, allow_truncated: bool = False) -> int:
        """Synchronise and raise on any error a kernel reported.  With
        ``allow_truncated`` the notice that a frontier was longer than the caller's
        rows (E_TRUNCATED: heads written, counts true) is returned instead of raised."""
        rc = self.status()
        if not (allow_truncated and rc == E_TRUNCATED):
            _check(rc, "ps_status")
        return rc

    def space(self, space: dict) -> "Space":
        return Space(self, space)

    def check_composition(self, shape: np.ndarray, N, T, K, D, code_tp, code_pp, code_dp,
                          act_variant=0, cap_bytes=NO_LIMIT, tp_max_valid=8, tp_coll_per_layer=4,
                          comm_kind=COMM_PAPER_PLUS_EXT) -> dict:
        shape = np.ascontiguousarray(shape)
        out = np.zeros(1, dtype=ENTRY_DTYPE)
        _check(_lib.ps_check_composition(self._h, shape.ctypes.data, N, T, K, D, code_tp, code_pp,
                                         code_dp, act_variant, cap_bytes, tp_max_valid,
                                         tp_coll_per_layer, comm_kind, out.ctypes.data),
               "ps_check_composition")
        return {k: int(out[0][k]) for k in ("mem", "comm", "host", "flags")}

    def select_into(self, d_queries: torch.Tensor, n: int, d_out: torch.Tensor, headroom=(7, 10),
                    layer=(3, 10), tp_degree=8):
        """ps_select on device buffers (uint8 tensors of 32-byte records)."""
        _check(_lib.ps_select(self._h, _dptr(d_queries), n, headroom[0], headroom[1], layer[0], layer[1],
                              tp_degree, _dptr(d_out)), "ps_select")

    def select(self, queries: np.ndarray, headroom=(7, 10), layer=(3, 10), tp_degree=8) -> np.ndarray:
        """Algorithm 1 for a structured array of SELECT_QUERY_DTYPE; returns SELECT_RESULT_DTYPE."""
        q = np.ascontiguousarray(queries)
        assert q.dtype.itemsize == 32
        d_q = torch.from_numpy(q.view(np.uint8).reshape(-1).copy()).to(self.torch_device)
        d_o = torch.empty(max(len(q), 1) * 32, dtype=torch.uint8, device=self.torch_device)
        self.select_into(d_q, len(q), d_o, headroom, layer, tp_degree)
        self.check_status()
        return d_o.cpu().numpy()[:len(q) * 32].view(SELECT_RESULT_DTYPE)

    def verify_batch(self, shape: dict, cases: np.ndarray, data: np.ndarray, want_theta: bool = False):
        """ps_verify_batch: `cases` a VERIFY_CASE_DTYPE array, `data` a float64 array holding every
        case's problem; returns VERIFY_RESULT_DTYPE records (and the final parameters)."""
        sh = _VerifyShape(shape["units"], shape["h"], shape["b"], shape.get("accum", 1), shape.get("steps", 3),
                          shape.get("gather_buffers", 1), shape.get("w_theta", 2), shape.get("w_omega", 12),
                          shape.get("w_grad", 2), 0, shape.get("lr", 0.05), shape.get("beta1", 0.9),
                          shape.get("beta2", 0.999), shape.get("eps", 1e-8), shape.get("rtol", 1e-12),
                          shape.get("atol", 1e-14))
        cases = np.ascontiguousarray(cases)
        assert cases.dtype.itemsize == 16
        data = np.ascontiguousarray(data, dtype=np.float64)
        n = len(cases)
        dev = self.torch_device
        d_cases = torch.from_numpy(cases.view(np.uint8).reshape(-1).copy()).to(dev)
        d_data = torch.from_numpy(data).to(dev)
        d_out = torch.zeros(max(n, 1) * 40, dtype=torch.uint8, device=dev)
        P = shape["units"] * shape["h"]
        d_theta = torch.zeros(max(n, 1) * P, dtype=torch.float64, device=dev) if want_theta else None
        _check(_lib.ps_verify_batch(self._h, C.byref(sh), _dptr(d_cases), n, _dptr(d_data), len(data),
                                    _dptr(d_out), _dptr(d_theta)), "ps_verify_batch")
        self.check_status()
        res = d_out.cpu().numpy()[:n * 40].view(VERIFY_RESULT_DTYPE)
        if want_theta:
            return res, d_theta.cpu().numpy().reshape(-1, P)[:n]
        return res

    def int_peak(self, blocks: int, iters: int, sink: torch.Tensor) -> int:
        ops = C.c_uint64()
        _check(_lib.ps_int_peak(self._h, blocks, iters, _dptr(sink), C.byref(ops)), "ps_int_peak")
        return ops.value


class Space:
    """ps_space: the device copy of a model table plus the enumeration."""

    def __init__(self, ctx: Context, space: dict):
        self.ctx = ctx
        models = np.ascontiguousarray(space["models"])
        assert models.dtype.itemsize == 48
        n_values = np.ascontiguousarray(space["n_values"], dtype=np.uint32)
        desc = _SpaceDesc(models.ctypes.data, len(models), n_values.ctypes.data, len(n_values),
                          space["t_enum_max"], space["k_enum_max"], space["tp_max_valid"],
                          space["n_act_variants"], space["n_tpa_variants"], space["mode_mask"],
                          space["tp_coll_per_layer"], space.get("sstar_units", 1),
                          space.get("grad_accum_steps", 1), space.get("replication_k", 1))
        handle = C.c_void_p()
        _check(_lib.ps_space_create(ctx._h, C.byref(desc), C.byref(handle)), "ps_space_create")
        self._h = handle
        self.n_models = len(models)

    def close(self):
        if getattr(self, "_h", None) and getattr(self.ctx, "_h", None) and _lib is not None:
            _lib.ps_space_destroy(self._h)
        self._h = None

    __del__ = close

    @property
    def size(self) -> int:
        return _lib.ps_space_size(self._h)

    @property
    def points_per_model(self) -> int:
        return _lib.ps_space_points_per_model(self._h)

    def decode(self, idx: int) -> dict:
        p = _Point()
        _check(_lib.ps_space_decode(self._h, idx, C.byref(p)), "ps_space_decode")
        return {f: getattr(p, f) for f, _ in _Point._fields_ if f != "pad"}

    def set_models(self, models_host) -> None:
        """Replace the shape table from host memory (numpy array or a pinned torch
        uint8 tensor of 48-byte records)."""
        if isinstance(models_host, torch.Tensor):
            ptr, n = models_host.data_ptr(), models_host.numel() * models_host.element_size() // 48
        else:
            models_host = np.ascontiguousarray(models_host)
            ptr, n = models_host.ctypes.data, len(models_host)
        _check(_lib.ps_space_set_models(self._h, ptr, n), "ps_space_set_models")

    def rederive(self) -> None:
        _check(_lib.ps_space_rederive(self._h), "ps_space_rederive")

    # ---- ps_eval_batch
    def eval_batch_into(self, first: int, count: int, out: dict, filt: dict | None = None,
                        idx_out: torch.Tensor | None = None, n_out: torch.Tensor | None = None):
        """Raw call: `out` maps any of mem/comm_paper/comm_ext/host/flags to device tensors."""
        soa = _OutSoa(*(None if out.get(k) is None else out[k].data_ptr()
                        for k in ("mem", "comm_paper", "comm_ext", "host", "flags")))
        f = _mk_filter(filt) if filt is not None else None
        _check(_lib.ps_eval_batch(self.ctx._h, self._h, first, count,
                                  C.byref(f) if f is not None else None, soa, _dptr(idx_out),
                                  _dptr(n_out)), "ps_eval_batch")

    def alloc_outputs(self, count: int, fields=("mem", "comm_paper", "comm_ext", "host", "flags")):
        dev = self.ctx.torch_device
        out = {}
        for k in fields:
            dt = torch.int32 if k == "flags" else torch.int64
            out[k] = torch.empty(max(count, 1), dtype=dt, device=dev)
        return out

    def eval_batch(self, first: int, count: int,
                   fields=("mem", "comm_paper", "comm_ext", "host", "flags")) -> dict:
        """Materialise [first, first+count) and return numpy arrays (unsigned)."""
        out = self.alloc_outputs(count, fields)
        self.eval_batch_into(first, count, out)
        self.ctx.check_status()
        return {k: _to_unsigned(v[:count]) for k, v in out.items()}

    def compact(self, first: int, count: int, filt: dict,
                fields=("mem", "comm_paper", "comm_ext", "host", "flags")) -> dict:
        """Filter and compact; returns numpy arrays of the survivors incl. 'idx'."""
        dev = self.ctx.torch_device
        out = self.alloc_outputs(count, fields)
        idx = torch.empty(max(count, 1), dtype=torch.int64, device=dev)
        n = torch.zeros(1, dtype=torch.int64, device=dev)
        self.eval_batch_into(first, count, out, filt, idx, n)
        self.ctx.check_status()
        k = int(n.item())
        res = {name: _to_unsigned(v[:k]) for name, v in out.items()}
        res["idx"] = _to_unsigned(idx[:k])
        return res

    def compact_noalloc_into(self, first: int, count: int, out: dict, filt: dict,
                             idx_out: torch.Tensor | None, n_out: torch.Tensor):
        """ps_eval_compact_noalloc: same contract as the filtered eval_batch_into, but the
        library allocates nothing (fixed scratch; at most NOALLOC_MAX_GROUPS groups per
        call; calls on one device must not overlap)."""
        soa = _OutSoa(*(None if out.get(k) is None else out[k].data_ptr()
                        for k in ("mem", "comm_paper", "comm_ext", "host", "flags")))
        f = _mk_filter(filt)
        _check(_lib.ps_eval_compact_noalloc(self.ctx._h, self._h, first, count, C.byref(f), soa,
                                            _dptr(idx_out), _dptr(n_out)), "ps_eval_compact_noalloc")

    # ---- ps_sweep_pareto
    def sweep_into(self, filt: dict, caps, kind: int, max_entries: int, d_out: torch.Tensor,
                   d_counts: torch.Tensor):
        caps = np.ascontiguousarray(caps, dtype=np.uint64)
        f = _mk_filter(filt)
        _check(_lib.ps_sweep_pareto(self.ctx._h, self._h, C.byref(f), caps.ctypes.data, len(caps),
                                    kind, max_entries, _dptr(d_out), _dptr(d_counts)),
               "ps_sweep_pareto")

    def select_compare(self, n_index: int, device_bytes: int, filt: dict, d_frontier: torch.Tensor,
                       d_counts: torch.Tensor, n_caps: int, cap_index: int, max_entries: int, fast: int = 1,
                       headroom=(7, 10), layer=(3, 10), tp_degree: int = 8) -> np.ndarray:
        """ps_select_compare on the device outputs of a Pareto sweep; returns SELECT_COMPARE_DTYPE records."""
        d_out = torch.zeros(self.n_models * 72, dtype=torch.uint8, device=self.ctx.torch_device)
        f = _mk_filter(filt)
        _check(_lib.ps_select_compare(self.ctx._h, self._h, n_index, device_bytes, fast, headroom[0], headroom[1],
                                      layer[0], layer[1], tp_degree, C.byref(f), _dptr(d_frontier), _dptr(d_counts),
                                      n_caps, cap_index, max_entries, _dptr(d_out)), "ps_select_compare")
        self.ctx.check_status()
        return d_out.cpu().numpy().view(SELECT_COMPARE_DTYPE)

    def alloc_sweep(self, n_caps: int, max_entries: int):
        dev = self.ctx.torch_device
        d_out = torch.empty(self.n_models * n_caps * max_entries * 40, dtype=torch.uint8, device=dev)
        d_counts = torch.empty(self.n_models * n_caps, dtype=torch.int32, device=dev)
        return d_out, d_counts

    def sweep(self, filt: dict, caps, kind: int, max_entries: int):
        """Returns (entries[n_models, n_caps, max_entries] structured, counts[n_models, n_caps])."""
        d_out, d_counts = self.alloc_sweep(len(caps), max_entries)
        self.sweep_into(filt, caps, kind, max_entries, d_out, d_counts)
        self.last_sweep_status = self.ctx.check_status(allow_truncated=True)
        entries = d_out.cpu().numpy().view(ENTRY_DTYPE).reshape(self.n_models, len(caps), max_entries)
        counts = d_counts.cpu().numpy().view(np.uint32).reshape(self.n_models, len(caps))
        return entries, counts


def _to_unsigned(t: torch.Tensor) -> np.ndarray:
    a = t.cpu().numpy()
    return a.view(np.uint64 if a.dtype == np.int64 else np.uint32)
