"""Python binding of libslonn.so: the same calls as include/slonn.h, with torch
tensors (device memory) or numpy arrays (host memory) marshalled to raw
pointers.  No arithmetic happens here; without the compiled CUDA library every
call raises.
"""
import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np

SLONN_F32, SLONN_BF16 = 0, 1
SLONN_OK = 0
ERR = {"ARG": -1, "DIM": -2, "DTYPE": -3, "ALIGN": -4, "BUDGET": -5, "NOMEM": -6, "CUDA": -7,
       "TIMEOUT": -8, "WORKSPACE": -9}

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("SLONN_LIB", os.path.join(_HERE, "libslonn.so"))  # SLONN_LIB: another build of the library

EXPORTS = [
    "slonn_version", "slonn_strerror", "slonn_build", "slonn_model_info", "slonn_model_tables_to_host",
    "slonn_free", "slonn_active_capacity", "slonn_logit_stride", "slonn_workspace_bytes", "slonn_run",
    "slonn_run_timed", "slonn_run_static", "slonn_dense_layer", "slonn_serialized_bytes", "slonn_serialize",
    "slonn_deserialize", "slonn_lcao_budgets", "slonn_confidence_build", "slonn_confidence_to_host",
    "slonn_confidence_free", "slonn_aclo_budgets",
    "slonn_host_workspace_bytes", "slonn_run_host", "slonn_test_tc_wait_limit", "slonn_run_traced",
]


class SlonnError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


class _BuildDesc(C.Structure):
    _fields_ = [("n_layers", C.c_uint32), ("dims", C.c_void_p), ("has_activator", C.c_void_p),
                ("dtype", C.c_int32), ("K", C.c_uint32), ("L", C.c_uint32), ("list_cap", C.c_uint32),
                ("seed", C.c_uint64), ("first_layer_sparse", C.c_uint32),
                ("hash_nodes_override", C.c_void_p), ("free_hash_nodes", C.c_uint32)]


class _Rows(C.Structure):
    _fields_ = [("n_rows", C.c_uint32), ("dense", C.c_void_p), ("indptr", C.c_void_p),
                ("ids", C.c_void_p), ("vals", C.c_void_p)]


class _LaunchRecord(C.Structure):
    _fields_ = [("stage", C.c_uint32), ("layer", C.c_uint32), ("bp_lo", C.c_uint32), ("bp_hi", C.c_uint32),
                ("skips_full", C.c_uint32), ("cols_bp", C.c_uint32), ("ms", C.c_float)]


class _Batch(C.Structure):
    _fields_ = [("n_queries", C.c_uint32), ("x_dense", C.c_void_p), ("x_indptr", C.c_void_p),
                ("x_ids", C.c_void_p), ("x_vals", C.c_void_p), ("budget_bp", C.c_void_p),
                ("max_budget_bp", C.c_uint32), ("logits", C.c_void_p), ("logit_ids", C.c_void_p),
                ("pred", C.c_void_p), ("codes", C.c_void_p), ("active_indptr", C.c_void_p),
                ("active_ids", C.c_void_p), ("active_vals", C.c_void_p), ("status", C.c_void_p),
                ("flags", C.c_uint32), ("kernel_path", C.c_uint32)]


_lib = None


def lib():
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2204_08400_b200.build_ext` (there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        L.slonn_version.restype = C.c_int
        L.slonn_strerror.restype = C.c_char_p
        L.slonn_strerror.argtypes = [C.c_int]
        L.slonn_build.restype = C.c_int
        L.slonn_build.argtypes = [C.POINTER(_BuildDesc), C.c_void_p, C.c_void_p, C.POINTER(_Rows),
                                  C.c_void_p, C.POINTER(C.c_void_p)]
        L.slonn_model_info.restype = C.c_int
        L.slonn_model_info.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.POINTER(C.c_void_p),
                                       C.POINTER(C.c_uint64), C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
        L.slonn_model_tables_to_host.restype = C.c_int
        L.slonn_model_tables_to_host.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint64]
        L.slonn_serialized_bytes.restype = C.c_int
        L.slonn_serialized_bytes.argtypes = [C.c_void_p, C.POINTER(C.c_uint64)]
        L.slonn_serialize.restype = C.c_int
        L.slonn_serialize.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
        L.slonn_deserialize.restype = C.c_int
        L.slonn_deserialize.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.POINTER(C.c_void_p)]
        L.slonn_confidence_build.restype = C.c_int
        L.slonn_confidence_build.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p]
        L.slonn_confidence_to_host.restype = C.c_int
        L.slonn_confidence_to_host.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint64]
        L.slonn_confidence_free.restype = None
        L.slonn_confidence_free.argtypes = [C.c_void_p]
        L.slonn_aclo_budgets.restype = C.c_int
        L.slonn_aclo_budgets.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32,
                                         C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.slonn_lcao_budgets.restype = C.c_int
        L.slonn_lcao_budgets.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint32,
                                         C.c_void_p, C.c_void_p, C.c_void_p]
        L.slonn_free.restype = None
        L.slonn_free.argtypes = [C.c_void_p]
        L.slonn_active_capacity.restype = C.c_int
        L.slonn_active_capacity.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.POINTER(C.c_uint64)]
        L.slonn_logit_stride.restype = C.c_int
        L.slonn_logit_stride.argtypes = [C.c_void_p, C.c_uint32, C.POINTER(C.c_uint32)]
        L.slonn_workspace_bytes.restype = C.c_int
        L.slonn_workspace_bytes.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32, C.POINTER(C.c_uint64)]
        L.slonn_run.restype = C.c_int
        L.slonn_run.argtypes = [C.c_void_p, C.POINTER(_Batch), C.c_void_p, C.c_uint64, C.c_void_p]
        L.slonn_run_static.restype = C.c_int
        L.slonn_run_static.argtypes = [C.c_void_p, C.POINTER(_Batch), C.c_void_p]
        L.slonn_dense_layer.restype = C.c_int
        L.slonn_dense_layer.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32,
                                        C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.slonn_test_tc_wait_limit.restype = C.c_int
        L.slonn_test_tc_wait_limit.argtypes = [C.c_uint32]
        L.slonn_run_timed.restype = C.c_int
        L.slonn_run_timed.argtypes = [C.c_void_p, C.POINTER(_Batch), C.c_void_p, C.c_uint64, C.c_void_p,
                                      C.c_void_p, C.c_void_p]
        L.slonn_run_traced.restype = C.c_int
        L.slonn_run_traced.argtypes = [C.c_void_p, C.POINTER(_Batch), C.c_void_p, C.c_uint64, C.c_void_p,
                                       C.c_void_p, C.c_uint32, C.POINTER(C.c_uint32)]
        L.slonn_host_workspace_bytes.restype = C.c_int
        L.slonn_host_workspace_bytes.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint64,
                                                 C.POINTER(C.c_uint64)]
        L.slonn_run_host.restype = C.c_int
        L.slonn_run_host.argtypes = [C.c_void_p, C.POINTER(_Batch), C.c_void_p, C.c_uint64, C.c_void_p,
                                     C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
        _lib = L
    return _lib


def _ptr(t) -> Optional[int]:
    """Raw address of a torch tensor, numpy array, int or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        return None
    return stream if isinstance(stream, int) else stream.cuda_stream


def version() -> int:
    return lib().slonn_version()


def strerror(code: int) -> str:
    return lib().slonn_strerror(code).decode()


class Model:
    """Handle of a built model; keeps the referenced weight tensors alive."""

    def __init__(self, handle, keep, dims, has_activator, dtype, K, L, first_layer_sparse, free_hash_nodes=False):
        self.handle = handle
        self._keep = keep
        self.dims = list(dims)
        self.has_activator = list(has_activator)
        self.n_act = sum(1 for h in has_activator if h)
        self.dtype, self.K, self.L = dtype, K, L
        self.first_layer_sparse = first_layer_sparse
        self.free_hash_nodes = free_hash_nodes

    def free(self):
        if self.handle:
            lib().slonn_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def slonn_build(dims: Sequence[int], has_activator: Sequence[int], dtype: int, W: List, bias: List,
                calib_dense=None, calib_csr=None, K: int = 10, L: int = 2, list_cap: int = 0, seed: int = 0,
                first_layer_sparse: bool = False, hash_nodes_override=None, stream=None,
                free_hash_nodes: bool = False) -> Model:
    """W[l], bias[l], calib_*: device tensors (W as float32 or as uint16/bfloat16 bit patterns)."""
    n_layers = len(dims) - 1
    d = np.asarray(dims, dtype=np.uint32)
    h = np.asarray(has_activator, dtype=np.uint8)
    Wp = (C.c_void_p * n_layers)(*[_ptr(w) for w in W])
    bp = (C.c_void_p * n_layers)(*[_ptr(b) for b in bias])
    keep = [list(W), list(bias), d, h]
    desc = _BuildDesc()
    desc.n_layers = n_layers
    desc.dims = d.ctypes.data
    desc.has_activator = h.ctypes.data
    desc.dtype = dtype
    desc.K, desc.L, desc.list_cap, desc.seed = K, L, list_cap, seed
    desc.first_layer_sparse = int(bool(first_layer_sparse))
    desc.free_hash_nodes = int(bool(free_hash_nodes))
    ov_keep = []
    if hash_nodes_override is not None:
        ov = (C.c_void_p * n_layers)()
        for l in range(n_layers):
            if hash_nodes_override[l] is not None:
                a = np.ascontiguousarray(hash_nodes_override[l], dtype=np.uint32).reshape(-1)
                ov_keep.append(a)
                ov[l] = a.ctypes.data
        desc.hash_nodes_override = C.cast(ov, C.c_void_p)
        ov_keep.append(ov)
    rows = _Rows()
    if calib_csr is not None:
        indptr, ids, vals = calib_csr
        rows.n_rows = indptr.numel() - 1
        rows.indptr, rows.ids, rows.vals = _ptr(indptr), _ptr(ids), _ptr(vals)
    elif calib_dense is not None:
        rows.n_rows = calib_dense.shape[0]
        rows.dense = _ptr(calib_dense)
    out = C.c_void_p()
    rc = lib().slonn_build(C.byref(desc), C.cast(Wp, C.c_void_p), C.cast(bp, C.c_void_p), C.byref(rows),
                           _stream_ptr(stream), C.byref(out))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_build")
    return Model(out.value, keep, dims, has_activator, dtype, K, L, bool(first_layer_sparse), bool(free_hash_nodes))


def slonn_serialize(model: Model) -> np.ndarray:
    """The trained activator (configuration, hash nodes, tables) as a byte array; weights not included."""
    nb = C.c_uint64()
    rc = lib().slonn_serialized_bytes(model.handle, C.byref(nb))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_serialized_bytes")
    buf = np.empty(nb.value, dtype=np.uint8)
    rc = lib().slonn_serialize(model.handle, buf.ctypes.data, buf.nbytes)
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_serialize")
    return buf


def slonn_deserialize(blob: np.ndarray, W: List, bias: List, stream=None) -> Model:
    """Rebuilds a model from slonn_serialize's bytes and the (device) weights it was trained on."""
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    n_layers = len(W)
    Wp = (C.c_void_p * n_layers)(*[_ptr(w) for w in W])
    bp = (C.c_void_p * n_layers)(*[_ptr(b) for b in bias])
    out = C.c_void_p()
    rc = lib().slonn_deserialize(blob.ctypes.data, blob.nbytes, C.cast(Wp, C.c_void_p), C.cast(bp, C.c_void_p),
                                 _stream_ptr(stream), C.byref(out))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_deserialize")
    hdr = np.frombuffer(blob[:36].tobytes(), dtype=np.uint32)
    n_l, dtype, K, L, first_sparse, free_hash = (int(hdr[2]), int(hdr[3]), int(hdr[4]), int(hdr[5]), int(hdr[7]),
                                                 int(hdr[8]))
    dims = np.frombuffer(blob[36:36 + 4 * 17].tobytes(), dtype=np.uint32)[: n_l + 1].tolist()
    has_act = blob[36 + 4 * 17: 36 + 4 * 17 + n_l].tolist()
    return Model(out.value, [list(W), list(bias)], dims, has_act, dtype, K, L, bool(first_sparse), bool(free_hash))


def slonn_lcao_budgets(profile_bp, profile_ms, t0, tau, budget_bp, feasible=None, stream=None) -> None:
    """Eq. 3 on the device: budget_bp[q] = largest profiled k with t0[q] + T(k) <= tau[q]."""
    rc = lib().slonn_lcao_budgets(_ptr(profile_bp), _ptr(profile_ms), int(profile_bp.numel()), _ptr(t0), _ptr(tau),
                                  int(t0.numel()), _ptr(budget_bp), _ptr(feasible), _stream_ptr(stream))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_lcao_budgets")


class Confidence:
    """Handle of trained Confidence LSH tables."""

    def __init__(self, handle, K, L, profile_bp):
        self.handle, self.K, self.L = handle, K, L
        self.profile_bp = np.asarray(profile_bp, dtype=np.uint16).copy()

    def free(self):
        if self.handle:
            lib().slonn_confidence_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def slonn_confidence_build(model: Model, rows_dense, profile_bp, stream=None) -> Confidence:
    """rows_dense: device tensor [n_rows, D0]; profile_bp: host sequence, strictly ascending."""
    pb = np.ascontiguousarray(profile_bp, dtype=np.uint16)
    rows = _Rows()
    rows.n_rows = rows_dense.shape[0]
    rows.dense = _ptr(rows_dense)
    out = C.c_void_p()
    rc = lib().slonn_confidence_build(model.handle, C.byref(rows), pb.ctypes.data, int(pb.size), _stream_ptr(stream),
                                      C.byref(out))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_confidence_build")
    return Confidence(out.value, model.K, model.L, pb)


def slonn_confidence_to_host(conf: Confidence):
    """(sum [L, 2^K, n_k] float64, count [L, 2^K] uint32)."""
    s = np.zeros((conf.L, 1 << conf.K, conf.profile_bp.size), np.float64)
    c = np.zeros((conf.L, 1 << conf.K), np.uint32)
    rc = lib().slonn_confidence_to_host(conf.handle, s.ctypes.data, s.size, c.ctypes.data, c.size)
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_confidence_to_host")
    return s, c


def slonn_confidence_free(conf: Confidence) -> None:
    conf.free()


def slonn_aclo_budgets(model: Model, conf: Confidence, x_dense, threshold, budget_bp, target=None, met=None,
                       estimate=None, status=None, stream=None) -> None:
    """Eq. 2 on the device; threshold: device tensor [n_targets, n_k] float32; outputs are device tensors."""
    rc = lib().slonn_aclo_budgets(model.handle, conf.handle, _ptr(x_dense), int(x_dense.shape[0]), _ptr(threshold),
                                  int(threshold.shape[0]), _ptr(target), _ptr(budget_bp), _ptr(met), _ptr(estimate),
                                  _ptr(status), _stream_ptr(stream))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_aclo_budgets")


def slonn_free(model: Model) -> None:
    model.free()


def slonn_model_info(model: Model, layer: int) -> dict:
    hn = np.zeros(model.K * model.L, dtype=np.uint32)
    tables = C.c_void_p()
    tb = C.c_uint64()
    ib = C.c_uint32()
    cap = C.c_uint32()
    rc = lib().slonn_model_info(model.handle, layer, hn.ctypes.data, C.byref(tables), C.byref(tb),
                                C.byref(ib), C.byref(cap))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_model_info")
    return {"hash_nodes": hn.reshape(model.L, model.K), "tables_dev": tables.value, "table_bytes": tb.value,
            "id_bytes": ib.value, "cap": cap.value}


def slonn_model_tables_to_host(model: Model, layer: int) -> np.ndarray:
    info = slonn_model_info(model, layer)
    dt = np.uint16 if info["id_bytes"] == 2 else np.uint32
    out = np.empty((model.L, 1 << model.K, info["cap"]), dtype=dt)
    rc = lib().slonn_model_tables_to_host(model.handle, layer, out.ctypes.data, out.nbytes)
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_model_tables_to_host")
    return out


def slonn_active_capacity(model: Model, n_queries: int, max_budget_bp: int = 0) -> int:
    v = C.c_uint64()
    rc = lib().slonn_active_capacity(model.handle, n_queries, max_budget_bp, C.byref(v))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_active_capacity")
    return v.value


def slonn_logit_stride(model: Model, max_budget_bp: int = 0) -> int:
    v = C.c_uint32()
    rc = lib().slonn_logit_stride(model.handle, max_budget_bp, C.byref(v))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_logit_stride")
    return v.value


def slonn_workspace_bytes(model: Model, n_queries: int, max_budget_bp: int = 0, flags: int = 0) -> int:
    v = C.c_uint64()
    rc = lib().slonn_workspace_bytes(model.handle, n_queries, max_budget_bp, flags, C.byref(v))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_workspace_bytes")
    return v.value


def slonn_host_workspace_bytes(model: Model, n_queries: int, max_budget_bp: int = 0, x_nnz: int = 0,
                               flags: int = 0) -> int:
    v = C.c_uint64()
    rc = lib().slonn_host_workspace_bytes(model.handle, n_queries, max_budget_bp, flags, x_nnz, C.byref(v))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_host_workspace_bytes")
    return v.value


def make_batch(n_queries: int, budget_bp, logits, status, x_dense=None, x_csr=None, max_budget_bp: int = 0,
               logit_ids=None, pred=None, codes=None, active_indptr=None, active_ids=None,
               active_vals=None, kernel_path: int = 0, flags: int = 0) -> _Batch:
    """Fills a slonn_batch from tensors/arrays (device for slonn_run, host for slonn_run_host)."""
    b = _Batch()
    b.n_queries = n_queries
    b.x_dense = _ptr(x_dense)
    if x_csr is not None:
        b.x_indptr, b.x_ids, b.x_vals = _ptr(x_csr[0]), _ptr(x_csr[1]), _ptr(x_csr[2])
    b.budget_bp = _ptr(budget_bp)
    b.max_budget_bp = max_budget_bp
    b.logits, b.logit_ids, b.pred, b.codes = _ptr(logits), _ptr(logit_ids), _ptr(pred), _ptr(codes)
    b.active_indptr, b.active_ids, b.active_vals = _ptr(active_indptr), _ptr(active_ids), _ptr(active_vals)
    b.status = _ptr(status)
    b.kernel_path = kernel_path
    b.flags = flags
    return b


def slonn_run(model: Model, batch: _Batch, workspace, workspace_bytes: int, stream=None) -> None:
    rc = lib().slonn_run(model.handle, C.byref(batch), _ptr(workspace), workspace_bytes, _stream_ptr(stream))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_run")


def slonn_dense_layer(x_bf16, w_bf16, bias, M: int, N: int, D: int, relu: bool, out_f32=None, out_bf16=None,
                      status=None, stream=None) -> None:
    """out = act(X W^T + bias) on the tensor cores; device tensors, bf16 bit patterns for X, W, out_bf16."""
    rc = lib().slonn_dense_layer(_ptr(x_bf16), _ptr(w_bf16), _ptr(bias), M, N, D, int(bool(relu)), _ptr(out_f32),
                                 _ptr(out_bf16), _ptr(status), _stream_ptr(stream))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_dense_layer")


def slonn_test_tc_wait_limit(polls: int) -> None:
    """Testing aid: polls != 0 makes later tensor-core launches give up on their first wait after that many
    polls (status[0] = 8, nothing computed); 0 restores normal operation."""
    rc = lib().slonn_test_tc_wait_limit(int(polls))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_test_tc_wait_limit")


STATIC_WORKSPACE_BYTES = 16 << 20


def slonn_run_static(model: Model, batch: _Batch, stream=None) -> None:
    """slonn_run for callers that may not allocate device memory: no workspace argument, the
    library's built-in scratch area (STATIC_WORKSPACE_BYTES) is used instead.  Raises
    SlonnError(SLONN_ERR_WORKSPACE) when the batch needs more than that.  Calls on one device
    share the scratch area, so keep them on one stream; make the first call before any stream
    capture starts."""
    rc = lib().slonn_run_static(model.handle, C.byref(batch), _stream_ptr(stream))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_run_static")


STAGES = ("plan", "hash_select", "gather_dot", "sparse_first", "argmax", "fused", "dense_tc", "cluster", "gather_cols", "layer_cols", "full_rows",
          "group_rows")
COLS_MAX_BP = 3500   # SLONN_COLS_MAX_BP
FLAG_DENSE_TC = 1
FLAG_ROW_KERNELS = 2
FLAG_COLUMN_KERNELS = 4
FLAG_UNGROUPED_ROWS = 8
PATH_AUTO, PATH_STAGED, PATH_FUSED, PATH_CLUSTER, PATH_BLOCK = 0, 1, 2, 3, 4


def slonn_run_timed(model: Model, batch: _Batch, workspace, workspace_bytes: int, stream=None):
    """Returns ({stage: ms}, {stage: launches}) for this run; synchronises the stream."""
    ms = np.zeros(len(STAGES), dtype=np.float32)
    cnt = np.zeros(len(STAGES), dtype=np.uint32)
    rc = lib().slonn_run_timed(model.handle, C.byref(batch), _ptr(workspace), workspace_bytes,
                               _stream_ptr(stream), ms.ctypes.data, cnt.ctypes.data)
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_run_timed")
    return dict(zip(STAGES, ms.tolist())), dict(zip(STAGES, cnt.tolist()))


ALL_LAYERS = 0xFFFFFFFF
MAX_RECORDS = 160


def slonn_run_traced(model: Model, batch: _Batch, workspace, workspace_bytes: int, stream=None) -> List[dict]:
    """One run with an event pair around every launch; returns the launch records in order, each a dict
    with stage (name), layer (None = every layer), bp_lo, bp_hi, skips_full, cols_bp, ms."""
    rec = (_LaunchRecord * MAX_RECORDS)()
    n = C.c_uint32()
    rc = lib().slonn_run_traced(model.handle, C.byref(batch), _ptr(workspace), workspace_bytes,
                                _stream_ptr(stream), C.addressof(rec), MAX_RECORDS, C.byref(n))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_run_traced")
    return [dict(stage=STAGES[r.stage], layer=None if r.layer == ALL_LAYERS else int(r.layer), bp_lo=int(r.bp_lo),
                 bp_hi=int(r.bp_hi), skips_full=bool(r.skips_full), cols_bp=int(r.cols_bp), ms=float(r.ms))
            for r in rec[: n.value]]


def slonn_run_host(model: Model, host_batch: _Batch, workspace, workspace_bytes: int, stream=None):
    """Returns (h2d_bytes, d2h_bytes)."""
    up, down = C.c_uint64(), C.c_uint64()
    rc = lib().slonn_run_host(model.handle, C.byref(host_batch), _ptr(workspace), workspace_bytes,
                              _stream_ptr(stream), C.byref(up), C.byref(down))
    if rc != SLONN_OK:
        raise SlonnError(rc, "slonn_run_host")
    return up.value, down.value
