"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE, not product code).

Marshals numpy arrays to oracle/libslonn_oracle.so.  Nothing here is imported
by the CUDA library or its Python binding.
"""
import ctypes as C
import os

import numpy as np

from . import build_oracle

CANON32, REF64 = 0, 1

_lib = None


class _Batch(C.Structure):
    _fields_ = [
        ("n_queries", C.c_uint32),
        ("x_dense", C.c_void_p),
        ("x_indptr", C.c_void_p),
        ("x_ids", C.c_void_p),
        ("x_vals", C.c_void_p),
        ("budget_bp", C.c_void_p),
        ("mode", C.c_int),
        ("logit_stride", C.c_uint32),
        ("logits32", C.c_void_p),
        ("logits64", C.c_void_p),
        ("logit_ids", C.c_void_p),
        ("pred", C.c_void_p),
        ("codes", C.c_void_p),
        ("active_indptr", C.c_void_p),
        ("active_ids", C.c_void_p),
        ("active_vals32", C.c_void_p),
        ("active_vals64", C.c_void_p),
    ]


def lib():
    global _lib
    if _lib is None:
        # SLONN_ORACLE_LIB: another build of the oracle (the mutation tests point it at broken copies)
        path = os.environ.get("SLONN_ORACLE_LIB") or build_oracle.build()
        L = C.CDLL(path)
        L.orc_dot_canon32.restype = C.c_float
        L.orc_dot_canon32.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_float]
        L.orc_dot_ref64.restype = C.c_double
        L.orc_dot_ref64.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_float]
        L.orc_budget_nodes.restype = C.c_uint32
        L.orc_budget_nodes.argtypes = [C.c_uint32, C.c_uint32]
        L.orc_splitmix64.restype = C.c_uint64
        L.orc_splitmix64.argtypes = [C.POINTER(C.c_uint64)]
        L.orc_model_new.restype = C.c_void_p
        L.orc_model_new.argtypes = [C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint32,
                                    C.c_uint32, C.c_uint32, C.c_int]
        L.orc_model_set_layer.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p]
        L.orc_model_keep_scores.argtypes = [C.c_void_p, C.c_int]
        L.orc_model_set_free_hash_nodes.argtypes = [C.c_void_p, C.c_int]
        L.orc_layer_nodes.restype = C.c_uint32
        L.orc_layer_nodes.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32]
        L.orc_model_free.argtypes = [C.c_void_p]
        for name, rt in (("orc_model_hash_nodes", C.c_void_p), ("orc_model_rank", C.c_void_p),
                         ("orc_model_var", C.c_void_p), ("orc_model_score", C.c_void_p),
                         ("orc_model_bucket_count", C.c_void_p), ("orc_model_cap", C.c_uint32)):
            f = getattr(L, name)
            f.restype = rt
            f.argtypes = [C.c_void_p, C.c_uint32]
        L.orc_model_set_tables.restype = C.c_int
        L.orc_model_set_tables.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint32]
        L.orc_sample_hash_nodes.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint64,
                                            C.c_uint32, C.c_void_p]
        L.orc_build.restype = C.c_int
        L.orc_build.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                C.c_uint32, C.c_uint64, C.c_void_p]
        L.orc_run.restype = C.c_int
        L.orc_run.argtypes = [C.c_void_p, C.POINTER(_Batch)]
        L.orc_lcao_budgets.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint32,
                                       C.c_void_p, C.c_void_p]
        L.orc_threads.restype = C.c_int
        L.orc_confidence.restype = C.c_double
        L.orc_confidence.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32]
        L.orc_confidence_build.restype = C.c_int
        L.orc_confidence_build.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.c_void_p,
                                           C.c_void_p]
        L.orc_aclo_budgets.restype = C.c_int
        L.orc_aclo_budgets.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p,
                                       C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data


def _arr(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


def dot_canon32(w, x, V, bias=0.0):
    w = _arr(w, np.float32); x = _arr(x, np.float32)
    return float(lib().orc_dot_canon32(_p(w), _p(x), w.size, V, np.float32(bias)))


def dot_ref64(w, x, bias=0.0):
    w = _arr(w, np.float32); x = _arr(x, np.float64)
    return float(lib().orc_dot_ref64(_p(w), _p(x), w.size, np.float32(bias)))


def budget_nodes(bp, N):
    return int(lib().orc_budget_nodes(int(bp), int(N)))


def splitmix64(state):
    """Returns (output, new_state)."""
    s = C.c_uint64(state)
    out = lib().orc_splitmix64(C.byref(s))
    return int(out), int(s.value)


def sample_hash_nodes(var, H, seed, layer):
    var = _arr(var, np.float64)
    out = np.empty(H, dtype=np.uint32)
    lib().orc_sample_hash_nodes(_p(var), var.size, H, seed, layer, _p(out))
    return out


def lcao_budgets(profile_bp, profile_ms, t0, tau):
    """Eq. 3: per query the largest profiled k with t0 + T(k) <= tau; returns (budget_bp, feasible)."""
    pb = _arr(profile_bp, np.uint16); pm = _arr(profile_ms, np.float32)
    t0 = _arr(t0, np.float32); tau = _arr(tau, np.float32)
    out = np.zeros(t0.size, np.uint16); ok = np.zeros(t0.size, np.uint8)
    lib().orc_lcao_budgets(_p(pb), _p(pm), pb.size, _p(t0), _p(tau), t0.size, _p(out), _p(ok))
    return out, ok


def threads():
    return int(lib().orc_threads())


def confidence(z_full, z_k):
    """Eq. 1 with the cross-entropy as distance: c = sum_j softmax(z_full)_j * log softmax(z_k)_j."""
    a = _arr(z_full, np.float32); b = _arr(z_k, np.float32)
    assert a.shape == b.shape and a.ndim == 1
    return float(lib().orc_confidence(_p(a), _p(b), a.size))


class OracleModel:
    """dims = [D0, N1, ..., N_out]; W[l] float32 [N_l, D_l] (bf16 weights widened
    exactly); V = 4 for fp32 storage, 8 for bf16 storage.  free_hash_nodes: the variant in which
    a layer's K*L hash nodes are always active and are left out of its ranked lists."""

    def __init__(self, dims, has_act, W, bias, V, K=10, L=2, list_cap=0, first_sparse=False,
                 free_hash_nodes=False):
        self.dims = [int(d) for d in dims]
        self.n_layers = len(self.dims) - 1
        self.has_act = [int(bool(h)) for h in has_act]
        self.n_act = sum(self.has_act)
        self.K, self.L, self.V = int(K), int(L), int(V)
        self.first_sparse = bool(first_sparse)
        self.free_hash_nodes = bool(free_hash_nodes)
        self.W = [_arr(w, np.float32) for w in W]
        self.bias = [_arr(b, np.float32) for b in bias]
        for l in range(self.n_layers):
            assert self.W[l].shape == (self.dims[l + 1], self.dims[l])
            assert self.bias[l].shape == (self.dims[l + 1],)
        d = np.asarray(self.dims, dtype=np.uint32)
        h = np.asarray(self.has_act, dtype=np.uint8)
        self._m = lib().orc_model_new(self.n_layers, _p(d), _p(h), self.V, self.K, self.L,
                                      int(list_cap), int(self.first_sparse))
        if not self._m:
            raise ValueError("orc_model_new rejected the arguments")
        for l in range(self.n_layers):
            lib().orc_model_set_layer(self._m, l, _p(self.W[l]), _p(self.bias[l]))
        lib().orc_model_set_free_hash_nodes(self._m, int(self.free_hash_nodes))

    def __del__(self):
        if getattr(self, "_m", None):
            lib().orc_model_free(self._m)
            self._m = None

    # ---- build -----------------------------------------------------------
    def build(self, calib_dense=None, calib_csr=None, seed=0, hash_override=None, keep_scores=False):
        lib().orc_model_keep_scores(self._m, int(keep_scores))
        ov = None
        keep = []
        if hash_override is not None:
            ptrs = (C.c_void_p * self.n_layers)()
            for l in range(self.n_layers):
                if hash_override[l] is None:
                    ptrs[l] = None
                else:
                    a = _arr(hash_override[l], np.uint32)
                    assert a.size == self.K * self.L
                    keep.append(a)
                    ptrs[l] = a.ctypes.data
            ov = C.cast(ptrs, C.c_void_p)
        if self.first_sparse:
            indptr, ids, vals = calib_csr
            indptr = _arr(indptr, np.uint64); ids = _arr(ids, np.uint32); vals = _arr(vals, np.float32)
            n_cal = indptr.size - 1
            rc = lib().orc_build(self._m, None, _p(indptr), _p(ids), _p(vals), n_cal, seed, ov)
        else:
            cd = _arr(calib_dense, np.float32)
            assert cd.ndim == 2 and cd.shape[1] == self.dims[0]
            rc = lib().orc_build(self._m, _p(cd), None, None, None, cd.shape[0], seed, ov)
        if rc != 0:
            raise RuntimeError(f"orc_build failed: {rc}")

    def _view(self, fn, l, shape, ctype, dtype):
        ptr = fn(self._m, l)
        if not ptr:
            return None
        n = int(np.prod(shape))
        buf = (ctype * n).from_address(ptr)
        return np.frombuffer(buf, dtype=dtype).reshape(shape).copy()

    def cap(self, l):
        return int(lib().orc_model_cap(self._m, l))

    def hash_nodes(self, l):
        return self._view(lib().orc_model_hash_nodes, l, (self.L, self.K), C.c_uint32, np.uint32)

    def rank(self, l):
        return self._view(lib().orc_model_rank, l, (self.L, 1 << self.K, self.cap(l)), C.c_uint32, np.uint32)

    def var(self, l):
        return self._view(lib().orc_model_var, l, (self.dims[l + 1],), C.c_double, np.float64)

    def score(self, l):
        return self._view(lib().orc_model_score, l, (self.L, 1 << self.K, self.dims[l + 1]), C.c_double, np.float64)

    def bucket_count(self, l):
        return self._view(lib().orc_model_bucket_count, l, (self.L, 1 << self.K), C.c_uint32, np.uint32)

    def set_tables(self, l, hash_nodes, rank):
        hn = _arr(hash_nodes, np.uint32); rk = _arr(rank, np.uint32)
        assert hn.size == self.K * self.L and rk.shape[:2] == (self.L, 1 << self.K)
        rc = lib().orc_model_set_tables(self._m, l, _p(hn), _p(rk), rk.shape[2])
        if rc != 0:
            raise RuntimeError(f"orc_model_set_tables failed: {rc}")

    # ---- confidence tables, ACLO -------------------------------------------
    def confidence_build(self, calib_dense, profile_bp):
        """Confidence LSH tables: (sum [L, 2^K, n_k] float64, count [L, 2^K] uint32)."""
        cd = _arr(calib_dense, np.float32); pb = _arr(profile_bp, np.uint16)
        s = np.zeros((self.L, 1 << self.K, pb.size), np.float64)
        c = np.zeros((self.L, 1 << self.K), np.uint32)
        rc = lib().orc_confidence_build(self._m, _p(cd), cd.shape[0], _p(pb), pb.size, _p(s), _p(c))
        if rc != 0:
            raise RuntimeError(f"orc_confidence_build failed: {rc}")
        return s, c

    def aclo_budgets(self, conf_sum, conf_count, profile_bp, x_dense, threshold, target=None):
        """Eq. 2: (budget_bp [n] uint16, met [n] uint8, estimate [n, n_k] float64)."""
        s = _arr(conf_sum, np.float64); c = _arr(conf_count, np.uint32); pb = _arr(profile_bp, np.uint16)
        xd = _arr(x_dense, np.float32); th = _arr(np.atleast_2d(threshold), np.float32)
        tg = _arr(target, np.uint32)
        n = xd.shape[0]
        assert th.shape[1] == pb.size and s.shape == (self.L, 1 << self.K, pb.size)
        out = np.zeros(n, np.uint16); met = np.zeros(n, np.uint8); est = np.zeros((n, pb.size), np.float64)
        rc = lib().orc_aclo_budgets(self._m, _p(s), _p(c), _p(pb), pb.size, _p(xd), n, _p(th), _p(tg), _p(out),
                                    _p(met), _p(est))
        if rc != 0:
            raise RuntimeError(f"orc_aclo_budgets failed: {rc}")
        return out, met, est

    # ---- run -------------------------------------------------------------
    def budgets(self, budget_bp):
        """[n, n_act] node counts per query and activator layer."""
        act_N = [self.dims[l + 1] for l in range(self.n_layers) if self.has_act[l]]
        return np.array([[int(lib().orc_layer_nodes(self._m, int(bp), N)) for N in act_N] for bp in np.asarray(budget_bp)],
                        dtype=np.int64).reshape(len(budget_bp), len(act_N))

    def run(self, budget_bp, x_dense=None, x_csr=None, mode=CANON32):
        bp = _arr(budget_bp, np.uint16)
        n = bp.size
        last_budgeted = bool(self.has_act[-1])
        Bs = self.budgets(bp)
        N_out = self.dims[-1]
        stride = int(Bs[:, -1].max()) if (last_budgeted and n) else N_out
        total = int(Bs.sum())
        res = {
            "pred": np.zeros(n, np.uint32),
            "codes": np.zeros((n, self.n_act, self.L), np.uint16),
            "active_indptr": np.zeros(n * self.n_act + 1, np.uint64),
            "active_ids": np.zeros(total, np.uint32),
            "logit_ids": np.zeros((n, stride), np.uint32) if last_budgeted else None,
            "logit_stride": stride,
        }
        if mode == CANON32:
            res["logits"] = np.zeros((n, stride), np.float32)
            res["active_vals"] = np.zeros(total, np.float32)
        else:
            res["logits"] = np.zeros((n, stride), np.float64)
            res["active_vals"] = np.zeros(total, np.float64)
        b = _Batch()
        b.n_queries = n
        keep = []
        if self.first_sparse:
            indptr, ids, vals = x_csr
            indptr = _arr(indptr, np.uint64); ids = _arr(ids, np.uint32); vals = _arr(vals, np.float32)
            assert indptr.size == n + 1
            keep += [indptr, ids, vals]
            b.x_indptr, b.x_ids, b.x_vals = _p(indptr), _p(ids), _p(vals)
        else:
            xd = _arr(x_dense, np.float32)
            assert xd.shape == (n, self.dims[0])
            keep.append(xd)
            b.x_dense = _p(xd)
        b.budget_bp = _p(bp)
        b.mode = mode
        b.logit_stride = stride
        if mode == CANON32:
            b.logits32 = _p(res["logits"]); b.active_vals32 = _p(res["active_vals"])
        else:
            b.logits64 = _p(res["logits"]); b.active_vals64 = _p(res["active_vals"])
        b.logit_ids = _p(res["logit_ids"])
        b.pred = _p(res["pred"])
        b.codes = _p(res["codes"])
        b.active_indptr = _p(res["active_indptr"])
        b.active_ids = _p(res["active_ids"])
        rc = lib().orc_run(self._m, C.byref(b))
        if rc != 0:
            raise RuntimeError(f"orc_run failed: {rc}")
        return res
