"""Device-side plumbing shared by the tests, the benchmark and the smoke check:
uploads a workload with torch, calls the binding, brings results back as numpy.
torch is used for device memory and streams only."""
import time
from typing import Optional

import numpy as np
import torch

from . import binding as sl
from .workloads import Workload


def _dev(a: np.ndarray, device) -> torch.Tensor:
    """Upload a numpy array keeping its bits (uint16/uint32/uint64 go up as same-width ints)."""
    a = np.ascontiguousarray(a)
    view = {np.dtype(np.uint16): np.int16, np.dtype(np.uint32): np.int32, np.dtype(np.uint64): np.int64}
    if a.dtype in view:
        a = a.view(view[a.dtype])
    return torch.from_numpy(a).to(device)


class DeviceModel:
    """A workload's weights on the device plus the built SLO-NN model."""

    def __init__(self, wl: Workload, device="cuda:0", n_cal: Optional[int] = None, hash_nodes_override=None):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required; this library has no CPU path")
        self.wl = wl
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.W = [_dev(w, self.device) for w in wl.W_store]
        self.bias = [_dev(b, self.device) for b in wl.bias]
        dtype = sl.SLONN_BF16 if wl.dtype == "bf16" else sl.SLONN_F32
        calib_dense = calib_csr = None
        if wl.first_sparse:
            ip, ids, vals = wl.calib
            if n_cal is not None:
                ip = ip[: n_cal + 1]
                ids, vals = ids[: int(ip[-1])], vals[: int(ip[-1])]
            calib_csr = (_dev(ip, self.device), _dev(ids, self.device), _dev(vals, self.device))
        else:
            c = wl.calib if n_cal is None else wl.calib[:n_cal]
            calib_dense = _dev(c, self.device)
        torch.cuda.synchronize(self.device)
        t0 = time.perf_counter()
        self.model = sl.slonn_build(wl.dims, wl.has_act, dtype, self.W, self.bias, calib_dense=calib_dense,
                                    calib_csr=calib_csr, K=wl.K, L=wl.L, list_cap=wl.list_cap, seed=wl.seed,
                                    first_layer_sparse=wl.first_sparse, hash_nodes_override=hash_nodes_override,
                                    free_hash_nodes=wl.free_hash_nodes)
        torch.cuda.synchronize(self.device)
        self.build_ms = (time.perf_counter() - t0) * 1e3   # slonn_build synchronises before it returns
        self.n_cal = int(calib_csr[0].numel() - 1) if calib_csr is not None else int(calib_dense.shape[0])

    def hash_nodes(self, layer: int) -> np.ndarray:
        return sl.slonn_model_info(self.model, layer)["hash_nodes"]

    def tables(self, layer: int) -> np.ndarray:
        return sl.slonn_model_tables_to_host(self.model, layer)

    def table_bytes(self) -> int:
        return sum(sl.slonn_model_info(self.model, l)["table_bytes"] for l in range(len(self.wl.dims) - 1))

    def free(self):
        sl.slonn_free(self.model)


class DeviceBatch:
    """Device buffers of one batch: inputs uploaded once, outputs preallocated."""

    def __init__(self, dm: DeviceModel, x, budget_bp: np.ndarray, max_budget_bp: int = 0, full_outputs=True,
                 kernel_path: int = 0, flags: int = 0):
        dev = dm.device
        self.dm = dm
        m = dm.model
        self.n = int(budget_bp.size)
        self.max_bp = int(max_budget_bp) if max_budget_bp else int(budget_bp.max()) if self.n else 10000
        self.x_dense = self.x_csr = None
        if dm.wl.first_sparse:
            self.x_csr = tuple(_dev(a, dev) for a in x)
        else:
            self.x_dense = _dev(x, dev)
        self.bp = _dev(np.ascontiguousarray(budget_bp, dtype=np.uint16), dev)
        self.stride = sl.slonn_logit_stride(m, self.max_bp)
        self.cap = sl.slonn_active_capacity(m, self.n, self.max_bp)
        self.last_budgeted = bool(dm.wl.has_act[-1])
        n = max(self.n, 1)
        self.logits = torch.zeros((n, self.stride), dtype=torch.float32, device=dev)
        self.logit_ids = torch.zeros((n, self.stride), dtype=torch.int32, device=dev) if self.last_budgeted else None
        self.pred = torch.zeros(n, dtype=torch.int32, device=dev)
        self.status = torch.zeros(4, dtype=torch.int32, device=dev)
        self.codes = self.indptr = self.ids = self.vals = None
        if full_outputs:
            self.codes = torch.zeros((n, max(m.n_act, 1), m.L), dtype=torch.int16, device=dev)
            self.indptr = torch.zeros(n * m.n_act + 1, dtype=torch.int64, device=dev)
            self.ids = torch.zeros(max(self.cap, 1), dtype=torch.int32, device=dev)
            self.vals = torch.zeros(max(self.cap, 1), dtype=torch.float32, device=dev)
        self.ws_bytes = sl.slonn_workspace_bytes(m, self.n, self.max_bp, flags)
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device=dev)
        self.batch = sl.make_batch(self.n, self.bp, self.logits, self.status, x_dense=self.x_dense,
                                   x_csr=self.x_csr, max_budget_bp=self.max_bp, logit_ids=self.logit_ids,
                                   pred=self.pred, codes=self.codes, active_indptr=self.indptr,
                                   active_ids=self.ids, active_vals=self.vals, kernel_path=kernel_path, flags=flags)

    def run(self, stream=None):
        sl.slonn_run(self.dm.model, self.batch, self.ws, self.ws_bytes, stream)

    def results(self) -> dict:
        torch.cuda.synchronize(self.dm.device)
        m = self.dm.model
        out = {
            "status": self.status.cpu().numpy().view(np.uint32),
            "logits": self.logits.cpu().numpy()[: self.n],
            "pred": self.pred.cpu().numpy().view(np.uint32)[: self.n],
            "logit_stride": self.stride,
        }
        if self.logit_ids is not None:
            out["logit_ids"] = self.logit_ids.cpu().numpy().view(np.uint32)[: self.n]
        if self.codes is not None:
            out["codes"] = self.codes.cpu().numpy().view(np.uint16)[: self.n, : m.n_act]
            out["active_indptr"] = self.indptr.cpu().numpy().view(np.uint64)
            total = int(out["active_indptr"][-1])
            out["active_ids"] = self.ids.cpu().numpy().view(np.uint32)[:total]
            out["active_vals"] = self.vals.cpu().numpy()[:total]
        return out


def run_once(dm: DeviceModel, x, budget_bp: np.ndarray, max_budget_bp: int = 0, kernel_path: int = 0,
             flags: int = 0) -> dict:
    b = DeviceBatch(dm, x, budget_bp, max_budget_bp, kernel_path=kernel_path, flags=flags)
    b.run()
    return b.results()
