"""Helpers shared by the GPU parity tests: move workload inputs to the device, run libcsat through its
C-ABI binding, fetch results as float64 numpy, and the error metric of the parity bar."""
import numpy as np
import torch

from paper_2507_02957_b200 import binding, workloads as wl

TOL = {"bf16": 2e-2, "fp32": 1e-4}     # max|gpu - oracle| / max|oracle|


def to_dev(x: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    return t if dtype == "fp32" else t.to(torch.bfloat16)   # exact: values are already bf16-representable


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def rel_err(gpu: np.ndarray, ref: np.ndarray) -> float:
    den = np.abs(ref).max()
    return float(np.abs(gpu - ref).max() / den) if den > 0 else float(np.abs(gpu).max())


def make_ctx(w: wl.Workload, **kw) -> binding.Csat:
    args = dict(B=w.B, n_q=w.n_q, dtype=w.dtype, T=w.T, lam=w.lam)
    args.update(kw)
    return binding.Csat(w.n, w.m, w.d, w.H, w.phi_seed, **args)


def device_inputs(w: wl.Workload, inp: dict):
    Q, K, V = (to_dev(inp[k], w.dtype) for k in "QKV")
    Psi = None if inp.get("Psi") is None else to_dev(inp["Psi"], w.dtype)
    return Q, K, V, Psi
