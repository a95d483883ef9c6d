"""Test infrastructure: the CPU oracle on many tensors at once.

The oracle is single-threaded numpy; a 100 M-element tensor takes it about a minute.  Tensors are
independent, so the full-shape parity tests hand each one to its own worker process.  Workers are
spawned (never forked: a forked child of a process that has touched CUDA hangs) and get their
inputs as .npy files in a scratch directory, so nothing large goes through a pipe.  Every job
returns the oracle's record bytes, unchanged; the comparison happens in the test."""
from __future__ import annotations

import multiprocessing as mp
import os
import shutil
import tempfile

import numpy as np

_POOL = None
_DIR = None
_COUNTER = 0


def workers() -> int:
    return max(1, min(os.cpu_count() or 1, 32))


def _scratch_root() -> str:
    shm = "/dev/shm"
    try:
        if os.path.isdir(shm) and shutil.disk_usage(shm).free > 24e9:
            return shm
    except OSError:
        pass
    return tempfile.gettempdir()


def pool():
    global _POOL, _DIR
    if _POOL is None:
        _DIR = tempfile.mkdtemp(prefix="excp_oracle_", dir=_scratch_root())
        _POOL = mp.get_context("spawn").Pool(workers())
    return _POOL


def shutdown() -> None:
    global _POOL, _DIR
    if _POOL is not None:
        _POOL.terminate()
        _POOL.join()
        _POOL = None
    if _DIR is not None:
        shutil.rmtree(_DIR, ignore_errors=True)
        _DIR = None


def _save(arrays) -> list[str]:
    global _COUNTER
    pool()
    paths = []
    for a in arrays:
        _COUNTER += 1
        path = os.path.join(_DIR, f"a{_COUNTER}.npy")
        np.save(path, np.ascontiguousarray(a))
        paths.append(path)
    return paths


def _load(paths):
    out = [np.load(p) for p in paths]
    for p in paths:
        try:
            os.unlink(p)
        except OSError:
            pass
    return out


def _compress_job(paths, params, tensor_index: int, want_decode: bool):
    from oracle import excp_oracle as orc
    w_t, w_prev, ea, eas = _load(paths)
    outs = []
    for prm in (params if isinstance(params, list) else [params]):
        rec, info = orc.compress_tensor(w_t, w_prev, ea, eas, orc.Params(**prm), tensor_index=tensor_index)
        out = {"record": rec, "nnz_w": info["nnz_w"], "nnz_o": info["nnz_o"],
               "median": np.float32(info["median"]), "mean_abs_ea": np.float32(info["mean_abs_ea"]),
               "thr_w": np.float32(info["thr_w"]), "thr_o": np.float32(info["thr_o"])}
        if want_decode:
            out["decoded"] = orc.decompress_tensor(rec, w_prev)
        outs.append(out)
    return outs if isinstance(params, list) else outs[0]


def _chain_job(w0_path, step_paths, params: dict, tensor_index: int):
    """Section 3.4 / Algorithm 3 for one tensor: every residual is taken against the previous
    reconstruction; returns each step's record and the reconstruction after the last step."""
    from oracle import excp_oracle as orc
    (w_hat,) = _load([w0_path])
    records = []
    ea_hat = eas_hat = None
    for paths in step_paths:
        w_t, ea, eas = _load(paths)
        rec, _ = orc.compress_tensor(w_t, w_hat, ea, eas, orc.Params(**params), tensor_index=tensor_index)
        w_hat, ea_hat, eas_hat = orc.decompress_tensor(rec, w_hat)
        records.append(rec)
    return {"records": records, "w_hat": w_hat, "ea_hat": ea_hat, "eas_hat": eas_hat}


def submit_compress(quad_np, params, tensor_index: int, want_decode: bool = False):
    """quad_np = (w_t, w_prev, ea, eas) as numpy arrays; params = the keyword arguments of the oracle's Params, or
    a list of them (one result per entry, same inputs); returns an AsyncResult (.get())."""
    return pool().apply_async(_compress_job, (_save(quad_np), params, tensor_index, want_decode))


def submit_chain(w0, steps, params: dict, tensor_index: int):
    """steps = [(w_t, ea, eas), ...] in order; returns an AsyncResult."""
    (w0_path,) = _save([w0])
    return pool().apply_async(_chain_job, (w0_path, [_save(s) for s in steps], params, tensor_index))
