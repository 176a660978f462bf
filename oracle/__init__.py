"""ctypes loader for the float64 CPU oracle (oracle/plora_oracle.c).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's
CPU-baseline leg import this; the product package never does.  Nothing here
touches CUDA or the product package.

Arrays are numpy: bf16 tensors as uint16 bit patterns, ids int32, y_in fp32,
results float64.  Adapters are passed as Python lists of per-adapter arrays in
the paper's logical layout, A_a [d_in, r_a] and B_a [r_a, d_out] (Section II-A).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_DIR = Path(__file__).resolve().parent
_SRC = _DIR / "plora_oracle.c"
_LIB = _DIR / "_build" / "libplora_oracle.so"

OK = 0
ERR_INVALID_ARG = -1
ERR_BAD_ADAPTER_ID = -3

_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (-O2 -fopenmp).  Rebuilds when the source is newer."""
    if not force and _LIB.exists() and _LIB.stat().st_mtime >= _SRC.stat().st_mtime:
        return _LIB
    _LIB.parent.mkdir(exist_ok=True)
    tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
    cmd = ["gcc", "-O2", "-fopenmp", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off",
           "-Wall", "-o", str(tmp), str(_SRC), "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        i32, p = ctypes.c_int32, ctypes.c_void_p
        lib.plora_oracle_bucket.argtypes = [p, i32, i32, p, p, p, p, p]
        lib.plora_oracle_shrink.argtypes = [p, p, i32, i32, i32, p, p, p, i32]
        lib.plora_oracle_expand.argtypes = [p, i32, p, i32, i32, i32, p, p, p, p, p]
        lib.plora_oracle_lora_delta.argtypes = [p, p, i32, i32, i32, i32, p, p, p, p, p, p]
        for f in (lib.plora_oracle_bucket, lib.plora_oracle_shrink, lib.plora_oracle_expand,
                  lib.plora_oracle_lora_delta, lib.plora_oracle_threads):
            f.restype = ctypes.c_int
        _lib = lib
    return _lib


def set_input_type(fp16: bool) -> None:
    """x, A and B are read as IEEE half (True) or bf16 (False, the default) from now on."""
    _load().plora_oracle_set_input_type(1 if fp16 else 0)


def input_to_double(bits) -> np.ndarray:
    """The float64 value of every 16-bit pattern under the current input type (exact)."""
    lib = _load()
    lib.plora_oracle_input_to_double.restype = ctypes.c_double
    lib.plora_oracle_input_to_double.argtypes = [ctypes.c_uint16]
    flat = np.ascontiguousarray(bits, np.uint16).ravel()
    return np.array([lib.plora_oracle_input_to_double(int(b)) for b in flat], np.float64).reshape(np.shape(bits))


def threads() -> int:
    """Threads an oracle call will use (OpenMP default: the cores available to the process)."""
    return int(_load().plora_oracle_threads())


class OracleError(ValueError):
    def __init__(self, code: int):
        super().__init__(f"oracle status {code}")
        self.code = code


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _ptr_table(mats, ranks, inner_first: bool, other_dim: int):
    """Array of per-adapter data pointers; checks each matrix has its adapter's shape."""
    n = len(mats)
    keep = []
    tab = (ctypes.c_void_p * n)()
    for a, m in enumerate(mats):
        if m is None:  # adapter not materialised: legal as long as no token uses it
            tab[a] = None
            continue
        m = np.ascontiguousarray(m, dtype=np.uint16)
        want = (other_dim, int(ranks[a])) if inner_first else (int(ranks[a]), other_dim)
        if m.shape != want:
            raise ValueError(f"adapter {a}: shape {m.shape}, expected {want}")
        keep.append(m)
        tab[a] = m.ctypes.data
    return tab, keep


def _check_present(ids, mats):
    for a in np.unique(ids[ids >= 0]):
        if a < len(mats) and mats[int(a)] is None:
            raise ValueError(f"adapter {int(a)} is used by a token but was not supplied")


def bucket(ids, n_adapters: int):
    """Stable bucketing of tokens by adapter id.

    Returns dict(perm, seg_adapter, seg_start, n_seg, n_active); array lengths
    T, min(T,N), min(T,N)+1 with the tail conventions of the C function.
    """
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    T = int(ids.shape[0])
    cap = min(T, int(n_adapters))
    perm = np.empty(T, np.int32)
    seg_adapter = np.empty(cap, np.int32)
    seg_start = np.empty(cap + 1, np.int32)
    n_seg = ctypes.c_int32(0)
    n_active = ctypes.c_int32(0)
    rc = _load().plora_oracle_bucket(_ptr(ids), T, int(n_adapters), _ptr(perm), _ptr(seg_adapter),
                                     _ptr(seg_start), ctypes.byref(n_seg), ctypes.byref(n_active))
    if rc != OK:
        raise OracleError(rc)
    return dict(perm=perm, seg_adapter=seg_adapter, seg_start=seg_start,
                n_seg=int(n_seg.value), n_active=int(n_active.value))


def shrink(x_bits, ids, ranks, A, ldm: int | None = None):
    """m = x A[a_t] per token, float64 [T, ldm] (ldm defaults to the largest rank)."""
    x_bits = np.ascontiguousarray(x_bits, dtype=np.uint16)
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    ranks = np.ascontiguousarray(ranks, dtype=np.int32)
    T, d_in = x_bits.shape
    N = len(A)
    ldm = int(ranks.max()) if ldm is None else int(ldm)
    _check_present(ids, A)
    tabA, keep = _ptr_table(A, ranks, True, d_in)
    m = np.empty((T, ldm), np.float64)
    rc = _load().plora_oracle_shrink(_ptr(x_bits), _ptr(ids), T, d_in, N, _ptr(ranks), tabA, _ptr(m), ldm)
    del keep
    if rc != OK:
        raise OracleError(rc)
    return m


def expand(m, ids, ranks, scales, B, d_out: int, y_in=None):
    """y_out = y_in + s_a (m_t B[a_t]), float64 [T, d_out]."""
    m = np.ascontiguousarray(m, dtype=np.float64)
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    ranks = np.ascontiguousarray(ranks, dtype=np.int32)
    scales = np.ascontiguousarray(scales, dtype=np.float32)
    T, ldm = m.shape
    N = len(B)
    _check_present(ids, B)
    tabB, keep = _ptr_table(B, ranks, False, d_out)
    if y_in is not None:
        y_in = np.ascontiguousarray(y_in, dtype=np.float32)
        assert y_in.shape == (T, d_out)
    y = np.empty((T, d_out), np.float64)
    rc = _load().plora_oracle_expand(_ptr(m), ldm, _ptr(ids), T, d_out, N, _ptr(ranks), _ptr(scales), tabB,
                                     _ptr(y_in), _ptr(y))
    del keep
    if rc != OK:
        raise OracleError(rc)
    return y


def lora_delta(x_bits, ids, ranks, scales, A, B, d_out: int, y_in=None):
    """y_out = y_in + s_a ((x_t A[a_t]) B[a_t]), float64 [T, d_out]; id -1 leaves y_in."""
    x_bits = np.ascontiguousarray(x_bits, dtype=np.uint16)
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    ranks = np.ascontiguousarray(ranks, dtype=np.int32)
    scales = np.ascontiguousarray(scales, dtype=np.float32)
    T, d_in = x_bits.shape
    N = len(A)
    assert len(B) == N and ranks.shape == (N,) and scales.shape == (N,)
    _check_present(ids, A)
    _check_present(ids, B)
    tabA, keepA = _ptr_table(A, ranks, True, d_in)
    tabB, keepB = _ptr_table(B, ranks, False, d_out)
    if y_in is not None:
        y_in = np.ascontiguousarray(y_in, dtype=np.float32)
        assert y_in.shape == (T, d_out)
    y = np.empty((T, d_out), np.float64)
    rc = _load().plora_oracle_lora_delta(_ptr(x_bits), _ptr(ids), T, d_in, d_out, N, _ptr(ranks), _ptr(scales),
                                         tabA, tabB, _ptr(y_in), _ptr(y))
    del keepA, keepB
    if rc != OK:
        raise OracleError(rc)
    return y
