"""ctypes wrapper around the fp64 CPU oracle (``treewy_oracle.c``).

TEST INFRASTRUCTURE.  Only ``tests/``, the smoke check and the bench's
CPU-baseline legs may import this module; the product (the CUDA library and its
Python binding) never does, and this module imports nothing from the product.

The C source is compiled with the host ``gcc`` on first use (or by
``build()``); no ``-march`` flag is given so the object runs on any x86-64 host.
All arrays cross the boundary as C-contiguous fp64 / int32 / uint64 numpy arrays;
storage dtypes (bf16, fp32) are widened exactly by the caller before the call.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "treewy_oracle.c")
_LIB = os.path.join(_HERE, "libtreewy_oracle.so")

SEQ_BAD_PARENT = 1
SEQ_TOO_MANY_NODES = 2
SEQ_BAD_ACCEPTED = 4
SEQ_BAD_OFFSETS = 32

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle into ``libtreewy_oracle.so`` next to its source."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        cmd = ["gcc", "-O3", "-std=c11", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
               _SRC, "-o", _LIB, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.treewy_oracle_num_threads.restype = ctypes.c_int
        lib.treewy_oracle_prepare.restype = ctypes.c_int
        lib.treewy_oracle_verify_commit.restype = ctypes.c_int
        _lib = lib
    return _lib


def set_max_nodes(n: int = 64) -> None:
    """Largest tree the oracle takes (default 64, the limit of the library's main calls)."""
    _load().treewy_oracle_set_max_nodes(ctypes.c_int32(int(n)))


def num_threads() -> int:
    """Threads the oracle's OpenMP loop uses (OMP_NUM_THREADS or the core count)."""
    return int(_load().treewy_oracle_num_threads())


def _arr(x, dtype):
    a = np.ascontiguousarray(np.asarray(x), dtype=dtype)
    return a


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


@dataclass
class OracleTree:
    depth: np.ndarray        # int32 [T]
    anc_mask: np.ndarray     # uint64 [T], bit j = local node j is ancestor-or-self
    cum_log_gate: np.ndarray  # float64 [T, H_v]
    level_order: np.ndarray  # uint8 [T], each sequence's nodes sorted by (depth, index)
    seq_status: np.ndarray   # int32 [B]


@dataclass
class OracleResult:
    O: np.ndarray            # float64 [T, H_v, d_v]
    U: np.ndarray            # float64 [T, H_v, d_v]
    S_commit: np.ndarray     # float64 [B, H_v, d_v, d_k]
    seq_status: np.ndarray   # int32 [B]
    Snap: np.ndarray | None  # float64 [T, H_v, d_v, d_k] when requested


def prepare(node_offsets, parent, alpha, T_declared: int | None = None) -> OracleTree:
    """depth, ancestor-or-self masks and cumulative log-gates of a packed batch of trees.
    T_declared: the packed node count the tree declares (default: the arrays' length); a sequence whose
    node range leaves 0..T_declared is flagged and skipped."""
    lib = _load()
    off = _arr(node_offsets, np.int32)
    par = _arr(parent, np.int32)
    al = _arr(alpha, np.float64)
    B, T = off.shape[0] - 1, par.shape[0]
    assert al.ndim == 2 and al.shape[0] == T
    H_v = al.shape[1]
    depth = np.full(T, -1, np.int32)
    mask = np.zeros(T, np.uint64)
    L = np.zeros((T, H_v), np.float64)
    order = np.zeros(T, np.uint8)
    status = np.zeros(B, np.int32)
    Td = T if T_declared is None else int(T_declared)
    assert 0 <= Td <= T
    rc = lib.treewy_oracle_prepare(ctypes.c_int32(B), ctypes.c_int32(Td), ctypes.c_int32(H_v), _ptr(off), _ptr(par),
                                   _ptr(al), _ptr(depth), _ptr(mask), _ptr(L), _ptr(order),
                                   _ptr(status))
    assert rc == 0
    return OracleTree(depth, mask, L, order, status)


def verify_commit(node_offsets, parent, S0, q, k, v, alpha, beta, accepted,
                  want_snapshots: bool = False, T_declared: int | None = None) -> OracleResult:
    """Outputs, pseudo-values and the committed state by walking Eq. 1 along every path."""
    lib = _load()
    off = _arr(node_offsets, np.int32)
    par = _arr(parent, np.int32)
    S0 = _arr(S0, np.float64)
    q = _arr(q, np.float64)
    k = _arr(k, np.float64)
    v = _arr(v, np.float64)
    al = _arr(alpha, np.float64)
    be = _arr(beta, np.float64)
    acc = _arr(accepted, np.int32)
    B, T = off.shape[0] - 1, par.shape[0]
    _, H_v, d_v, d_k = S0.shape
    H_qk = q.shape[1]
    assert S0.shape[0] == B and q.shape == (T, H_qk, d_k) and k.shape == q.shape
    assert v.shape == (T, H_v, d_v) and al.shape == (T, H_v) and be.shape == (T, H_v)
    assert acc.shape == (B,)
    O = np.zeros((T, H_v, d_v), np.float64)
    U = np.zeros((T, H_v, d_v), np.float64)
    Sc = np.zeros((B, H_v, d_v, d_k), np.float64)
    Snap = np.zeros((T, H_v, d_v, d_k), np.float64) if want_snapshots else None
    status = np.zeros(B, np.int32)
    rc = lib.treewy_oracle_verify_commit(
        ctypes.c_int32(B), ctypes.c_int32(T if T_declared is None else int(T_declared)),
        ctypes.c_int32(H_v), ctypes.c_int32(H_qk), ctypes.c_int32(d_k),
        ctypes.c_int32(d_v), _ptr(off), _ptr(par), _ptr(S0), _ptr(q), _ptr(k), _ptr(v), _ptr(al),
        _ptr(be), _ptr(acc), _ptr(O), _ptr(U), _ptr(Sc), _ptr(Snap), _ptr(status))
    if rc != 0:
        raise RuntimeError(f"treewy_oracle_verify_commit failed with code {rc}")
    return OracleResult(O, U, Sc, status, Snap)
