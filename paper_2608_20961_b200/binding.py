"""Thin ctypes binding of libtreewy's C ABI (``include/treewy.h``).

Argument marshalling only: torch tensors supply device memory and the stream, every
step of verify / commit runs inside the library's CUDA kernels.  There is no CPU or
PyTorch fallback -- if ``libtreewy.so`` cannot be loaded the import of a function fails
loudly.  Function names and argument order follow the C header.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libtreewy.so")

TREEWY_OK, TREEWY_ERR_INVALID_ARG, TREEWY_ERR_UNSUPPORTED, TREEWY_ERR_CUDA = 0, 1, 2, 3
TREEWY_F32, TREEWY_BF16 = 0, 1
SEQ_BAD_PARENT, SEQ_TOO_MANY_NODES, SEQ_BAD_ACCEPTED, SEQ_TIMEOUT, SEQ_BAD_STATE, SEQ_BAD_OFFSETS = 1, 2, 4, 8, 16, 32
D = 128
MAX_NODES = 64

_DTYPES = {torch.float32: TREEWY_F32, torch.bfloat16: TREEWY_BF16}


class TreeStruct(ctypes.Structure):
    """Mirror of ``treewy_tree_t``."""
    _fields_ = [
        ("B", ctypes.c_int32), ("T", ctypes.c_int32), ("H_v", ctypes.c_int32),
        ("max_nodes", ctypes.c_int32),
        ("node_offsets", ctypes.c_void_p), ("parent", ctypes.c_void_p),
        ("depth", ctypes.c_void_p), ("anc_mask", ctypes.c_void_p),
        ("cum_log_gate", ctypes.c_void_p), ("level_order", ctypes.c_void_p),
    ]


class PoolStruct(ctypes.Structure):
    """Mirror of ``treewy_state_pool_t``."""
    _fields_ = [("states", ctypes.c_void_p), ("state_index", ctypes.c_void_p), ("n_states", ctypes.c_int32)]


class TreewyError(RuntimeError):
    def __init__(self, fn: str, code: int):
        self.code = code
        super().__init__(f"{fn} returned {code} ({status_string(code)})")


_lib = None


def load_library(path: str | None = None):
    """Load ``libtreewy.so`` (built in-tree by ``build.py``); raises if it is absent."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise ImportError(
            f"{path} not found: build it with `python -m paper_2608_20961_b200.build` "
            "(nvcc, sm_100a). libtreewy has no CPU fallback.")
    lib = ctypes.CDLL(path)
    vp, i32 = ctypes.c_void_p, ctypes.c_int32
    lib.treewy_tree_prepare.argtypes = [ctypes.POINTER(TreeStruct), vp, vp, vp]
    lib.treewy_tree_prepare.restype = ctypes.c_int
    lib.treewy_tree_prepare_log.argtypes = [ctypes.POINTER(TreeStruct), vp, vp, vp]
    lib.treewy_tree_prepare_log.restype = ctypes.c_int
    lib.treewy_verify_pool.argtypes = [ctypes.POINTER(PoolStruct), vp, vp, vp, vp, ctypes.POINTER(TreeStruct), i32,
                                       ctypes.c_int, ctypes.c_int, vp, vp, vp, vp]
    lib.treewy_verify_pool.restype = ctypes.c_int
    lib.treewy_commit_pool.argtypes = [ctypes.POINTER(PoolStruct), vp, vp, ctypes.POINTER(TreeStruct), i32, vp,
                                       ctypes.c_int, vp, vp]
    lib.treewy_commit_pool.restype = ctypes.c_int
    verify_args = [vp, vp, vp, vp, vp, ctypes.POINTER(TreeStruct), i32, ctypes.c_int, ctypes.c_int,
                   vp, vp, vp, vp]
    lib.treewy_verify.argtypes = verify_args
    lib.treewy_verify.restype = ctypes.c_int
    lib.treewy_verify_generic.argtypes = verify_args
    lib.treewy_verify_generic.restype = ctypes.c_int
    lib.treewy_commit.argtypes = [vp, vp, vp, ctypes.POINTER(TreeStruct), i32, vp, ctypes.c_int,
                                  vp, vp, vp]
    lib.treewy_commit.restype = ctypes.c_int
    lib.treewy_verify_half_u.argtypes = verify_args
    lib.treewy_verify_half_u.restype = ctypes.c_int
    lib.treewy_commit_half_u.argtypes = lib.treewy_commit.argtypes
    lib.treewy_commit_half_u.restype = ctypes.c_int
    lib.treewy_tree_prepare_wide.argtypes = [ctypes.POINTER(TreeStruct), vp, vp, vp]
    lib.treewy_tree_prepare_wide.restype = ctypes.c_int
    lib.treewy_verify_wide.argtypes = verify_args
    lib.treewy_verify_wide.restype = ctypes.c_int
    lib.treewy_commit_wide.argtypes = lib.treewy_commit.argtypes
    lib.treewy_commit_wide.restype = ctypes.c_int
    lib.treewy_commit_verify.argtypes = [vp, vp, vp, ctypes.POINTER(TreeStruct), vp, vp, vp, vp, vp,
                                         ctypes.POINTER(TreeStruct), i32, ctypes.c_int, ctypes.c_int, vp, vp, i32, vp, vp]
    lib.treewy_commit_verify.restype = ctypes.c_int
    lib.treewy_commit_verify_pool.argtypes = [ctypes.POINTER(PoolStruct), vp, vp, ctypes.POINTER(TreeStruct), vp, vp,
                                              vp, vp, vp, ctypes.POINTER(TreeStruct), i32, ctypes.c_int, ctypes.c_int,
                                              vp, vp, i32, vp, vp]
    lib.treewy_commit_verify_pool.restype = ctypes.c_int
    lib.treewy_snapshot_all.argtypes = [vp, vp, vp, ctypes.POINTER(TreeStruct), i32, ctypes.c_int, vp, vp, vp]
    lib.treewy_snapshot_all.restype = ctypes.c_int
    lib.treewy_debug_inject.argtypes = [ctypes.c_int64, ctypes.c_int32]
    lib.treewy_debug_inject.restype = None
    lib.treewy_status_string.argtypes = [ctypes.c_int]
    lib.treewy_status_string.restype = ctypes.c_char_p
    lib.treewy_version.restype = ctypes.c_int
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().treewy_status_string(int(code)).decode()


def version() -> int:
    return int(load_library().treewy_version())


def treewy_debug_inject(wait_cycles: int = 0, skip_item: int = -1) -> None:
    """Test hook: limit of the kernels' bounded waits (SM clocks, 0 = default) and the one item whose
    loads the tree-verify kernel never issues (-1 = none).  Process-wide; tests only."""
    load_library().treewy_debug_inject(int(wait_cycles), int(skip_item))


def _p(t: torch.Tensor | None):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check(fn: str, code: int):
    if code != TREEWY_OK:
        raise TreewyError(fn, code)


_recording: list | None = None


def _call(name: str, cfunc, *cargs):
    """Invoke one C entry point with marshalled arguments (or, inside ``prebound``, record it)."""
    if _recording is not None:
        _recording.append((name, cfunc, cargs))
        return
    _check(name, cfunc(*cargs))


class Prebound:
    """C calls with their arguments already marshalled: calling the object enqueues them again on
    the stream(s) they were recorded with.  For loops that call the library with the same buffers
    step after step (a decoding loop over fixed device buffers): the per-call Python work of
    building structs and pointer objects is done once."""

    def __init__(self, calls, keep):
        self._calls, self._keep = calls, keep

    def __call__(self) -> None:
        for name, cfunc, cargs in self._calls:
            code = cfunc(*cargs)
            if code != TREEWY_OK:
                raise TreewyError(name, code)


def prebound(fn, *args, **kwargs) -> Prebound:
    """Marshal ``fn(*args, **kwargs)`` (any function of this module, or a callable that makes several
    such calls) once and return a ``Prebound`` that replays the C call(s).  Tensors and trees passed in
    are kept alive by the returned object; the stream is the one current (or passed) at this time."""
    global _recording
    assert _recording is None, "prebound() does not nest"
    _recording = []
    try:
        fn(*args, **kwargs)
        calls = _recording
    finally:
        _recording = None
    return Prebound(calls, (args, kwargs))


@dataclass
class Tree:
    """Device-side ``treewy_tree_t``: topology in, depth / mask / log-gates out."""
    B: int
    T: int
    H_v: int
    max_nodes: int
    node_offsets: torch.Tensor   # int32 [B+1]
    parent: torch.Tensor         # int32 [T]
    depth: torch.Tensor          # int32 [T]
    anc_mask: torch.Tensor       # int64 storage of the uint64 masks [T]
    cum_log_gate: torch.Tensor   # fp32 [T, H_v]
    level_order: torch.Tensor    # uint8 [T]

    @classmethod
    def empty(cls, node_offsets: torch.Tensor, parent: torch.Tensor, H_v: int,
              max_nodes: int = 0) -> "Tree":
        dev = parent.device
        T = int(parent.numel())
        return cls(B=int(node_offsets.numel()) - 1, T=T, H_v=H_v, max_nodes=max_nodes,
                   node_offsets=node_offsets, parent=parent,
                   depth=torch.full((max(T, 1),), -1, dtype=torch.int32, device=dev),
                   anc_mask=torch.zeros((max(T, 1),), dtype=torch.int64, device=dev),
                   cum_log_gate=torch.zeros((max(T, 1), H_v), dtype=torch.float32, device=dev),
                   level_order=torch.zeros((max(T, 1),), dtype=torch.uint8, device=dev))

    def struct(self) -> TreeStruct:
        return TreeStruct(self.B, self.T, self.H_v, self.max_nodes,
                          self.node_offsets.data_ptr(), self.parent.data_ptr(),
                          self.depth.data_ptr(), self.anc_mask.data_ptr(),
                          self.cum_log_gate.data_ptr(), self.level_order.data_ptr())


def treewy_tree_prepare(tree: Tree, alpha: torch.Tensor, seq_status: torch.Tensor | None = None,
                        stream=None) -> None:
    lib = load_library()
    ts = tree.struct()
    _call("treewy_tree_prepare", lib.treewy_tree_prepare, ctypes.byref(ts), _p(alpha), _p(seq_status), _stream(stream))


def treewy_tree_prepare_log(tree: Tree, log_alpha: torch.Tensor, seq_status: torch.Tensor | None = None,
                            stream=None) -> None:
    """As treewy_tree_prepare, with the gates given as logarithms (log alpha <= 0)."""
    lib = load_library()
    ts = tree.struct()
    _call("treewy_tree_prepare_log", lib.treewy_tree_prepare_log, ctypes.byref(ts), _p(log_alpha), _p(seq_status), _stream(stream))


def _pool(states: torch.Tensor, state_index: torch.Tensor) -> PoolStruct:
    assert state_index.dtype == torch.int32
    return PoolStruct(states.data_ptr(), state_index.data_ptr(), int(states.shape[0]))


def treewy_verify_pool(states, state_index, q, k, v, beta, tree: Tree, H_qk: int, O: torch.Tensor,
                       U: torch.Tensor, seq_status: torch.Tensor | None = None, stream=None) -> None:
    """treewy_verify with sequence b's state at states[state_index[b]] (block-pool addressing)."""
    lib = load_library()
    ts, ps = tree.struct(), _pool(states, state_index)
    _call("treewy_verify_pool", lib.treewy_verify_pool, ctypes.byref(ps), _p(q), _p(k), _p(v), _p(beta), ctypes.byref(ts), H_qk,
                                  _DTYPES[states.dtype], _DTYPES[O.dtype], _p(O), _p(U), _p(seq_status), _stream(stream))


def treewy_commit_pool(states, state_index, U, k, tree: Tree, H_qk: int, accepted: torch.Tensor,
                       seq_status: torch.Tensor | None = None, stream=None) -> None:
    """treewy_commit, in place, with sequence b's state at states[state_index[b]]."""
    lib = load_library()
    ts, ps = tree.struct(), _pool(states, state_index)
    _call("treewy_commit_pool", lib.treewy_commit_pool, ctypes.byref(ps), _p(U), _p(k), ctypes.byref(ts), H_qk, _p(accepted),
                                  _DTYPES[states.dtype], _p(seq_status), _stream(stream))


def treewy_verify(S0, q, k, v, beta, tree: Tree, H_qk: int, O: torch.Tensor, U: torch.Tensor,
                  seq_status: torch.Tensor | None = None, stream=None, generic: bool = False) -> None:
    """O and U are written in place; io dtype comes from S0, the output dtype from O."""
    lib = load_library()
    ts = tree.struct()
    fn = lib.treewy_verify_generic if generic else lib.treewy_verify
    assert q.dtype == S0.dtype and k.dtype == S0.dtype and v.dtype == S0.dtype
    _call("treewy_verify_generic" if generic else "treewy_verify", fn, _p(S0), _p(q), _p(k), _p(v), _p(beta), ctypes.byref(ts), int(H_qk),
              _DTYPES[S0.dtype], _DTYPES[O.dtype], _p(O), _p(U), _p(seq_status), _stream(stream))


def treewy_commit(S0, U, k, tree: Tree, H_qk: int, accepted, S_out_f32: torch.Tensor | None = None,
                  seq_status: torch.Tensor | None = None, stream=None) -> None:
    """S0 is updated in place; S_out_f32, when given, also receives the unrounded state."""
    lib = load_library()
    ts = tree.struct()
    _call("treewy_commit", lib.treewy_commit, _p(S0), _p(U), _p(k), ctypes.byref(ts), int(H_qk), _p(accepted),
                             _DTYPES[S0.dtype], _p(S_out_f32), _p(seq_status), _stream(stream))


def treewy_verify_half_u(S0, q, k, v, beta, tree: Tree, H_qk: int, O: torch.Tensor, U16: torch.Tensor,
                         seq_status: torch.Tensor | None = None, stream=None) -> None:
    """treewy_verify with the pseudo-values written as fp16."""
    lib = load_library()
    ts = tree.struct()
    assert U16.dtype == torch.float16 and q.dtype == S0.dtype and k.dtype == S0.dtype and v.dtype == S0.dtype
    _call("treewy_verify_half_u", lib.treewy_verify_half_u, _p(S0), _p(q), _p(k), _p(v), _p(beta), ctypes.byref(ts), int(H_qk),
                                    _DTYPES[S0.dtype], _DTYPES[O.dtype], _p(O), _p(U16), _p(seq_status),
                                    _stream(stream))


def treewy_commit_half_u(S0, U16, k, tree: Tree, H_qk: int, accepted, S_out_f32: torch.Tensor | None = None,
                         seq_status: torch.Tensor | None = None, stream=None) -> None:
    """treewy_commit reading fp16 pseudo-values."""
    lib = load_library()
    ts = tree.struct()
    assert U16.dtype == torch.float16
    _call("treewy_commit_half_u", lib.treewy_commit_half_u, _p(S0), _p(U16), _p(k), ctypes.byref(ts), int(H_qk), _p(accepted),
                                    _DTYPES[S0.dtype], _p(S_out_f32), _p(seq_status), _stream(stream))


def treewy_tree_prepare_wide(tree: Tree, alpha: torch.Tensor, seq_status: torch.Tensor | None = None, stream=None) -> None:
    """treewy_tree_prepare for trees of up to 128 nodes (no ancestor masks are written)."""
    ts = tree.struct()
    _call("treewy_tree_prepare_wide", load_library().treewy_tree_prepare_wide, ctypes.byref(ts), _p(alpha), _p(seq_status), _stream(stream))


def treewy_verify_wide(S0, q, k, v, beta, tree: Tree, H_qk: int, O: torch.Tensor, U: torch.Tensor,
                       seq_status: torch.Tensor | None = None, stream=None) -> None:
    ts = tree.struct()
    assert q.dtype == S0.dtype and k.dtype == S0.dtype and v.dtype == S0.dtype
    _call("treewy_verify_wide", load_library().treewy_verify_wide, _p(S0), _p(q), _p(k), _p(v), _p(beta), ctypes.byref(ts), int(H_qk),
                                             _DTYPES[S0.dtype], _DTYPES[O.dtype], _p(O), _p(U), _p(seq_status),
                                             _stream(stream))


def treewy_commit_wide(S0, U, k, tree: Tree, H_qk: int, accepted, S_out_f32: torch.Tensor | None = None,
                       seq_status: torch.Tensor | None = None, stream=None) -> None:
    ts = tree.struct()
    _call("treewy_commit_wide", load_library().treewy_commit_wide, _p(S0), _p(U), _p(k), ctypes.byref(ts), int(H_qk), _p(accepted),
                                             _DTYPES[S0.dtype], _p(S_out_f32), _p(seq_status), _stream(stream))


def treewy_commit_verify(S0, U_prev, k_prev, tree_prev: Tree, accepted_prev, q, k, v, beta, tree: Tree,
                         H_qk: int, O: torch.Tensor, U: torch.Tensor, single_kernel: bool = False,
                         seq_status: torch.Tensor | None = None, stream=None) -> None:
    """Commit the previous round's accepted nodes into S0 and verify the new trees: the two stand-alone
    kernels, or (single_kernel) the fused kernel that reads and writes the state once."""
    lib = load_library()
    tp, ts = tree_prev.struct(), tree.struct()
    _call("treewy_commit_verify", lib.treewy_commit_verify, _p(S0), _p(U_prev), _p(k_prev), ctypes.byref(tp), _p(accepted_prev), _p(q),
                                    _p(k), _p(v), _p(beta), ctypes.byref(ts), int(H_qk), _DTYPES[S0.dtype],
                                    _DTYPES[O.dtype], _p(O), _p(U), int(bool(single_kernel)), _p(seq_status),
                                    _stream(stream))


def treewy_commit_verify_pool(states, state_index, U_prev, k_prev, tree_prev: Tree, accepted_prev, q, k, v, beta,
                              tree: Tree, H_qk: int, O: torch.Tensor, U: torch.Tensor, single_kernel: bool = False,
                              seq_status: torch.Tensor | None = None, stream=None) -> None:
    """treewy_commit_verify with sequence b's state at states[state_index[b]]."""
    lib = load_library()
    tp, ts, ps = tree_prev.struct(), tree.struct(), _pool(states, state_index)
    _call("treewy_commit_verify_pool", lib.treewy_commit_verify_pool, ctypes.byref(ps), _p(U_prev), _p(k_prev), ctypes.byref(tp), _p(accepted_prev),
                                         _p(q), _p(k), _p(v), _p(beta), ctypes.byref(ts), int(H_qk),
                                         _DTYPES[states.dtype], _DTYPES[O.dtype], _p(O), _p(U),
                                         int(bool(single_kernel)), _p(seq_status), _stream(stream))


def treewy_snapshot_all(S0, U, k, tree: Tree, H_qk: int, Snap: torch.Tensor,
                        seq_status: torch.Tensor | None = None, stream=None) -> None:
    """Every node's state into Snap [T, H_v, 128, 128] (the snapshotting comparator); S0 is read only."""
    lib = load_library()
    ts = tree.struct()
    _call("treewy_snapshot_all", lib.treewy_snapshot_all, _p(S0), _p(U), _p(k), ctypes.byref(ts), int(H_qk), _DTYPES[S0.dtype],
                                   _p(Snap), _p(seq_status), _stream(stream))


# --------------------------------------------------------------------------- user-level step

class _StepBuffers:
    """Device-side inputs and outputs of one in-flight step."""

    def __init__(self, B, H_v, H_qk, max_T, io, o_dtype, dev):
        z = lambda shape, dt: torch.empty(shape, dtype=dt, device=dev)
        self.q, self.k = z((max_T, H_qk, D), io), z((max_T, H_qk, D), io)
        self.v = z((max_T, H_v, D), io)
        self.alpha, self.beta = z((max_T, H_v), torch.float32), z((max_T, H_v), torch.float32)
        self.node_offsets = z((B + 1,), torch.int32)
        self.parent = z((max_T,), torch.int32)
        self.accepted = z((B,), torch.int32)
        self.O = z((max_T, H_v, D), o_dtype)
        self.U = z((max_T, H_v, D), torch.float32)
        self.depth = z((max_T,), torch.int32)
        self.anc_mask = z((max_T,), torch.int64)
        self.cum_log_gate = z((max_T, H_v), torch.float32)
        self.level_order = z((max_T,), torch.uint8)
        self.uploaded = torch.cuda.Event()
        self.verified = torch.cuda.Event()
        self.computed = torch.cuda.Event()
        self.downloaded = torch.cuda.Event()


class VerifyCommitLayer:
    """One GDN layer's speculative state on a device: the committed state lives in HBM across
    steps; each step uploads the draft window's inputs, verifies, returns the outputs to the
    host, and commits the accepted node.  This is the call a serving loop makes.

    ``step`` runs everything on the current stream.  ``step_async`` pipelines consecutive steps
    over three streams (upload / compute / download) with double-buffered inputs and outputs:
    the upload of step i+1 and the download of step i overlap the kernels, which stay in order
    because every step reads and writes the same committed state."""

    def __init__(self, S0: torch.Tensor, H_qk: int, max_T: int, max_nodes: int = 0,
                 o_dtype: torch.dtype | None = None):
        dev = S0.device
        self.S0 = S0
        self.B, self.H_v = int(S0.shape[0]), int(S0.shape[1])
        self.H_qk, self.max_nodes = H_qk, max_nodes
        o_dtype = o_dtype or S0.dtype
        self.bufs = [_StepBuffers(self.B, self.H_v, H_qk, max_T, S0.dtype, o_dtype, dev)
                     for _ in range(2)]
        self.status = torch.zeros((self.B,), dtype=torch.int32, device=dev)
        self.s_up, self.s_run, self.s_down = (torch.cuda.Stream(dev) for _ in range(3))
        self._n = 0

    @property
    def O(self) -> torch.Tensor:
        return self.bufs[0].O

    def _tree(self, b: _StepBuffers, T: int) -> Tree:
        return Tree(self.B, T, self.H_v, self.max_nodes, b.node_offsets, b.parent, b.depth,
                    b.anc_mask, b.cum_log_gate, b.level_order)

    @staticmethod
    def _upload(b: _StepBuffers, host: dict) -> int:
        T = int(host["parent"].numel())
        for name in ("q", "k", "v", "alpha", "beta", "parent"):
            getattr(b, name)[:T].copy_(host[name], non_blocking=True)
        b.node_offsets.copy_(host["node_offsets"], non_blocking=True)
        b.accepted.copy_(host["accepted"], non_blocking=True)
        return T

    def _run(self, b: _StepBuffers, T: int, stream=None) -> None:
        tree = self._tree(b, T)
        wide = self.max_nodes > 64                      # trees of more than 64 nodes: the wide-tree calls
        (treewy_tree_prepare_wide if wide else treewy_tree_prepare)(tree, b.alpha, self.status, stream)
        (treewy_verify_wide if wide else treewy_verify)(self.S0, b.q, b.k, b.v, b.beta, tree, self.H_qk, b.O, b.U,
                                                        self.status, stream)
        b.verified.record(stream)
        (treewy_commit_wide if wide else treewy_commit)(self.S0, b.U, b.k, tree, self.H_qk, b.accepted, None,
                                                        self.status, stream)

    def step(self, host: dict, O_host: torch.Tensor) -> None:
        """upload -> prepare -> verify -> outputs to host -> commit, all on the current stream."""
        b = self.bufs[0]
        T = self._upload(b, host)
        self._run(b, T, torch.cuda.current_stream())
        O_host[:T].copy_(b.O[:T], non_blocking=True)

    def step_async(self, host: dict, O_host: torch.Tensor) -> None:
        """Enqueue one step; returns at once.  ``host`` and ``O_host`` must be pinned and must not
        be reused before the second-next ``step_async`` (or ``synchronize``)."""
        b = self.bufs[self._n & 1]
        self._n += 1
        with torch.cuda.stream(self.s_up):
            self.s_up.wait_event(b.computed)     # the kernels that last read this buffer set
            T = self._upload(b, host)
            b.uploaded.record(self.s_up)
        with torch.cuda.stream(self.s_run):
            self.s_run.wait_event(b.uploaded)
            self.s_run.wait_event(b.downloaded)  # O of this buffer set has left for the host
            self._run(b, T, self.s_run)
            b.computed.record(self.s_run)
        with torch.cuda.stream(self.s_down):
            self.s_down.wait_event(b.verified)
            O_host[:T].copy_(b.O[:T], non_blocking=True)
            b.downloaded.record(self.s_down)

    def synchronize(self) -> None:
        for s in (self.s_up, self.s_run, self.s_down):
            s.synchronize()
