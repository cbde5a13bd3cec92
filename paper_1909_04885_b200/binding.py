"""ctypes binding over ``libchicle.so`` (the C ABI in ``include/chicle.h``), same names, argument marshalling only.

Every step of a round runs in the library's CUDA kernels. PyTorch is used for device memory (the library's
allocations are routed through torch's caching allocator) and for the stream. There is no host fallback: if the
shared library is missing, loading fails with an error.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("CHICLE_LIB_PATH") or os.path.join(_HERE, "libchicle.so")

OK, ERR_INVALID_ARG, ERR_BAD_STATE, ERR_OOM, ERR_CUDA, ERR_UNSUPPORTED, ERR_NUMERIC, ERR_TIMEOUT, ERR_INTERNAL = range(9)
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "BAD_STATE", 3: "OOM", 4: "CUDA", 5: "UNSUPPORTED", 6: "NUMERIC", 7: "TIMEOUT",
                8: "INTERNAL"}
LOSS = {"hinge": 0, "logistic": 1, "ridge": 2}
FMT = {"dense": 0, "csr": 1, "csc": 2}
MEM_HOST, MEM_DEVICE = 0, 1

EXPORTED = ["chicle_glm_create", "chicle_partition", "chicle_cocoa_round", "chicle_duality_gap", "chicle_get_alpha",
            "chicle_get_v", "chicle_get_partition", "chicle_get_permutation", "chicle_set_state", "chicle_get_info",
            "chicle_last_error", "chicle_glm_destroy", "chicle_partition_noalloc", "chicle_partition_sizes",
            "chicle_cocoa_round_steps", "chicle_chunks_cut", "chicle_chunks_assign", "chicle_chunks_scale_in",
            "chicle_chunks_scale_out", "chicle_chunks_rebalance_step", "chicle_partition_chunks", "chicle_cocoa_round_delta",
            "chicle_apply_deltas", "chicle_export_state_of", "chicle_import_state"]


class ChicleError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("chicle: %s: %s" % (STATUS_NAMES.get(status, status), message))
        self.status = status


class Matrix(C.Structure):
    _fields_ = [("fmt", C.c_int), ("space", C.c_int), ("n_rows", C.c_int64), ("n_cols", C.c_int64), ("nnz", C.c_int64),
                ("ld", C.c_int64), ("indptr", C.c_void_p), ("indices", C.c_void_p), ("values", C.c_void_p)]


ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_void_p, C.c_size_t)
FREE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)


class Allocator(C.Structure):
    _fields_ = [("alloc", ALLOC_FN), ("free", FREE_FN), ("ctx", C.c_void_p)]


class RoundStats(C.Structure):
    _fields_ = [("ms_permutation", C.c_float), ("ms_local", C.c_float), ("ms_reduce", C.c_float), ("ms_total", C.c_float),
                ("steps", C.c_int64), ("solver_variant", C.c_int32), ("ms_prepare", C.c_float),
                ("solver_slices", C.c_int32), ("cluster_ctas", C.c_int32), ("solver_launches", C.c_int32),
                ("order_launches", C.c_int32)]


_lib = None


def load():
    """Loads the shared library; raises if it has not been built (``python -m paper_1909_04885_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libchicle.so is missing (%s): build it with `python -m paper_1909_04885_b200.build`; "
                           "there is no CPU path" % LIB_PATH)
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, u64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_float
    lib.chicle_glm_create.restype = C.c_int
    lib.chicle_glm_create.argtypes = [C.POINTER(Matrix), vp, f32, C.c_int, C.c_int, vp, C.POINTER(Allocator), C.POINTER(vp)]
    lib.chicle_partition.restype = C.c_int
    lib.chicle_partition.argtypes = [vp, i32, u64]
    lib.chicle_partition_sizes.restype = C.c_int
    lib.chicle_partition_sizes.argtypes = [vp, i32, u64, vp]
    lib.chicle_cocoa_round.restype = C.c_int
    lib.chicle_cocoa_round.argtypes = [vp, i64, f32, C.POINTER(RoundStats)]
    lib.chicle_cocoa_round_steps.restype = C.c_int
    lib.chicle_cocoa_round_steps.argtypes = [vp, vp, f32, C.POINTER(RoundStats)]
    lib.chicle_cocoa_round_delta.restype = C.c_int
    lib.chicle_cocoa_round_delta.argtypes = [vp, vp, f32, vp, i64, C.POINTER(RoundStats)]
    lib.chicle_apply_deltas.restype = C.c_int
    lib.chicle_apply_deltas.argtypes = [vp, vp, i32, i64]
    lib.chicle_export_state_of.restype = C.c_int
    lib.chicle_export_state_of.argtypes = [vp, vp, vp, i64]
    lib.chicle_import_state.restype = C.c_int
    lib.chicle_import_state.argtypes = [vp, vp, i64]
    lib.chicle_chunks_cut.restype = i64
    lib.chicle_chunks_cut.argtypes = [i64, vp, i64, i64, vp]
    lib.chicle_chunks_assign.restype = C.c_int
    lib.chicle_chunks_assign.argtypes = [i64, i32, C.c_uint64, vp]
    lib.chicle_chunks_scale_in.restype = C.c_int
    lib.chicle_chunks_scale_in.argtypes = [i64, i32, i32, vp]
    lib.chicle_chunks_scale_out.restype = C.c_int
    lib.chicle_chunks_scale_out.argtypes = [i64, i32, i32, C.c_uint64, vp]
    lib.chicle_chunks_rebalance_step.restype = C.c_int
    lib.chicle_chunks_rebalance_step.argtypes = [i64, vp, i32, vp, vp]
    lib.chicle_partition_chunks.restype = C.c_int
    lib.chicle_partition_chunks.argtypes = [vp, i32, C.c_uint64, i64, vp, vp]
    lib.chicle_duality_gap.restype = C.c_int
    lib.chicle_duality_gap.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_double)]
    for name in ("chicle_get_alpha", "chicle_get_v"):
        fn = getattr(lib, name)
        fn.restype = C.c_int
        fn.argtypes = [vp, vp, i64, C.c_int]
    lib.chicle_get_partition.restype = C.c_int
    lib.chicle_get_partition.argtypes = [vp, vp, i64]
    lib.chicle_get_permutation.restype = C.c_int
    lib.chicle_get_permutation.argtypes = [vp, i64, i32, vp, i64]
    lib.chicle_set_state.restype = C.c_int
    lib.chicle_set_state.argtypes = [vp, vp, vp, i64]
    lib.chicle_get_info.restype = C.c_int
    lib.chicle_get_info.argtypes = [vp, C.POINTER(i64), C.POINTER(i32), C.POINTER(i64), C.POINTER(i64)]
    lib.chicle_last_error.restype = C.c_char_p
    lib.chicle_last_error.argtypes = [vp]
    lib.chicle_glm_destroy.restype = None
    lib.chicle_glm_destroy.argtypes = [vp]
    lib.chicle_partition_noalloc.restype = C.c_int
    lib.chicle_partition_noalloc.argtypes = [C.c_int, vp, i64, i32, u64, vp, vp, C.c_char_p, C.c_size_t]
    _lib = lib
    return lib


def _stats_dict(rs) -> dict:
    return {"ms_permutation": rs.ms_permutation, "ms_local": rs.ms_local, "ms_reduce": rs.ms_reduce,
            "ms_total": rs.ms_total, "steps": rs.steps, "solver_variant": rs.solver_variant,
            "ms_prepare": rs.ms_prepare, "solver_slices": rs.solver_slices, "cluster_ctas": rs.cluster_ctas,
            "solver_launches": rs.solver_launches, "order_launches": rs.order_launches}


def _is_torch(x) -> bool:
    return x is not None and type(x).__module__.startswith("torch")


def _ptr(x):
    if x is None:
        return None
    if _is_torch(x):
        return C.c_void_p(x.data_ptr())
    return x.ctypes.data_as(C.c_void_p)


class _TorchAllocator:
    """Routes the library's device allocations through torch's caching allocator."""

    def __init__(self, device: int):
        import torch
        self._torch = torch
        self._device = torch.device("cuda", device)
        self._live = {}
        self.fail = False   # True: every request is refused (the callback returns NULL), to exercise the library's OOM paths
        self._alloc_cb = ALLOC_FN(self._alloc)
        self._free_cb = FREE_FN(self._free)
        self.struct = Allocator(self._alloc_cb, self._free_cb, None)

    def _alloc(self, _ctx, nbytes):
        if self.fail:
            return None
        try:
            t = self._torch.empty(int(nbytes), dtype=self._torch.uint8, device=self._device)
        except Exception:
            return None
        self._live[t.data_ptr()] = t
        return t.data_ptr()

    def _free(self, _ctx, ptr):
        self._live.pop(ptr, None)

    @property
    def bytes_live(self) -> int:
        return sum(t.numel() for t in self._live.values())


class Glm:
    """One training problem on one GPU. ``values``/``indptr``/``indices``/``labels`` are numpy arrays (host) or
    torch CUDA tensors (device), all in the same place. fp32 values and labels, int64 indptr, int32 indices."""

    def __init__(self, loss: str, fmt: str, n_rows: int, n_cols: int, values, labels, lam: float, indptr=None,
                 indices=None, device: int = 0, stream: Optional[int] = None, torch_allocator: bool = True,
                 ld: Optional[int] = None):
        self._lib = load()
        self._h = C.c_void_p(None)
        on_dev = _is_torch(values)
        if on_dev:
            import torch
            assert values.is_cuda and values.dtype == torch.float32 and values.is_contiguous()
            assert labels.is_cuda and labels.dtype == torch.float32
            if indptr is not None:
                assert indptr.dtype == torch.int64 and indices.dtype == torch.int32
            nvals = values.numel()
        else:
            values = np.ascontiguousarray(values, np.float32).reshape(-1)
            labels = np.ascontiguousarray(labels, np.float32)
            indptr = None if indptr is None else np.ascontiguousarray(indptr, np.int64)
            indices = None if indices is None else np.ascontiguousarray(indices, np.int32)
            nvals = values.size
        self._keep = (values, labels, indptr, indices)
        m = Matrix(FMT[fmt], MEM_DEVICE if on_dev else MEM_HOST, n_rows, n_cols, 0 if fmt == "dense" else nvals,
                   (ld or n_cols) if fmt == "dense" else 0, _ptr(indptr), _ptr(indices), _ptr(values))
        self._alloc = None
        alloc_ref = None
        if torch_allocator:
            self._alloc = _TorchAllocator(device)
            alloc_ref = C.byref(self._alloc.struct)
        if stream is None:
            import torch
            with torch.cuda.device(device):
                stream = torch.cuda.current_stream().cuda_stream
        self.stream = stream
        self.device = device
        self.loss, self.fmt = loss, fmt
        st = self._lib.chicle_glm_create(C.byref(m), _ptr(labels), C.c_float(lam), LOSS[loss], device,
                                         C.c_void_p(stream), alloc_ref, C.byref(self._h))
        if st != OK:
            raise ChicleError(st, self._lib.chicle_last_error(None).decode())
        self._keep = None
        self.n_coord = n_cols if loss == "ridge" else n_rows
        self.dim = n_rows if loss == "ridge" else n_cols
        self.K = 0

    # -- helpers
    def _check(self, st: int):
        if st != OK:
            raise ChicleError(st, self._lib.chicle_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.chicle_glm_destroy(self._h)
            self._h = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # -- the ABI, one method per entry point
    def partition(self, K: int, seed: int, sizes=None):
        """``chicle_partition``, or ``chicle_partition_sizes`` when ``sizes`` (K positive integers summing to the number
        of coordinates) is given."""
        if sizes is None:
            self._check(self._lib.chicle_partition(self._h, K, C.c_uint64(seed & (2**64 - 1))))
        else:
            sz = np.ascontiguousarray(sizes, np.int64)
            if sz.size != K:
                raise ValueError("sizes must have K entries")
            self._check(self._lib.chicle_partition_sizes(self._h, K, C.c_uint64(seed & (2**64 - 1)), _ptr(sz)))
        self.K = K

    def partition_chunks(self, K: int, seed: int, chunk_off, chunk_task):
        """``chicle_partition_chunks``: the partition that a placement of data chunks on K tasks induces."""
        off = np.ascontiguousarray(chunk_off, np.int64)
        task = np.ascontiguousarray(chunk_task, np.int32)
        if off.size != task.size + 1:
            raise ValueError("chunk_off must have one entry more than chunk_task")
        self._check(self._lib.chicle_partition_chunks(self._h, K, C.c_uint64(seed & (2**64 - 1)), task.size, _ptr(off), _ptr(task)))
        self.K = K

    def cocoa_round(self, H: int = 0, sigma_prime: Optional[float] = None, stats: bool = False, steps=None):
        """One round; ``steps`` (K integers, 0 <= steps[k] <= size of partition k) gives each partition its own budget."""
        sp = float(self.K if sigma_prime is None else sigma_prime)
        rs = RoundStats() if stats else None
        ref = C.byref(rs) if stats else None
        if steps is not None:
            st = np.ascontiguousarray(steps, np.int64)
            if st.size != self.K:
                raise ValueError("steps must have K entries")
            self._check(self._lib.chicle_cocoa_round_steps(self._h, st.ctypes.data, C.c_float(sp), ref))
        else:
            self._check(self._lib.chicle_cocoa_round(self._h, H, C.c_float(sp), ref))
        return _stats_dict(rs) if stats else None

    def cocoa_round_delta(self, steps, sigma_prime: float, delta_out, stats: bool = False):
        """``chicle_cocoa_round_delta``: the round with budgets ``steps``; the summed update goes to ``delta_out`` (a
        CUDA tensor of ``dim`` floats on this handle's device) and v is left alone."""
        st = np.ascontiguousarray(steps, np.int64)
        if st.size != self.K:
            raise ValueError("steps must have K entries")
        rs = RoundStats() if stats else None
        self._check(self._lib.chicle_cocoa_round_delta(self._h, st.ctypes.data, C.c_float(float(sigma_prime)), _ptr(delta_out),
                                                       delta_out.numel(), C.byref(rs) if stats else None))
        return _stats_dict(rs) if stats else None

    def apply_deltas(self, deltas):
        """``chicle_apply_deltas``: ``deltas`` is a contiguous CUDA tensor of shape (count, dim)."""
        count = deltas.numel() // self.dim
        self._check(self._lib.chicle_apply_deltas(self._h, _ptr(deltas), count, self.dim))

    def export_state_of(self, keep, out):
        """``chicle_export_state_of``: ``keep`` holds K flags, ``out`` is a CUDA tensor of one float per coordinate."""
        kp = np.ascontiguousarray(keep, np.uint8)
        if kp.size != self.K:
            raise ValueError("keep must have K entries")
        self._check(self._lib.chicle_export_state_of(self._h, kp.ctypes.data, _ptr(out), out.numel()))

    def import_state(self, state):
        """``chicle_import_state``: ``state`` is a CUDA tensor of one float per coordinate."""
        self._check(self._lib.chicle_import_state(self._h, _ptr(state), state.numel()))

    def fail_allocations(self, on: bool):
        """Makes the allocator callback that the library was given refuse every request (return NULL) from now on, or
        serve them again: a way to see the library's out-of-memory behaviour without exhausting the device."""
        if self._alloc is None:
            raise RuntimeError("this handle allocates with cudaMalloc, not through a callback")
        self._alloc.fail = bool(on)

    def duality_gap(self):
        g, p, d = C.c_double(), C.c_double(), C.c_double()
        self._check(self._lib.chicle_duality_gap(self._h, C.byref(g), C.byref(p), C.byref(d)))
        return {"gap": g.value, "primal": p.value, "dual": d.value}

    def get_alpha(self, out=None) -> np.ndarray:
        return self._get(self._lib.chicle_get_alpha, self.n_coord, out)

    def get_v(self, out=None) -> np.ndarray:
        return self._get(self._lib.chicle_get_v, self.dim, out)

    def _get(self, fn, n, out):
        if out is None:
            out = np.empty(n, np.float32)
        space = MEM_DEVICE if _is_torch(out) else MEM_HOST
        self._check(fn(self._h, _ptr(out), n, space))
        return out

    def get_partition(self) -> np.ndarray:
        out = np.empty(self.n_coord, np.int32)
        self._check(self._lib.chicle_get_partition(self._h, _ptr(out), out.size))
        return out

    def get_permutation(self, rnd: int, k: int, n_k: int) -> np.ndarray:
        out = np.empty(n_k, np.int32)
        self._check(self._lib.chicle_get_permutation(self._h, rnd, k, _ptr(out), n_k))
        return out

    def set_state(self, alpha: np.ndarray, v: Optional[np.ndarray], rnd: int):
        alpha = np.ascontiguousarray(alpha, np.float32)
        v = None if v is None else np.ascontiguousarray(v, np.float32)
        assert alpha.size == self.n_coord and (v is None or v.size == self.dim)
        self._check(self._lib.chicle_set_state(self._h, _ptr(alpha), _ptr(v), rnd))

    def info(self):
        r, K, n, d = C.c_int64(), C.c_int32(), C.c_int64(), C.c_int64()
        self._check(self._lib.chicle_get_info(self._h, C.byref(r), C.byref(K), C.byref(n), C.byref(d)))
        return {"round": r.value, "K": K.value, "n_coord": n.value, "dim": d.value}


def from_workload(w, device: int = 0, on_device: bool = False, **kw) -> Glm:
    """Builds a ``Glm`` from a ``datagen.Workload`` (host arrays by default; ``on_device`` uploads them with torch
    first so that creation copies device to device)."""
    vals, labels, indptr, indices = w.values, w.labels, w.indptr, w.indices
    if on_device:
        import torch
        dev = torch.device("cuda", device)
        vals = torch.from_numpy(vals).to(dev)
        labels = torch.from_numpy(labels).to(dev)
        indptr = None if indptr is None else torch.from_numpy(indptr).to(dev)
        indices = None if indices is None else torch.from_numpy(indices).to(dev)
    return Glm(w.loss, w.fmt, w.n_rows, w.n_cols, vals, labels, w.lam, indptr, indices, device=device, **kw)


def partition_noalloc(n_coord: int, K: int, seed: int, owner_out, members_out, device: int = 0, stream: int = 0):
    """``chicle_partition_noalloc``: fills two caller-owned int32 CUDA tensors of ``n_coord`` entries with the partition
    map and the grouped member list, using the library's built-in workspace instead of allocating one. Meant for
    callers that may not touch a device allocator at this point (frozen memory pools, serving loops). Asynchronous on
    ``stream``; raises ``ChicleError`` with the library's message when the size is beyond the built-in limit."""
    lib = load()
    buf = C.create_string_buffer(256)
    st = lib.chicle_partition_noalloc(device, C.c_void_p(stream), n_coord, K, C.c_uint64(seed & (2**64 - 1)),
                                      C.c_void_p(owner_out.data_ptr()), C.c_void_p(members_out.data_ptr()), buf, 256)
    if st != OK:
        raise ChicleError(st, buf.value.decode())


# ---- mobile data chunks: host-side placement logic of the library (argument marshalling only) -------------------
def chunks_cut(n_coord: int, chunk_bytes: int, indptr=None, dense_dim: int = 0) -> np.ndarray:
    """``chicle_chunks_cut``: chunk offsets for chunks of at most ``chunk_bytes``."""
    off = np.empty(n_coord + 1, np.int64)
    ip = None if indptr is None else np.ascontiguousarray(indptr, np.int64)
    c = load().chicle_chunks_cut(n_coord, None if ip is None else _ptr(ip), dense_dim, chunk_bytes, _ptr(off))
    if c < 0:
        raise ValueError("chicle_chunks_cut: bad arguments")
    return off[:c + 1].copy()


def chunks_assign(n_chunks: int, K: int, seed: int) -> np.ndarray:
    task = np.empty(n_chunks, np.int32)
    st = load().chicle_chunks_assign(n_chunks, K, C.c_uint64(seed & (2**64 - 1)), _ptr(task))
    if st != OK:
        raise ChicleError(st, "chicle_chunks_assign: need 1 <= K <= number of chunks")
    return task


def chunks_scale_in(task, K_old: int, K_new: int) -> np.ndarray:
    out = np.array(task, np.int32, copy=True)
    st = load().chicle_chunks_scale_in(out.size, K_old, K_new, _ptr(out))
    if st != OK:
        raise ChicleError(st, "chicle_chunks_scale_in: need 1 <= K_new <= K_old")
    return out


def chunks_scale_out(task, K_old: int, K_new: int, seed: int) -> np.ndarray:
    out = np.array(task, np.int32, copy=True)
    st = load().chicle_chunks_scale_out(out.size, K_old, K_new, C.c_uint64(seed & (2**64 - 1)), _ptr(out))
    if st != OK:
        raise ChicleError(st, "chicle_chunks_scale_out: need 1 <= K_old <= K_new and tasks in [0, K_old)")
    return out


def chunks_rebalance_step(task, chunk_off, K: int, time_per_sample):
    """Returns (new placement, whether a chunk moved)."""
    out = np.array(task, np.int32, copy=True)
    off = np.ascontiguousarray(chunk_off, np.int64)
    t = np.ascontiguousarray(time_per_sample, np.float64)
    if off.size != out.size + 1 or t.size != K:
        raise ValueError("chunk_off needs one entry more than task, time_per_sample K entries")
    r = load().chicle_chunks_rebalance_step(out.size, _ptr(off), K, _ptr(t), _ptr(out))
    if r < 0:
        raise ValueError("chicle_chunks_rebalance_step: bad arguments")
    return out, bool(r)
