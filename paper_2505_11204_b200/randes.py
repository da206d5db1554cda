"""Thin binding over the CUDA C-ABI library (``include/randes.h``).

Argument marshalling only: every step of the path runs in the library's
kernels.  PyTorch supplies device memory and the stream.  There is no CPU
fallback: if the compiled library is missing, loading raises.

Two levels:

* module functions ``randes_plan``, ``randes_compress``, ``randes_add_model``,
  ``randes_remove_model``, ``randes_retrieve`` ... with the C names, taking
  ctypes pointer arrays / raw addresses;
* ``Plan``: the same calls on lists of torch CUDA tensors.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

F32 = 0
BF16 = 1
SHUFFLE = 1
FLIP = 2
SHIFT = 4
GAUSS = 1 << 16   # RANDES_GAUSS: Gaussian-like diagonal context (the paper's "RD" ablation) instead of the +-1 one


def SKIP(k: int) -> int:
    """Group flag bits of RANDES_SKIP(k): only every k-th member of the group takes part."""
    return (int(k) & 0xFF) << 8

OK = 0
INVALID_ARGUMENT = -1
SHAPE_MISMATCH = -2
UNKNOWN_TASK = -3
DUPLICATE_TASK = -4
WORKSPACE_TOO_SMALL = -5
UNSUPPORTED_DTYPE = -6
MISALIGNED = -7
CAPACITY = -8
CUDA_ERROR = -9
OUT_OF_MEMORY = -10

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librandes.so")
_lib = None


class RandesError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__("randes error %d: %s" % (code, message))
        self.code = code


class Layer(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_uint32), ("cols", ctypes.c_uint32), ("group", ctypes.c_uint32)]


class Group(ctypes.Structure):
    _fields_ = [("flags", ctypes.c_uint32)]


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "%s is missing: build it with `python -m paper_2505_11204_b200.build` "
                "(there is no CPU fallback)" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, u32, u64, sz = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_size_t
        L.randes_plan_workspace_bytes.argtypes = [vp, u32, u32]
        L.randes_plan_workspace_bytes.restype = sz
        L.randes_plan_workspace_bytes_groups.argtypes = [vp, u32, vp, u32, u32]
        L.randes_plan_workspace_bytes_groups.restype = sz
        L.randes_plan.argtypes = [vp, u32, vp, u32, ctypes.c_int, ctypes.c_int, vp, vp, u32, u32, vp, sz, vp,
                                  ctypes.POINTER(vp)]
        L.randes_plan.restype = ctypes.c_int
        L.randes_plan_destroy.argtypes = [vp]
        L.randes_plan_destroy.restype = None
        L.randes_plan_validate.argtypes = [vp]
        L.randes_plan_validate.restype = ctypes.c_int
        L.randes_debug_violation.argtypes = [ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_int)]
        L.randes_debug_violation.restype = ctypes.c_int
        L.randes_superposition_bytes.argtypes = [vp]
        L.randes_superposition_bytes.restype = sz
        L.randes_layer_offset.argtypes = [vp, u32]
        L.randes_layer_offset.restype = sz
        L.randes_num_layers.argtypes = [vp]
        L.randes_num_layers.restype = u32
        L.randes_num_tasks.argtypes = [vp]
        L.randes_num_tasks.restype = u32
        L.randes_task_list.argtypes = [vp, vp, vp]
        L.randes_task_list.restype = ctypes.c_int
        L.randes_task_tables.argtypes = [vp, u32, vp, vp]
        L.randes_task_tables.restype = ctypes.c_int
        L.randes_compress.argtypes = [vp, vp, vp, vp, vp]
        L.randes_compress.restype = ctypes.c_int
        L.randes_add_model.argtypes = [vp, u32, u64, vp, vp, vp, vp]
        L.randes_add_model.restype = ctypes.c_int
        L.randes_add_models.argtypes = [vp, vp, vp, u32, vp, vp, vp, vp]
        L.randes_add_models.restype = ctypes.c_int
        L.randes_remove_model.argtypes = [vp, u32, vp, vp, vp, vp]
        L.randes_remove_model.restype = ctypes.c_int
        L.randes_retrieve.argtypes = [vp, u32, ctypes.c_float, ctypes.c_int, vp, vp, vp, vp]
        L.randes_retrieve.restype = ctypes.c_int
        L.randes_plan_serialize.argtypes = [vp, vp, sz]
        L.randes_plan_serialize.restype = sz
        L.randes_plan_deserialize.argtypes = [vp, sz, u32, vp, sz, vp, ctypes.POINTER(vp)]
        L.randes_plan_deserialize.restype = ctypes.c_int
        L.randes_plan_workspace_needed.argtypes = [vp]
        L.randes_plan_workspace_needed.restype = sz
        L.randes_delta_gram_scratch_bytes.argtypes = [vp]
        L.randes_delta_gram_scratch_bytes.restype = sz
        L.randes_delta_gram.argtypes = [vp, vp, vp, vp, vp, sz, vp]
        L.randes_delta_gram.restype = ctypes.c_int
        L.randes_interference_norm.argtypes = [vp, u32, u32, ctypes.c_double, ctypes.POINTER(ctypes.c_double)]
        L.randes_interference_norm.restype = ctypes.c_int
        L.randes_pairwise_cosines.argtypes = [vp, u32, ctypes.c_int32, vp, ctypes.POINTER(ctypes.c_double)]
        L.randes_pairwise_cosines.restype = ctypes.c_int
        L.randes_retrieve_batch.argtypes = [vp, vp, u32, ctypes.c_float, ctypes.c_int, vp, vp, vp, vp]
        L.randes_retrieve_batch.restype = ctypes.c_int
        L.randes_retrieve_static.argtypes = [vp, u32, ctypes.c_float, ctypes.c_int, vp, vp, vp, vp]
        L.randes_retrieve_static.restype = ctypes.c_int
        L.randes_linear.argtypes = [vp, u32, ctypes.c_float, u32, vp, u32, vp, vp, vp, ctypes.c_int, vp]
        L.randes_linear.restype = ctypes.c_int
        L.randes_linear_gated.argtypes = [vp, u32, ctypes.c_float, u32, vp, u32, vp, vp, vp, ctypes.c_int, vp, u64, vp]
        L.randes_linear_gated.restype = ctypes.c_int
        L.randes_linear_giveups.argtypes = [ctypes.POINTER(ctypes.c_uint)]
        L.randes_linear_giveups.restype = ctypes.c_int
        L.randes_launch_count.argtypes = []
        L.randes_launch_count.restype = u64
        L.randes_last_error.argtypes = []
        L.randes_last_error.restype = ctypes.c_char_p
        _lib = L
    return _lib


EXPORTS = [
    "randes_plan_workspace_bytes", "randes_plan_workspace_bytes_groups", "randes_plan", "randes_plan_destroy", "randes_plan_validate", "randes_debug_violation", "randes_superposition_bytes",
    "randes_layer_offset", "randes_num_layers", "randes_num_tasks", "randes_task_list",
    "randes_task_tables", "randes_plan_serialize", "randes_plan_workspace_needed", "randes_plan_deserialize", "randes_compress", "randes_add_model", "randes_add_models", "randes_remove_model",
    "randes_retrieve", "randes_delta_gram_scratch_bytes", "randes_delta_gram", "randes_interference_norm", "randes_pairwise_cosines", "randes_retrieve_batch", "randes_retrieve_static", "randes_linear", "randes_linear_gated", "randes_linear_giveups", "randes_launch_count", "randes_last_error",
]


def randes_last_error() -> str:
    return lib().randes_last_error().decode()


def _check(rc: int) -> None:
    if rc != OK:
        raise RandesError(rc, randes_last_error())


def _addr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, ctypes.Array):
        return ctypes.addressof(x)
    return int(x.data_ptr())  # torch tensor


# ---- C-named entry points (raw addresses / ctypes arrays) ----------------------------------
def randes_plan_workspace_bytes(layers, n_layers: int, max_tasks: int) -> int:
    return int(lib().randes_plan_workspace_bytes(_addr(layers), n_layers, max_tasks))


def randes_plan_workspace_bytes_groups(layers, n_layers: int, groups, n_groups: int, max_tasks: int) -> int:
    """Workspace bytes of a plan with these groups (larger than the plain figure only with a RANDES_GAUSS group)."""
    return int(lib().randes_plan_workspace_bytes_groups(_addr(layers), n_layers, _addr(groups), n_groups, max_tasks))


def randes_plan(layers, n_layers, groups, n_groups, storage_dtype, m_dtype, task_ids, seeds, n_tasks, max_tasks,
                dev_workspace, dev_workspace_bytes, stream) -> int:
    """Returns the plan handle (an address); raises RandesError on failure."""
    out = ctypes.c_void_p()
    _check(lib().randes_plan(_addr(layers), n_layers, _addr(groups), n_groups, storage_dtype, m_dtype,
                             _addr(task_ids), _addr(seeds), n_tasks, max_tasks, _addr(dev_workspace),
                             dev_workspace_bytes, stream, ctypes.byref(out)))
    return out.value


def randes_plan_serialize(plan) -> bytes:
    """The plan's shapes, flags, element types and (id, seed) pairs as a self-contained blob."""
    n = int(lib().randes_plan_serialize(plan, None, 0))
    if n == 0:
        raise RandesError(INVALID_ARGUMENT, randes_last_error())
    buf = ctypes.create_string_buffer(n)
    if int(lib().randes_plan_serialize(plan, ctypes.addressof(buf), n)) != n:
        raise RandesError(INVALID_ARGUMENT, randes_last_error())
    return buf.raw


def randes_plan_workspace_needed(plan) -> int:
    """Workspace bytes a plan equal to this one needs (also answered by a host-only plan)."""
    return int(lib().randes_plan_workspace_needed(plan))


def randes_plan_deserialize(blob: bytes, max_tasks: int = 0, dev_workspace=None, dev_workspace_bytes: int = 0, stream=None) -> int:
    """A plan handle rebuilt from randes_plan_serialize's blob (host-only without a workspace)."""
    out = ctypes.c_void_p()
    buf = ctypes.create_string_buffer(blob, len(blob))
    _check(lib().randes_plan_deserialize(ctypes.addressof(buf), len(blob), max_tasks, _addr(dev_workspace), dev_workspace_bytes,
                                         stream, ctypes.byref(out)))
    return out.value


def randes_plan_destroy(plan) -> None:
    lib().randes_plan_destroy(plan)


def randes_plan_validate(plan) -> None:
    """Host-side self-check of a plan's tables; raises RandesError naming the first violation."""
    _check(lib().randes_plan_validate(plan))


def randes_debug_violation():
    """(word, checked_build): the first bounds violation recorded by a checked build's kernels (0 = none)."""
    word, flag = ctypes.c_uint64(0), ctypes.c_int(0)
    _check(lib().randes_debug_violation(ctypes.byref(word), ctypes.byref(flag)))
    return int(word.value), bool(flag.value)


def randes_superposition_bytes(plan) -> int:
    return int(lib().randes_superposition_bytes(plan))


def randes_layer_offset(plan, layer: int) -> int:
    return int(lib().randes_layer_offset(plan, layer))


def randes_num_layers(plan) -> int:
    return int(lib().randes_num_layers(plan))


def randes_num_tasks(plan) -> int:
    return int(lib().randes_num_tasks(plan))


def randes_compress(plan, base, tasks, M, stream) -> None:
    _check(lib().randes_compress(plan, _addr(base), _addr(tasks), _addr(M), stream))


def randes_add_model(plan, task_id, seed, base, task, M, stream) -> None:
    _check(lib().randes_add_model(plan, task_id, seed, _addr(base), _addr(task), _addr(M), stream))


def randes_add_models(plan, task_ids, seeds, base, tasks, M, stream) -> None:
    """Several models added in one pass over M; ``tasks`` holds n_tasks * n_layers pointers, task-major."""
    n = len(task_ids)
    ids = (ctypes.c_uint32 * max(n, 1))(*[int(t) for t in task_ids])
    sds = (ctypes.c_uint64 * max(n, 1))(*[int(t) for t in seeds])
    _check(lib().randes_add_models(plan, ctypes.addressof(ids), ctypes.addressof(sds), n, _addr(base), _addr(tasks), _addr(M), stream))


def randes_remove_model(plan, task_id, base, task, M, stream) -> None:
    _check(lib().randes_remove_model(plan, task_id, _addr(base), _addr(task), _addr(M), stream))


def randes_retrieve(plan, task_id, lam, out_dtype, base, M, out, stream) -> None:
    _check(lib().randes_retrieve(plan, task_id, lam, out_dtype, _addr(base), _addr(M), _addr(out), stream))


def randes_delta_gram_scratch_bytes(plan) -> int:
    return int(lib().randes_delta_gram_scratch_bytes(plan))


def randes_delta_gram(plan, base, tasks, gram, scratch, scratch_bytes, stream) -> None:
    _check(lib().randes_delta_gram(plan, _addr(base), _addr(tasks), _addr(gram), _addr(scratch), scratch_bytes, stream))


def randes_retrieve_batch(plan, task_ids, lam, out_dtype, base, M, out, stream) -> None:
    """Several tasks in one pass; ``out`` holds n_tasks * n_layers pointers, task-major."""
    ids = (ctypes.c_uint32 * len(task_ids))(*[int(t) for t in task_ids])
    _check(lib().randes_retrieve_batch(plan, ctypes.addressof(ids), len(task_ids), lam, out_dtype, _addr(base), _addr(M),
                                       _addr(out), stream))


def randes_retrieve_static(plan, task_id, lam, out_dtype, base, M, out, stream) -> None:
    """retrieve with the kernel's tables in the library's built-in device array (no workspace)."""
    _check(lib().randes_retrieve_static(plan, task_id, lam, out_dtype, _addr(base), _addr(M), _addr(out), stream))


def randes_linear(plan, task_id, lam, layer, x, n_tokens, base, M, y, stream, y_dtype: int = F32) -> None:
    """y = x What_t[layer]^T on the tensor cores, the retrieved weight never written to memory."""
    _check(lib().randes_linear(plan, task_id, lam, layer, _addr(x), n_tokens, _addr(base), _addr(M), _addr(y), y_dtype, stream))


def randes_linear_gated(plan, task_id, lam, layer, x, n_tokens, base, M, y, gate, wait_ns, stream, y_dtype: int = F32) -> None:
    """randes_linear whose thread blocks first wait (at most wait_ns nanoseconds; 0 = one second) for the device word
    ``gate`` to become non-zero; blocks whose wait runs out write nothing and count in randes_linear_giveups()."""
    _check(lib().randes_linear_gated(plan, task_id, lam, layer, _addr(x), n_tokens, _addr(base), _addr(M), _addr(y), y_dtype,
                                     _addr(gate), int(wait_ns), stream))


def randes_linear_giveups() -> int:
    """Thread blocks of randes_linear that gave up on a bounded wait (0 in a healthy run); synchronises."""
    n = ctypes.c_uint(0)
    _check(lib().randes_linear_giveups(ctypes.byref(n)))
    return int(n.value)


def randes_launch_count() -> int:
    return int(lib().randes_launch_count())


def ptr_array(tensors: Sequence) -> ctypes.Array:
    """Host array of device addresses, one per tensor (nested lists are flattened)."""
    flat = []
    for t in tensors:
        if isinstance(t, (list, tuple)):
            flat.extend(t)
        else:
            flat.append(t)
    arr = (ctypes.c_void_p * max(len(flat), 1))()
    for i, t in enumerate(flat):
        arr[i] = None if t is None else (t if isinstance(t, int) else int(t.data_ptr()))
    return arr


def _as_ptrs(x):
    if x is None or isinstance(x, ctypes.Array):
        return x
    return ptr_array(x)


def _host_gram(gram):
    """An [n, n] Gram matrix (torch tensor, numpy array or nested lists) as a host array of doubles."""
    if hasattr(gram, "detach"):
        gram = gram.detach().cpu().tolist()
    elif hasattr(gram, "tolist"):
        gram = gram.tolist()
    n = len(gram)
    return (ctypes.c_double * max(n * n, 1))(*[float(v) for row in gram for v in row]), n


def randes_interference_norm(gram, t: int, lam: float) -> float:
    """|| lam * sum_{j != t} T_t^-1 T_j d_j || from the Gram matrix; computed by the library."""
    g, n = _host_gram(gram)
    out = ctypes.c_double(0.0)
    _check(lib().randes_interference_norm(ctypes.addressof(g), n, int(t), float(lam), ctypes.byref(out)))
    return float(out.value)


def randes_pairwise_cosines(gram, exclude: int = -1):
    """(cosines as n lists of n floats, mean over pairs j < l that leave `exclude` out); computed by the library."""
    g, n = _host_gram(gram)
    cos = (ctypes.c_double * max(n * n, 1))()
    mean = ctypes.c_double(0.0)
    _check(lib().randes_pairwise_cosines(ctypes.addressof(g), n, -1 if exclude is None else int(exclude), ctypes.addressof(cos),
                                         ctypes.byref(mean)))
    return [[float(cos[j * n + l]) for l in range(n)] for j in range(n)], float(mean.value)


# ---- convenience object over torch tensors --------------------------------------------------
class Plan:
    """A plan plus the device workspace it lives in.

    ``rows, cols, group`` describe the layers, ``gflags`` the groups (see
    ``include/randes.h``).  Tensors passed to the methods are torch CUDA tensors
    of the storage dtype (float32 or bfloat16), one per layer.
    """

    def __init__(self, rows, cols, group, gflags, storage: int = F32, task_ids=(), seeds=(),
                 max_tasks: Optional[int] = None, device="cuda", host_only: bool = False, m_dtype: int = F32):
        n_layers, n_groups = len(rows), len(gflags)
        self._layers = (Layer * max(n_layers, 1))()
        for l in range(n_layers):
            self._layers[l] = Layer(int(rows[l]), int(cols[l]), int(group[l]))
        self._groups = (Group * max(n_groups, 1))()
        for g in range(n_groups):
            self._groups[g] = Group(int(gflags[g]))
        n_tasks = len(task_ids)
        if max_tasks is None:
            max_tasks = max(1, n_tasks + 8)
        ids = (ctypes.c_uint32 * max(n_tasks, 1))(*[int(t) for t in task_ids])
        sds = (ctypes.c_uint64 * max(n_tasks, 1))(*[int(s) for s in seeds])
        self.n_layers = n_layers
        self.rows, self.cols = [int(r) for r in rows], [int(c) for c in cols]
        self.storage = storage
        self.m_dtype = m_dtype
        self.handle = None
        self.workspace = None
        self.device = device
        ws_ptr, ws_bytes, stream = None, 0, None
        if not host_only:
            import torch

            ws_bytes = randes_plan_workspace_bytes_groups(self._layers, n_layers, self._groups, n_groups, max_tasks)
            if ws_bytes == 0:
                raise RandesError(INVALID_ARGUMENT, randes_last_error())
            self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=device)
            ws_ptr = self.workspace.data_ptr()
            stream = self._stream()
        self.handle = randes_plan(self._layers, n_layers, self._groups, n_groups, storage, m_dtype, ids, sds, n_tasks,
                                  max_tasks, ws_ptr, ws_bytes, stream)
        self.m_bytes = randes_superposition_bytes(self.handle)
        self.offsets = [randes_layer_offset(self.handle, l) for l in range(n_layers)]

    @classmethod
    def from_workload(cls, w, **kw) -> "Plan":
        kw.setdefault("task_ids", w.task_ids)
        kw.setdefault("seeds", w.seeds)
        return cls(w.rows, w.cols, w.group, w.gflags, storage=w.storage, **kw)

    def _stream(self):
        import torch

        return torch.cuda.current_stream(self.device).cuda_stream

    def close(self) -> None:
        if self.handle is not None:
            randes_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- queries
    @property
    def n_tasks(self) -> int:
        return randes_num_tasks(self.handle)

    def task_list(self):
        n = self.n_tasks
        ids = (ctypes.c_uint32 * max(n, 1))()
        sds = (ctypes.c_uint64 * max(n, 1))()
        _check(lib().randes_task_list(self.handle, ctypes.addressof(ids), ctypes.addressof(sds)))
        return [int(x) for x in ids[:n]], [int(x) for x in sds[:n]]

    def task_tables(self, task_id: int):
        src = (ctypes.c_uint32 * max(self.n_layers, 1))()
        pos = (ctypes.c_uint32 * max(self.n_layers, 1))()
        _check(lib().randes_task_tables(self.handle, task_id, ctypes.addressof(src), ctypes.addressof(pos)))
        return [int(x) for x in src[:self.n_layers]], [int(x) for x in pos[:self.n_layers]]

    # -- device buffers
    def new_superposition(self):
        import torch

        if self.m_dtype == BF16:
            return torch.empty(self.m_bytes // 2, dtype=torch.bfloat16, device=self.device)
        return torch.empty(self.m_bytes // 4, dtype=torch.float32, device=self.device)

    def slot(self, M, layer: int):
        """View of slot ``layer`` of the arena M as a [rows, cols] tensor."""
        o = self.offsets[layer] // (2 if self.m_dtype == BF16 else 4)
        n = self.rows[layer] * self.cols[layer]
        return M[o:o + n].view(self.rows[layer], self.cols[layer])

    def new_output(self, out_dtype: int = F32):
        import torch

        dt = torch.bfloat16 if out_dtype == BF16 else torch.float32
        return [torch.empty(r, c, dtype=dt, device=self.device) for r, c in zip(self.rows, self.cols)]

    # -- the path
    def compress(self, base, tasks, M=None):
        if M is None:
            M = self.new_superposition()
        randes_compress(self.handle, _as_ptrs(base), _as_ptrs(tasks), M, self._stream())
        return M

    def add_model(self, task_id: int, seed: int, base, task, M):
        randes_add_model(self.handle, task_id, seed, _as_ptrs(base), _as_ptrs(task), M, self._stream())
        return M

    def add_models(self, task_ids, seeds, base, tasks, M):
        randes_add_models(self.handle, task_ids, seeds, _as_ptrs(base), _as_ptrs(tasks), M, self._stream())
        return M

    def remove_model(self, task_id: int, base, task, M):
        randes_remove_model(self.handle, task_id, _as_ptrs(base), _as_ptrs(task), M, self._stream())
        return M

    def delta_gram(self, base, tasks):
        """Gram matrix of the transformed deltas as an [n, n] float64 CUDA tensor (see include/randes.h)."""
        import torch

        n = self.n_tasks
        gram = torch.empty(n, n, dtype=torch.float64, device=self.device)
        nbytes = randes_delta_gram_scratch_bytes(self.handle)
        scratch = torch.empty(nbytes // 8, dtype=torch.float64, device=self.device)
        randes_delta_gram(self.handle, _as_ptrs(base), _as_ptrs(tasks), gram, scratch, nbytes, self._stream())
        return gram

    def retrieve_batch(self, task_ids, lam: float, base, M, out=None, out_dtype: int = F32):
        """Rebuild several tasks in one launch; returns a list (per task) of lists of tensors."""
        out_lists = None
        if out is None:
            out = out_lists = [self.new_output(out_dtype) for _ in task_ids]
        elif not isinstance(out, ctypes.Array):
            out_lists = out
        randes_retrieve_batch(self.handle, task_ids, lam, out_dtype, _as_ptrs(base), M, _as_ptrs(out), self._stream())
        return out_lists

    def linear(self, task_id: int, lam: float, layer: int, x, base, M, y=None, y_dtype: int = F32):
        """x: [n_tokens, cols] bf16 CUDA tensor; returns y [n_tokens, rows], fp32 or bf16."""
        import torch

        if y is None:
            y = torch.empty((x.shape[0], self.rows[layer]), dtype=torch.bfloat16 if y_dtype == BF16 else torch.float32, device=x.device)
        else:
            y_dtype = BF16 if y.dtype == torch.bfloat16 else F32
        randes_linear(self.handle, task_id, lam, layer, x, int(x.shape[0]), _as_ptrs(base), M, y, self._stream(), y_dtype)
        return y

    def retrieve(self, task_id: int, lam: float, base, M, out=None, out_dtype: int = F32):
        out_list = None
        if out is None:
            out = out_list = self.new_output(out_dtype)
        elif not isinstance(out, ctypes.Array):
            out_list = out
        randes_retrieve(self.handle, task_id, lam, out_dtype, _as_ptrs(base), M, _as_ptrs(out), self._stream())
        return out_list
