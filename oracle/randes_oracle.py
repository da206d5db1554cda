"""ctypes front end of the RanDeS CPU oracle (``randes_oracle.c``).

TEST INFRASTRUCTURE.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this module; the CUDA library never does, and this
module never imports the CUDA library.  All arithmetic lives in the C file;
this file only marshals numpy arrays.

Conventions
-----------
* A model is a list of ``L`` row-major 2-D numpy arrays (1-D parameters are
  ``[1, cols]``), dtype float32 or uint16 (bf16 bit patterns).
* ``spec`` = ``(rows, cols, group, gflags)``: per-layer shapes and group ids,
  per-group flag words (bit 0 = shuffle, bit 1 = column sign flip).
* ``M`` is a list of ``L`` float32 arrays, one per slot (Section 4 of the
  paper: the superposed delta; always fp32).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence, Tuple

import numpy as np

F32 = 0
BF16 = 1
SHUFFLE = 1
FLIP = 2
SHIFT = 4
GAUSS = 1 << 16   # Gaussian-like diagonal context (Section 5.5, "RD") instead of the +-1 one


def SKIP(k: int) -> int:
    """Group flag bits for 'only every k-th member takes part'."""
    return (int(k) & 0xFF) << 8

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "randes_oracle.c")
_LIB = os.path.join(_HERE, "librandes_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no FMA contraction, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u32p = ctypes.POINTER(ctypes.c_uint32)
        lib.ro_philox4x32_10.argtypes = [u32p, u32p, u32p]
        lib.ro_philox4x32_10.restype = None
        lib.ro_permutation.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32,
                                       ctypes.c_uint32, u32p]
        lib.ro_permutation.restype = None
        lib.ro_sign.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32]
        lib.ro_sign.restype = ctypes.c_int
        lib.ro_sign_row.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32,
                                    ctypes.c_uint32, ctypes.c_void_p]
        lib.ro_sign_row.restype = None
        lib.ro_gauss.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32]
        lib.ro_gauss.restype = ctypes.c_float
        lib.ro_f32_to_bf16.argtypes = [ctypes.c_float]
        lib.ro_f32_to_bf16.restype = ctypes.c_uint16
        lib.ro_task_tables.restype = ctypes.c_int
        lib.ro_compress.restype = ctypes.c_int
        lib.ro_add_model.restype = ctypes.c_int
        lib.ro_add_models.restype = ctypes.c_int
        lib.ro_remove_model.restype = ctypes.c_int
        lib.ro_retrieve.restype = ctypes.c_int
        lib.ro_linear.restype = ctypes.c_int
        lib.ro_delta_gram.restype = ctypes.c_int
        lib.ro_num_threads.restype = ctypes.c_int
        lib.ro_set_num_threads.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


# --------------------------------------------------------------------------- primitives
def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> Tuple[int, int, int, int]:
    lib = _load()
    c = (ctypes.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (ctypes.c_uint32 * 4)()
    lib.ro_philox4x32_10(c, k, o)
    return tuple(int(x) for x in o)


def permutation(seed: int, task_id: int, group_index: int, G: int) -> np.ndarray:
    """sigma for one (task, group): slot k receives member sigma[k] (Section 4.3)."""
    lib = _load()
    out = np.zeros(max(G, 1), dtype=np.uint32)
    lib.ro_permutation(seed, task_id, group_index, G,
                       out.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32)))
    return out[:G]


def sign(seed: int, task_id: int, slot: int, col: int) -> int:
    return int(_load().ro_sign(seed, task_id, slot, col))


def sign_row(seed: int, task_id: int, slot: int, cols: int) -> np.ndarray:
    """Diagonal of D for one (task, slot) as an int8 vector of +-1 (Section 4.4)."""
    out = np.zeros(max(cols, 1), dtype=np.int8)
    _load().ro_sign_row(seed, task_id, slot, cols, out.ctypes.data_as(ctypes.c_void_p))
    return out[:cols]


def gauss(seed: int, task_id: int, slot: int, col: int) -> float:
    """Diagonal entry of the Gaussian-like context (Section 5.5, "RD") for (task, slot, column)."""
    return float(_load().ro_gauss(seed, task_id, slot, col))


def f32_to_bf16(x: float) -> int:
    return int(_load().ro_f32_to_bf16(ctypes.c_float(x)))


def num_threads() -> int:
    return int(_load().ro_num_threads())


def set_num_threads(n: int) -> None:
    _load().ro_set_num_threads(int(n))


# --------------------------------------------------------------------------- marshalling
def _u32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.uint32))


def _spec_args(spec):
    rows, cols, group, gflags = (_u32(x) for x in spec)
    assert rows.shape == cols.shape == group.shape
    keep = (rows, cols, group, gflags)
    p = ctypes.c_void_p
    args = [ctypes.c_uint32(rows.size), p(rows.ctypes.data), p(cols.ctypes.data),
            p(group.ctypes.data), ctypes.c_uint32(gflags.size), p(gflags.ctypes.data)]
    return args, keep


def _ptr_array(arrs: Sequence[np.ndarray]):
    pa = (ctypes.c_void_p * max(len(arrs), 1))()
    for i, a in enumerate(arrs):
        if a is None:   # a layer the masked computation never touches
            pa[i] = None
            continue
        assert a.flags["C_CONTIGUOUS"]
        pa[i] = a.ctypes.data
    return pa


def _mask(mask, n) -> Tuple[ctypes.c_void_p, Optional[np.ndarray]]:
    if mask is None:
        return ctypes.c_void_p(None), None
    m = np.zeros(n, dtype=np.uint8)
    m[np.asarray(list(mask), dtype=np.int64)] = 1
    return ctypes.c_void_p(m.ctypes.data), m


def _check_layers(spec, layers, dtype):
    rows, cols = spec[0], spec[1]
    want = np.uint16 if dtype == BF16 else np.float32
    assert len(layers) == len(rows)
    for l, a in enumerate(layers):
        if a is None:
            continue
        assert a.dtype == want, (l, a.dtype, want)
        assert a.size == int(rows[l]) * int(cols[l]), (l, a.shape)


def task_tables(spec, seed: int, task_id: int) -> Tuple[np.ndarray, np.ndarray]:
    """(src_of_slot, slot_of_pos) = (sigma, sigma^-1) over the whole layer list."""
    lib = _load()
    _, _, group, gflags = (_u32(x) for x in spec)
    L = group.size
    src = np.zeros(max(L, 1), dtype=np.uint32)
    pos = np.zeros(max(L, 1), dtype=np.uint32)
    p = ctypes.c_void_p
    rc = lib.ro_task_tables(ctypes.c_uint32(L), p(group.ctypes.data), ctypes.c_uint32(gflags.size),
                            p(gflags.ctypes.data), ctypes.c_uint64(seed), ctypes.c_uint32(task_id),
                            p(src.ctypes.data), p(pos.ctypes.data))
    if rc:
        raise ValueError("ro_task_tables failed: %d" % rc)
    return src[:L], pos[:L]


def new_superposition(spec, slots=None, m_dtype: int = F32) -> List[np.ndarray]:
    """One zeroed array per slot (fp32, or uint16 bf16 bits); with ``slots`` given, only those are allocated."""
    keep = None if slots is None else set(int(x) for x in slots)
    mdt = np.uint16 if m_dtype == BF16 else np.float32
    return [np.zeros((int(r), int(c)), dtype=mdt) if keep is None or l in keep else None
            for l, (r, c) in enumerate(zip(spec[0], spec[1]))]


def _sum_models(fn_name, spec, dtype, task_ids, seeds, base, tasks, slots, M, m_dtype):
    lib = _load()
    sargs, keep = _spec_args(spec)
    L = keep[0].size
    K = len(task_ids)
    assert len(tasks) == K and len(seeds) == K
    if base is not None:
        _check_layers(spec, base, dtype)
    flat = []
    for t in tasks:
        _check_layers(spec, t, dtype)
        flat.extend(t)
    if M is None:
        M = new_superposition(spec, slots, m_dtype)
    ids = _u32(task_ids)
    sd = np.ascontiguousarray(np.asarray(seeds, dtype=np.uint64))
    mptr, mkeep = _mask(slots, L)
    p = ctypes.c_void_p
    base_pa = _ptr_array(base) if base is not None else None
    rc = getattr(lib, fn_name)(*sargs, ctypes.c_int(dtype), ctypes.c_int(m_dtype), ctypes.c_uint32(K), p(ids.ctypes.data),
                               p(sd.ctypes.data), base_pa, _ptr_array(flat), _ptr_array(M), mptr)
    if rc:
        raise ValueError("%s failed: %d" % (fn_name, rc))
    return M


def compress(spec, dtype: int, task_ids: Sequence[int], seeds: Sequence[int],
             base: Optional[Sequence[np.ndarray]], tasks: Sequence[Sequence[np.ndarray]],
             slots=None, M: Optional[List[np.ndarray]] = None, m_dtype: int = F32) -> List[np.ndarray]:
    """M = sum_i T_i(W_i - W_0) in the given task order.  base=None: tasks hold deltas.
    m_dtype=BF16: the fp32 sum is rounded once to bf16 bit patterns."""
    return _sum_models("ro_compress", spec, dtype, task_ids, seeds, base, tasks, slots, M, m_dtype)


def add_models(spec, dtype: int, task_ids: Sequence[int], seeds: Sequence[int],
               base: Optional[Sequence[np.ndarray]], tasks: Sequence[Sequence[np.ndarray]], M: List[np.ndarray],
               slots=None, m_dtype: int = F32) -> List[np.ndarray]:
    """M <- M + sum_i T_i(W_i - W_0), in place: several models added in one step (Section 5.7).  The sum runs in
    fp32 from M's values in the given order; a bf16 M is rounded once, at the end."""
    return _sum_models("ro_add_models", spec, dtype, task_ids, seeds, base, tasks, slots, M, m_dtype)


def delta_gram(spec, dtype: int, task_ids: Sequence[int], seeds: Sequence[int],
               base: Optional[Sequence[np.ndarray]], tasks: Sequence[Sequence[np.ndarray]]) -> np.ndarray:
    """gram[i, j] = <T_i d_i, T_j d_j> in float64 (Section 3; the interfering deltas' inner products)."""
    lib = _load()
    sargs, keep = _spec_args(spec)
    K = len(task_ids)
    if base is not None:
        _check_layers(spec, base, dtype)
    flat = []
    for t in tasks:
        _check_layers(spec, t, dtype)
        flat.extend(t)
    ids = _u32(task_ids)
    sd = np.ascontiguousarray(np.asarray(seeds, dtype=np.uint64))
    gram = np.zeros((K, K), dtype=np.float64)
    p = ctypes.c_void_p
    base_pa = _ptr_array(base) if base is not None else None
    rc = lib.ro_delta_gram(*sargs, ctypes.c_int(dtype), ctypes.c_uint32(K), p(ids.ctypes.data), p(sd.ctypes.data),
                           base_pa, _ptr_array(flat), p(gram.ctypes.data))
    if rc:
        raise ValueError("ro_delta_gram failed: %d" % rc)
    return gram


def _swap(fn_name, spec, dtype, task_id, seed, base, task, M, slots, m_dtype):
    lib = _load()
    sargs, keep = _spec_args(spec)
    L = keep[0].size
    if base is not None:
        _check_layers(spec, base, dtype)
    _check_layers(spec, task, dtype)
    mptr, mkeep = _mask(slots, L)
    base_pa = _ptr_array(base) if base is not None else None
    rc = getattr(lib, fn_name)(*sargs, ctypes.c_int(dtype), ctypes.c_int(m_dtype), ctypes.c_uint32(task_id),
                               ctypes.c_uint64(seed), base_pa, _ptr_array(task),
                               _ptr_array(M), mptr)
    if rc:
        raise ValueError("%s failed: %d" % (fn_name, rc))
    return M


def add_model(spec, dtype, task_id, seed, base, task, M, slots=None, m_dtype: int = F32):
    """M <- M + T_j(W_j - W_0), in place (Section 5.7, model hot swapping)."""
    return _swap("ro_add_model", spec, dtype, task_id, seed, base, task, M, slots, m_dtype)


def remove_model(spec, dtype, task_id, seed, base, task, M, slots=None, m_dtype: int = F32):
    """M <- M - T_j(W_j - W_0), in place."""
    return _swap("ro_remove_model", spec, dtype, task_id, seed, base, task, M, slots, m_dtype)


def retrieve(spec, dtype: int, out_dtype: int, task_id: int, seed: int, lam: float,
             base: Sequence[np.ndarray], M: Sequence[np.ndarray], positions=None, m_dtype: int = F32) -> List[np.ndarray]:
    """What_t = W_0 + lambda * T_t^-1(M) (Section 4); out fp32 or bf16 bit patterns."""
    lib = _load()
    sargs, keep = _spec_args(spec)
    L = keep[0].size
    _check_layers(spec, base, dtype)
    _check_layers(spec, M, m_dtype)
    odt = np.uint16 if out_dtype == BF16 else np.float32
    wanted = None if positions is None else set(int(x) for x in positions)
    out = [np.zeros((int(r), int(c)), dtype=odt) if wanted is None or l in wanted else None
           for l, (r, c) in enumerate(zip(spec[0], spec[1]))]
    mptr, mkeep = _mask(positions, L)
    rc = lib.ro_retrieve(*sargs, ctypes.c_int(dtype), ctypes.c_int(m_dtype), ctypes.c_int(out_dtype),
                         ctypes.c_uint32(task_id), ctypes.c_uint64(seed), ctypes.c_float(lam),
                         _ptr_array(base), _ptr_array(M), _ptr_array(out), mptr)
    if rc:
        raise ValueError("ro_retrieve failed: %d" % rc)
    return out


def linear(spec, dtype: int, task_id: int, seed: int, lam: float, layer: int, x: np.ndarray,
           base: Sequence[np.ndarray], M: Sequence[np.ndarray], m_dtype: int = F32) -> Tuple[np.ndarray, np.ndarray]:
    """y = x What_t[layer]^T with What = W_0 + lambda * T_t^-1(M) (Section 4) never formed: fp64 from the
    definition.  x is [n_tokens, cols] in the storage type.  Returns (y, y_abs), both [n_tokens, rows] float64;
    y_abs = sum_c |x| (|W_0| + |lambda M|) is the scale for judging a finite-precision result."""
    lib = _load()
    sargs, keep = _spec_args(spec)
    _check_layers(spec, base, dtype)
    _check_layers(spec, M, m_dtype)
    rows, cols = int(spec[0][layer]), int(spec[1][layer])
    want = np.uint16 if dtype == BF16 else np.float32
    x = np.ascontiguousarray(x)
    if x.dtype != want or x.ndim != 2 or x.shape[1] != cols:
        raise ValueError("x must be [n_tokens, %d] of %s" % (cols, want))
    y = np.zeros((x.shape[0], rows), dtype=np.float64)
    y_abs = np.zeros_like(y)
    rc = lib.ro_linear(*sargs, ctypes.c_int(dtype), ctypes.c_int(m_dtype), ctypes.c_uint32(task_id),
                       ctypes.c_uint64(seed), ctypes.c_float(lam), ctypes.c_uint32(layer),
                       x.ctypes.data_as(ctypes.c_void_p), ctypes.c_uint32(x.shape[0]),
                       _ptr_array(base), _ptr_array(M),
                       y.ctypes.data_as(ctypes.c_void_p), y_abs.ctypes.data_as(ctypes.c_void_p))
    if rc:
        raise ValueError("ro_linear failed: %d" % rc)
    return y, y_abs
