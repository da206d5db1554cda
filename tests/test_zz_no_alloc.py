"""randes_retrieve_static: retrieve for callers that must not allocate device memory.

Some users of this library are given the weight tensors and a stream but own no
allocator: a plug-in inside a serving process whose memory pool belongs to the
host framework, or a handler that swaps models in a latency-critical loop where
cudaMalloc would stall the device.  For them the library keeps the retrieve
kernel's tables in a fixed device array of its own, so the call needs no
workspace.  This file checks, through the C ABI, that the variant returns
exactly what the ordinary entry point returns -- and what the CPU oracle
computes -- on two calls in a row (the second call reuses the array the first
one filled), that the device's free memory does not shrink across a call, that
the library's sources name no device allocator at all, and that a model too
large for the array is refused cleanly.  It is collected last on purpose.
"""
import ctypes
import glob
import os
import re

import numpy as np
import pytest

from oracle import randes_oracle as ro
from paper_2505_11204_b200 import build, randes, workloads as wl

from gpu_util import assert_bits_equal, from_dev, model_to_dev, poison

S, F = randes.SHUFFLE, randes.FLIP


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def small_workload(storage):
    shapes = [(40, 256, 3), (1, 256, 3), (33, 132, 2), (7, 12, 1), (64, 1024, 2)]
    names, rows, cols, group = [], [], [], []
    for k in range(3):
        for g, (r, c, n) in enumerate(shapes):
            if k < n:
                names.append("g%d.%d" % (g, k)); rows.append(r); cols.append(c); group.append(g)
    gflags = [S | F, S, S | F, F, S | F]
    return wl.Workload(name="no_alloc_case", layer_names=names, rows=rows, cols=cols, group=group, gflags=gflags,
                       storage=storage, n_tasks=3, task_ids=[0, 1, 2], seeds=[42, 43, 44], scale=1e-3, lam=0.3,
                       data_seed=11)


@pytest.mark.gpu
@pytest.mark.parametrize("storage", [wl.F32, wl.BF16])
def test_static_retrieve_matches_retrieve_on_two_calls_in_a_row(storage):
    import torch

    w = small_workload(storage)
    base, tasks = wl.model_set(w)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w)                      # ordinary plan, with a workspace
    host_plan = randes.Plan.from_workload(w, host_only=True)  # what a caller without an allocator builds
    M = plan.compress(d_base, d_tasks)
    M_ref = ro.compress(w.spec, w.storage, w.task_ids, w.seeds, base, tasks)
    p_base = randes.ptr_array(d_base)
    stream = torch.cuda.current_stream().cuda_stream
    calls = 0
    for out_dtype in (wl.F32, wl.BF16):
        for task in (2, 0):                                   # two calls in a row, different permutations and signs
            want = plan.retrieve(task, w.lam, d_base, M, out_dtype=out_dtype)
            ref = ro.retrieve(w.spec, w.storage, out_dtype, task, w.seeds[task], w.lam, base, M_ref)
            got = [poison(o) for o in plan.new_output(out_dtype)]
            p_got = randes.ptr_array(got)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]       # the device's own count, not torch's allocator
            p_base_call = randes.ptr_array(d_base)
            randes.randes_retrieve_static(host_plan.handle, task, w.lam, out_dtype, p_base_call, M, p_got, stream)
            # the pointer arrays are the caller's again as soon as the call returns: scribble over them before the
            # kernel has (necessarily) run -- the library works from its own copy of the tables
            ctypes.memset(ctypes.addressof(p_base_call), 0xFF, ctypes.sizeof(p_base_call))
            ctypes.memset(ctypes.addressof(p_got), 0xFF, ctypes.sizeof(p_got))
            torch.cuda.synchronize()
            calls += 1
            if calls > 1:                                     # the first call on a device may load the module with its array
                assert torch.cuda.mem_get_info()[0] >= free_before
            for l in range(w.n_layers):
                assert_bits_equal(from_dev(got[l]), from_dev(want[l]), "static retrieve task %d layer %d" % (task, l))
                assert_bits_equal(from_dev(got[l]), ref[l], "static retrieve against the oracle, task %d layer %d" % (task, l))
    # the ordinary plan's handle works too, and argument checks are the same
    got = plan.new_output(wl.F32)
    randes.randes_retrieve_static(plan.handle, 1, w.lam, wl.F32, p_base, M, randes.ptr_array(got), stream)
    want = plan.retrieve(1, w.lam, d_base, M)
    for l in range(w.n_layers):
        assert_bits_equal(from_dev(got[l]), from_dev(want[l]), "static retrieve via full plan, layer %d" % l)
    with pytest.raises(randes.RandesError) as e:
        randes.randes_retrieve_static(host_plan.handle, 9, w.lam, wl.F32, p_base, M, randes.ptr_array(got), stream)
    assert e.value.code == randes.UNKNOWN_TASK
    plan.close()
    host_plan.close()


def test_library_sources_name_no_device_allocator():
    """No entry point of the library may allocate or free device memory (callers own every buffer): the CUDA
    sources must not even name the runtime's or the driver's allocation routines."""
    here = os.path.dirname(os.path.abspath(build.__file__))
    banned = re.compile(r"\b(cudaMalloc\w*|cudaFree\w*|cudaHostAlloc|cuMemAlloc\w*|cuMemFree\w*|cuMemCreate|cudaMemPool\w*)\b")
    sources = sorted(glob.glob(os.path.join(here, "csrc", "*")))
    assert len(sources) >= 8
    for path in sources:
        hits = banned.findall(open(path).read())
        assert not hits, (os.path.basename(path), hits)


def test_static_retrieve_refuses_models_beyond_its_scratch():
    # 100k rows x 1024 columns x 12 layers: more tile descriptors than the 1 MiB array holds.
    # The check happens on the host before anything is launched, so this needs no GPU.
    n = 12
    plan = randes.Plan([100_000] * n, [1024] * n, [0] * n, [S | F], task_ids=[0], seeds=[1], host_only=True)
    # (addresses only, a GiB apart so that the 410 MB tensors do not overlap: nothing is ever dereferenced)
    fake = (ctypes.c_void_p * n)(*[(i + 1) << 30 for i in range(n)])
    fake_out = (ctypes.c_void_p * n)(*[(i + 100) << 30 for i in range(n)])
    with pytest.raises(randes.RandesError) as e:
        randes.randes_retrieve_static(plan.handle, 0, 1.0, randes.F32, fake, 1 << 50, fake_out, None)
    assert e.value.code == randes.CAPACITY
    assert "scratch" in str(e.value)
    plan.close()
