"""Full-size parity on the ViT-L/14-shaped set (304 M parameters, K = 20), in the launch
configuration the benchmark times: compress all 20, a retrieve sweep over all tasks, then a
streaming add / remove of further models, one by one and all in one pass.

The oracle cannot redo 26 models x 304 M parameters in seconds, so it computes whole sampled
slots of M (one or two of every kind of tensor) and the layers that those slots feed at
retrieval; these are compared bit for bit.  Inputs are generated layer by layer on the host
(seeded), streamed to the device, and kept on the host only where the sampled slots need them:
no oracle input ever comes from the GPU.
"""
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest

from oracle import randes_oracle as ro
from paper_2505_11204_b200 import build, randes, workloads as wl

from gpu_util import assert_bits_equal, from_dev, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def sampled_slots(w):
    """One early and one late member of every repeated tensor kind, and every unrepeated tensor."""
    by_group = {}
    for l, g in enumerate(w.group):
        by_group.setdefault(g, []).append(l)
    slots = []
    for g, mem in by_group.items():
        if len(mem) == 1:
            slots.append(mem[0])
        else:
            big = w.rows[mem[0]] > 1
            slots.append(mem[5 % len(mem)])
            if big and g % 2 == 0:
                slots.append(mem[-1])
    return sorted(slots)


def run_full_size(storage, n_swap):
    import torch

    w = wl.vit_l14(storage=storage)
    K, L = w.n_tasks, w.n_layers
    ids, seeds = list(w.task_ids), list(w.seeds)
    swap_ids = [K + j for j in range(n_swap)]
    swap_seeds = [seeds[0] + K + j for j in range(n_swap)]
    all_ids, all_seeds = ids + swap_ids, seeds + swap_seeds
    src_of = {t: ro.task_tables(w.spec, s, t)[0] for t, s in zip(all_ids, all_seeds)}
    slots = sampled_slots(w)
    need_base, need_task = set(), set()
    for l in slots:
        for t in all_ids:
            src = int(src_of[t][l])
            need_base.add(src)
            need_task.add((t, src))

    base_h = [None] * L
    tasks_h = {t: [None] * L for t in all_ids}
    d_base = [None] * L
    d_tasks = {t: [None] * L for t in all_ids}
    with ThreadPoolExecutor(max_workers=16) as ex:
        for l, (b, ts) in enumerate(ex.map(lambda l: wl.layer_all_tasks(w, l, all_ids), range(L))):
            d_base[l] = to_dev(b)
            if l in need_base:
                base_h[l] = b
            for t, a in zip(all_ids, ts):
                d_tasks[t][l] = to_dev(a)
                if (t, l) in need_task:
                    tasks_h[t][l] = a

    # the benchmark's launch configuration
    plan = randes.Plan.from_workload(w, max_tasks=K + max(n_swap, 1))
    M = plan.new_superposition().zero_()       # padding between slots is never written: keep it finite
    out = plan.new_output(wl.F32)
    p_base = randes.ptr_array(d_base)
    p_out = randes.ptr_array(out)
    sh = torch.cuda.current_stream().cuda_stream

    def check_m(tag):
        for l in slots:
            assert_bits_equal(from_dev(plan.slot(M, l)), M_ref[l], "%s slot %d (%s)" % (tag, l, w.layer_names[l]))

    randes.randes_compress(plan.handle, p_base, randes.ptr_array([d_tasks[t] for t in ids]), M, sh)
    M_ref = ro.compress(w.spec, storage, ids, seeds, base_h, [tasks_h[t] for t in ids], slots=slots)
    check_m("compress")

    def check_retrieve(t, s, tag):
        randes.randes_retrieve(plan.handle, t, w.lam, wl.F32, p_base, M, p_out, sh)
        pos = sorted(set(int(src_of[t][l]) for l in slots))      # the layers fed by the sampled slots
        ref = ro.retrieve(w.spec, storage, wl.F32, t, s, w.lam, base_h, M_ref, positions=pos)
        for p in pos:
            assert_bits_equal(from_dev(out[p]), ref[p], "%s retrieve task %d layer %d (%s)" % (tag, t, p, w.layer_names[p]))

    for t, s in zip(ids, seeds):
        check_retrieve(t, s, "sweep")
    if storage == wl.F32:
        # all 20 tasks in one launch: the same sampled layers, against the same oracle results
        outs = [plan.new_output(wl.F32) for _ in ids]
        randes.randes_retrieve_batch(plan.handle, ids, w.lam, wl.F32, p_base, M, randes.ptr_array(outs), sh)
        for b, (t, s) in enumerate(zip(ids, seeds)):
            pos = sorted(set(int(src_of[t][l]) for l in slots))
            ref = ro.retrieve(w.spec, storage, wl.F32, t, s, w.lam, base_h, M_ref, positions=pos)
            for p in pos:
                assert_bits_equal(from_dev(outs[b][p]), ref[p], "batched retrieve task %d layer %d" % (t, p))
        del outs
        torch.cuda.empty_cache()
    if storage == wl.F32:
        # Gram matrix of the transformed deltas at full size, checked through what holds at any size:
        # orthogonality keeps every delta's norm, sum_ij G_ij = ||M||^2, and the transforms remove the
        # cosine of 0.25 that the input recipe puts between any two deltas.
        task_ptrs = randes.ptr_array([d_tasks[t] for t in ids])
        G = plan.delta_gram(p_base, task_ptrs).cpu().numpy()
        for i in (0, 7, 19):
            n2 = sum(float(((a.double() - b.double()) ** 2).sum()) for a, b in zip(d_tasks[ids[i]], d_base))
            assert abs(G[i, i] - n2) <= 1e-9 * n2
        m2 = sum(float((plan.slot(M, l).double() ** 2).sum()) for l in range(L))
        assert abs(G.sum() - m2) <= 1e-5 * m2
        assert abs(randes.randes_pairwise_cosines(G)[1]) < 2e-3
        w0 = wl.Workload(**{**w.__dict__})
        w0.gflags = [0] * len(w.gflags)
        plain = randes.Plan.from_workload(w0)
        G0 = plain.delta_gram(p_base, task_ptrs).cpu().numpy()
        assert abs(randes.randes_pairwise_cosines(G0)[1] - 0.25) < 5e-3
        assert np.allclose(np.diag(G0), np.diag(G), rtol=1e-12)
        plain.close()
    for t, s in zip(swap_ids, swap_seeds):
        randes.randes_add_model(plan.handle, t, s, p_base, randes.ptr_array(d_tasks[t]), M, sh)
        ro.add_model(w.spec, storage, t, s, base_h, tasks_h[t], M_ref, slots=slots)
        check_m("add %d" % t)
    if swap_ids:
        check_retrieve(swap_ids[-1], swap_seeds[-1], "after adds")
    for t, s in zip(swap_ids, swap_seeds):
        randes.randes_remove_model(plan.handle, t, p_base, randes.ptr_array(d_tasks[t]), M, sh)
        ro.remove_model(w.spec, storage, t, s, base_h, tasks_h[t], M_ref, slots=slots)
        check_m("remove %d" % t)
    if len(swap_ids) > 1:
        # the same models again, now in one pass over M
        randes.randes_add_models(plan.handle, swap_ids, swap_seeds, p_base, randes.ptr_array([d_tasks[t] for t in swap_ids]), M, sh)
        ro.add_models(w.spec, storage, swap_ids, swap_seeds, base_h, [tasks_h[t] for t in swap_ids], M_ref, slots=slots)
        check_m("add_models")
        for t, s in zip(swap_ids, swap_seeds):
            randes.randes_remove_model(plan.handle, t, p_base, randes.ptr_array(d_tasks[t]), M, sh)
            ro.remove_model(w.spec, storage, t, s, base_h, tasks_h[t], M_ref, slots=slots)
        check_m("removes after add_models")
    check_retrieve(ids[7], seeds[7], "after removes")
    # properties that hold at any size: M is finite everywhere and no slot was left untouched
    assert bool(torch.isfinite(M).all())
    torch.cuda.synchronize()
    plan.close()


def test_vit_l14_shaped_fp32_full_size_sampled():
    run_full_size(wl.F32, n_swap=5)


def test_vit_l14_shaped_bf16_full_size_sampled():
    run_full_size(wl.BF16, n_swap=2)


def test_gaussian_context_full_size_sampled():
    """The Gaussian-diagonal ("RD") context of Section 5.5 on the ViT-L/14-shaped set (fp32, 3 tasks + 1 added and
    removed): plans with such a group get taller tiles on large models (up to 128 rows per warp), which the small
    parity cases never reach.  Sampled slots of M and the layers they feed are compared with the oracle bit for bit."""
    import torch

    w = wl.vit_l14(storage=wl.F32).with_tasks(3)
    w.gflags = [(f & ~wl.FLIP) | randes.GAUSS if f & wl.FLIP else f for f in w.gflags]
    L = w.n_layers
    ids, seeds = list(w.task_ids), list(w.seeds)
    all_ids, all_seeds = ids + [9], seeds + [1234]
    src_of = {t: ro.task_tables(w.spec, s, t)[0] for t, s in zip(all_ids, all_seeds)}
    slots = sampled_slots(w)[::2]
    need_base, need_task = set(), set()
    for l in slots:
        for t in all_ids:
            src = int(src_of[t][l])
            need_base.add(src)
            need_task.add((t, src))
    base_h, tasks_h = [None] * L, {t: [None] * L for t in all_ids}
    d_base, d_tasks = [None] * L, {t: [None] * L for t in all_ids}
    with ThreadPoolExecutor(max_workers=16) as ex:
        for l, (b, ts) in enumerate(ex.map(lambda l: wl.layer_all_tasks(w, l, all_ids), range(L))):
            d_base[l] = to_dev(b)
            if l in need_base:
                base_h[l] = b
            for t, a in zip(all_ids, ts):
                d_tasks[t][l] = to_dev(a)
                if (t, l) in need_task:
                    tasks_h[t][l] = a
    plan = randes.Plan.from_workload(w, max_tasks=4)
    randes.randes_plan_validate(plan.handle)
    M = plan.new_superposition().zero_()
    out = plan.new_output(wl.F32)
    p_base, p_out = randes.ptr_array(d_base), randes.ptr_array(out)
    sh = torch.cuda.current_stream().cuda_stream

    def check_m(tag):
        for l in slots:
            assert_bits_equal(from_dev(plan.slot(M, l)), M_ref[l], "%s slot %d (%s)" % (tag, l, w.layer_names[l]))

    def check_retrieve(t, s, tag):
        randes.randes_retrieve(plan.handle, t, w.lam, wl.F32, p_base, M, p_out, sh)
        pos = sorted(set(int(src_of[t][l]) for l in slots))
        ref = ro.retrieve(w.spec, wl.F32, wl.F32, t, s, w.lam, base_h, M_ref, positions=pos)
        for p in pos:
            assert_bits_equal(from_dev(out[p]), ref[p], "%s retrieve task %d layer %d (%s)" % (tag, t, p, w.layer_names[p]))

    randes.randes_compress(plan.handle, p_base, randes.ptr_array([d_tasks[t] for t in ids]), M, sh)
    M_ref = ro.compress(w.spec, wl.F32, ids, seeds, base_h, [tasks_h[t] for t in ids], slots=slots)
    check_m("compress")
    for t, s in zip(ids, seeds):
        check_retrieve(t, s, "sweep")
    randes.randes_add_model(plan.handle, 9, 1234, p_base, randes.ptr_array(d_tasks[9]), M, sh)
    ro.add_model(w.spec, wl.F32, 9, 1234, base_h, tasks_h[9], M_ref, slots=slots)
    check_m("add")
    check_retrieve(9, 1234, "after add")
    randes.randes_remove_model(plan.handle, 1, p_base, randes.ptr_array(d_tasks[1]), M, sh)
    ro.remove_model(w.spec, wl.F32, 1, seeds[1], base_h, tasks_h[1], M_ref, slots=slots)
    check_m("remove")
    assert bool(torch.isfinite(M).all())
    torch.cuda.synchronize()
    plan.close()
