"""Parity of the CUDA library (through its C ABI) with the CPU oracle.

Bars: permutation tables, sign bits and the fp32 superposition M are bit-exact;
fp32 outputs of retrieve are bit-exact (one fused multiply-add on both sides;
the accepted bound would be 1e-6 * max|W|); bf16 outputs are bit-exact (accepted
bound: 1 bf16 ulp).  All inputs are seeded and synthetic.
"""
import ctypes

import numpy as np
import pytest

from oracle import randes_oracle as ro
from paper_2505_11204_b200 import build, randes, workloads as wl

from gpu_util import (assert_bits_equal, check_model, check_superposition, from_dev, model_to_dev, poison,
                      to_dev)

pytestmark = pytest.mark.gpu
S, F = randes.SHUFFLE, randes.FLIP


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def make_workload(shapes, flags=S | F, storage=wl.F32, n_tasks=3, seed0=42, data_seed=7, interleave=True):
    """shapes: list of (rows, cols, group_size).  Layers of different groups are
    interleaved so that group-local and global indices differ."""
    names, rows, cols, group = [], [], [], []
    maxg = max(s[2] for s in shapes)
    order = [(k, g) for k in range(maxg) for g in range(len(shapes)) if k < shapes[g][2]] if interleave else \
            [(k, g) for g in range(len(shapes)) for k in range(shapes[g][2])]
    for k, g in order:
        names.append("g%d.%d" % (g, k)); rows.append(shapes[g][0]); cols.append(shapes[g][1]); group.append(g)
    gflags = [flags if isinstance(flags, int) else flags[g] for g in range(len(shapes))]
    return wl.Workload(name="case", layer_names=names, rows=rows, cols=cols, group=group, gflags=gflags,
                       storage=storage, n_tasks=n_tasks, task_ids=list(range(n_tasks)),
                       seeds=[seed0 + i for i in range(n_tasks)], scale=1e-3, lam=0.3, data_seed=data_seed)


def run_full_cycle(w, out_dtypes=(wl.F32, wl.BF16), lam=None, extra_task=True, m_dtype=wl.F32):
    """compress -> retrieve all -> add -> retrieve -> remove -> retrieve, each
    step compared with the oracle replaying the same calls."""
    import torch

    lam = w.lam if lam is None else lam
    ids, seeds = list(w.task_ids), list(w.seeds)
    all_ids = ids + ([max(ids) + 5] if extra_task else [])
    base, tasks = wl.model_set(w, all_ids)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w, max_tasks=len(all_ids) + 1, m_dtype=m_dtype)
    K = len(ids)
    msz = 2 if m_dtype == wl.BF16 else 4

    M_dev = poison(plan.new_superposition())
    plan.compress(d_base, d_tasks[:K], M_dev)
    M_ref = ro.compress(w.spec, w.storage, ids, seeds, base, tasks[:K], m_dtype=m_dtype)
    check_superposition(plan, M_dev, M_ref, "compress")
    # padding between slots is never written
    raw = M_dev.view(torch.int16 if m_dtype == wl.BF16 else torch.int32)
    for l in range(w.n_layers):
        end = plan.offsets[l] // msz + w.rows[l] * w.cols[l]
        nxt = plan.offsets[l + 1] // msz if l + 1 < w.n_layers else plan.m_bytes // msz
        assert bool((raw[end:nxt] == -1).all()), "padding after slot %d was written" % l

    def retrieve_all(tag):
        cur_ids, cur_seeds = plan.task_list()
        for od in out_dtypes:
            for t, s in zip(cur_ids, cur_seeds):
                out = [poison(o) for o in plan.new_output(od)]
                plan.retrieve(t, lam, d_base, M_dev, out=out, out_dtype=od)
                ref = ro.retrieve(w.spec, w.storage, od, t, s, lam, base, M_ref, m_dtype=m_dtype)
                check_model(out, ref, "%s retrieve task %d dtype %d" % (tag, t, od))

    retrieve_all("after compress")
    if extra_task:
        new_id, new_seed = all_ids[-1], 100
        plan.add_model(new_id, new_seed, d_base, d_tasks[K], M_dev)
        ro.add_model(w.spec, w.storage, new_id, new_seed, base, tasks[K], M_ref, m_dtype=m_dtype)
        check_superposition(plan, M_dev, M_ref, "add")
        assert plan.task_list() == (ids + [new_id], seeds + [new_seed])
        retrieve_all("after add")
        gone = ids[len(ids) // 2]
        j = ids.index(gone)
        plan.remove_model(gone, d_base, d_tasks[j], M_dev)
        ro.remove_model(w.spec, w.storage, gone, seeds[j], base, tasks[j], M_ref, m_dtype=m_dtype)
        check_superposition(plan, M_dev, M_ref, "remove")
        assert gone not in plan.task_list()[0]
        retrieve_all("after remove")
    torch.cuda.synchronize()
    plan.close()


# --------------------------------------------------------------------------- small cases
def test_toy_config_all_steps():
    run_full_cycle(wl.toy())


RAGGED = [(1, 1, 3), (5, 3, 3), (37, 12, 2), (3, 127, 3), (2, 129, 4), (7, 130, 2), (19, 260, 3),
          (1, 4100, 2), (33, 768, 3), (50, 640, 1), (130, 256, 2), (1, 4096, 5), (17, 384, 2)]


@pytest.mark.parametrize("storage", [wl.F32, wl.BF16])
def test_ragged_shapes_span_tiles_and_tails(storage):
    run_full_cycle(make_workload(RAGGED, storage=storage, n_tasks=3))


@pytest.mark.parametrize("storage", [wl.F32, wl.BF16])
def test_bf16_superposition(storage):
    # M stored as bf16: sums in fp32, one rounding per element at the end of compress, again after add / remove
    run_full_cycle(make_workload(RAGGED, storage=storage, n_tasks=4), m_dtype=wl.BF16)
    # more than 32 tasks would need the partial sum to pass through the bf16 arena: refused
    w = make_workload([(5, 260, 3), (1, 33, 2)], storage=storage, n_tasks=35)
    base, tasks = wl.model_set(w)
    plan = randes.Plan.from_workload(w, m_dtype=wl.BF16)
    with pytest.raises(randes.RandesError) as e:
        plan.compress(model_to_dev(base), [model_to_dev(t) for t in tasks])
    assert e.value.code == randes.CAPACITY
    plan.close()


def test_bf16_superposition_batched_and_static_retrieve():
    import torch

    w = make_workload(RAGGED, storage=wl.BF16, n_tasks=5)
    base, tasks = wl.model_set(w)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w, m_dtype=wl.BF16)
    assert plan.m_bytes <= 2 * w.n_params + 256 * w.n_layers
    M = plan.compress(d_base, d_tasks)
    M_ref = ro.compress(w.spec, w.storage, w.task_ids, w.seeds, base, tasks, m_dtype=wl.BF16)
    outs = plan.retrieve_batch([3, 0, 4], w.lam, d_base, M, out_dtype=wl.BF16)
    for b, t in enumerate([3, 0, 4]):
        check_model(outs[b], ro.retrieve(w.spec, w.storage, wl.BF16, t, w.seeds[t], w.lam, base, M_ref, m_dtype=wl.BF16),
                    "batched retrieve from bf16 M, task %d" % t)
    got = plan.new_output(wl.F32)
    randes.randes_retrieve_static(plan.handle, 2, w.lam, wl.F32, randes.ptr_array(d_base), M, randes.ptr_array(got),
                                  torch.cuda.current_stream().cuda_stream)
    check_model(got, ro.retrieve(w.spec, w.storage, wl.F32, 2, w.seeds[2], w.lam, base, M_ref, m_dtype=wl.BF16), "static retrieve from bf16 M")
    plan.close()


@pytest.mark.parametrize("flags", [0, S, F])
def test_single_transform_modes(flags):
    run_full_cycle(make_workload(RAGGED[3:10], flags=flags, n_tasks=2), out_dtypes=(wl.F32,))


def test_mixed_group_flags():
    shapes = [(9, 132, 3), (1, 132, 3), (4, 256, 1), (6, 20, 4)]
    run_full_cycle(make_workload(shapes, flags=[S | F, S, F, 0], n_tasks=4), out_dtypes=(wl.F32,))


def test_shift_and_skip_rate_variants():
    # layer shifting and skip rates of the paper's appendix: plan-level variants of the same kernels
    shapes = [(9, 132, 7), (1, 132, 7), (4, 256, 1), (6, 20, 5)]
    SH, K = randes.SHIFT, randes.SKIP
    for flags in ([SH | F, SH, F, SH | F | K(2)], [S | F | K(2), S | K(3), F | K(2), S | F | K(4)]):
        run_full_cycle(make_workload(shapes, flags=flags, n_tasks=4), out_dtypes=(wl.F32,))


def test_more_tasks_than_one_chunk():
    # 40 tasks: the kernel holds 32 task descriptors at a time
    run_full_cycle(make_workload([(5, 260, 3), (1, 33, 2), (24, 128, 2)], n_tasks=40), out_dtypes=(wl.F32,),
                   extra_task=True)


def test_single_task_round_trip_and_lambda_one():
    w = make_workload(RAGGED[2:9], n_tasks=1)
    base, tasks = wl.model_set(w)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w)
    M = plan.compress(d_base, d_tasks)
    out = plan.retrieve(0, 1.0, d_base, M)
    for b, t, o in zip(base, tasks[0], out):
        want = (b + (t - b).astype(np.float32)).astype(np.float32)
        assert_bits_equal(from_dev(o), want, "K=1 round trip")
    plan.close()


@pytest.mark.parametrize("storage,shapes", [(wl.F32, [(16, 768, 3), (768, 16, 2), (1, 100, 2)]),
                                            (wl.BF16, [(16, 768, 3), (768, 16, 2), (1, 104, 2)])])
def test_delta_input_without_base(storage, shapes):
    # adapter deltas given directly (Section 5.8): base = NULL (bf16: all widths multiples of 8, the add / remove
    # kernel with 4 + 4 columns per lane)
    w = make_workload(shapes, n_tasks=3, storage=storage)
    deltas = [[wl.lora_delta_layer(w, l, t) for l in range(w.n_layers)] for t in w.task_ids]
    d_deltas = [model_to_dev(d) for d in deltas]
    plan = randes.Plan.from_workload(w)
    M = plan.compress(None, d_deltas)
    M_ref = ro.compress(w.spec, w.storage, w.task_ids, w.seeds, None, deltas)
    check_superposition(plan, M, M_ref, "delta compress")
    extra = [wl.lora_delta_layer(w, l, 9) for l in range(w.n_layers)]
    plan.add_model(9, 77, None, model_to_dev(extra), M)
    ro.add_model(w.spec, w.storage, 9, 77, None, extra, M_ref)
    check_superposition(plan, M, M_ref, "delta add")
    plan.remove_model(1, None, d_deltas[1], M)
    ro.remove_model(w.spec, w.storage, 1, w.seeds[1], None, deltas[1], M_ref)
    check_superposition(plan, M, M_ref, "delta remove")
    plan.close()


def test_sign_bits_and_permutation_seen_through_the_kernels():
    # delta == 1 everywhere except a per-layer tag: M exposes s_i(l, c) and sigma_i(l) directly
    w = make_workload([(3, 300, 5)], n_tasks=1)
    ones = [np.full((r, c), float(l + 1), dtype=np.float32) for l, (r, c) in enumerate(zip(w.rows, w.cols))]
    plan = randes.Plan.from_workload(w)
    M = plan.compress(None, [model_to_dev(ones)])
    src, _ = ro.task_tables(w.spec, w.seeds[0], 0)
    for l in range(w.n_layers):
        want = np.tile(ro.sign_row(w.seeds[0], 0, l, w.cols[l]).astype(np.float32) * float(src[l] + 1), (w.rows[l], 1))
        assert_bits_equal(from_dev(plan.slot(M, l)), want, "sign/perm slot %d" % l)
    plan.close()


def test_unaligned_tensors_take_the_scalar_path():
    import torch

    for storage in (wl.F32, wl.BF16):
        w = make_workload([(6, 132, 3), (3, 260, 2)], storage=storage, n_tasks=2)
        base, tasks = wl.model_set(w)

        def shifted(a, k):  # same values, start address off by k elements
            t = to_dev(a)
            buf = torch.empty(a.size + 8, dtype=t.dtype, device="cuda")
            v = buf[k:k + a.size].view(a.shape)
            v.copy_(t)
            return v

        d_base = [shifted(a, 1 + (l % 3)) for l, a in enumerate(base)]
        d_tasks = [[shifted(a, 1 + ((l + i) % 2)) for l, a in enumerate(t)] for i, t in enumerate(tasks)]
        plan = randes.Plan.from_workload(w)
        M = plan.compress(d_base, d_tasks)
        M_ref = ro.compress(w.spec, storage, w.task_ids, w.seeds, base, tasks)
        check_superposition(plan, M, M_ref, "unaligned compress")
        for od in (wl.F32, wl.BF16):
            dt = torch.bfloat16 if od == wl.BF16 else torch.float32
            bufs = [torch.empty(r * c + 8, dtype=dt, device="cuda") for r, c in zip(w.rows, w.cols)]
            out = [b[1:1 + r * c].view(r, c) for b, r, c in zip(bufs, w.rows, w.cols)]
            plan.retrieve(1, 0.3, d_base, M, out=out, out_dtype=od)
            ref = ro.retrieve(w.spec, storage, od, 1, w.seeds[1], 0.3, base, M_ref)
            check_model(out, ref, "unaligned retrieve")
        plan.close()


@pytest.mark.parametrize("storage", [wl.F32, wl.BF16])
def test_batched_retrieve_equals_single_retrieves(storage):
    # several tasks rebuilt in one pass over W_0: bit-identical to one call per task
    w = make_workload(RAGGED, storage=storage, n_tasks=6)
    base, tasks = wl.model_set(w)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w)
    M = plan.compress(d_base, d_tasks)
    M_ref = ro.compress(w.spec, storage, w.task_ids, w.seeds, base, tasks)
    for od in (wl.F32, wl.BF16):
        for batch in ([4, 0, 5, 2, 1, 3], [3], [5, 1]):
            outs = [[poison(o) for o in plan.new_output(od)] for _ in batch]
            plan.retrieve_batch(batch, w.lam, d_base, M, out=outs, out_dtype=od)
            for b, t in enumerate(batch):
                ref = ro.retrieve(w.spec, storage, od, t, w.seeds[t], w.lam, base, M_ref)
                check_model(outs[b], ref, "batched retrieve task %d dtype %d" % (t, od))
    with pytest.raises(randes.RandesError) as e:
        plan.retrieve_batch([1, 1], w.lam, d_base, M)
    assert e.value.code == randes.DUPLICATE_TASK
    with pytest.raises(randes.RandesError) as e:
        plan.retrieve_batch([1, 77], w.lam, d_base, M)
    assert e.value.code == randes.UNKNOWN_TASK
    plan.close()


@pytest.mark.parametrize("storage", [wl.F32, wl.BF16])
def test_delta_gram_matches_oracle(storage):
    """Gram matrix of the transformed deltas (interference diagnostics).  Products are exact in fp64 on both
    sides; only the order of the fp64 additions differs, so |dG_ij| <= N * 2^-53 * sum|x_i x_j|
    <= N * 2^-53 * sqrt(G_ii G_jj) with N the number of parameters."""
    import torch

    w = make_workload(RAGGED, storage=storage, n_tasks=6)
    base, tasks = wl.model_set(w)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w)
    N = w.n_params
    for use_base in (True, False):
        G = plan.delta_gram(d_base if use_base else None, d_tasks).cpu().numpy()
        ref = ro.delta_gram(w.spec, storage, w.task_ids, w.seeds, base if use_base else None, tasks)
        scale = np.sqrt(np.outer(np.diag(ref), np.diag(ref)))
        assert np.all(np.abs(G - ref) <= N * 2.0 ** -53 * scale), np.max(np.abs(G - ref) / scale)
        G2 = plan.delta_gram(d_base if use_base else None, d_tasks).cpu().numpy()
        assert np.array_equal(G, G2)                      # fixed summation order: reproducible bit for bit
    # helpers on top of the matrix
    M_ref = ro.compress(w.spec, storage, w.task_ids, w.seeds, base, tasks)
    G = plan.delta_gram(d_base, d_tasks).cpu().numpy()
    m2 = sum(float((m.astype(np.float64) ** 2).sum()) for m in M_ref)
    assert abs(G.sum() - m2) <= 1e-5 * m2                  # ||M||^2 = sum_ij G_ij up to M's fp32 rounding
    t = 2
    out = ro.retrieve(w.spec, storage, wl.F32, t, w.seeds[t], 1.0, base, M_ref)
    f32 = (lambda a: wl.bf16_bits_to_f32(a) if a.dtype == np.uint16 else a)
    inter = np.concatenate([(o.astype(np.float64) - f32(b).astype(np.float64) - (f32(x).astype(np.float64) - f32(b).astype(np.float64))).ravel()
                            for o, b, x in zip(out, base, tasks[t])])
    assert abs(randes.randes_interference_norm(G, t, 1.0) - float(np.sqrt(inter @ inter))) <= 1e-3 * float(np.sqrt(inter @ inter))
    assert abs(randes.randes_pairwise_cosines(G)[1]) < 0.2       # decorrelated (raw cosine of this recipe: 0.25)
    plan.close()


@pytest.mark.parametrize("storage,m_dtype,n_new", [(wl.F32, wl.F32, 3), (wl.F32, wl.F32, 1), (wl.BF16, wl.F32, 5),
                                                   (wl.F32, wl.BF16, 4), (wl.BF16, wl.BF16, 2), (wl.F32, wl.F32, 37)])
def test_adding_several_models_in_one_pass(storage, m_dtype, n_new):
    """M <- M + sum of the new models' transformed deltas, one launch; with an fp32 M also equal to separate adds."""
    import torch

    shapes = RAGGED if n_new < 10 else [(19, 260, 3), (1, 4100, 2), (37, 12, 2), (5, 3, 3)]
    w = make_workload(shapes, storage=storage, n_tasks=2)
    new_ids = [10 + 3 * j for j in range(n_new)]
    new_seeds = [1000 + j for j in range(n_new)]
    base, tasks = wl.model_set(w, list(w.task_ids) + new_ids)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w, max_tasks=2 + n_new, m_dtype=m_dtype)
    M_dev = poison(plan.new_superposition())
    plan.compress(d_base, d_tasks[:2], M_dev)
    M_ref = ro.compress(w.spec, storage, w.task_ids, w.seeds, base, tasks[:2], m_dtype=m_dtype)
    if m_dtype == wl.F32:
        one_by_one = M_dev.clone()
    plan.add_models(new_ids, new_seeds, d_base, d_tasks[2:], M_dev)
    ro.add_models(w.spec, storage, new_ids, new_seeds, base, tasks[2:], M_ref, m_dtype=m_dtype)
    check_superposition(plan, M_dev, M_ref, "add_models")
    assert plan.task_list() == (list(w.task_ids) + new_ids, list(w.seeds) + new_seeds)
    # the new tasks are retrievable and removable like any other
    t, s_ = new_ids[-1], new_seeds[-1]
    out = plan.retrieve(t, 0.3, d_base, M_dev)
    check_model(out, ro.retrieve(w.spec, storage, wl.F32, t, s_, 0.3, base, M_ref, m_dtype=m_dtype), "retrieve of an added model")
    if m_dtype == wl.F32:
        other = randes.Plan.from_workload(w, max_tasks=2 + n_new)
        for i, sd, dt in zip(new_ids, new_seeds, d_tasks[2:]):
            other.add_model(i, sd, d_base, dt, one_by_one)
        assert torch.equal(one_by_one.view(torch.int32), M_dev.view(torch.int32))
        other.close()
    # nothing is registered when the call is refused
    before = plan.task_list()
    with pytest.raises(randes.RandesError) as e:
        plan.add_models([500, new_ids[0]], [1, 2], d_base, d_tasks[:2], M_dev)
    assert e.value.code == randes.DUPLICATE_TASK
    with pytest.raises(randes.RandesError) as e:
        plan.add_models([500, 500], [1, 2], d_base, d_tasks[:2], M_dev)
    assert e.value.code == randes.DUPLICATE_TASK
    with pytest.raises(randes.RandesError) as e:
        plan.add_models([500], [1], d_base, d_tasks[:1], M_dev)
    assert e.value.code == randes.CAPACITY
    plan.add_models([], [], d_base, [], M_dev)
    assert plan.task_list() == before
    check_superposition(plan, M_dev, M_ref, "after refused calls")
    torch.cuda.synchronize()
    plan.close()


def test_empty_layers_and_degenerate_plans():
    import torch

    # a model with empty tensors (zero rows or zero columns) among ordinary ones
    w = wl.Workload(name="empties", layer_names=list("abcde"), rows=[4, 0, 3, 5, 0], cols=[128, 64, 0, 20, 0], group=[0, 1, 2, 3, 4],
                    gflags=[F, F, F, F, F], storage=wl.F32, n_tasks=2, task_ids=[0, 1], seeds=[5, 6], scale=1e-3,
                    lam=0.5, data_seed=3)
    base, tasks = wl.model_set(w)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w)
    M = plan.compress(d_base, d_tasks)
    M_ref = ro.compress(w.spec, w.storage, w.task_ids, w.seeds, base, tasks)
    check_superposition(plan, M, M_ref, "compress with empty layers")
    out = plan.retrieve(1, w.lam, d_base, M)
    check_model(out, ro.retrieve(w.spec, w.storage, wl.F32, 1, 6, w.lam, base, M_ref), "retrieve with empty layers")
    plan.close()
    # nothing but empty layers: every call succeeds and launches nothing
    w0 = wl.Workload(name="nothing", layer_names=["x", "y"], rows=[0, 7], cols=[9, 0], group=[0, 1], gflags=[F, F],
                     storage=wl.F32, n_tasks=1, task_ids=[0], seeds=[1], scale=1e-3, lam=1.0, data_seed=3)
    base, tasks = wl.model_set(w0)
    plan = randes.Plan.from_workload(w0)
    before = randes.randes_launch_count()
    M = torch.zeros(64, dtype=torch.float32, device="cuda")
    plan.compress(model_to_dev(base), [model_to_dev(tasks[0])], M)
    plan.retrieve(0, 1.0, model_to_dev(base), M, out=plan.new_output())
    assert randes.randes_launch_count() == before
    plan.close()


def test_lambda_zero_and_bf16_ties():
    import torch

    # lambda = 0 gives back W_0 bit for bit; lambda = 1 on W_0 = 0 exposes +-M, whose values sit on
    # bf16 rounding ties, just above and just below them
    w = make_workload([(8, 128, 1)], flags=F, n_tasks=1)
    base, tasks = wl.model_set(w)
    plan = randes.Plan.from_workload(w)
    d_base = model_to_dev(base)
    M = plan.compress(d_base, [model_to_dev(tasks[0])])
    out = plan.retrieve(0, 0.0, d_base, M)
    assert_bits_equal(from_dev(out[0]), base[0], "lambda = 0")
    rng = np.random.default_rng(4)
    hi = rng.integers(0x3C00, 0x4400, size=(8, 128)).astype(np.uint32) << 16
    lo = rng.choice(np.array([0x8000, 0x7FFF, 0x8001, 0x0000, 0xFFFF], dtype=np.uint32), size=(8, 128))
    m_vals = (hi | lo).view(np.float32)
    M_dev = plan.new_superposition().zero_()
    plan.slot(M_dev, 0).copy_(to_dev(m_vals))
    zero = [torch.zeros(8, 128, device="cuda")]
    out = plan.retrieve(0, 1.0, zero, M_dev, out_dtype=wl.BF16)
    ref = ro.retrieve(w.spec, wl.F32, wl.BF16, 0, w.seeds[0], 1.0, [np.zeros((8, 128), np.float32)], [m_vals])
    assert_bits_equal(from_dev(out[0]), ref[0], "bf16 ties")
    plan.close()


def test_thirty_two_tasks_exactly_and_wide_single_row():
    run_full_cycle(make_workload([(1, 100000, 1), (3, 4096, 2)], n_tasks=32), out_dtypes=(wl.F32,), extra_task=False)


@pytest.mark.parametrize("storage", [wl.F32, wl.BF16])
@pytest.mark.parametrize("n_tasks", [2, 5, 32])
def test_large_and_partly_shuffled_groups(n_tasks, storage):
    """Compress of shuffled groups runs over group units (W_0 of all members staged in shared memory):
    groups of 30, 48 and 50 members (3, 2 and 1 rows per unit with fp32 weights; 2, 1 and 1 with bf16),
    97 members (too large: per-layer path), a group where only every second member is shuffled, ragged rows
    and widths (with bf16 weights the widths that are no multiple of 8 take the element-wise path); 2 to 32
    tasks (32 tasks x 48 members exceed the tables that fit beside two resident CTAs)."""
    shapes = [(9, 132, 30), (5, 256, 50), (3, 128, 97), (6, 260, 48), (11, 520, 7), (21, 128, 4), (2, 4, 24), (7, 264, 48)]
    flags = [S | F, S | F, S | F, S, S | F | randes.SKIP(2), S | F, S | F, S | F]
    run_full_cycle(make_workload(shapes, flags=flags, n_tasks=n_tasks, storage=storage), out_dtypes=(wl.F32,), extra_task=False)


@pytest.mark.parametrize("storage", [wl.F32, wl.BF16])
@pytest.mark.parametrize("n_tasks", [24, 30])
def test_group_compress_with_shallower_rings(storage, n_tasks):
    """Many tasks x many members: the per-(slot, task) records take the room of ring stages (fp32: 24 tasks x 30 members
    leave 5 stages, 30 x 30 leave 4; bf16: 3) while two CTAs still fit an SM."""
    shapes = [(8, 128, 24), (6, 256, 30), (4, 64, 1)]
    run_full_cycle(make_workload(shapes, flags=[S | F, S | F, F], storage=storage, n_tasks=n_tasks), out_dtypes=(wl.F32,), extra_task=False)


def test_batched_retrieve_of_many_tasks_and_members():
    """32 tasks x 30 members: the records of the grouped batched retrieve no longer fit beside two resident CTAs."""
    import torch

    w = make_workload([(6, 256, 30), (5, 132, 24), (3, 64, 1)], flags=[S | F, S | F, F], n_tasks=32)
    base, tasks = wl.model_set(w, w.task_ids)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w, max_tasks=32)
    M = plan.compress(d_base, d_tasks)
    M_ref = ro.compress(w.spec, w.storage, w.task_ids, w.seeds, base, tasks)
    check_superposition(plan, M, M_ref, "compress")
    outs = plan.retrieve_batch(list(w.task_ids), w.lam, d_base, M)
    for b, (t, s_) in enumerate(zip(w.task_ids, w.seeds)):
        check_model(outs[b], ro.retrieve(w.spec, w.storage, wl.F32, t, s_, w.lam, base, M_ref), "batch task %d" % t)
    torch.cuda.synchronize()
    plan.close()


def test_bf16_weights_with_widths_that_are_multiples_of_eight():
    """bf16 weights whose every width is a multiple of 8: add / remove and retrieve then take the kernels in which a lane
    owns 4 + 4 columns of the two halves of a 256-column block (ragged last blocks: 8, 264, 1032 columns)."""
    shapes = [(9, 256, 3), (5, 264, 2), (17, 1032, 2), (1, 8, 4), (40, 520, 1), (3, 128, 5)]
    flags = [S | F, S | F, F, S, F, S | F | randes.SKIP(2)]
    run_full_cycle(make_workload(shapes, flags=flags, storage=wl.BF16, n_tasks=4))
    run_full_cycle(make_workload(shapes, flags=flags, storage=wl.BF16, n_tasks=2), m_dtype=wl.BF16, out_dtypes=(wl.BF16,))


@pytest.mark.parametrize("storage", [wl.F32, wl.BF16])
@pytest.mark.parametrize("n_tasks", [3, 10])
def test_gaussian_diagonal_context(storage, n_tasks):
    """The "RD" ablation of Section 5.5 (a nearly normal diagonal instead of +-1; compress multiplies, retrieve divides):
    every step bit for bit against the oracle, alone, under a shuffle, with a skip rate, and beside groups that keep
    the sign flip or no context (a plan with one such group runs all its layers through the plain kernels);
    10 tasks = two passes of 8 and 2 through M."""
    G = randes.GAUSS
    shapes = [(9, 132, 3), (5, 256, 4), (17, 520, 2), (1, 300, 5), (33, 64, 3), (3, 2100, 2), (7, 131, 2), (4, 6, 3), (21, 1030, 2)]
    flags = [G | S, G, S | F, G | S | randes.SKIP(2), S, G | S, G | S, G, S | F]     # (widths 131, 6, 1030: the element-wise path)
    run_full_cycle(make_workload(shapes, flags=flags, storage=storage, n_tasks=n_tasks), extra_task=True)


@pytest.mark.parametrize("storage", [wl.F32, wl.BF16])
def test_gaussian_diagonal_context_registry_changes(storage):
    """The factors of the RD context are kept per registered task in a table in the plan's workspace.  A remove shifts the
    later tasks up one row, a batched add appends rows: after each change every remaining task must still be retrieved
    with ITS factors, and the sums must equal the oracle's replay of the same calls (six tasks = two passes of four and
    two; the batched add continues from M)."""
    G = randes.GAUSS
    w = make_workload([(9, 132, 3), (6, 257, 2), (17, 520, 2), (1, 300, 4)], flags=[G | S, G | S, S | F, G], storage=storage, n_tasks=6)
    ids, seeds = list(w.task_ids), list(w.seeds)
    new_ids, new_seeds = [40, 41, 42], [900, 901, 902]
    base, tasks = wl.model_set(w, ids + new_ids)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w, max_tasks=9)
    M_dev = poison(plan.new_superposition())
    plan.compress(d_base, d_tasks[:6], M_dev)
    M_ref = ro.compress(w.spec, storage, ids, seeds, base, tasks[:6])
    check_superposition(plan, M_dev, M_ref, "compress")
    # remove the second task: rows 2 .. 5 of the table move up
    plan.remove_model(ids[1], d_base, d_tasks[1], M_dev)
    ro.remove_model(w.spec, storage, ids[1], seeds[1], base, tasks[1], M_ref)
    check_superposition(plan, M_dev, M_ref, "remove of a middle task")
    for t in (0, 2, 5):
        check_model(plan.retrieve(ids[t], 0.3, d_base, M_dev), ro.retrieve(w.spec, storage, wl.F32, ids[t], seeds[t], 0.3, base, M_ref),
                    "retrieve of task %d after the shift" % ids[t])
    # three more in one pass, then one of the old ones leaves
    plan.add_models(new_ids, new_seeds, d_base, d_tasks[6:], M_dev)
    ro.add_models(w.spec, storage, new_ids, new_seeds, base, tasks[6:], M_ref)
    check_superposition(plan, M_dev, M_ref, "add_models")
    plan.remove_model(ids[4], d_base, d_tasks[4], M_dev)
    ro.remove_model(w.spec, storage, ids[4], seeds[4], base, tasks[4], M_ref)
    check_superposition(plan, M_dev, M_ref, "second remove")
    for t, sd in ((ids[5], seeds[5]), (new_ids[0], new_seeds[0]), (new_ids[2], new_seeds[2])):
        check_model(plan.retrieve(t, 0.3, d_base, M_dev, out_dtype=wl.BF16), ro.retrieve(w.spec, storage, wl.BF16, t, sd, 0.3, base, M_ref),
                    "retrieve of task %d after the second shift" % t)
    plan.close()


def test_plan_rebuilt_from_its_blob_on_the_device():
    """A plan kept as a blob comes back in two steps: deserialized host-only it tells the workspace it needs, deserialized
    again with that memory it computes the same bits as the original -- also for a plan whose workspace holds the factor
    table of the Gaussian-like context."""
    import torch

    G = randes.GAUSS
    for flags in ([S | F, S, F], [G | S, G, S | F]):
        w = make_workload([(9, 132, 3), (5, 256, 2), (17, 520, 2)], flags=flags, n_tasks=3)
        base, tasks = wl.model_set(w, w.task_ids)
        d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
        plan = randes.Plan.from_workload(w, max_tasks=4)
        M_a = plan.compress(d_base, d_tasks)
        blob = randes.randes_plan_serialize(plan.handle)
        host = randes.randes_plan_deserialize(blob, max_tasks=4)
        need = randes.randes_plan_workspace_needed(host)
        randes.randes_plan_destroy(host)
        assert 0 < need <= plan.workspace.numel()
        stream = torch.cuda.current_stream().cuda_stream
        ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        with pytest.raises(randes.RandesError) as e:
            randes.randes_plan_deserialize(blob, 4, ws.data_ptr(), need - 256, stream)
        assert e.value.code == randes.WORKSPACE_TOO_SMALL
        twin = randes.randes_plan_deserialize(blob, 4, ws.data_ptr(), need, stream)
        try:
            M_b = poison(plan.new_superposition())
            randes.randes_compress(twin, randes.ptr_array(d_base), randes.ptr_array(d_tasks), M_b, stream)
            for l in range(w.n_layers):          # slot by slot: the lead-in and the padding between slots are never written
                assert torch.equal(plan.slot(M_a, l).view(torch.int32), plan.slot(M_b, l).view(torch.int32)), "slot %d" % l
            out_a = plan.retrieve(w.task_ids[1], 0.3, d_base, M_a)
            out_b = plan.new_output(wl.F32)
            randes.randes_retrieve(twin, w.task_ids[1], 0.3, wl.F32, randes.ptr_array(d_base), M_b, randes.ptr_array(out_b), stream)
            assert all(torch.equal(a.view(torch.int32), b.view(torch.int32)) for a, b in zip(out_a, out_b))
        finally:
            randes.randes_plan_destroy(twin)
        plan.close()


def test_gaussian_diagonal_context_limits():
    G = randes.GAUSS
    w = make_workload([(8, 64, 2)], flags=[G | S], n_tasks=2)
    base, tasks = wl.model_set(w, w.task_ids)
    d_base = model_to_dev(base)
    with pytest.raises(randes.RandesError) as e:
        randes.Plan.from_workload(w, max_tasks=2, m_dtype=wl.BF16)
    assert e.value.code == randes.UNSUPPORTED_DTYPE
    with pytest.raises(randes.RandesError) as e:
        randes.Plan.from_workload(make_workload([(8, 64, 2)], flags=[G | F], n_tasks=2), max_tasks=2)
    assert e.value.code == randes.INVALID_ARGUMENT
    plan = randes.Plan.from_workload(w, max_tasks=2)
    import torch

    # the plan keeps a table of its factors in the workspace: the plain workspace figure is refused, with a message that
    # names the query to use
    small = randes.randes_plan_workspace_bytes(plan._layers, w.n_layers, 2)
    assert small < randes.randes_plan_workspace_bytes_groups(plan._layers, w.n_layers, plan._groups, len(w.gflags), 2) == plan.workspace.numel()
    ids = (ctypes.c_uint32 * 2)(*w.task_ids)
    sds = (ctypes.c_uint64 * 2)(*w.seeds)
    ws = torch.empty(small, dtype=torch.uint8, device="cuda")
    with pytest.raises(randes.RandesError) as e:
        randes.randes_plan(plan._layers, w.n_layers, plan._groups, len(w.gflags), w.storage, wl.F32, ids, sds, 2, 2, ws.data_ptr(), small,
                           torch.cuda.current_stream().cuda_stream)
    assert e.value.code == randes.WORKSPACE_TOO_SMALL and "randes_plan_workspace_bytes_groups" in str(e.value)
    M = plan.compress(d_base, [model_to_dev(t) for t in tasks])
    before = randes.randes_launch_count()
    for call in (lambda: plan.retrieve_batch(list(w.task_ids), 0.3, d_base, M),
                 lambda: plan.delta_gram(d_base, [model_to_dev(t) for t in tasks]),
                 lambda: randes.randes_retrieve_static(plan.handle, w.task_ids[0], 0.3, wl.F32, randes.ptr_array(d_base), M,
                                                       randes.ptr_array(plan.new_output(wl.F32)), 0)):
        with pytest.raises(randes.RandesError) as e:
            call()
        assert e.value.code == randes.INVALID_ARGUMENT
    assert randes.randes_launch_count() == before
    plan.close()


def test_random_plans():
    """Seeded random models: shapes, group sizes, flags (shuffle / shift / flip / skip), task counts, ids,
    seeds and storage types drawn at random; every step of the path against the oracle."""
    rng = np.random.default_rng(2024)
    SH, SK = randes.SHIFT, randes.SKIP
    for case in range(12):
        n_groups = int(rng.integers(1, 6))
        shapes, flags = [], []
        for _ in range(n_groups):
            rows = int(rng.choice([1, 1, 2, 7, 16, 17, 40, 130]))
            cols = int(rng.choice([1, 4, 8, 12, 100, 128, 132, 256, 384, 520, 1024, 1032]))
            shapes.append((rows, cols, int(rng.integers(1, 7))))
            f = int(rng.choice([0, S, SH])) | (F if rng.random() < 0.7 else 0)
            if rng.random() < 0.3:
                f |= SK(int(rng.integers(2, 4)))
            flags.append(f)
        w = make_workload(shapes, flags=flags, storage=int(rng.integers(0, 2)), n_tasks=int(rng.integers(1, 7)),
                          seed0=int(rng.integers(0, 2**62)), data_seed=100 + case, interleave=bool(rng.integers(0, 2)))
        w.task_ids = [int(x) for x in rng.choice(1000, size=w.n_tasks, replace=False)]
        run_full_cycle(w, out_dtypes=(int(rng.integers(0, 2)),), lam=float(rng.choice([0.1, 0.3, 1.0, 2.0])))


def test_random_plans_with_a_gaussian_context():
    """The same draw with the Gaussian-like diagonal in some groups (such a plan runs all its layers, flipped or not,
    through the kernels of the general context; up to twelve tasks = three passes of four): every step against the oracle."""
    rng = np.random.default_rng(4711)
    SH, SK, G = randes.SHIFT, randes.SKIP, randes.GAUSS
    for case in range(10):
        n_groups = int(rng.integers(1, 5))
        shapes, flags = [], []
        for g in range(n_groups):
            rows = int(rng.choice([1, 2, 5, 16, 17, 33, 70]))
            cols = int(rng.choice([4, 6, 12, 64, 130, 136, 256, 264, 520, 1024, 1032, 2056]))
            shapes.append((rows, cols, int(rng.choice([1, 2, 3, 5, 12]))))
            f = int(rng.choice([0, S, S, SH]))
            if g == 0 or rng.random() < 0.6:
                f |= G
            elif rng.random() < 0.7:
                f |= F
            if rng.random() < 0.25:
                f |= SK(int(rng.integers(2, 4)))
            flags.append(f)
        w = make_workload(shapes, flags=flags, storage=int(rng.integers(0, 2)), n_tasks=int(rng.choice([1, 2, 4, 5, 9, 12])),
                          seed0=int(rng.integers(0, 2**62)), data_seed=300 + case, interleave=bool(rng.integers(0, 2)))
        w.task_ids = [int(x) for x in rng.choice(1000, size=w.n_tasks, replace=False)]
        run_full_cycle(w, out_dtypes=(int(rng.integers(0, 2)),), lam=float(rng.choice([0.1, 0.3, 1.0])))


def test_row_slices_shard_without_exchange():
    # what each of several GPUs would hold under row-slice sharding, run here one slice after the other
    w = make_workload([(37, 256, 3), (1, 256, 3), (50, 132, 2)], n_tasks=3)
    base, tasks = wl.model_set(w)
    M_ref = ro.compress(w.spec, w.storage, w.task_ids, w.seeds, base, tasks)
    out_ref = ro.retrieve(w.spec, w.storage, wl.F32, 2, w.seeds[2], w.lam, base, M_ref)
    parts = 2
    for part in range(parts):
        ws, bounds = wl.row_slice(w, part, parts)
        cut = lambda model: [np.ascontiguousarray(a[lo:hi]) for a, (lo, hi) in zip(model, bounds)]
        plan = randes.Plan.from_workload(ws)
        d_base = model_to_dev(cut(base))
        M = plan.compress(d_base, [model_to_dev(cut(t)) for t in tasks])
        out = plan.retrieve(2, w.lam, d_base, M)
        for l, (lo, hi) in enumerate(bounds):
            if hi > lo:
                assert_bits_equal(from_dev(plan.slot(M, l)), M_ref[l][lo:hi], "slice %d of M, slot %d" % (part, l))
                assert_bits_equal(from_dev(out[l]), out_ref[l][lo:hi], "slice %d of the retrieved model, layer %d" % (part, l))
        plan.close()


def test_two_plans_on_two_streams_do_not_disturb_each_other():
    """Calls on one plan are ordered on the stream they are given; distinct plans share nothing.  Two plans (fp32 and
    bf16 weights) are driven on two CUDA streams with their calls interleaved on the host -- compress, adds, removes
    and retrieves of one plan enqueued between those of the other, nothing synchronised in between -- and every result
    equals the oracle's bit for bit."""
    import torch

    ws = [wl.toy(n_tasks=3, width=384, n_blocks=5), wl.toy(n_tasks=4, width=256, n_blocks=7).with_storage(wl.BF16)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    st = []
    for w in ws:
        ids = list(w.task_ids) + [77]
        base, models = wl.model_set(w, ids)
        st.append({"w": w, "base": base, "tasks": models[:w.n_tasks], "extra": models[w.n_tasks],
                   "d_base": model_to_dev(base), "d_tasks": [model_to_dev(t) for t in models[:w.n_tasks]],
                   "d_extra": model_to_dev(models[w.n_tasks])})
    torch.cuda.synchronize()
    for s_, q in zip(streams, st):
        with torch.cuda.stream(s_):
            q["plan"] = randes.Plan.from_workload(q["w"], max_tasks=q["w"].n_tasks + 1)
            q["M"] = q["plan"].new_superposition()
            q["outs"] = {}
    order = ["compress", "retrieve0", "add", "retrieve77", "remove", "retrieve1"]
    for step in order:
        for s_, q in zip(streams, st):                       # plan A's call, then plan B's, never a synchronisation
            w, plan = q["w"], q["plan"]
            with torch.cuda.stream(s_):
                if step == "compress":
                    plan.compress(q["d_base"], q["d_tasks"], q["M"])
                elif step == "add":
                    plan.add_model(77, 1234, q["d_base"], q["d_extra"], q["M"])
                elif step == "remove":
                    plan.remove_model(w.task_ids[0], q["d_base"], q["d_tasks"][0], q["M"])
                else:
                    t = int(step[len("retrieve"):])
                    q["outs"][step] = plan.retrieve(t, w.lam, q["d_base"], q["M"])
    torch.cuda.synchronize()
    for q in st:
        w = q["w"]
        M_ref = ro.compress(w.spec, w.storage, w.task_ids, w.seeds, q["base"], q["tasks"])
        check_model(q["outs"]["retrieve0"], ro.retrieve(w.spec, w.storage, wl.F32, 0, w.seeds[0], w.lam, q["base"], M_ref), "retrieve 0")
        ro.add_model(w.spec, w.storage, 77, 1234, q["base"], q["extra"], M_ref)
        check_model(q["outs"]["retrieve77"], ro.retrieve(w.spec, w.storage, wl.F32, 77, 1234, w.lam, q["base"], M_ref), "retrieve 77")
        ro.remove_model(w.spec, w.storage, w.task_ids[0], w.seeds[0], q["base"], q["tasks"][0], M_ref)
        check_model(q["outs"]["retrieve1"], ro.retrieve(w.spec, w.storage, wl.F32, 1, w.seeds[1], w.lam, q["base"], M_ref), "retrieve 1")
        check_superposition(q["plan"], q["M"], M_ref, "final M")
        q["plan"].close()


def test_gpu_argument_validation():
    import torch

    w = make_workload([(4, 128, 2)], n_tasks=1)
    base, tasks = wl.model_set(w)
    d_base, d_task = model_to_dev(base), model_to_dev(tasks[0])
    plan = randes.Plan.from_workload(w, max_tasks=2)
    M = plan.compress(d_base, [d_task])

    def expect(code, fn):
        with pytest.raises(randes.RandesError) as e:
            fn()
        assert e.value.code == code, str(e.value)

    before = randes.randes_launch_count()
    expect(randes.UNKNOWN_TASK, lambda: plan.retrieve(5, 1.0, d_base, M))
    expect(randes.UNSUPPORTED_DTYPE, lambda: plan.retrieve(0, 1.0, d_base, M, out=plan.new_output(), out_dtype=3))
    expect(randes.INVALID_ARGUMENT, lambda: plan.retrieve(0, 1.0, d_base, M, out=d_base))          # aliases base
    expect(randes.INVALID_ARGUMENT, lambda: plan.retrieve(0, 1.0, d_base, M, out=[plan.slot(M, 0), plan.slot(M, 1)]))
    expect(randes.MISALIGNED, lambda: plan.compress(d_base, [d_task], M[1:]))
    expect(randes.INVALID_ARGUMENT, lambda: randes.randes_compress(plan.handle, randes.ptr_array(d_base),
                                                                   randes.ptr_array(d_task), None, None))
    expect(randes.DUPLICATE_TASK, lambda: plan.add_model(0, 9, d_base, d_task, M))
    expect(randes.UNKNOWN_TASK, lambda: plan.remove_model(4, d_base, d_task, M))
    odd = torch.empty(4 * 128 * 4 + 2, dtype=torch.uint8, device="cuda")[1:1 + 4 * 128 * 4]
    expect(randes.MISALIGNED, lambda: plan.compress([odd, d_base[1]], [d_task], M))
    plan.add_model(1, 9, d_base, d_task, M)
    expect(randes.CAPACITY, lambda: plan.add_model(2, 9, d_base, d_task, M))
    assert randes.randes_launch_count() == before + 1      # only the valid add launched
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(randes.RandesError) as e:
        randes.randes_plan(plan._layers, 2, plan._groups, 1, 0, 0, None, None, 0, 1, small, 256, None)
    assert e.value.code == randes.WORKSPACE_TOO_SMALL
    plan.close()


# --------------------------------------------------------------------------- the paper-shaped configs, full size
def test_vit_b32_shaped_full():
    w = wl.vit_b32()
    run_full_cycle(w, out_dtypes=(wl.F32,), extra_task=False)


def test_gpt2_shaped_bf16_hot_swap_full():
    # K = 7 in bf16 storage; then remove task 3 and add task 7 (seed 100), retrieving every task after each change
    import torch

    w = wl.gpt2_small()
    ids, seeds = list(w.task_ids), list(w.seeds)
    base, tasks = wl.model_set(w, ids + [7])
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w, max_tasks=9)
    M = plan.compress(d_base, d_tasks[:7])
    M_ref = ro.compress(w.spec, w.storage, ids, seeds, base, tasks[:7])
    check_superposition(plan, M, M_ref, "compress")

    def sweep(tag):
        cur_ids, cur_seeds = plan.task_list()
        out = plan.new_output(wl.BF16)
        for t, s in zip(cur_ids, cur_seeds):
            plan.retrieve(t, w.lam, d_base, M, out=out, out_dtype=wl.BF16)
            ref = ro.retrieve(w.spec, w.storage, wl.BF16, t, s, w.lam, base, M_ref)
            check_model(out, ref, "%s task %d" % (tag, t))

    sweep("initial")
    plan.remove_model(3, d_base, d_tasks[3], M)
    ro.remove_model(w.spec, w.storage, 3, seeds[3], base, tasks[3], M_ref)
    check_superposition(plan, M, M_ref, "remove 3")
    sweep("after remove")
    plan.add_model(7, 100, d_base, d_tasks[7], M)
    ro.add_model(w.spec, w.storage, 7, 100, base, tasks[7], M_ref)
    check_superposition(plan, M, M_ref, "add 7")
    sweep("after add")
    torch.cuda.synchronize()
    plan.close()


def test_flan_t5_shaped_full_and_lora_variant():
    w = wl.flan_t5_base()
    base, tasks = wl.model_set(w)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w)
    M = plan.compress(d_base, d_tasks)
    M_ref = ro.compress(w.spec, w.storage, w.task_ids, w.seeds, base, tasks)
    check_superposition(plan, M, M_ref, "compress")
    for t in (0, 5):
        out = plan.retrieve(t, w.lam, d_base, M)
        ref = ro.retrieve(w.spec, w.storage, wl.F32, t, w.seeds[t], w.lam, base, M_ref)
        check_model(out, ref, "retrieve %d" % t)
    plan.close()
    del d_tasks, tasks, M
    # rank-16 adapters on q and v of every attention module, materialised, plan over those 72 matrices only
    targets = wl.flan_t5_lora_targets(w)
    assert len(targets) == 72
    wlora = wl.subset(w, targets, "flan_t5_base_lora")
    deltas = [[wl.lora_delta_layer(wlora, l, t) for l in range(wlora.n_layers)] for t in wlora.task_ids]
    lbase = [base[l] for l in targets]
    plan = randes.Plan.from_workload(wlora)
    M = plan.compress(None, [model_to_dev(d) for d in deltas])
    M_ref = ro.compress(wlora.spec, wlora.storage, wlora.task_ids, wlora.seeds, None, deltas)
    check_superposition(plan, M, M_ref, "lora compress")
    out = plan.retrieve(2, w.lam, model_to_dev(lbase), M)
    ref = ro.retrieve(wlora.spec, wlora.storage, wl.F32, 2, wlora.seeds[2], w.lam, lbase, M_ref)
    check_model(out, ref, "lora retrieve")
    plan.close()
    # the other form of the same case: the plan of the WHOLE model, every layer without an adapter given as a zero
    # tensor (one zero tensor per shape, shared by all tasks).  M is zero there, and retrieval returns W_0 itself.
    is_target = set(targets)
    zeros_h, zeros_d = {}, {}
    for l in range(w.n_layers):
        shape = (w.rows[l], w.cols[l])
        if l not in is_target and shape not in zeros_h:
            zeros_h[shape] = np.zeros(shape, dtype=np.float32)
            zeros_d[shape] = to_dev(zeros_h[shape])
    pos = {l: k for k, l in enumerate(targets)}
    full_h = [[deltas[i][pos[l]] if l in is_target else zeros_h[(w.rows[l], w.cols[l])] for l in range(w.n_layers)]
              for i in range(w.n_tasks)]
    d_deltas = [model_to_dev(d) for d in deltas]
    full_d = [[d_deltas[i][pos[l]] if l in is_target else zeros_d[(w.rows[l], w.cols[l])] for l in range(w.n_layers)]
              for i in range(w.n_tasks)]
    plan = randes.Plan.from_workload(w)
    M = plan.compress(None, full_d)
    M_ref = ro.compress(w.spec, w.storage, w.task_ids, w.seeds, None, full_h)
    check_superposition(plan, M, M_ref, "lora compress, whole model with zero tensors")
    out = plan.retrieve(2, w.lam, d_base, M)
    ref = ro.retrieve(w.spec, w.storage, wl.F32, 2, w.seeds[2], w.lam, base, M_ref)
    check_model(out, ref, "lora retrieve, whole model")
    for l in range(w.n_layers):
        if l not in is_target:
            # (equal as numbers: a -0.0 of W_0 comes back as +0.0, because fma(lambda, +0, -0) = +0)
            assert np.array_equal(from_dev(out[l]), base[l]), "layer %d has no adapter: retrieval must return W_0" % l
    plan.close()
