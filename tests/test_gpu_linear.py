"""GPU parity of randes_linear (a linear layer on the retrieved weight, never written to memory; tensor cores)
against the CPU oracle's fp64 definition.

Tolerance: the kernel multiplies bf16 operands exactly and accumulates 2 * cols products per output in fp32, in an
order the hardware chooses, then applies lambda with one fused multiply-add; any such evaluation differs from the
exact sum by at most 2 * cols * 2^-24 * sum_c |x| (|W_0| + |lambda M|) (plus one rounding of the result)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import randes_oracle as ro                      # noqa: E402
from paper_2505_11204_b200 import build, randes, workloads as wl   # noqa: E402
from gpu_util import model_to_dev, to_dev, check_superposition   # noqa: E402

S, F = wl.SHUFFLE, wl.FLIP


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _workload(shapes, flags, n_tasks=3):
    names, rows, cols, group = [], [], [], []
    maxg = max(s[2] for s in shapes)
    for k in range(maxg):
        for g, (r, c, n) in enumerate(shapes):
            if k < n:
                names.append("g%d.%d" % (g, k)); rows.append(r); cols.append(c); group.append(g)
    return wl.Workload(name="linear-case", layer_names=names, rows=rows, cols=cols, group=group, gflags=list(flags),
                       storage=wl.BF16, n_tasks=n_tasks, task_ids=[3, 0, 8][:n_tasks], seeds=[42, 43, 2**35 + 1][:n_tasks],
                       scale=1e-3, lam=0.3, data_seed=21)


def _bf16_normal(rng, shape):
    return wl.to_bf16_bits(rng.standard_normal(shape).astype(np.float32))


def _run(w, token_counts, layers=None):
    ids, seeds = list(w.task_ids), list(w.seeds)
    base, tasks = wl.model_set(w, ids)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w, max_tasks=len(ids), m_dtype=wl.BF16)
    M_dev = plan.compress(d_base, d_tasks)
    M_ref = ro.compress(w.spec, w.storage, ids, seeds, base, tasks, m_dtype=wl.BF16)
    check_superposition(plan, M_dev, M_ref, "compress")
    rng = np.random.default_rng(5)
    before = randes.randes_linear_giveups()
    for p in (range(w.n_layers) if layers is None else layers):
        rows, cols = w.rows[p], w.cols[p]
        for n_tok in token_counts:
            for t, s in zip(ids, seeds):
                x = _bf16_normal(rng, (n_tok, cols))
                y = torch.full((n_tok, rows), float("nan"), dtype=torch.float32, device="cuda")
                plan.linear(t, w.lam, p, to_dev(x), d_base, M_dev, y=y)
                y_ref, y_abs = ro.linear(w.spec, w.storage, t, s, w.lam, p, x, base, M_ref, m_dtype=wl.BF16)
                got = y.cpu().numpy().astype(np.float64)
                tol = (2 * cols + 2) * 2.0 ** -24 * y_abs + 1e-30
                bad = np.abs(got - y_ref) > tol
                assert not bad.any(), "layer %d (%dx%d), %d tokens, task %d: %d outputs off, worst %.3g x tolerance" % (
                    p, rows, cols, n_tok, t, int(bad.sum()), float(np.nanmax(np.abs(got - y_ref) / tol)))
    torch.cuda.synchronize()
    assert randes.randes_linear_giveups() == before
    plan.close()


def test_linear_small_shapes_ragged_tokens_and_features():
    # one k-step, several k-steps with a ragged last one, feature and token counts off the 128-tile
    w = _workload([(128, 64, 3), (200, 192, 2), (72, 520, 3), (1, 256, 1)], [S | F, S | F, F, F])
    _run(w, [1, 37, 128, 300])


def test_linear_bf16_output_is_the_fp32_result_rounded_once():
    w = _workload([(200, 192, 2), (7, 72, 2)], [S | F, F], n_tasks=2)
    ids, seeds = list(w.task_ids), list(w.seeds)
    base, tasks = wl.model_set(w, ids)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w, max_tasks=2, m_dtype=wl.BF16)
    M_dev = plan.compress(d_base, d_tasks)
    rng = np.random.default_rng(6)
    for p in range(w.n_layers):
        x = to_dev(_bf16_normal(rng, (150, w.cols[p])))
        y32 = plan.linear(ids[0], w.lam, p, x, d_base, M_dev)
        y16 = plan.linear(ids[0], w.lam, p, x, d_base, M_dev, y_dtype=wl.BF16)
        assert y16.dtype == torch.bfloat16
        assert torch.equal(y16, y32.to(torch.bfloat16))           # same accumulators, one rounding to nearest even
    assert randes.randes_linear_giveups() == 0
    plan.close()


def test_linear_without_flip_and_without_shuffle():
    w = _workload([(136, 128, 3), (64, 72, 2)], [S, 0])
    _run(w, [5, 130])


def test_linear_blocks_of_256_tokens():
    # enough tiles (16 feature tiles x 10 blocks of 256 tokens >= the SM count) for the 256-token CTA, whose second
    # block of 128 tokens has accumulators of its own; ragged token count, ragged last k-step, bf16 and fp32 output
    w = _workload([(2048, 136, 2)], [S | F], n_tasks=2)
    _run(w, [2500], layers=[0])
    ids = list(w.task_ids)
    base, tasks = wl.model_set(w, ids)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w, max_tasks=2, m_dtype=wl.BF16)
    M_dev = plan.compress(d_base, d_tasks)
    x = to_dev(_bf16_normal(np.random.default_rng(8), (2500, 136)))
    y32 = plan.linear(ids[1], w.lam, 1, x, d_base, M_dev)
    y16 = plan.linear(ids[1], w.lam, 1, x, d_base, M_dev, y_dtype=wl.BF16)
    assert torch.equal(y16, y32.to(torch.bfloat16))
    plan.close()


def test_linear_wide_layer_many_k_steps():
    # 16 k-steps: every stage of the ring is reused several times
    w = _workload([(384, 1024, 2)], [S | F], n_tasks=2)
    _run(w, [257], layers=[1])


def test_linear_unaligned_output_zero_tokens_and_host_only_plan():
    """y only 4-byte aligned (element-wise stores), no tokens (nothing launched), and a plan built without a device
    workspace (the call needs none)."""
    w = _workload([(136, 128, 2)], [S | F], n_tasks=2)
    ids, seeds = list(w.task_ids), list(w.seeds)
    base, tasks = wl.model_set(w, ids)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w, max_tasks=2, m_dtype=wl.BF16)
    M_dev = plan.compress(d_base, d_tasks)
    M_ref = ro.compress(w.spec, w.storage, ids, seeds, base, tasks, m_dtype=wl.BF16)
    host_plan = randes.Plan.from_workload(w, max_tasks=2, m_dtype=wl.BF16, host_only=True)
    x = _bf16_normal(np.random.default_rng(9), (45, 128))
    buf = torch.full((45 * 136 + 1,), float("nan"), dtype=torch.float32, device="cuda")
    y = buf[1:].view(45, 136)                                  # 4 bytes past a 16-byte boundary
    before = randes.randes_launch_count()
    host_plan.linear(ids[1], 0.3, 1, to_dev(x), d_base, M_dev, y=y)
    assert randes.randes_launch_count() == before + 1
    y_ref, y_abs = ro.linear(w.spec, w.storage, ids[1], seeds[1], 0.3, 1, x, base, M_ref, m_dtype=wl.BF16)
    assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - y_ref) <= (2 * 128 + 2) * 2.0 ** -24 * y_abs + 1e-30)
    assert bool(torch.isnan(buf[0]))                           # nothing before y was written
    empty = torch.zeros((0, 128), dtype=torch.bfloat16, device="cuda")
    randes.randes_linear(plan.handle, ids[0], 0.3, 0, empty, 0, randes.ptr_array(d_base), M_dev, y, torch.cuda.current_stream().cuda_stream, wl.F32)
    assert randes.randes_launch_count() == before + 1          # no tokens: no launch
    with pytest.raises(randes.RandesError) as e:
        plan.linear(77, 0.3, 0, to_dev(x), d_base, M_dev)
    assert e.value.code == randes.UNKNOWN_TASK
    assert randes.randes_linear_giveups() == 0
    plan.close(); host_plan.close()


def test_linear_rejects_what_it_cannot_run():
    w = _workload([(16, 12, 1)], [F], n_tasks=1)           # cols not a multiple of 8
    base, tasks = wl.model_set(w, w.task_ids)
    d_base = model_to_dev(base)
    plan = randes.Plan.from_workload(w, max_tasks=1, m_dtype=wl.BF16)
    M = plan.new_superposition()
    x = torch.zeros((4, 12), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(randes.RandesError) as e:
        plan.linear(w.task_ids[0], 0.3, 0, x, d_base, M)
    assert e.value.code == randes.INVALID_ARGUMENT
    plan.close()
    w32 = wl.toy()
    plan32 = randes.Plan.from_workload(w32, max_tasks=4)
    b32 = model_to_dev(wl.model_set(w32, [])[0])
    with pytest.raises(randes.RandesError) as e:
        plan32.linear(0, 1.0, 0, torch.zeros((4, 512), dtype=torch.bfloat16, device="cuda"), b32, plan32.new_superposition())
    assert e.value.code == randes.UNSUPPORTED_DTYPE
    plan32.close()
