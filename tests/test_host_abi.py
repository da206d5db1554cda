"""Host-side checks of the C-ABI library that need no GPU: it loads, exports what
the header declares, validates arguments, and draws the same permutations as
the oracle (two independent implementations of the seed -> sigma rule)."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import randes_oracle as ro
from paper_2505_11204_b200 import build, randes, workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "randes.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(randes_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 15
    L = ctypes.CDLL(randes.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n
    assert sorted(randes.EXPORTS) == names


def test_host_only_plan_tables_match_oracle():
    for w in (wl.toy(), wl.vit_b32(), wl.gpt2_small(), wl.flan_t5_base(), wl.vit_l14()):
        ids = list(range(w.n_tasks)) + [1000]
        seeds = w.seeds + [2**63 + 12345]
        p = randes.Plan(w.rows, w.cols, w.group, w.gflags, storage=w.storage, task_ids=ids, seeds=seeds,
                        host_only=True)
        for t, s in zip(ids, seeds):
            src, pos = p.task_tables(t)
            osrc, opos = ro.task_tables(w.spec, s, t)
            assert src == osrc.tolist() and pos == opos.tolist()
        assert p.task_list() == (ids, seeds)
        p.close()


def test_sigma_agrees_for_many_seeds_and_group_sizes():
    rng = np.random.default_rng(5)
    for _ in range(300):
        G = int(rng.integers(1, 40))
        seed = int(rng.integers(0, 2**63))
        tid = int(rng.integers(0, 2**32))
        n_pad = int(rng.integers(0, 3))   # singleton groups before the one under test shift its index
        rows = [1] * n_pad + [2] * G
        cols = [3 + i for i in range(n_pad)] + [8] * G
        group = list(range(n_pad)) + [n_pad] * G
        gflags = [randes.FLIP] * n_pad + [randes.SHUFFLE]
        p = randes.Plan(rows, cols, group, gflags, task_ids=[tid], seeds=[seed], host_only=True)
        src, pos = p.task_tables(tid)
        sigma = ro.permutation(seed, tid, n_pad, G)
        assert src[n_pad:] == [n_pad + int(s) for s in sigma]
        assert all(pos[src[l]] == l for l in range(len(rows)))
        p.close()


def test_shift_and_skip_tables_match_oracle():
    S, F, SH = randes.SHUFFLE, randes.FLIP, randes.SHIFT
    rows = [2] * 9 + [1] * 7
    cols = [8] * 9 + [5] * 7
    group = [0] * 9 + [1] * 7
    for gflags in ([SH | F, SH], [S | F | randes.SKIP(2), SH | randes.SKIP(3)], [F | randes.SKIP(4), S | randes.SKIP(2)]):
        ids, seeds = [0, 1, 5, 11], [3, 4, 5, 6]
        p = randes.Plan(rows, cols, group, gflags, task_ids=ids, seeds=seeds, host_only=True)
        for t, s in zip(ids, seeds):
            src, pos = p.task_tables(t)
            osrc, opos = ro.task_tables((rows, cols, group, gflags), s, t)
            assert src == osrc.tolist() and pos == opos.tolist()
        p.close()
    with pytest.raises(randes.RandesError) as e:
        randes.Plan(rows, cols, group, [S | SH, 0], task_ids=[0], seeds=[0], host_only=True)
    assert e.value.code == randes.INVALID_ARGUMENT


def test_superposition_layout_is_one_fp32_copy_independent_of_task_count():
    w = wl.vit_b32()
    p1 = randes.Plan.from_workload(w.with_tasks(1), host_only=True)
    p8 = randes.Plan.from_workload(w, host_only=True)
    assert p1.m_bytes == p8.m_bytes
    assert p1.offsets == p8.offsets
    assert all(o % 256 == 0 for o in p8.offsets)
    raw = 4 * w.n_params
    assert raw <= p8.m_bytes <= raw + 256 * w.n_layers
    for l in range(w.n_layers - 1):
        assert p8.offsets[l + 1] - p8.offsets[l] >= 4 * w.rows[l] * w.cols[l]
    assert randes.randes_layer_offset(p8.handle, w.n_layers) == 2**64 - 1
    # a bf16 superposition takes half the bytes (up to slot padding)
    ph = randes.Plan.from_workload(w, host_only=True, m_dtype=randes.BF16)
    assert 2 * w.n_params <= ph.m_bytes <= 2 * w.n_params + 256 * w.n_layers and all(o % 256 == 0 for o in ph.offsets)
    # memory figures of the paper's first results table: 0.564 -> 0.89 (GiB) is one fp32 copy of the encoder
    assert abs(0.564 + raw / 2**30 - 0.89) < 0.005


def test_workspace_size_grows_with_capacity_and_rejects_bad_input():
    w = wl.toy()
    p = randes.Plan.from_workload(w, host_only=True)
    a = randes.randes_plan_workspace_bytes(p._layers, w.n_layers, 4)
    b = randes.randes_plan_workspace_bytes(p._layers, w.n_layers, 64)
    assert 0 < a < b
    assert randes.randes_plan_workspace_bytes(p._layers, w.n_layers, 0) == 0
    assert randes.randes_plan_workspace_bytes(None, 3, 4) == 0
    # the group-aware figure: the same without a RANDES_GAUSS group; with one, larger by at least the table of factors
    # (4 bytes per task and column of every layer)
    n_groups = len(w.gflags)
    assert randes.randes_plan_workspace_bytes_groups(p._layers, w.n_layers, p._groups, n_groups, 4) == a
    assert randes.randes_plan_workspace_bytes_groups(p._layers, w.n_layers, None, 0, 4) == a
    assert randes.randes_plan_workspace_bytes_groups(p._layers, w.n_layers, p._groups, n_groups, 0) == 0
    wg = wl.Workload(**{**w.__dict__})
    wg.gflags = [(f & ~wl.FLIP) | randes.GAUSS if f & wl.FLIP else f for f in w.gflags]
    assert any(f & randes.GAUSS for f in wg.gflags)
    pg = randes.Plan.from_workload(wg, host_only=True)
    for cap in (4, 64):
        plain = randes.randes_plan_workspace_bytes(pg._layers, wg.n_layers, cap)
        with_table = randes.randes_plan_workspace_bytes_groups(pg._layers, wg.n_layers, pg._groups, n_groups, cap)
        assert with_table >= plain + 4 * cap * sum(wg.cols)
        assert with_table <= plain + 4 * cap * sum(c + 3 for c in wg.cols) + 4 * wg.n_layers + 1024


def test_plan_round_trips_through_its_serialized_form():
    w = wl.gpt2_small()
    gflags = list(w.gflags)
    gflags[2] |= randes.SKIP(2)
    p = randes.Plan(w.rows, w.cols, w.group, gflags, storage=w.storage, task_ids=[3, 0, 9], seeds=[2**63 + 1, 42, 7],
                    host_only=True, m_dtype=randes.BF16)
    blob = randes.randes_plan_serialize(p.handle)
    q = randes.randes_plan_deserialize(blob)
    try:
        assert randes.randes_num_layers(q) == w.n_layers and randes.randes_num_tasks(q) == 3
        assert randes.randes_superposition_bytes(q) == p.m_bytes
        L = w.n_layers
        for t in (3, 0, 9):
            a = (ctypes.c_uint32 * L)(); b = (ctypes.c_uint32 * L)()
            assert randes.lib().randes_task_tables(q, t, ctypes.addressof(a), ctypes.addressof(b)) == 0
            assert (list(a), list(b)) == p.task_tables(t)
        assert randes.randes_plan_serialize(q) == blob
        # a host-only plan already tells what workspace its device twin needs: no more than the a-priori figure
        need = randes.randes_plan_workspace_needed(q)
        assert 0 < need <= randes.randes_plan_workspace_needed(p.handle)       # (q holds room for its 3 tasks only)
        assert need <= randes.randes_plan_workspace_bytes_groups(p._layers, L, p._groups, len(gflags), 3)
        assert randes.randes_plan_workspace_needed(None) == 0
    finally:
        randes.randes_plan_destroy(q)
    for bad in (blob[:20], b"\0" * len(blob), blob[:-8]):
        with pytest.raises(randes.RandesError) as e:
            randes.randes_plan_deserialize(bad)
        assert e.value.code == randes.INVALID_ARGUMENT
    p.close()


def _expect(code, fn):
    with pytest.raises(randes.RandesError) as e:
        fn()
    assert e.value.code == code, (e.value.code, str(e.value))
    assert randes.randes_last_error()


def test_plan_argument_validation():
    S, F = randes.SHUFFLE, randes.FLIP
    mk = lambda **kw: randes.Plan(kw.get("rows", [2, 2]), kw.get("cols", [4, 4]), kw.get("group", [0, 0]),
                                  kw.get("gflags", [S | F]), storage=kw.get("storage", randes.F32),
                                  task_ids=kw.get("ids", [0]), seeds=kw.get("seeds", [1]),
                                  max_tasks=kw.get("max_tasks", 4), host_only=True)
    mk().close()
    _expect(randes.SHAPE_MISMATCH, lambda: mk(cols=[4, 5]))
    _expect(randes.DUPLICATE_TASK, lambda: mk(ids=[3, 3], seeds=[1, 2]))
    _expect(randes.INVALID_ARGUMENT, lambda: mk(group=[0, 1]))          # group id out of range
    _expect(randes.INVALID_ARGUMENT, lambda: mk(gflags=[8]))            # unknown flag bit
    _expect(randes.INVALID_ARGUMENT, lambda: mk(max_tasks=0, ids=[], seeds=[]))
    _expect(randes.INVALID_ARGUMENT, lambda: mk(ids=[0, 1, 2], seeds=[0, 1, 2], max_tasks=2))
    _expect(randes.UNSUPPORTED_DTYPE, lambda: mk(storage=7))
    _expect(randes.INVALID_ARGUMENT, lambda: mk(rows=[70000, 70000], cols=[70000, 70000]))   # >= 2^32 elements per layer
    with pytest.raises(randes.RandesError) as e:
        randes.Plan([2], [4], [0], [0], task_ids=[0], seeds=[1], host_only=True, m_dtype=5)
    assert e.value.code == randes.UNSUPPORTED_DTYPE
    p = mk()
    _expect(randes.UNKNOWN_TASK, lambda: p.task_tables(99))
    # a host-only plan cannot compute
    arr = (ctypes.c_void_p * 2)(256, 512)
    _expect(randes.INVALID_ARGUMENT, lambda: randes.randes_compress(p.handle, arr, arr, 256, None))
    _expect(randes.INVALID_ARGUMENT, lambda: randes.randes_retrieve(p.handle, 0, 1.0, randes.F32, arr, 256, arr, None))
    _expect(randes.INVALID_ARGUMENT, lambda: randes.randes_add_model(p.handle, 5, 5, arr, arr, 256, None))
    _expect(randes.INVALID_ARGUMENT, lambda: randes.randes_remove_model(p.handle, 0, arr, arr, 256, None))
    _expect(randes.INVALID_ARGUMENT, lambda: randes.randes_add_models(p.handle, [5, 6], [5, 6], arr, arr, 256, None))
    p.close()


def test_interference_norm_and_cosines_against_the_oracle():
    """randes_interference_norm / randes_pairwise_cosines (host entry points) against what the oracle gives:
    the norm of the interference is measured on the oracle's own retrieved model (Section 4, second display:
    What_t - W_0 - lambda d_t is the interference), the cosines on the transformed deltas themselves
    (a one-task compress is T_i d_i).  Dyadic inputs: the Gram matrix and every sum are exact."""
    S, F = randes.SHUFFLE, randes.FLIP
    rows, cols, group = [4, 2, 4, 2, 4, 2], [8, 5, 8, 5, 8, 5], [0, 1, 0, 1, 0, 1]
    spec = (rows, cols, group, [S | F, S])
    rng = np.random.default_rng(77)
    model = lambda: [(rng.integers(-512, 513, size=(r, c)) / 1024.0).astype(np.float32) for r, c in zip(rows, cols)]
    base = model()
    ids, seeds = [4, 0, 9, 2], [11, 12, 13, 14]
    tasks = [model() for _ in ids]
    G = ro.delta_gram(spec, ro.F32, ids, seeds, base, tasks)
    flat = lambda m: np.concatenate([np.asarray(a, dtype=np.float64).ravel() for a in m])
    M = ro.compress(spec, ro.F32, ids, seeds, base, tasks)
    for lam in (1.0, 0.25):
        for t in range(len(ids)):
            what = ro.retrieve(spec, ro.F32, ro.F32, ids[t], seeds[t], lam, base, M)
            inter = flat(what) - flat(base) - lam * (flat(tasks[t]) - flat(base))
            want = float(np.sqrt(inter @ inter))
            got = randes.randes_interference_norm(G, t, lam)
            assert abs(got - want) <= 4 * np.finfo(np.float64).eps * want, (t, got, want)
    X = [flat(ro.compress(spec, ro.F32, [i], [s], base, [tk])) for i, s, tk in zip(ids, seeds, tasks)]
    cos, mean = randes.randes_pairwise_cosines(G)
    n = len(ids)
    for j in range(n):
        for l in range(n):
            want = 1.0 if j == l else float(X[j] @ X[l]) / float(np.sqrt((X[j] @ X[j]) * (X[l] @ X[l])))
            assert abs(cos[j][l] - want) <= 1e-15, (j, l)
    pairs = [(j, l) for j in range(n) for l in range(j + 1, n)]
    assert abs(mean - sum(cos[j][l] for j, l in pairs) / len(pairs)) <= 1e-15
    _, mean_wo = randes.randes_pairwise_cosines(G, exclude=1)
    kept = [(j, l) for j, l in pairs if 1 not in (j, l)]
    assert abs(mean_wo - sum(cos[j][l] for j, l in kept) / len(kept)) <= 1e-15
    # degenerate inputs: one task (no pair, nothing interferes), a zero delta, bad arguments
    assert randes.randes_pairwise_cosines([[2.0]])[1] == 0.0
    assert randes.randes_interference_norm([[2.0]], 0, 1.0) == 0.0
    assert randes.randes_pairwise_cosines([[0.0, 0.0], [0.0, 4.0]])[0] == [[1.0, 0.0], [0.0, 1.0]]
    _expect(randes.INVALID_ARGUMENT, lambda: randes.randes_interference_norm(G, n, 1.0))
    _expect(randes.INVALID_ARGUMENT, lambda: randes.randes_pairwise_cosines(G, exclude=n))
    out = ctypes.c_double()
    assert randes.lib().randes_interference_norm(None, 2, 0, 1.0, ctypes.byref(out)) == randes.INVALID_ARGUMENT
    assert randes.lib().randes_pairwise_cosines(None, 2, -1, None, None) == randes.INVALID_ARGUMENT


def test_outputs_that_overlap_an_input_or_each_other_are_refused():
    """out may overlap neither base, nor M, nor another output tensor -- not even part-way.  The check runs on the
    host before anything is launched (shown here through the entry point that accepts a host-only plan)."""
    n, rows, cols = 3, 4, 8
    nbytes = rows * cols * 4
    plan = randes.Plan([rows] * n, [cols] * n, [0] * n, [randes.SHUFFLE | randes.FLIP], task_ids=[0], seeds=[1], host_only=True)
    arr = lambda xs: (ctypes.c_void_p * n)(*xs)
    base = arr([0x10000 + i * 0x1000 for i in range(n)])
    M = 0x100000
    call = lambda out: randes.randes_retrieve_static(plan.handle, 0, 1.0, randes.F32, base, M, arr(out), None)
    good = [0x20000 + i * 0x1000 for i in range(n)]
    cases = {
        "a base tensor": [good[0], 0x10000 + 0x1000 + nbytes - 4, good[2]],          # last element of base[1], from another layer
        "M": [good[0], good[1], M + plan.m_bytes - 4],
        "another output tensor": [good[0], good[0] + nbytes - 16, good[2]],
    }
    for what, out in cases.items():
        with pytest.raises(randes.RandesError) as e:
            call(out)
        assert e.value.code == randes.INVALID_ARGUMENT and what in str(e.value), (what, str(e.value))
    plan.close()


def test_every_plan_passes_its_self_check():
    """randes_plan_validate: permutations are bijections inside groups, slots of M are disjoint, and every tile
    list covers every (row, column block) of every layer exactly once -- on the five paper-shaped sets in both
    storage types, with the skip / shift / Gaussian-context variants, and on ragged random shapes."""
    S, F = randes.SHUFFLE, randes.FLIP
    for make in (wl.toy, wl.vit_b32, wl.gpt2_small, wl.flan_t5_base, wl.vit_l14):
        for storage in (wl.F32, wl.BF16):
            for m_dtype in (wl.F32, wl.BF16):
                w = make().with_storage(storage)
                p = randes.Plan.from_workload(w, host_only=True, m_dtype=m_dtype)
                randes.randes_plan_validate(p.handle)
                p.close()
    w = wl.vit_b32()
    for variant in (lambda f: f | randes.SKIP(2), lambda f: (f & ~S) | randes.SHIFT if f & S else f,
                    lambda f: (f & ~F) | randes.GAUSS if f & F else f):
        p = randes.Plan(w.rows, w.cols, w.group, [variant(f) for f in w.gflags], task_ids=[0, 5], seeds=[1, 2], host_only=True)
        randes.randes_plan_validate(p.handle)
        p.close()
    rng = np.random.default_rng(3)
    for _ in range(40):
        n_groups = int(rng.integers(1, 5))
        rows, cols, group = [], [], []
        for g in range(n_groups):
            r, c, n = int(rng.integers(1, 300)), int(rng.integers(1, 2100)), int(rng.integers(1, 30))
            rows += [r] * n; cols += [c] * n; group += [g] * n
        order = rng.permutation(len(rows))
        rows, cols, group = [rows[i] for i in order], [cols[i] for i in order], [group[i] for i in order]
        flags = [int(rng.choice([0, S, F, S | F])) for _ in range(n_groups)]
        p = randes.Plan(rows, cols, group, flags, storage=int(rng.integers(0, 2)), task_ids=[3, 9, 4], seeds=[7, 8, 9], host_only=True)
        randes.randes_plan_validate(p.handle)
        p.close()
    assert randes.lib().randes_plan_validate(None) == randes.INVALID_ARGUMENT


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(randes, "_lib", None)
    monkeypatch.setattr(randes, "LIB_PATH", str(tmp_path / "absent.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        randes.lib()
