"""GPU parity of randes_linear (a linear layer on the retrieved weight, never written to memory; tensor cores)
against the CPU oracle's fp64 definition.

Two kinds of comparison.

* Dyadic inputs (x, W_0, M multiples of 1/16 of magnitude <= 1/2, lambda = 1/4): every product and every partial sum
  of the 2 * cols products is exactly representable in fp32, whatever order the tensor core adds them in, so the
  kernel must return the bits of the oracle's fp64 result.  A wrong sign, a wrong slot, a stale or half-flipped tile
  changes the exact sum and fails the comparison.
* Gaussian inputs: the kernel multiplies bf16 operands exactly and accumulates 2 * cols products per output in fp32
  in an order the hardware chooses, then applies lambda with one fused multiply-add.  The worst case of such an
  evaluation is (2 * cols + 2) * 2^-24 * y_abs with y_abs = sum_c |x| (|W_0| + |lambda M|); that bound grows like
  cols^2 in absolute terms and would hide a whole wrong column at wide layers.  The accepted tolerance is therefore
  the random-walk form sqrt(2 * cols + 2) * 2^-24 * y_abs: each of the n = 2 * cols additions errs by at most
  2^-24 of a partial sum, partial sums of these zero-mean products stay near y_abs / sqrt(n), and independent errors
  add in quadrature, so the bound sits far out in the tail (and still several times above an accumulation that
  truncates instead of rounding, whose bias adds linearly over the cols / 8 accumulator updates).  Measured on
  B200 at 64 to 4096 columns, the worst error of 76 800 outputs was 0.09 to 0.17 of this tolerance, growing like
  sqrt(cols) as the model says.  At every tested width the test also
  shows that it can see one wrong column: the oracle is run again with the sign of one column of M flipped, and the
  kernel's result must NOT pass against that."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import randes_oracle as ro                      # noqa: E402
from paper_2505_11204_b200 import build, randes, workloads as wl   # noqa: E402
from gpu_util import model_to_dev, to_dev, check_superposition, assert_bits_equal   # noqa: E402

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


def _tolerance(cols, y_abs):
    return np.sqrt(2.0 * cols + 2.0) * 2.0 ** -24 * y_abs + 1e-30


def _flip_one_column(M_ref, slot, col):
    """A copy of the oracle's superposition with the sign of one column of one slot flipped (bf16 bit patterns)."""
    bad = [m for m in M_ref]
    bad[slot] = M_ref[slot].copy()
    bad[slot][:, col] ^= np.uint16(0x8000)
    return bad


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
                tol = _tolerance(cols, y_abs)
                bad = np.abs(got - y_ref) > tol
                assert not bad.any(), "layer %d (%dx%d), %d tokens, task %d: %d outputs off, worst %.3g x tolerance" % (
                    p, rows, cols, n_tok, t, int(bad.sum()), float(np.nanmax(np.abs(got - y_ref) / tol)))
                # the tolerance can see one wrong column: a planted sign error in the oracle must not pass
                slot = int(ro.task_tables(w.spec, s, t)[1][p])
                if rows * n_tok >= 64 and (w.gflags[w.group[p]] & F):
                    col = int(rng.integers(0, cols))
                    y_bad, _ = ro.linear(w.spec, w.storage, t, s, w.lam, p, x, base, _flip_one_column(M_ref, slot, col), m_dtype=wl.BF16)
                    assert (np.abs(got - y_bad) > tol).any(), "layer %d (%dx%d): a wrong sign in column %d passes" % (p, rows, cols, col)
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
    giveups = randes.randes_linear_giveups()
    for p in range(w.n_layers):
        x = to_dev(_bf16_normal(rng, (150, w.cols[p])))
        y32 = plan.linear(ids[0], w.lam, p, x, d_base, M_dev)
        y16 = plan.linear(ids[0], w.lam, p, x, d_base, M_dev, y_dtype=wl.BF16)
        assert y16.dtype == torch.bfloat16
        assert torch.equal(y16, y32.to(torch.bfloat16))           # same accumulators, one rounding to nearest even
    assert randes.randes_linear_giveups() == giveups
    plan.close()


def test_linear_without_flip_and_without_shuffle():
    w = _workload([(136, 128, 3), (64, 72, 2)], [S, 0])
    _run(w, [5, 130])


def test_linear_blocks_of_256_tokens():
    # 16 feature tiles x 9 blocks of 256 tokens (one wave of 256-token CTAs, whose second block of 128 tokens has
    # accumulators of its own) and the ragged rest in 128-token CTAs; ragged last k-step, bf16 and fp32 output
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


def _dyadic_bits(rng, shape, kmax=8):
    """Multiples of 1/16 in [-kmax/16, kmax/16] as bf16 bit patterns (exact in bf16)."""
    return wl.to_bf16_bits((rng.integers(-kmax, kmax + 1, size=shape) / 16.0).astype(np.float32))


def _lead_tokens(rows, n_tok):
    """The library's choice of CTA shapes: the first `lead` tokens (a multiple of 256, or all of them) go to 256-token
    tiles, the rest to 128-token tiles; a 128-token tile costs about 3/4 of a 256-token tile, and the split with the lowest
    sum of (number of waves over the SMs) x (cost of a tile) wins, the larger lead on a tie."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    feature_tiles = (rows + 127) // 128
    best, lead = None, 0
    for b in range((n_tok + 255) // 256 + 1):
        rest = max(0, n_tok - 256 * b)
        cost = -(-feature_tiles * b // sms) * 4 + -(-feature_tiles * ((rest + 127) // 128) // sms) * 3
        if best is None or cost <= best:
            best, lead = cost, min(256 * b, n_tok)
    return lead


def _run_dyadic(shape, gflag, n_tok, sample_tokens, want_lead, lam=0.25, members=2):
    """Bit equality with the oracle on dyadic inputs: layer [rows, cols], `members` same-shape layers in one group
    (so that the shuffle picks a slot), x [n_tok, cols].  The oracle runs on `sample_tokens` rows of x; every row
    is also checked against an fp32 library product on the weight formed from the oracle's slot and sign row
    (exact for these inputs in any order, so it must give the same bits: a check that holds at any size)."""
    rows, cols = shape
    w = _workload([(rows, cols, members)], [gflag], n_tasks=2)
    ids, seeds = list(w.task_ids), list(w.seeds)
    assert _lead_tokens(rows, n_tok) == want_lead                          # tokens covered by 256-token tiles
    n_k = (cols + 63) // 64
    assert n_k >= (2 * 3 + 1 if want_lead else 2 * 4 + 1), "every stage of the operand ring must be reused"
    rng = np.random.default_rng(rows * 7 + cols)
    base = [_dyadic_bits(rng, (rows, cols)) for _ in range(w.n_layers)]
    M_ref = [_dyadic_bits(rng, (rows, cols)) for _ in range(w.n_layers)]
    d_base = model_to_dev(base)
    plan = randes.Plan.from_workload(w, max_tasks=2, m_dtype=wl.BF16)
    M_dev = plan.new_superposition()
    M_dev.zero_()
    for l in range(w.n_layers):
        plan.slot(M_dev, l).copy_(to_dev(M_ref[l]))
    x = _dyadic_bits(rng, (n_tok, cols))
    d_x = to_dev(x)
    before = randes.randes_linear_giveups()
    sample = sorted(set(int(t) for t in sample_tokens if 0 <= t < n_tok))
    for p in range(w.n_layers):
        for t, s in zip(ids, seeds):
            y = torch.full((n_tok, rows), float("nan"), dtype=torch.float32, device="cuda")
            launches = randes.randes_launch_count()
            plan.linear(t, lam, p, d_x, d_base, M_dev, y=y)
            assert randes.randes_launch_count() - launches == (want_lead > 0) + (want_lead < n_tok)
            got = y.cpu().numpy()
            y_ref, _ = ro.linear(w.spec, w.storage, t, s, lam, p, np.ascontiguousarray(x[sample]), base, M_ref, m_dtype=wl.BF16)
            want = y_ref.astype(np.float32)
            assert np.array_equal(want.astype(np.float64), y_ref)          # the exact result is an fp32 number
            assert_bits_equal(got[sample], want, "dyadic linear, layer %d task %d, sampled tokens" % (p, t))
            # all tokens: the weight formed from the oracle's tables, multiplied by a library GEMM in fp32
            slot = int(ro.task_tables(w.spec, s, t)[1][p])
            sg = ro.sign_row(s, t, slot, cols).astype(np.float32) if (gflag & F) else np.ones(cols, np.float32)
            what = wl.bf16_bits_to_f32(base[p]) + np.float32(lam) * sg[None, :] * wl.bf16_bits_to_f32(M_ref[slot])
            full = (d_x.float() @ torch.from_numpy(what).cuda().T).cpu().numpy()
            assert np.array_equal(full[sample], want)                      # the library product agrees with the oracle
            assert_bits_equal(got, full, "dyadic linear, layer %d task %d, all tokens" % (p, t))
    torch.cuda.synchronize()
    assert randes.randes_linear_giveups() == before
    plan.close()


def _block_edges(n_tok):
    """Token rows at both 128-token halves of the first, a middle and the last 256-token block."""
    edges = [0, 1, 31, 32, 95, 127, 128, 129, 191, 255, 256, 257]
    mid = (n_tok // 512) * 256
    last = ((n_tok - 1) // 256) * 256
    for b in (mid, last):
        edges += [b, b + 1, b + 127, b + 128, b + 129, b + 255]
    return edges + [n_tok - 1, n_tok - 2]


def test_linear_bit_exact_on_dyadic_inputs_in_the_benchmarked_shape():
    # [1024 x 4096] x 8192 tokens: 256-token CTAs, 64 k-steps through the 3-stage ring (every stage reused 21 times)
    _run_dyadic((1024, 4096), S | F, 8192, _block_edges(8192), want_lead=8192, members=2)


def test_linear_bit_exact_on_dyadic_inputs_256_token_blocks_ragged():
    # 256-token CTAs alone (16 feature tiles x 9 token blocks: one wave) with a ragged last k-step (648 = 10 x 64 + 8),
    # ragged token and feature counts
    _run_dyadic((2000, 648), S | F, 2300, _block_edges(2300), want_lead=2300)


def test_linear_bit_exact_on_dyadic_inputs_two_tile_shapes_in_one_call():
    # the first 2304 tokens in one wave of 256-token CTAs, the ragged rest in 128-token CTAs (a second launch whose
    # token offset is not zero); with and without flip
    _run_dyadic((2000, 648), S | F, 2500, _block_edges(2500) + list(range(2296, 2312)), want_lead=2304)
    _run_dyadic((2048, 456), S, 2400, _block_edges(2400) + list(range(2296, 2312)), want_lead=2304)


def test_linear_bit_exact_on_dyadic_inputs_two_tile_shapes_vit_b32_mlp():
    # [768 x 3072] x 8192 tokens: 6144 tokens in one wave of 144 256-token CTAs, 2048 tokens in 96 128-token CTAs
    edges = _block_edges(8192) + [6143, 6144, 6145, 6271, 6272, 8063, 8064]
    _run_dyadic((768, 3072), S | F, 8192, edges, want_lead=6144, members=2)


def test_linear_bit_exact_on_dyadic_inputs_128_token_blocks():
    # 128-token CTAs (too few tiles for the wider shape), 17 and 9 k-steps through the 4-stage ring, ragged last k-step
    _run_dyadic((384, 1032), S | F, 257, range(257), want_lead=0)
    _run_dyadic((200, 576), S, 130, range(130), want_lead=0)
    _run_dyadic((136, 4096), F, 100, range(100), want_lead=0, members=1)


def test_linear_gaussian_inputs_wide_layers_see_one_wrong_column():
    # the random-walk tolerance at the widths of the paper-shaped sets, each with the planted wrong-sign column
    w = _workload([(256, 3072, 2), (128, 4096, 2)], [S | F, S | F], n_tasks=2)
    _run(w, [192])


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
    giveups = randes.randes_linear_giveups()
    host_plan.linear(ids[1], 0.3, 1, to_dev(x), d_base, M_dev, y=y)
    assert randes.randes_launch_count() == before + 1
    y_ref, y_abs = ro.linear(w.spec, w.storage, ids[1], seeds[1], 0.3, 1, x, base, M_ref, m_dtype=wl.BF16)
    assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - y_ref) <= _tolerance(128, y_abs))
    assert bool(torch.isnan(buf[0]))                           # nothing before y was written
    empty = torch.zeros((0, 128), dtype=torch.bfloat16, device="cuda")
    randes.randes_linear(plan.handle, ids[0], 0.3, 0, empty, 0, randes.ptr_array(d_base), M_dev, y, torch.cuda.current_stream().cuda_stream, wl.F32)
    assert randes.randes_launch_count() == before + 1          # no tokens: no launch
    with pytest.raises(randes.RandesError) as e:
        plan.linear(77, 0.3, 0, to_dev(x), d_base, M_dev)
    assert e.value.code == randes.UNKNOWN_TASK
    assert randes.randes_linear_giveups() == giveups
    plan.close(); host_plan.close()


@pytest.mark.parametrize("gflag", [S | F, S])
def test_linear_behind_a_gate_that_nothing_opens_gives_up_and_leaves_the_context_usable(gflag):
    """Failure detection of the one kernel that waits.  The gated call makes every thread block wait for a device
    word; here nothing sets it, so the (3 ms) wait runs out in all 3 x 2 blocks: each must return without a copy,
    a product or a store (y keeps its poison), count itself in randes_linear_giveups, and leave the context healthy.
    With the gate open the same call computes the layer, and the ordinary call still works afterwards."""
    w = _workload([(300, 192, 2)], [gflag], n_tasks=2)
    ids, seeds = list(w.task_ids), list(w.seeds)
    base, tasks = wl.model_set(w, ids)
    d_base, d_tasks = model_to_dev(base), [model_to_dev(t) for t in tasks]
    plan = randes.Plan.from_workload(w, max_tasks=2, m_dtype=wl.BF16)
    M_dev = plan.compress(d_base, d_tasks)
    M_ref = ro.compress(w.spec, w.storage, ids, seeds, base, tasks, m_dtype=wl.BF16)
    n_tok, p, t, s = 200, 1, ids[1], seeds[1]
    x = _bf16_normal(np.random.default_rng(12), (n_tok, 192))
    d_x, p_base = to_dev(x), randes.ptr_array(d_base)
    stream = torch.cuda.current_stream().cuda_stream
    gate = torch.zeros(1, dtype=torch.int32, device="cuda")
    guard = torch.full((n_tok + 2, 300), float("nan"), dtype=torch.float32, device="cuda")
    y = guard[1:-1]
    before = randes.randes_linear_giveups()
    randes.randes_linear_gated(plan.handle, t, w.lam, p, d_x, n_tok, p_base, M_dev, y, gate, 3_000_000, stream)
    torch.cuda.synchronize()                                   # returns: the kernel ended by itself
    assert randes.randes_linear_giveups() - before == 3 * 2    # ceil(300 / 128) feature tiles x ceil(200 / 128) token blocks
    assert bool(torch.isnan(guard).all())                      # nothing was written, inside or around y
    gate.fill_(1)
    y_ref, y_abs = ro.linear(w.spec, w.storage, t, s, w.lam, p, x, base, M_ref, m_dtype=wl.BF16)
    tol = _tolerance(192, y_abs)
    randes.randes_linear_gated(plan.handle, t, w.lam, p, d_x, n_tok, p_base, M_dev, y, gate, 0, stream)
    assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - y_ref) <= tol)
    y2 = plan.linear(t, w.lam, p, d_x, d_base, M_dev)
    assert torch.equal(y2, y)                                  # the ordinary call, same bits
    assert bool(torch.isnan(guard[0]).all()) and bool(torch.isnan(guard[-1]).all())
    assert randes.randes_linear_giveups() - before == 6        # no further give-ups
    with pytest.raises(randes.RandesError) as e:
        randes.randes_linear_gated(plan.handle, t, w.lam, p, d_x, n_tok, p_base, M_dev, y, None, 0, stream)
    assert e.value.code == randes.INVALID_ARGUMENT
    plan.close()


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
    w8 = _workload([(16, 8, 1)], [F], n_tasks=1)
    d8 = model_to_dev(wl.model_set(w8, w8.task_ids)[0])
    plan8 = randes.Plan.from_workload(w8, max_tasks=1, m_dtype=wl.BF16)
    M8 = plan8.new_superposition()
    x8 = torch.zeros((4, 8), dtype=torch.bfloat16, device="cuda")
    y8 = torch.zeros((4, 16), dtype=torch.float32, device="cuda")
    before = randes.randes_launch_count()
    with pytest.raises(randes.RandesError) as e:           # more tokens than the grid can hold: refused before any launch
        randes.randes_linear(plan8.handle, w8.task_ids[0], 0.3, 0, x8, 65535 * 128 + 1, randes.ptr_array(d8), M8, y8,
                             torch.cuda.current_stream().cuda_stream, wl.F32)
    assert e.value.code == randes.INVALID_ARGUMENT and randes.randes_launch_count() == before
    plan8.close()
    w32 = wl.toy()
    plan32 = randes.Plan.from_workload(w32, max_tasks=4)
    b32 = model_to_dev(wl.model_set(w32, [])[0])
    with pytest.raises(randes.RandesError) as e:
        plan32.linear(0, 1.0, 0, torch.zeros((4, 512), dtype=torch.bfloat16, device="cuda"), b32, plan32.new_superposition())
    assert e.value.code == randes.UNSUPPORTED_DTYPE
    plan32.close()
