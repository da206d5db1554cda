"""Pins of the CPU oracle to facts fixed by the paper and by mathematics.

Each test compares the oracle with something that is not the oracle: published
known-answer vectors, dense signed-permutation matrices built from the paper's
printed definitions, closed forms in exact rational arithmetic, library
routines, or statistical laws.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import randes_oracle as ro
from paper_2505_11204_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
SHUFFLE, FLIP = ro.SHUFFLE, ro.FLIP


# --------------------------------------------------------------------------- helpers
def tiny_spec(flags=SHUFFLE | FLIP, n_a=3, n_b=3, shape_a=(4, 8), shape_b=(2, 5)):
    """Two groups, interleaved in layer order, so that group-local and global
    indices differ."""
    rows, cols, group = [], [], []
    for k in range(max(n_a, n_b)):
        if k < n_a:
            rows.append(shape_a[0]); cols.append(shape_a[1]); group.append(0)
        if k < n_b:
            rows.append(shape_b[0]); cols.append(shape_b[1]); group.append(1)
    return (rows, cols, group, [flags, flags])


def rand_model(spec, rng, scale=1.0, dyadic=False):
    out = []
    for r, c in zip(spec[0], spec[1]):
        if dyadic:
            out.append((rng.integers(-1024, 1025, size=(r, c)) / 1024.0).astype(np.float32))
        else:
            out.append((rng.standard_normal((r, c)) * scale).astype(np.float32))
    return out


def members_of(spec, g):
    return [l for l, gg in enumerate(spec[2]) if gg == g]


def dense_transform(spec, seed, task_id):
    """T = D P as an explicit d x d matrix over the concatenated, flattened
    layers, built from the paper's definitions: (P delta)[slot k] =
    delta[sigma(k)] (Section 4.3, first display) and each slot's matrix
    right-multiplied by a +-1 diagonal (Section 4.4, first display)."""
    rows, cols, group, gflags = spec
    L = len(rows)
    sizes = [r * c for r, c in zip(rows, cols)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    d = int(offs[-1])
    P = np.zeros((d, d))
    # identity on every layer, then overwrite shuffled groups
    src_of_slot = list(range(L))
    takes_part = [False] * L
    for g, fl in enumerate(gflags):
        skip = max(1, (fl >> 8) & 0xFF)
        mem = members_of(spec, g)[::skip]          # every skip-th member of the group takes part
        for m in mem:
            takes_part[m] = True
        if len(mem) >= 2 and (fl & SHUFFLE):
            sigma = ro.permutation(seed, task_id, g, len(mem))
            for k, m in enumerate(mem):
                src_of_slot[m] = mem[int(sigma[k])]
        elif len(mem) >= 2 and (fl & ro.SHIFT):
            shift = 1 + task_id % (len(mem) - 1)   # one or more positions deeper, with wrap-around
            for k, m in enumerate(mem):
                src_of_slot[mem[(k + shift) % len(mem)]] = m
    for l in range(L):
        s = src_of_slot[l]
        P[offs[l]:offs[l + 1], offs[s]:offs[s + 1]] = np.eye(sizes[l])
    D = np.zeros((d, d))
    for l in range(L):
        if (gflags[group[l]] & FLIP) and takes_part[l]:
            diag = ro.sign_row(seed, task_id, l, cols[l]).astype(np.float64)
        elif (gflags[group[l]] & ro.GAUSS) and takes_part[l]:
            diag = np.array([ro.gauss(seed, task_id, l, c) for c in range(cols[l])], dtype=np.float64)
        else:
            diag = np.ones(cols[l])
        # vec(X diag(s)) for row-major X [rows, cols] = tile(s, rows) * vec(X)
        full = np.tile(diag, rows[l])
        D[offs[l]:offs[l + 1], offs[l]:offs[l + 1]] = np.diag(full)
    return D @ P, offs


def flat(model):
    return np.concatenate([np.asarray(a, dtype=np.float64).ravel() for a in model])


def unflat(v, spec, offs):
    return [v[offs[l]:offs[l + 1]].reshape(spec[0][l], spec[1][l]) for l in range(len(spec[0]))]


def round_fraction_to_f32(v: Fraction) -> np.float32:
    """Correctly rounded (nearest, ties to even) fp32 of an exact rational."""
    if v == 0:
        return np.float32(0.0)
    approx = np.float32(float(v))
    cands = {approx, np.nextafter(approx, np.float32(np.inf)), np.nextafter(approx, np.float32(-np.inf))}
    best = None
    for c in cands:
        err = abs(Fraction(float(c)) - v)
        even = (np.float32(c).view(np.uint32) & 1) == 0
        key = (err, 0 if even else 1)
        if best is None or key < best[0]:
            best = (key, np.float32(c))
    return best[1]


# --------------------------------------------------------------------------- Philox
def test_philox_known_answers():
    n = 0
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert ro.philox4x32_10(w[0:4], w[4:6]) == tuple(w[6:10])
        n += 1
    assert n == 3


def test_philox_is_a_bijection_of_the_counter_and_avalanches():
    # distinct counters -> distinct blocks (Philox is a permutation per key);
    # one flipped input bit changes about half of the 128 output bits
    rng = np.random.default_rng(1)
    seen = set()
    for n in range(2000):
        seen.add(ro.philox4x32_10((n, 0, 0, 0), (7, 9)))
    assert len(seen) == 2000
    flips = []
    for _ in range(300):
        ctr = [int(x) for x in rng.integers(0, 2**32, 4)]
        key = [int(x) for x in rng.integers(0, 2**32, 2)]
        a = ro.philox4x32_10(ctr, key)
        w = int(rng.integers(0, 6)); b = int(rng.integers(0, 32))
        if w < 4:
            ctr[w] ^= 1 << b
        else:
            key[w - 4] ^= 1 << b
        c = ro.philox4x32_10(ctr, key)
        flips.append(sum(bin(x ^ y).count("1") for x, y in zip(a, c)))
    assert 60 < np.mean(flips) < 68


# --------------------------------------------------------------------------- permutation
def test_sigma_is_a_bijection_and_tables_invert():
    for G in (1, 2, 3, 7, 24, 100):
        for seed in (0, 42, 2**40 + 5):
            s = ro.permutation(seed, 3, 1, G)
            assert sorted(s.tolist()) == list(range(G))
    w = wl.vit_b32()
    src, pos = ro.task_tables(w.spec, 42, 0)
    L = w.n_layers
    assert sorted(src.tolist()) == list(range(L))
    assert all(pos[src[l]] == l for l in range(L))
    assert all(src[pos[p]] == p for p in range(L))
    # a layer only ever moves inside its own group
    assert all(w.group[src[l]] == w.group[l] for l in range(L))
    # something does move
    assert sum(src[l] != l for l in range(L)) > L // 2


def test_sigma_uniform_over_the_symmetric_group():
    # Section 4.3: sigma ~ S_K.  Chi-square over all G! outcomes.
    for G, n in ((3, 12000), (4, 24000)):
        counts = {}
        for seed in range(n):
            s = tuple(ro.permutation(seed, 0, 0, G).tolist())
            counts[s] = counts.get(s, 0) + 1
        nperm = math.factorial(G)
        assert len(counts) == nperm
        exp = n / nperm
        chi2 = sum((c - exp) ** 2 / exp for c in counts.values())
        # dof = nperm-1; 99.99% quantiles: 5 dof -> 25.7, 23 dof -> 58.6
        assert chi2 < (25.7 if G == 3 else 58.6), chi2


def test_sigma_depends_on_task_group_and_seed_only_through_the_counter():
    a = ro.permutation(42, 0, 0, 24)
    assert not np.array_equal(a, ro.permutation(42, 1, 0, 24))
    assert not np.array_equal(a, ro.permutation(42, 0, 1, 24))
    assert not np.array_equal(a, ro.permutation(43, 0, 0, 24))
    assert np.array_equal(a, ro.permutation(42, 0, 0, 24))


def test_fisher_yates_consumes_philox_words_in_order():
    # replay with exact integers from raw Philox blocks
    seed, task, g, G = 0x1234567890, 5, 2, 11
    key = (seed & 0xFFFFFFFF, seed >> 32)
    words = []
    for n in range(3):
        words.extend(ro.philox4x32_10((n, g, 0x5045524D, task), key))
    p = list(range(G))
    it = iter(words)
    for k in range(G - 1, 0, -1):
        j = (next(it) * (k + 1)) >> 32
        p[k], p[j] = p[j], p[k]
    assert p == ro.permutation(seed, task, g, G).tolist()


def test_no_shuffle_flag_or_singleton_is_identity():
    spec = tiny_spec(flags=FLIP)
    src, pos = ro.task_tables(spec, 9, 1)
    assert src.tolist() == list(range(6)) and pos.tolist() == list(range(6))
    spec1 = ([3, 3], [4, 4], [0, 1], [SHUFFLE | FLIP, SHUFFLE | FLIP])
    src, pos = ro.task_tables(spec1, 9, 1)
    assert src.tolist() == [0, 1]


# --------------------------------------------------------------------------- signs
def test_sign_bits_are_balanced_and_independent():
    # Section 4.4: diagonal entries +1 / -1 with equal probability
    n = 1 << 15
    s = ro.sign_row(42, 0, 7, n).astype(np.int64)
    assert set(np.unique(s)) == {-1, 1}
    assert abs(s.sum()) < 5 * math.sqrt(n)
    for other in (ro.sign_row(42, 1, 7, n), ro.sign_row(42, 0, 8, n), ro.sign_row(43, 0, 7, n)):
        assert abs(int((s * other).sum())) < 5 * math.sqrt(n)
    # no short-range structure along the columns
    for lag in (1, 2, 32, 128):
        assert abs(int((s[:-lag] * s[lag:]).sum())) < 5 * math.sqrt(n)


def test_sign_bit_layout_in_the_philox_block():
    seed, task, slot = 2**35 + 17, 4, 9
    key = (seed & 0xFFFFFFFF, seed >> 32)
    row = ro.sign_row(seed, task, slot, 300)
    for c in (0, 1, 31, 32, 127, 128, 129, 255, 256, 299):
        blk = ro.philox4x32_10((c >> 7, slot, 0x5349474E, task), key)
        bit = (blk[(c >> 5) & 3] >> (c & 31)) & 1
        assert row[c] == (-1 if bit else 1)
        assert ro.sign(seed, task, slot, c) == row[c]


# --------------------------------------------------------------------------- bf16
def test_bf16_rounding_matches_library_conversion():
    import torch

    rng = np.random.default_rng(3)
    bits = rng.integers(0, 2**32, 20000, dtype=np.uint64).astype(np.uint32)
    special = np.array([0x00000000, 0x80000000, 0x3F808000, 0x3F818000, 0x3F807FFF, 0x3F808001,
                        0x7F7FFFFF, 0x7F7F8000, 0x7F800000, 0xFF800000, 0x00000001, 0x00008000,
                        0x00018000, 0x7F7F7FFF], dtype=np.uint32)
    bits = np.concatenate([bits, special])
    x = bits.view(np.float32)
    want = torch.from_numpy(x.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    for xi, wi in zip(x, want):
        got = ro.f32_to_bf16(float(xi)) if not np.isnan(xi) else None
        if got is None:
            continue
        assert got == int(wi), (hex(int(np.float32(xi).view(np.uint32))), hex(got), hex(int(wi)))
    # NaN stays NaN
    nan_bits = ro.f32_to_bf16(float("nan"))
    assert (nan_bits & 0x7F80) == 0x7F80 and (nan_bits & 0x7F) != 0


# --------------------------------------------------------------------------- dense brute force
@pytest.mark.parametrize("flags", [SHUFFLE, FLIP, SHUFFLE | FLIP, 0])
def test_transform_is_orthogonal_and_compress_retrieve_match_dense_matrices(flags):
    """Section 4: M = sum_i O_i Delta_i and What_t = W_0 + lambda O_t^-1 M with
    O_t^-1 = O_t^T, against d x d matrices in double precision.  Dyadic inputs
    make every fp32 sum exact, so equality is bit for bit."""
    spec = tiny_spec(flags)
    rng = np.random.default_rng(11)
    K = 3
    ids, seeds = [5, 0, 9], [100, 7, 2**33]
    base = rand_model(spec, rng, dyadic=True)
    tasks = [rand_model(spec, rng, dyadic=True) for _ in range(K)]
    Ts = []
    for i in range(K):
        T, offs = dense_transform(spec, seeds[i], ids[i])
        assert np.array_equal(T.T @ T, np.eye(T.shape[0]))  # orthogonal, literally
        Ts.append(T)
    if flags == 0:
        assert all(np.array_equal(T, np.eye(T.shape[0])) for T in Ts)
    else:
        assert not np.array_equal(Ts[0], Ts[1])
    deltas = [flat(t) - flat(base) for t in tasks]
    M_dense = sum(T @ d for T, d in zip(Ts, deltas))
    M = ro.compress(spec, ro.F32, ids, seeds, base, tasks)
    assert np.array_equal(flat(M), M_dense)
    lam = 0.5  # dyadic
    for t in range(K):
        what_dense = flat(base) + lam * (Ts[t].T @ M_dense)
        what = ro.retrieve(spec, ro.F32, ro.F32, ids[t], seeds[t], lam, base, M)
        assert np.array_equal(flat(what), what_dense)
        # Section 4, second display: own delta unchanged + transformed interference
        interference = sum(Ts[t].T @ (Ts[j] @ deltas[j]) for j in range(K) if j != t)
        assert np.array_equal(flat(what) - flat(base) - lam * deltas[t], lam * interference)


@pytest.mark.parametrize("flags", [ro.SHIFT | FLIP, ro.SHIFT, SHUFFLE | FLIP | ro.SKIP(2), ro.SHIFT | FLIP | ro.SKIP(3),
                                   FLIP | ro.SKIP(2), SHUFFLE | ro.SKIP(4)])
def test_shift_and_skip_rate_variants_match_dense_matrices(flags):
    """The appendix's layer shifting and skip rate: still orthogonal, still exact on dyadic inputs."""
    spec = tiny_spec(flags, n_a=7, n_b=5, shape_a=(2, 6), shape_b=(1, 5))
    rng = np.random.default_rng(31)
    ids, seeds = [0, 3, 4], [5, 6, 7]
    base = rand_model(spec, rng, dyadic=True)
    tasks = [rand_model(spec, rng, dyadic=True) for _ in ids]
    Ts = []
    for t, s in zip(ids, seeds):
        T, _ = dense_transform(spec, s, t)
        assert np.array_equal(T.T @ T, np.eye(T.shape[0]))
        Ts.append(T)
    deltas = [flat(t) - flat(base) for t in tasks]
    M_dense = sum(T @ d for T, d in zip(Ts, deltas))
    M = ro.compress(spec, ro.F32, ids, seeds, base, tasks)
    assert np.array_equal(flat(M), M_dense)
    for j in range(len(ids)):
        what = ro.retrieve(spec, ro.F32, ro.F32, ids[j], seeds[j], 0.5, base, M)
        assert np.array_equal(flat(what), flat(base) + 0.5 * (Ts[j].T @ M_dense))


def test_shift_moves_layers_one_position_deeper_and_skip_leaves_the_rest():
    rng = np.random.default_rng(32)
    G = 5
    spec = ([2] * G, [4] * G, [0] * G, [ro.SHIFT])
    delta = rand_model(spec, rng)
    M = ro.compress(spec, ro.F32, [0], [9], None, [delta])          # task 0: one position
    for k in range(G):
        assert np.array_equal(M[(k + 1) % G], delta[k])
    M = ro.compress(spec, ro.F32, [2], [9], None, [delta])          # task 2: three positions
    for k in range(G):
        assert np.array_equal(M[(k + 3) % G], delta[k])
    # skip rate 2: members 1 and 3 neither move nor flip
    spec2 = ([2] * G, [4] * G, [0] * G, [SHUFFLE | FLIP | ro.SKIP(2)])
    for seed in range(6):
        M = ro.compress(spec2, ro.F32, [1], [seed], None, [delta])
        assert np.array_equal(M[1], delta[1]) and np.array_equal(M[3], delta[3])
        src, _ = ro.task_tables(spec2, seed, 1)
        assert sorted(int(src[k]) for k in (0, 2, 4)) == [0, 2, 4]
    with pytest.raises(ValueError):
        ro.compress(([2, 2], [4, 4], [0, 0], [SHUFFLE | ro.SHIFT]), ro.F32, [0], [0], None, [delta[:2]])


def test_gaussian_inputs_match_dense_matrices_within_rounding():
    spec = tiny_spec(SHUFFLE | FLIP)
    rng = np.random.default_rng(12)
    K = 4
    ids, seeds = list(range(K)), [42 + i for i in range(K)]
    base = rand_model(spec, rng, 0.02)
    tasks = [[b + d for b, d in zip(base, rand_model(spec, rng, 1e-3))] for _ in range(K)]
    Ts = [dense_transform(spec, seeds[i], ids[i])[0] for i in range(K)]
    M_dense = sum(T @ (flat(t) - flat(base)) for T, t in zip(Ts, tasks))
    M = ro.compress(spec, ro.F32, ids, seeds, base, tasks)
    # W_i - W_0 is rounded at the magnitude of W (about 0.02 * 4 sigma), then K sums
    tol = 2.0 ** -24 * (0.1 + K * 8e-3) * 2
    assert np.max(np.abs(flat(M) - M_dense)) < tol
    what = ro.retrieve(spec, ro.F32, ro.F32, ids[2], seeds[2], 0.3, base, M)
    what_dense = flat(base) + float(np.float32(0.3)) * (Ts[2].T @ flat(M))
    assert np.max(np.abs(flat(what) - what_dense)) <= 2.0 ** -24 * 0.2


# --------------------------------------------------------------------------- closed forms
def test_single_model_round_trip_is_exact_in_every_mode():
    # K = 1, lambda = 1: T^-1 T = I, so What = fl(W_0 + fl(W_1 - W_0))
    rng = np.random.default_rng(13)
    for flags in (SHUFFLE, FLIP, SHUFFLE | FLIP):
        spec = tiny_spec(flags, shape_a=(5, 130), shape_b=(1, 33))
        base = rand_model(spec, rng, 0.02)
        task = [b + d for b, d in zip(base, rand_model(spec, rng, 1e-3))]
        M = ro.compress(spec, ro.F32, [3], [77], base, [task])
        out = ro.retrieve(spec, ro.F32, ro.F32, 3, 77, 1.0, base, M)
        for b, t, o in zip(base, task, out):
            want = (b + (t - b).astype(np.float32)).astype(np.float32)
            assert np.array_equal(o, want)
        # and M really is transformed (not the plain delta) when a transform is on
        plain = [(t - b).astype(np.float32) for b, t in zip(base, task)]
        assert any(not np.array_equal(m, p) for m, p in zip(M, plain))
        # a wrong seed does not bring the model back
        bad = ro.retrieve(spec, ro.F32, ro.F32, 3, 78, 1.0, base, M)
        assert any(not np.array_equal(o, x) for o, x in zip(out, bad))


def test_single_model_any_lambda_is_one_fused_multiply_add():
    rng = np.random.default_rng(14)
    spec = tiny_spec(SHUFFLE | FLIP)
    base = rand_model(spec, rng, 0.02)
    task = [b + d for b, d in zip(base, rand_model(spec, rng, 1e-3))]
    lam = 0.3
    M = ro.compress(spec, ro.F32, [0], [42], base, [task])
    out = ro.retrieve(spec, ro.F32, ro.F32, 0, 42, lam, base, M)
    lam32 = Fraction(float(np.float32(lam)))
    n_checked = 0
    for b, t, o in zip(base, task, out):
        d = (t - b).astype(np.float32)
        for idx in np.ndindex(b.shape):
            exact = lam32 * Fraction(float(d[idx])) + Fraction(float(b[idx]))
            assert o[idx] == round_fraction_to_f32(exact)
            n_checked += 1
    assert n_checked > 100


def test_identity_plan_is_task_arithmetic():
    # all T_i = I: M = sum of deltas in order, What = W_0 + lambda * sum (Section 3, Eq. 1)
    rng = np.random.default_rng(15)
    spec = tiny_spec(0)
    K = 5
    base = rand_model(spec, rng, 0.02)
    tasks = [[b + d for b, d in zip(base, rand_model(spec, rng, 1e-3))] for _ in range(K)]
    M = ro.compress(spec, ro.F32, list(range(K)), list(range(K)), base, tasks)
    for l in range(len(base)):
        acc = np.zeros_like(base[l])
        for i in range(K):
            acc = (acc + (tasks[i][l] - base[l]).astype(np.float32)).astype(np.float32)
        assert np.array_equal(M[l], acc)


def test_task_order_is_the_given_order():
    rng = np.random.default_rng(16)
    spec = tiny_spec(0)
    base = rand_model(spec, rng, 0.02)
    tasks = [[b + d for b, d in zip(base, rand_model(spec, rng, s))] for s in (1.0, 1e-4, -1.0 + 2.0)]
    tasks[2] = [2 * b - t for b, t in zip(base, tasks[0])]  # delta_2 = -delta_0 (approximately)
    fwd = ro.compress(spec, ro.F32, [0, 1, 2], [0, 1, 2], base, tasks)
    rev = ro.compress(spec, ro.F32, [0, 2, 1], [0, 2, 1], base, [tasks[0], tasks[2], tasks[1]])
    assert any(not np.array_equal(a, b) for a, b in zip(fwd, rev))


def test_flip_is_an_involution_and_preserves_magnitudes():
    # D^-1 = D and |T delta| is a rearrangement of |delta| (orthogonality)
    rng = np.random.default_rng(17)
    spec = tiny_spec(SHUFFLE | FLIP, shape_a=(3, 200))
    delta = rand_model(spec, rng, 1e-3)
    M = ro.compress(spec, ro.F32, [2], [5], None, [delta])
    assert np.array_equal(np.sort(np.abs(flat(M))), np.sort(np.abs(flat(delta))))
    flip_only = (spec[0], spec[1], spec[2], [FLIP, FLIP])
    once = ro.compress(flip_only, ro.F32, [2], [5], None, [delta])
    twice = ro.compress(flip_only, ro.F32, [2], [5], None, [once])
    assert all(np.array_equal(a, b) for a, b in zip(twice, delta))
    assert any(not np.array_equal(a, b) for a, b in zip(once, delta))
    # the sign is a function of the column only: every row of a slot agrees
    for l in range(len(delta)):
        ratio = np.sign(once[l]) * np.sign(delta[l])
        assert np.all(ratio == ratio[0:1, :])


def test_delta_input_equals_weights_input():
    rng = np.random.default_rng(18)
    spec = tiny_spec(SHUFFLE | FLIP)
    base = rand_model(spec, rng, dyadic=True)
    tasks = [rand_model(spec, rng, dyadic=True) for _ in range(3)]
    deltas = [[(t - b).astype(np.float32) for t, b in zip(tk, base)] for tk in tasks]
    a = ro.compress(spec, ro.F32, [0, 1, 2], [1, 2, 3], base, tasks)
    b = ro.compress(spec, ro.F32, [0, 1, 2], [1, 2, 3], None, deltas)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))


# --------------------------------------------------------------------------- hot swapping
def test_add_then_remove_restores_superposition():
    # Section 5.7: transforms are independent of data, so models come and go
    rng = np.random.default_rng(19)
    spec = tiny_spec(SHUFFLE | FLIP)
    base = rand_model(spec, rng, dyadic=True)
    tasks = [rand_model(spec, rng, dyadic=True) for _ in range(4)]
    M = ro.compress(spec, ro.F32, [0, 1, 2], [10, 11, 12], base, tasks[:3])
    M0 = [m.copy() for m in M]
    ro.add_model(spec, ro.F32, 3, 13, base, tasks[3], M)
    M4 = ro.compress(spec, ro.F32, [0, 1, 2, 3], [10, 11, 12, 13], base, tasks)
    assert all(np.array_equal(a, b) for a, b in zip(M, M4))       # add == compress of the larger set
    ro.remove_model(spec, ro.F32, 3, 13, base, tasks[3], M)
    assert all(np.array_equal(a, b) for a, b in zip(M, M0))       # exact on the dyadic grid
    # remove an original member: equals compress of the rest
    ro.remove_model(spec, ro.F32, 1, 11, base, tasks[1], M)
    M_rest = ro.compress(spec, ro.F32, [0, 2], [10, 12], base, [tasks[0], tasks[2]])
    assert all(np.array_equal(a, b) for a, b in zip(M, M_rest))


def test_add_remove_on_gaussian_inputs_within_one_rounding():
    rng = np.random.default_rng(20)
    spec = tiny_spec(SHUFFLE | FLIP)
    base = rand_model(spec, rng, 0.02)
    tasks = [[b + d for b, d in zip(base, rand_model(spec, rng, 1e-3))] for _ in range(3)]
    M = ro.compress(spec, ro.F32, [0, 1], [1, 2], base, tasks[:2])
    M0 = [m.copy() for m in M]
    ro.add_model(spec, ro.F32, 2, 3, base, tasks[2], M)
    x = [np.abs(a - b) for a, b in zip(M, M0)]
    ro.remove_model(spec, ro.F32, 2, 3, base, tasks[2], M)
    for a, b, xx in zip(M, M0, x):
        assert np.all(np.abs(a - b) <= 2.0 ** -23 * (np.abs(b) + xx))


def test_adding_several_models_at_once_matches_dense_matrices_and_left_to_right_sums():
    # Section 5.7 applied to a set of models: M <- M + T_a d_a + T_b d_b + ..., in the given order
    rng = np.random.default_rng(23)
    spec = tiny_spec(SHUFFLE | FLIP)
    base = rand_model(spec, rng, dyadic=True)
    tasks = [rand_model(spec, rng, dyadic=True) for _ in range(5)]
    ids, seeds = [4, 0, 8, 2, 6], [40, 41, 2**35, 43, 44]
    M = ro.compress(spec, ro.F32, ids[:2], seeds[:2], base, tasks[:2])
    M_before = flat(M)
    ro.add_models(spec, ro.F32, ids[2:], seeds[2:], base, tasks[2:], M)
    dense = sum(dense_transform(spec, seeds[i], ids[i])[0] @ (flat(tasks[i]) - flat(base)) for i in range(2, 5))
    assert np.array_equal(flat(M), M_before + dense)              # exact on the dyadic grid
    M_all = ro.compress(spec, ro.F32, ids, seeds, base, tasks)
    assert np.array_equal(flat(M), flat(M_all))
    # Gaussian inputs: one fp32 rounding per term, left to right, starting from M
    base = rand_model(spec, rng, 0.02)
    tasks = [[b + d for b, d in zip(base, rand_model(spec, rng, 1e-3))] for _ in range(4)]
    M = ro.compress(spec, ro.F32, [1], [5], base, tasks[:1])
    terms = [ro.compress(spec, ro.F32, [i], [s], base, [t]) for i, s, t in zip([2, 3, 9], [6, 7, 8], tasks[1:])]
    want = [m.copy() for m in M]
    for x in terms:
        want = [(w + xx).astype(np.float32) for w, xx in zip(want, x)]
    ro.add_models(spec, ro.F32, [2, 3, 9], [6, 7, 8], base, tasks[1:], M)
    assert all(np.array_equal(a, b) for a, b in zip(M, want))
    # a bf16 M is widened once, summed in fp32 and rounded once: not what three separate adds give
    M16 = ro.compress(spec, ro.F32, [1], [5], base, tasks[:1], m_dtype=ro.BF16)
    want = [wl.bf16_bits_to_f32(m) for m in M16]
    for x in terms:
        want = [(w + xx).astype(np.float32) for w, xx in zip(want, x)]
    one_by_one = [m.copy() for m in M16]
    for i, s_, t in zip([2, 3, 9], [6, 7, 8], tasks[1:]):
        ro.add_model(spec, ro.F32, i, s_, base, t, one_by_one, m_dtype=ro.BF16)
    ro.add_models(spec, ro.F32, [2, 3, 9], [6, 7, 8], base, tasks[1:], M16, m_dtype=ro.BF16)
    assert all(np.array_equal(a, wl.to_bf16_bits(b)) for a, b in zip(M16, want))
    assert any(not np.array_equal(a, b) for a, b in zip(M16, one_by_one))
    # an empty set leaves M alone
    keep = [m.copy() for m in M]
    ro.add_models(spec, ro.F32, [], [], base, [], M)
    assert all(np.array_equal(a, b) for a, b in zip(M, keep))


# --------------------------------------------------------------------------- decorrelation
def test_sign_flip_decorrelates_with_the_predicted_variance():
    """For one m x n layer and tasks i != j: <A D_i, B D_j> = sum_c eps_c g_c with
    g_c = sum_r A_rc B_rc and eps_c i.i.d. +-1, so the mean is 0 and the variance
    is exactly sum_c g_c^2 (Section 3: interference falls with the cosine)."""
    rng = np.random.default_rng(21)
    m, n = 16, 64
    spec = ([m], [n], [0], [FLIP])
    shared = rng.standard_normal((m, n))
    A = (0.5 * shared + math.sqrt(0.75) * rng.standard_normal((m, n))).astype(np.float32)
    B = (0.5 * shared + math.sqrt(0.75) * rng.standard_normal((m, n))).astype(np.float32)
    g = (A.astype(np.float64) * B.astype(np.float64)).sum(axis=0)
    raw = float(g.sum())
    vals = []
    for seed in range(1500):
        TA = ro.compress(spec, ro.F32, [0], [seed], None, [[A]])[0].astype(np.float64)
        TB = ro.compress(spec, ro.F32, [1], [seed], None, [[B]])[0].astype(np.float64)
        vals.append(float((TA * TB).sum()))
    vals = np.array(vals)
    var_pred = float((g ** 2).sum())
    assert abs(vals.mean()) < 4 * math.sqrt(var_pred / len(vals))
    assert 0.85 < vals.var() / var_pred < 1.15
    # the cosine shrinks by about 1/sqrt(n) relative to the raw 0.25
    cos_raw = raw / (np.linalg.norm(A) * np.linalg.norm(B))
    cos_std = vals.std() / (np.linalg.norm(A) * np.linalg.norm(B))
    assert 0.15 < cos_raw < 0.35
    assert cos_std < 2.0 * cos_raw / math.sqrt(n) + 1.5 / math.sqrt(m * n)


def test_shuffle_aligns_shared_component_only_when_slots_coincide():
    # with shuffle alone, <P_i a, P_j b> over a group = sum_k <a[s_i(k)], b[s_j(k)]>
    rng = np.random.default_rng(22)
    G = 6
    spec = ([4] * G, [8] * G, [0] * G, [SHUFFLE])
    a = rand_model(spec, rng)
    b = rand_model(spec, rng)
    for seed in range(5):
        Ta = ro.compress(spec, ro.F32, [0], [seed], None, [a])
        Tb = ro.compress(spec, ro.F32, [1], [seed], None, [b])
        si = ro.permutation(seed, 0, 0, G)
        sj = ro.permutation(seed, 1, 0, G)
        want = sum(float((a[si[k]].astype(np.float64) * b[sj[k]].astype(np.float64)).sum()) for k in range(G))
        got = sum(float((x.astype(np.float64) * y.astype(np.float64)).sum()) for x, y in zip(Ta, Tb))
        assert abs(got - want) < 1e-9


def test_gram_of_transformed_deltas_matches_dense_matrices_and_the_interference_norm():
    """Section 3: || lambda sum_{j != i} Delta_j ||^2 = lambda^2 sum_{j,l != i} <Delta_j, Delta_l>; under
    RanDeS the interfering deltas are O_i^-1 O_j Delta_j, whose inner products are those of O_j Delta_j."""
    spec = tiny_spec(SHUFFLE | FLIP)
    rng = np.random.default_rng(33)
    ids, seeds = [0, 1, 2, 3], [42, 43, 44, 45]
    base = rand_model(spec, rng, dyadic=True)
    tasks = [rand_model(spec, rng, dyadic=True) for _ in ids]
    Ts = [dense_transform(spec, s, t)[0] for t, s in zip(ids, seeds)]
    X = [T @ (flat(t) - flat(base)) for T, t in zip(Ts, tasks)]
    want = np.array([[float(a @ b) for b in X] for a in X])
    G = ro.delta_gram(spec, ro.F32, ids, seeds, base, tasks)
    assert np.array_equal(G, want)              # dyadic inputs: every product and sum is exact in double
    assert np.array_equal(G, G.T)
    # the diagonal is the squared norm of the untouched delta (orthogonality)
    for i, t in enumerate(tasks):
        assert G[i, i] == float((flat(t) - flat(base)) @ (flat(t) - flat(base)))
    # interference norm at retrieval, against the retrieved model itself
    lam = 0.5
    M = ro.compress(spec, ro.F32, ids, seeds, base, tasks)
    for t in range(len(ids)):
        what = ro.retrieve(spec, ro.F32, ro.F32, ids[t], seeds[t], lam, base, M)
        interference = flat(what) - flat(base) - lam * (flat(tasks[t]) - flat(base))
        others = [j for j in range(len(ids)) if j != t]
        assert float(interference @ interference) == lam * lam * sum(G[j, l] for j in others for l in others)
    # the same without transforms is the plain Gram matrix of the deltas
    G0 = ro.delta_gram(tiny_spec(0), ro.F32, ids, seeds, base, tasks)
    D = [flat(t) - flat(base) for t in tasks]
    assert np.array_equal(G0, np.array([[float(a @ b) for b in D] for a in D]))
    assert np.array_equal(np.diag(G0), np.diag(G))


# --------------------------------------------------------------------------- bf16 storage
def test_bf16_storage_and_output():
    rng = np.random.default_rng(23)
    spec = tiny_spec(SHUFFLE | FLIP, shape_a=(3, 40))
    base32 = rand_model(spec, rng, 0.02)
    base = [wl.to_bf16_bits(b) for b in base32]
    tasks = [[wl.to_bf16_bits(wl.bf16_bits_to_f32(b) + d) for b, d in zip(base, rand_model(spec, rng, 1e-3))]
             for _ in range(3)]
    ids, seeds = [0, 1, 2], [4, 5, 6]
    M = ro.compress(spec, ro.BF16, ids, seeds, base, tasks)
    # same as the fp32 path on the widened inputs (bf16 -> fp32 is exact)
    M32 = ro.compress(spec, ro.F32, ids, seeds, [wl.bf16_bits_to_f32(b) for b in base],
                      [[wl.bf16_bits_to_f32(x) for x in t] for t in tasks])
    assert all(np.array_equal(a, b) for a, b in zip(M, M32))
    out16 = ro.retrieve(spec, ro.BF16, ro.BF16, 1, 5, 0.5, base, M)
    out32 = ro.retrieve(spec, ro.BF16, ro.F32, 1, 5, 0.5, base, M)
    for a, b in zip(out16, out32):
        assert a.dtype == np.uint16
        assert np.array_equal(a, wl.to_bf16_bits(b))


def test_bf16_superposition_is_the_fp32_sum_rounded_once():
    # the further compression of M that the paper's conclusion leaves open: M stored as bf16
    rng = np.random.default_rng(41)
    spec = tiny_spec(SHUFFLE | FLIP, shape_a=(3, 40))
    base = rand_model(spec, rng, 0.02)
    tasks = [[b + d for b, d in zip(base, rand_model(spec, rng, 1e-3))] for _ in range(4)]
    ids, seeds = [0, 1, 2], [4, 5, 6]
    M32 = ro.compress(spec, ro.F32, ids, seeds, base, tasks[:3])
    M16 = ro.compress(spec, ro.F32, ids, seeds, base, tasks[:3], m_dtype=ro.BF16)
    for a, b in zip(M16, M32):
        assert a.dtype == np.uint16 and np.array_equal(a, wl.to_bf16_bits(b))
    # retrieve widens the stored element: same as retrieving from the widened copy
    wide = [wl.bf16_bits_to_f32(m) for m in M16]
    out16 = ro.retrieve(spec, ro.F32, ro.F32, 1, 5, 0.3, base, M16, m_dtype=ro.BF16)
    out32 = ro.retrieve(spec, ro.F32, ro.F32, 1, 5, 0.3, base, wide)
    assert all(np.array_equal(a, b) for a, b in zip(out16, out32))
    # add: widen, add the transformed delta in fp32, round again
    x = ro.compress(spec, ro.F32, [7], [70], base, [tasks[3]])             # T_7(delta) alone
    ro.add_model(spec, ro.F32, 7, 70, base, tasks[3], M16, m_dtype=ro.BF16)
    for m, w_, xx in zip(M16, wide, x):
        assert np.array_equal(m, wl.to_bf16_bits((w_ + xx).astype(np.float32)))
    wide2 = [wl.bf16_bits_to_f32(m) for m in M16]
    ro.remove_model(spec, ro.F32, 7, 70, base, tasks[3], M16, m_dtype=ro.BF16)
    for m, w_, xx in zip(M16, wide2, x):
        assert np.array_equal(m, wl.to_bf16_bits((w_ - xx).astype(np.float32)))


# --------------------------------------------------------------------------- masks, errors
def test_slot_mask_limits_work_and_matches_full_result():
    rng = np.random.default_rng(24)
    spec = tiny_spec(SHUFFLE | FLIP)
    base = rand_model(spec, rng, 0.02)
    tasks = [[b + d for b, d in zip(base, rand_model(spec, rng, 1e-3))] for _ in range(3)]
    full = ro.compress(spec, ro.F32, [0, 1, 2], [1, 2, 3], base, tasks)
    part = ro.compress(spec, ro.F32, [0, 1, 2], [1, 2, 3], base, tasks, slots=[1, 4])
    assert np.array_equal(part[1], full[1]) and np.array_equal(part[4], full[4])
    assert part[0] is None and part[2] is None
    _, pos = ro.task_tables(spec, 2, 1)
    outp = ro.retrieve(spec, ro.F32, ro.F32, 1, 2, 0.3, base, full, positions=[2])
    outf = ro.retrieve(spec, ro.F32, ro.F32, 1, 2, 0.3, base, full)
    assert np.array_equal(outp[2], outf[2]) and outp[0] is None


def test_group_with_unequal_shapes_is_rejected():
    spec = ([4, 4], [8, 9], [0, 0], [SHUFFLE])
    base = [np.zeros((4, 8), np.float32), np.zeros((4, 9), np.float32)]
    with pytest.raises(ValueError):
        ro.compress(spec, ro.F32, [0], [0], base, [base])


# --------------------------------------------------------------------------- linear layer on the retrieved weight
@pytest.mark.parametrize("flags", [SHUFFLE | FLIP, FLIP, SHUFFLE, 0])
def test_linear_matches_dense_matrices_and_the_retrieved_weight(flags):
    """y = x What^T with What = W_0 + lambda O_t^T M (Section 4, second display) taken from d x d matrices:
    on dyadic inputs every product and sum is exact in double, so the oracle must agree bit for bit; it must
    also agree with a matrix product on the oracle's own retrieved weights."""
    spec = tiny_spec(flags)
    rng = np.random.default_rng(77)
    ids, seeds = [4, 1, 8], [11, 2**40 + 3, 5]
    base = rand_model(spec, rng, dyadic=True)
    tasks = [rand_model(spec, rng, dyadic=True) for _ in ids]
    M = ro.compress(spec, ro.F32, ids, seeds, base, tasks)
    lam = 0.25
    for t, s in zip(ids, seeds):
        T, offs = dense_transform(spec, s, t)
        what_dense = unflat(flat(base) + lam * (T.T @ flat(M)), spec, offs)
        what = ro.retrieve(spec, ro.F32, ro.F32, t, s, lam, base, M)
        for p in range(len(spec[0])):
            x = (rng.integers(-64, 65, size=(5, spec[1][p])) / 64.0).astype(np.float32)
            y, y_abs = ro.linear(spec, ro.F32, t, s, lam, p, x, base, M)
            assert np.array_equal(y, x.astype(np.float64) @ what_dense[p].T)
            assert np.array_equal(y, x.astype(np.float64) @ what[p].astype(np.float64).T)
            assert np.all(y_abs >= np.abs(y))


def test_linear_on_bf16_inputs_and_superposition_stays_close_to_the_retrieved_weight():
    """bf16 weights and a bf16 superposition: the unformed weight W_0 + lambda s M differs from the retrieved
    fp32 weight by one fp32 rounding per element, so the two products agree to 2^-24 of the magnitude sum; a
    single column with the wrong sign would move the result far beyond that."""
    rng = np.random.default_rng(78)
    spec = ([6] * 3, [40] * 3, [0] * 3, [SHUFFLE | FLIP])
    to_b = lambda a: np.array([ro.f32_to_bf16(float(v)) for v in a.ravel()], dtype=np.uint16).reshape(a.shape)
    widen = lambda b: (b.astype(np.uint32) << 16).view(np.float32)
    base = [to_b(a * 0.02) for a in rand_model(spec, rng)]
    M = [to_b(a * 0.003) for a in rand_model(spec, rng)]
    x = to_b(rng.standard_normal((7, 40)).astype(np.float32))
    lam, t, s = 0.3, 3, 99
    for p in range(3):
        y, y_abs = ro.linear(spec, ro.BF16, t, s, lam, p, x, base, M, m_dtype=ro.BF16)
        what = ro.retrieve(spec, ro.BF16, ro.F32, t, s, lam, base, M, positions=[p], m_dtype=ro.BF16)[p]
        y_ret = widen(x).astype(np.float64) @ what.astype(np.float64).T
        assert np.all(np.abs(y - y_ret) <= 2.0 ** -23 * y_abs)
        # flipping the sign of one column's superposition term changes y by 2 |x_c| lambda |M_c|
        _, slot_of_pos = ro.task_tables(spec, s, t)
        l = int(slot_of_pos[p])
        Mw = [m.copy() for m in M]
        Mw[l][:, 17] ^= 0x8000
        y_wrong, _ = ro.linear(spec, ro.BF16, t, s, lam, p, x, base, Mw, m_dtype=ro.BF16)
        want = -2.0 * float(np.float32(lam)) * ro.sign(s, t, l, 17) * np.outer(widen(x)[:, 17].astype(np.float64), widen(M[l])[:, 17].astype(np.float64))
        assert np.allclose(y_wrong - y, want, rtol=0, atol=1e-12)
        assert np.abs(y_wrong - y).max() > 2.0 ** -14 * y_abs.max()


@pytest.mark.parametrize("cols", [1024, 4096])
def test_linear_tolerance_of_the_gpu_test_sees_one_wrong_column_at_wide_layers(cols):
    """The GPU comparison accepts sqrt(2 cols + 2) 2^-24 y_abs.  With weights and a superposition of the
    magnitudes of the synthetic sets (W_0 ~ 0.02, M ~ 0.002, lambda = 0.3) one column of M with the wrong sign
    must move some output beyond that at the widths of the paper-shaped layers; the old worst-case bound
    (2 cols + 2) 2^-24 y_abs would not have seen it."""
    rng = np.random.default_rng(cols)
    spec = ([24], [cols], [0], [FLIP])
    base = [wl.to_bf16_bits((rng.standard_normal((24, cols)) * 0.02).astype(np.float32))]
    M = [wl.to_bf16_bits((rng.standard_normal((24, cols)) * 0.002).astype(np.float32))]
    x = wl.to_bf16_bits(rng.standard_normal((64, cols)).astype(np.float32))
    lam, t, s = 0.3, 1, 43
    y, y_abs = ro.linear(spec, ro.BF16, t, s, lam, 0, x, base, M, m_dtype=ro.BF16)
    Mw = [M[0].copy()]
    Mw[0][:, cols // 3] ^= 0x8000
    y_wrong, _ = ro.linear(spec, ro.BF16, t, s, lam, 0, x, base, Mw, m_dtype=ro.BF16)
    tol = np.sqrt(2.0 * cols + 2.0) * 2.0 ** -24 * y_abs
    assert (np.abs(y_wrong - y) > tol).mean() > 0.5          # most outputs, not just the tail
    assert (np.abs(y_wrong - y) > (2 * cols + 2) * 2.0 ** -24 * y_abs).mean() < 0.5   # the worst-case bound misses most


# --------------------------------------------------------------------------- Gaussian-like diagonal context ("RD", Section 5.5)
def test_gauss_entries_replay_the_stated_recipe_and_have_unit_variance():
    """Entry (task, slot, column) = sum of twelve uniforms minus six, uniforms = top 24 bits of the words of
    Philox blocks 3c .. 3c+2 of the "GAUS" stream, added left to right in fp32: replayed here from the oracle's
    Philox (itself pinned to published vectors); mean 0, variance 1, support inside (-6, 6)."""
    seed, task, slot = 2**40 + 5, 9, 3
    for c in (0, 1, 130, 4095):
        acc = np.float32(0.0)
        for b in range(3):
            blk = ro.philox4x32_10((3 * c + b, slot, 0x47415553, task), (seed & 0xFFFFFFFF, seed >> 32))
            for w in blk:
                acc = np.float32(acc + np.float32(w >> 8) * np.float32(2.0 ** -24))
        want = np.float32(acc - np.float32(6.0))
        assert np.float32(ro.gauss(seed, task, slot, c)) == (want if want != 0 else np.float32(1.0))
    g = np.array([ro.gauss(seed, task, slot, c) for c in range(40000)])
    assert abs(g.mean()) < 4 / np.sqrt(g.size) and abs(g.var() - 1.0) < 0.03
    assert np.abs(g).max() < 6.0 and np.all(g != 0.0)
    # fourth moment of the twelve-uniform sum: 3 - 6/(5*12) = 2.9
    assert abs(np.mean(g ** 4) - 2.9) < 0.15
    other = np.array([ro.gauss(seed, task + 1, slot, c) for c in range(4000)])
    assert abs(np.corrcoef(g[:4000], other)[0, 1]) < 0.06


@pytest.mark.parametrize("flags", [ro.GAUSS, ro.GAUSS | SHUFFLE, ro.GAUSS | SHUFFLE | ro.SKIP(2)])
def test_gauss_context_matches_dense_matrices_and_is_not_orthogonal(flags):
    """Section 5.5: with a Gaussian-like diagonal D the same formulas hold with D^-1 in place of D^T:
    M = sum_i D_i P_i delta_i, What_t = W_0 + lambda P_t^T D_t^-1 M; the transform is not orthogonal."""
    spec = tiny_spec(flags, n_a=4, n_b=3)
    rng = np.random.default_rng(91)
    ids, seeds = [2, 7, 5], [3, 2**35, 11]
    base = rand_model(spec, rng, scale=0.02)
    tasks = [[b + d for b, d in zip(base, rand_model(spec, rng, scale=1e-3))] for _ in ids]
    Ts = [dense_transform(spec, s, t)[0] for t, s in zip(ids, seeds)]
    assert not np.allclose(Ts[0].T @ Ts[0], np.eye(Ts[0].shape[0]))
    deltas = [flat([np.float32(a - b) for a, b in zip(t, base)]) for t in tasks]
    M_dense = sum(T @ d for T, d in zip(Ts, deltas))
    M = ro.compress(spec, ro.F32, ids, seeds, base, tasks)
    scale = sum(np.abs(T) @ np.abs(d) for T, d in zip(Ts, deltas))
    assert np.all(np.abs(flat(M) - M_dense) <= 2.0 ** -22 * scale + 1e-30)      # one rounding per product and per sum
    lam = 0.3
    for j, (t, s) in enumerate(zip(ids, seeds)):
        what = ro.retrieve(spec, ro.F32, ro.F32, t, s, lam, base, M)
        want = flat(base) + float(np.float32(lam)) * (np.linalg.inv(Ts[j]) @ flat(M))
        tol = 2.0 ** -22 * (np.abs(flat(base)) + lam * np.abs(np.linalg.inv(Ts[j])) @ np.abs(flat(M)))
        assert np.all(np.abs(flat(what) - want) <= tol + 1e-30)


def test_gauss_context_single_model_round_trip_and_larger_interference_than_sign_flips():
    """K = 1: (delta g) / g returns delta within two roundings.  K > 1: the paper's finding of Section 5.5 -- a
    diagonal that does not preserve magnitudes leaves more interference than the +-1 one on the same models."""
    rng = np.random.default_rng(92)
    spec_g = ([16] * 4, [64] * 4, [0] * 4, [ro.GAUSS])
    spec_f = ([16] * 4, [64] * 4, [0] * 4, [FLIP])
    base = rand_model(spec_g, rng, scale=0.02)
    deltas = [rand_model(spec_g, rng, scale=1e-3) for _ in range(6)]
    tasks = [[b + d for b, d in zip(base, dl)] for dl in deltas]
    M1 = ro.compress(spec_g, ro.F32, [4], [17], base, tasks[:1])
    back = ro.retrieve(spec_g, ro.F32, ro.F32, 4, 17, 1.0, base, M1)
    d0 = [np.float32(t - b) for t, b in zip(tasks[0], base)]
    for l in range(4):
        assert np.all(np.abs(back[l].astype(np.float64) - base[l] - d0[l]) <= 2.0 ** -22 * (np.abs(d0[l]) + np.abs(base[l])))
    ids, seeds = list(range(6)), [50 + i for i in range(6)]
    err = {}
    for name, spec in (("gauss", spec_g), ("flip", spec_f)):
        M = ro.compress(spec, ro.F32, ids, seeds, base, tasks)
        out = ro.retrieve(spec, ro.F32, ro.F32, 0, seeds[0], 1.0, base, M)
        err[name] = np.sqrt(sum(np.sum((o.astype(np.float64) - t) ** 2) for o, t in zip(out, tasks[0])))
    assert err["gauss"] > 2.0 * err["flip"]


def test_gauss_and_flip_exclude_each_other_and_diagnostics_refuse_the_gauss_context():
    spec = ([2, 2], [8, 8], [0, 0], [ro.GAUSS | FLIP])
    m = rand_model(spec, np.random.default_rng(1))
    with pytest.raises(ValueError):
        ro.compress(spec, ro.F32, [0], [1], None, [m])
    spec = ([2, 2], [8, 8], [0, 0], [ro.GAUSS])
    with pytest.raises(ValueError):
        ro.delta_gram(spec, ro.F32, [0, 1], [1, 2], None, [m, m])
