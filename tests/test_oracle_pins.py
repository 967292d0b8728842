"""Pins for the CPU oracle: what the paper and the mathematics fix, checked against the oracle (no GPU).

Each test cites the passage that fixes the expected value.  A dropped term, a wrong sign or index, or a transposed
operand anywhere in the oracle should fail at least one of these.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import (SCALE_E8M0_B32, AXIS_COL, AXIS_ROW, GRID_E1M2, GRID_E2M1, GRID_E2M1_MAX2, GRID_E2M1_MAX4, GRID_INT4, ROUND_RTNE, ROUND_SR, SCALE_E4M3_TENSOR,
                    SCALE_FP32, SCALE_POW2)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(a):
    """numpy float -> BF16 bit patterns (round to nearest even), via torch's converter."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.uint16).numpy().copy()


def bf16_vals(bits):
    return torch.from_numpy(bits.copy()).view(torch.bfloat16).to(torch.float64).numpy()


# ------------------------------------------------------------------ Philox (Salmon et al., SC'11 known answers)

def test_philox_known_answers():
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for w in rows:
        v = [int(t, 16) for t in w]
        out = oracle.philox4x32_10(v[0:4], v[4:6])
        assert out.tolist() == v[6:10]


def test_sr_bytes_are_little_endian_bytes_of_the_philox_block():
    seed, b, variant = 0x1234567890ABCDEF, (5 << 32) | 77, 1
    words = oracle.philox4x32_10([b & 0xFFFFFFFF, b >> 32, variant, 0x53520000], [seed & 0xFFFFFFFF, seed >> 32])
    expect = np.frombuffer(words.astype("<u4").tobytes(), dtype=np.uint8)
    assert oracle.sr_bytes(seed, b, variant).tolist() == expect.tolist()


# ------------------------------------------------------------------ Hadamard and RHT (Sec. 2.2)

@pytest.mark.parametrize("n", [1, 2, 4, 8, 16, 32, 64])
def test_hadamard_is_orthogonal(n):
    H = oracle.hadamard_matrix(n)
    tol = 0.0 if n in (1, 4, 16, 64) else 4e-16   # entries are +-2^-k exactly when n is a power of 4
    assert np.max(np.abs(H.T @ H - np.eye(n))) <= tol


def test_hadamard_16_entries_and_sylvester_structure():
    H = oracle.hadamard_matrix(16)
    assert set(np.unique(H).tolist()) == {-0.25, 0.25}
    # Sylvester order: entry (i, j) has sign (-1)^popcount(i & j); first row and column are all positive
    for i in range(16):
        for j in range(16):
            assert H[i, j] == 0.25 * (-1) ** bin(i & j).count("1")
    H8 = oracle.hadamard_matrix(8)
    c = 1 / np.sqrt(2.0)
    assert np.allclose(H, c * np.block([[H8, H8], [H8, -H8]]), atol=1e-16)


def test_butterfly_equals_row_vector_times_sign_times_hadamard():
    H = oracle.hadamard_matrix(16)
    for mask in (0, 0xFFFF, 0x36A6, 0x0001, 0x8000):
        eps = np.array([-1.0 if (mask >> i) & 1 else 1.0 for i in range(16)])
        Hp = np.diag(eps) @ H                      # H' = S H: signs are applied before the Hadamard transform
        for i in range(16):                        # basis vectors: exact in FP32
            e = np.zeros(16, dtype=np.float32)
            e[i] = 1.0
            assert np.array_equal(oracle.rht16_f32(e, mask).astype(np.float64), Hp[i])
        rng = np.random.default_rng(mask)
        x = rng.integers(-64, 64, size=16).astype(np.float32)     # small integers: every FP32 step is exact
        assert np.array_equal(oracle.rht16_f32(x, mask).astype(np.float64), x.astype(np.float64) @ Hp)
        x = rng.standard_normal(16).astype(np.float32)
        assert np.allclose(oracle.rht16_f32(x, mask), x.astype(np.float64) @ Hp, rtol=0, atol=2e-6)


def test_rht_is_invertible_and_preserves_the_gemm():
    rng = np.random.default_rng(3)
    mask = oracle.rht_sign_mask(1)
    eps = np.array([-1.0 if (mask >> i) & 1 else 1.0 for i in range(16)])
    Hp = np.diag(eps) @ oracle.hadamard_matrix(16)
    assert np.max(np.abs(Hp @ Hp.T - np.eye(16))) == 0.0
    X = rng.standard_normal((24, 64))
    W = rng.standard_normal((40, 64))
    B = np.kron(np.eye(4), Hp)                     # block-diagonal RHT along the shared dimension
    Y = X @ W.T
    Yr = (X @ B) @ (W @ B).T
    assert np.max(np.abs(Y - Yr)) <= 1e-12 * np.max(np.abs(Y))
    x = rng.standard_normal(16).astype(np.float32)
    back = oracle.rht16_f32(x, mask).astype(np.float64) @ Hp.T
    assert np.allclose(back, x, atol=1e-6)


@pytest.mark.parametrize("n", [32, 64, 128])
def test_wide_rht_equals_row_vector_times_sign_times_hadamard(n):
    """RHT block sizes 32 / 64 / 128 (App. B): v -> (v o eps) H_n with the Sylvester H_n, signs first; the 128 sign bits
    are the four Philox words whose first 16 bits are the 16-point mask."""
    H = oracle.hadamard_matrix(n)
    c32 = float(np.float32(1.0 / np.sqrt(n)))
    for seed in (0, 1, 0xDEADBEEFCAFEF00D):
        signs = oracle.rht_signs(seed)
        w = oracle.philox4x32_10([0, 0, 0, 0x52485400], [seed & 0xFFFFFFFF, seed >> 32])
        assert np.array_equal(signs, w) and int(signs[0]) & 0xFFFF == oracle.rht_sign_mask(seed)
        eps = np.array([-1.0 if (int(signs[i >> 5]) >> (i & 31)) & 1 else 1.0 for i in range(n)])
        Hp = np.diag(eps) @ H
        assert np.max(np.abs(Hp @ Hp.T - np.eye(n))) < 1e-15
        for i in (0, 1, 15, 16, 17, n // 2, n - 1):              # basis vectors: row i of H', up to the FP32 1/sqrt(n)
            e = np.zeros(n, dtype=np.float32)
            e[i] = 1.0
            assert np.array_equal(oracle.rht_f32(e, n, signs).astype(np.float64), np.sign(Hp[i]) * c32)
        rng = np.random.default_rng(seed & 0xFFFF)
        x = rng.integers(-64, 64, size=n).astype(np.float32)     # small integers: every butterfly step is exact
        want = (x.astype(np.float64) @ (np.sign(Hp))).astype(np.float32) * np.float32(c32)
        assert np.array_equal(oracle.rht_f32(x, n, signs), want.astype(np.float32))
        x = rng.standard_normal(n).astype(np.float32)
        assert np.allclose(oracle.rht_f32(x, n, signs), x.astype(np.float64) @ Hp, rtol=0, atol=4e-6)


@pytest.mark.parametrize("n", [32, 64, 128])
def test_wide_rht_quantizer_rotates_whole_chunks_then_quantizes_16_blocks(n):
    """Quantizing with RHT block n equals quantizing, without rotation, the tensor whose n-wide chunks along the
    reduction dimension were rotated beforehand (values that stay BF16-exact: small integers times a power of two, so
    that the pre-rotated tensor can be handed over in BF16), for both layouts; and the rotation preserves the product."""
    rng = np.random.default_rng(n)
    signs = oracle.rht_signs(5)
    rows, cols = 2 * n, 2 * n
    # entries in {-1, 0, 1} times 2^k: chunk sums stay below 2^8 in magnitude, exact in BF16 after the power-of-two part
    x = rng.integers(-1, 2, size=(rows, cols)).astype(np.float32)
    bits = bf16_bits(x)
    for axis in (AXIS_ROW, AXIS_COL):
        xs = x if axis == AXIS_ROW else x.T
        rot = np.stack([np.concatenate([oracle.rht_f32(r[c:c + n], n, signs) for c in range(0, r.size, n)]) for r in xs])
        if n == 64:                                   # 1/8 is exact: the rotated tensor is itself BF16-exact
            assert np.array_equal(bf16_vals(bf16_bits(rot)), rot.astype(np.float64))
            pre = bf16_bits(rot if axis == AXIS_ROW else rot.T)
            a = oracle.quantize(bits, axis, rht_block=n, seed_rht=5)
            b = oracle.quantize(pre, axis, rht_block=0)
            assert np.array_equal(a.codes, b.codes) and np.array_equal(a.scales, b.scales)
        # any n: the scale of every block is amax of the rotated values over g_max
        q = oracle.quantize(bits, axis, rht_block=n, seed_rht=5)
        amax = np.abs(rot).reshape(rot.shape[0], -1, 16).max(axis=2).astype(np.float32)
        assert np.array_equal(q.scales, (amax / np.float32(7.0)).astype(np.float32))
    # the rotation is orthogonal up to the rounding of 1/sqrt(n): products of rotated operands match the plain product
    X, W = rng.standard_normal((8, 2 * n)).astype(np.float32), rng.standard_normal((6, 2 * n)).astype(np.float32)
    rot = lambda M: np.stack([np.concatenate([oracle.rht_f32(r[c:c + n], n, signs) for c in range(0, r.size, n)]) for r in M])
    assert np.allclose(rot(X).astype(np.float64) @ rot(W).astype(np.float64).T, X.astype(np.float64) @ W.astype(np.float64).T, atol=2e-5)


def test_sign_mask_depends_on_seed_only_through_philox_word0():
    for seed in (0, 1, 2, 0xDEADBEEFCAFEF00D):
        w = oracle.philox4x32_10([0, 0, 0, 0x52485400], [seed & 0xFFFFFFFF, seed >> 32])
        assert oracle.rht_sign_mask(seed) == int(w[0]) & 0xFFFF


# ------------------------------------------------------------------ codebooks and RTNE bins (Sec. 2.1, Sec. 3.1)

def _golden_e2m1():
    levels, bins = None, []
    with open(os.path.join(GOLDEN, "e2m1_grid.txt")) as f:
        for ln in f:
            w = ln.split()
            if not w or w[0].startswith("#"):
                continue
            if w[0] == "levels":
                levels = [float(t) for t in w[1:]]
            elif w[0] == "bin":
                bins.append([float(t) for t in w[1:]])
    return levels, bins


def test_codebooks():
    levels, _ = _golden_e2m1()
    assert oracle.levels(GRID_E2M1).tolist() == levels
    for grid, gmax in ((GRID_INT4, 7.0), (GRID_E1M2, 1.75)):
        L = oracle.levels(grid)
        assert L[0] == 0 and L[-1] == gmax
        assert np.all(np.diff(L) == L[1])          # equal spacing: l_i = r_i in every bin
    assert np.array_equal(oracle.levels(GRID_E1M2) * 4, oracle.levels(GRID_INT4))


def test_nibble_encodings():
    # INT4: two's complement; E1M2 / E2M1: sign bit + 3-bit level index.  E1M2 = 1 sign, 1 exponent, 2 mantissa bits
    # with bias 1: exponent 0 is subnormal (0.mm), exponent 1 is 1.mm.
    for nib in range(16):
        q = nib - 16 if nib & 8 else nib
        assert oracle.nibble_value(GRID_INT4, nib) == q
        e, mm = (nib >> 2) & 1, nib & 3
        mag = (mm / 4.0) if e == 0 else (1.0 + mm / 4.0)
        assert oracle.nibble_value(GRID_E1M2, nib) == (-mag if nib & 8 else mag)
        ee, m = (nib >> 1) & 3, nib & 1          # E2M1: 2 exponent bits (bias 1), 1 mantissa bit
        mag = (m * 0.5) if ee == 0 else (1.0 + m * 0.5) * 2.0 ** (ee - 1)
        assert oracle.nibble_value(GRID_E2M1, nib) == (-mag if nib & 8 else mag)


def _exact_rtne(a: Fraction, levels):
    """Nearest level in exact rational arithmetic; ties to the even index."""
    best, best_d = 0, abs(a - levels[0])
    for i in range(1, len(levels)):
        d = abs(a - levels[i])
        if d < best_d or (d == best_d and i % 2 == 0):
            best, best_d = i, d
    return best


@pytest.mark.parametrize("grid", [GRID_INT4, GRID_E1M2, GRID_E2M1])
def test_rtne_bins_are_midpoint_bins(grid):
    """Eq. 1: the bin of interior level q_i is ((q_{i-1}+q_i)/2, (q_i+q_{i+1})/2)."""
    L = oracle.levels(grid)
    eps = 1e-9
    for i in range(1, 7):
        lo, hi = (L[i - 1] + L[i]) / 2, (L[i] + L[i + 1]) / 2
        for a in (lo + eps, L[i], hi - eps, (lo + hi) / 2):
            assert oracle.round_rtne(a, grid) == i
        assert oracle.round_rtne(lo - eps, grid) == i - 1
        assert oracle.round_rtne(hi + eps, grid) == i + 1
    assert oracle.round_rtne(0.0, grid) == 0
    assert oracle.round_rtne(L[7] * 1.5, grid) == 7      # above the grid: saturate
    # every BF16-representable magnitude in [0, 1.25 g_max], against exact rational arithmetic
    Lf = [Fraction(float(v)) for v in L]
    bits = np.arange(0, 0x7F80, dtype=np.uint16)
    vals = bf16_vals(bits)
    sel = vals[(vals <= 1.25 * L[7])]
    step = max(1, sel.size // 6000)
    for a in sel[::step]:
        assert oracle.round_rtne(float(a), grid) == _exact_rtne(Fraction(float(a)), Lf)


def test_rtne_ties_go_to_even_code():
    # uniform grid: IEEE round-half-even on the code integer (numpy's rint is the library statement of it)
    a = np.arange(0, 7.5, 0.125)
    got = np.array([oracle.round_rtne(float(v), GRID_INT4) for v in a])
    assert np.array_equal(got, np.rint(a).astype(int))
    got = np.array([oracle.round_rtne(float(v) / 4, GRID_E1M2) for v in a])
    assert np.array_equal(got, np.rint(a).astype(int))
    # E2M1 (1 mantissa bit): ties keep the mantissa bit even, i.e. the even code
    ties = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0}
    L = oracle.levels(GRID_E2M1)
    for t, expect in ties.items():
        assert L[oracle.round_rtne(t, GRID_E2M1)] == expect


def test_worked_example_bins_of_the_paper():
    """Footnote to Sec. 3.1: level 2 has bin (1.75, 2.5), l = 0.25, r = 0.5; level 4 the same at double the scale."""
    _, bins = _golden_e2m1()
    L = oracle.levels(GRID_E2M1)
    for level, lo, hi, l_w, r_w, bias in bins:
        i = L.tolist().index(level)
        assert (L[i - 1] + L[i]) / 2 == lo and (L[i] + L[i + 1]) / 2 == hi
        assert (L[i] - L[i - 1]) / 2 == l_w and (L[i + 1] - L[i]) / 2 == r_w
        assert (l_w - r_w) / 2 == bias
        t = np.linspace(lo, hi, 200001)[1:-1]
        got = np.array([L[oracle.round_rtne(float(v), GRID_E2M1)] for v in t[::40]])
        assert np.all(got == level)


@pytest.mark.parametrize("grid", [GRID_INT4, GRID_E1M2, GRID_E2M1])
def test_per_bin_bias_matches_closed_form(grid):
    """Eq. 2: E[rho(t) - t | t in B_i] = (2 q_i - q_{i-1} - q_{i+1}) / 4 under locally uniform density."""
    L = oracle.levels(grid)
    t = (np.arange(400000) + 0.5) / 400000 * L[7]          # uniform density on (0, g_max)
    idx = np.array([oracle.round_rtne(float(v), grid) for v in t])
    for i in range(1, 7):
        closed = (2 * L[i] - L[i - 1] - L[i + 1]) / 4
        measured = np.mean(L[idx[idx == i]] - t[idx == i])
        assert abs(measured - closed) < 2e-4 * L[7]
    if grid == GRID_E2M1:
        closed = [(2 * L[i] - L[i - 1] - L[i + 1]) / 4 for i in range(1, 7)]
        assert closed == [0, 0, 0, -0.125, 0, -0.25]      # the values the paper prints for levels 2 and 4
    else:
        assert all((2 * L[i] - L[i - 1] - L[i + 1]) == 0 for i in range(1, 7))


def test_bin_bias_through_the_quantizer_pipeline():
    """Same closed form, measured by orc_bin_bias on the y values the quantizer itself produced (RHT off)."""
    rng = np.random.default_rng(11)
    for grid, gmax in ((GRID_INT4, 7.0), (GRID_E2M1, 6.0)):
        n_blocks = 60000
        x = rng.uniform(0.0, 1.0, size=(n_blocks, 16)) * rng.choice([-1.0, 1.0], size=(n_blocks, 16))
        x[:, 0] = 1.0                                     # block amax = 1 exactly -> t = |x| * g_max
        q = oracle.quantize(bf16_bits(x), AXIS_ROW, rht_block=0, grid=grid, want_y=True)
        count, mean = oracle.bin_bias(q.y, q.codes, grid)
        L = oracle.levels(grid)
        assert count.sum() == n_blocks * 16
        for i in range(1, 7):
            closed = (2 * L[i] - L[i - 1] - L[i + 1]) / 4
            width = (L[i + 1] - L[i - 1]) / 2
            sigma = width / np.sqrt(12 * count[i])
            # BF16 input spacing (2^-8 relative) adds a small deterministic lumpiness on top of sampling noise
            assert abs(mean[i] - closed) < 4 * sigma + 2e-3 * gmax


# ------------------------------------------------------------------ stochastic rounding (Sec. 2.1)

@pytest.mark.parametrize("grid", [GRID_INT4, GRID_E1M2, GRID_E2M1])
def test_sr_probabilities_and_expectation(grid):
    """Pr[q = g_b] = (a - g_a)/(g_b - g_a): over the 256 equally likely random bytes the count of 'up' outcomes is
    p*256 rounded to an integer, so E[SR(a)] = a to within half a 1/256 step of the gap."""
    L = oracle.levels(grid)
    rng = np.random.default_rng(5)
    pts = np.concatenate([rng.uniform(0, L[7], 300), L, (L[:-1] + L[1:]) / 2, [L[7] * 1.01, L[7] * 2]])
    for a in pts:
        a = float(np.float32(a))
        out = np.array([oracle.round_sr(a, grid, r) for r in range(256)])
        if a >= L[7]:
            assert np.all(out == 7)
            continue
        lo = int(np.searchsorted(L, a, side="right") - 1)
        gap = L[lo + 1] - L[lo]
        assert set(out.tolist()) <= {lo, lo + 1}
        p = Fraction(a) - Fraction(float(L[lo]))
        p = p / Fraction(float(gap))
        n_up = int(np.sum(out == lo + 1))
        assert abs(Fraction(n_up, 256) - p) <= Fraction(1, 512)
        assert abs(np.mean(L[out]) - a) <= gap / 512 + 1e-12
        # monotone in r: small random bytes round up, large ones round down
        assert np.all(np.diff((out == lo + 1).astype(int)) <= 0)
    # exact levels never move
    for i in range(8):
        assert all(oracle.round_sr(float(L[i]), grid, r) == i for r in (0, 127, 255))


def test_sr_expectation_through_the_quantizer():
    """E[SR(x)] = x (Sec. 2.1) measured over many Philox-keyed blocks: |mean - x| <= 2^-9 step + 4 sigma."""
    n_blocks = 40000
    vals = np.array([1.0, 0.3, -0.55, 0.051, 0.77, -0.123, 0.9, 0.004, -0.31, 0.66, 0.5, -0.999, 0.25, 0.42, -0.8, 0.1])
    x = np.tile(vals, (n_blocks, 1))
    bits = bf16_bits(x)
    xv = bf16_vals(bits)[0]
    for grid, gmax in ((GRID_INT4, 7.0), (GRID_E2M1, 6.0)):
        q = oracle.quantize(bits, AXIS_ROW, rht_block=0, grid=grid, rounding=ROUND_SR, seed_sr=2)
        deq = oracle.dequantize(q)
        s = float(q.scales[0, 0])
        assert np.all(q.scales == np.float32(1.0) / np.float32(gmax))
        mean = deq.mean(axis=0)
        step = (2.0 if grid == GRID_E2M1 else 1.0) * s
        assert np.all(np.abs(mean - xv) <= step * (2.0 ** -9) + 4 * 0.5 * step / np.sqrt(n_blocks) + 1e-6)
        # different blocks see different random bytes
        assert len({bytes(q.codes[i]) for i in range(200)}) > 50
        # and a different seed gives different draws, the same seed the same draws
        q2 = oracle.quantize(bits, AXIS_ROW, rht_block=0, grid=grid, rounding=ROUND_SR, seed_sr=3)
        q3 = oracle.quantize(bits, AXIS_ROW, rht_block=0, grid=grid, rounding=ROUND_SR, seed_sr=2)
        assert not np.array_equal(q.codes, q2.codes) and np.array_equal(q.codes, q3.codes)


def test_sr_draws_are_keyed_by_block_index_and_variant():
    """Which random bytes a block sees: block b = o * (K/16) + kb of the variant's own scales array (o = output row,
    kb = block along the reduction axis), variant word 0 for the row layout and 1 for the col layout, element j of the
    block taking byte j.  The codes of a small tensor are rebuilt here from sr_bytes() and round_sr() alone, with the
    scale arithmetic written out in numpy; a transposed, shifted or swapped index in the quantizer would change them."""
    rows, cols = 32, 48
    rng = np.random.default_rng(77)
    bits = bf16_bits(rng.standard_normal((rows, cols)) * np.exp(rng.standard_normal((rows, 1))))
    x = bf16_vals(bits).astype(np.float32)
    seed_sr = 0x1234567_89ABCDEF
    for axis, variant in ((AXIS_ROW, 0), (AXIS_COL, 1)):
        v = x if axis == AXIS_ROW else np.ascontiguousarray(x.T)      # [output row o][reduction index]
        R, K = v.shape
        nkb = K // 16
        for grid, gmax in ((GRID_INT4, 7.0), (GRID_E2M1, 6.0)):
            q = oracle.quantize(bits, axis, rht_block=0, grid=grid, rounding=ROUND_SR, seed_sr=seed_sr)
            L = oracle.levels(grid)
            expect = np.zeros((R, K), dtype=np.int64)
            for o in range(R):
                for kb in range(nkb):
                    blk = v[o, 16 * kb:16 * kb + 16]
                    amax = np.float32(np.max(np.abs(blk)))
                    inv = np.float32(gmax) / amax
                    y = (blk * inv).astype(np.float32)
                    r = oracle.sr_bytes(seed_sr, o * nkb + kb, variant)
                    for j in range(16):
                        idx = oracle.round_sr(abs(float(y[j])), grid, int(r[j]))
                        if grid == GRID_INT4:
                            expect[o, 16 * kb + j] = (-idx if y[j] < 0 else idx) & 0xF
                        else:
                            expect[o, 16 * kb + j] = 0 if idx == 0 else ((8 if y[j] < 0 else 0) | idx)
            got = np.stack([q.codes & 0xF, q.codes >> 4], axis=-1).reshape(R, K)
            assert np.array_equal(got, expect)
            # the mapping matters on this input: the neighbouring block's bytes or the other variant's give other codes
            other = oracle.sr_bytes(seed_sr, 1, variant)
            assert not np.array_equal(other, oracle.sr_bytes(seed_sr, 0, variant))
            assert not np.array_equal(oracle.sr_bytes(seed_sr, 0, 0), oracle.sr_bytes(seed_sr, 0, 1))


def test_a_window_of_a_tensor_quantizes_like_that_part_of_the_whole():
    """orc_quantize_window on a band (row band for the row layout, column band for the col layout, and a band along the
    reduction axis) gives exactly the codes and scales the whole-tensor call gives there, SR draws included."""
    rows, cols = 96, 160
    bits = _rand_bits(rows, cols, 91)
    for rounding in (ROUND_RTNE, ROUND_SR):
        kw = dict(rht_block=16, grid=GRID_INT4, rounding=rounding, seed_rht=3, seed_sr=9)
        full_r = oracle.quantize(bits, AXIS_ROW, **kw)
        full_c = oracle.quantize(bits, AXIS_COL, **kw)
        # rows 32..79, columns 48..127 of the tensor
        r0, r1, c0, c1 = 32, 80, 48, 128
        part = np.ascontiguousarray(bits[r0:r1, c0:c1])
        w = oracle.quantize(part, AXIS_ROW, window=(r0, c0 // 16, cols // 16), **kw)
        assert np.array_equal(w.codes, full_r.codes[r0:r1, c0 // 2:c1 // 2]) and np.array_equal(w.scales, full_r.scales[r0:r1, c0 // 16:c1 // 16])
        w = oracle.quantize(part, AXIS_COL, window=(c0, r0 // 16, rows // 16), **kw)
        assert np.array_equal(w.codes, full_c.codes[c0:c1, r0 // 2:r1 // 2]) and np.array_equal(w.scales, full_c.scales[c0:c1, r0 // 16:r1 // 16])
        if rounding == ROUND_SR:     # and the window's place matters for SR
            w0 = oracle.quantize(part, AXIS_ROW, **kw)
            assert not np.array_equal(w0.codes, full_r.codes[r0:r1, c0 // 2:c1 // 2])


# ------------------------------------------------------------------ the blockwise quantizer (Sec. 2.1, Sec. 4)

def _rand_bits(rows, cols, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    return bf16_bits(rng.standard_normal((rows, cols)) * scale)


@pytest.mark.parametrize("grid,gmax", [(GRID_INT4, 7.0), (GRID_E1M2, 1.75), (GRID_E2M1, 6.0)])
def test_scale_is_amax_over_gmax_and_top_code_is_used(grid, gmax):
    bits = _rand_bits(48, 64, 21, 0.37)
    q = oracle.quantize(bits, AXIS_ROW, rht_block=0, grid=grid)
    amax = np.abs(bf16_vals(bits)).reshape(48, 4, 16).max(axis=2)
    assert np.array_equal(q.scales, (amax.astype(np.float32) / np.float32(gmax)).astype(np.float32))
    lo, hi = q.codes & 0xF, q.codes >> 4
    vals = np.vectorize(lambda n: abs(oracle.nibble_value(grid, int(n))))(np.stack([lo, hi], -1).reshape(48, 4, 16))
    assert np.all(vals.max(axis=2) == gmax)          # no clipping and s = amax / g_max: the top level is always hit


# ------------------------------------------------------------------ range-restricted E2M1 (Sec. 5.4; App. B, max_fpx)

@pytest.mark.parametrize("grid,max_fpx,kept", [(GRID_E2M1_MAX4, 4.0, [0, 0.5, 1, 1.5, 2, 3, 4]),
                                               (GRID_E2M1_MAX2, 2.0, [0, 0.5, 1, 1.5, 2])])
def test_range_restricted_e2m1_levels_scale_and_rounding(grid, max_fpx, kept):
    """Sec. 5.4: max_fpx = 2 keeps only {0, 0.5, 1, 1.5, 2}; the scale divides by max_fpx, the codes are E2M1 codes,
    nothing above max_fpx is ever emitted and the block maximum lands on max_fpx."""
    assert oracle.lib().orc_gmax(grid) == max_fpx
    assert list(oracle.levels(grid)) == list(oracle.levels(GRID_E2M1))          # same codebook behind the nibbles
    for n in range(16):
        assert oracle.nibble_value(grid, n) == oracle.nibble_value(GRID_E2M1, n)
    # rounding onto the kept levels only: brute force over a fine sweep, exact rational nearest-level search
    Lf = [Fraction(v) for v in kept]
    for a in np.linspace(0.0, 7.0, 1401):
        assert oracle.levels(grid)[oracle.round_rtne(float(a), grid)] == float(Lf[_exact_rtne(Fraction(float(a)), Lf)])
        out = {oracle.levels(grid)[oracle.round_sr(float(a), grid, r)] for r in (0, 100, 255)}
        lo = max(v for v in kept if v <= min(a, max_fpx))
        hi = min([v for v in kept if v > a] + [max_fpx])
        assert out <= {lo, hi}
    # through the quantizer
    bits = _rand_bits(48, 64, 31, 0.37)
    amax = np.abs(bf16_vals(bits)).reshape(48, 4, 16).max(axis=2)
    for rounding in (ROUND_RTNE, ROUND_SR):
        q = oracle.quantize(bits, AXIS_ROW, rht_block=0, grid=grid, rounding=rounding, seed_sr=4)
        assert np.array_equal(q.scales, (amax.astype(np.float32) / np.float32(max_fpx)).astype(np.float32))
        mags = np.abs(oracle.dequantize(q) / np.repeat(q.scales.astype(np.float64), 16, axis=1))
        assert set(np.unique(mags).tolist()) <= set(kept)
        assert np.all(mags.reshape(48, 4, 16).max(axis=2) == max_fpx)


def test_max_fpx_2_is_a_uniform_five_level_grid():
    """With max_fpx = 2 the kept levels are the integers 0..4 in half units: the quantizer must agree with a plain
    uniform quantizer, round-half-even of 2 x / s clipped to 4 (numpy's rint), in value and in E2M1 nibble."""
    bits = _rand_bits(40, 96, 32, 2.5)
    x = bf16_vals(bits).astype(np.float32)
    q = oracle.quantize(bits, AXIS_ROW, rht_block=0, grid=GRID_E2M1_MAX2)
    amax = np.abs(x).reshape(40, 6, 16).max(axis=2)
    inv = (np.float32(2.0) / amax.astype(np.float32)).astype(np.float32)
    y = (x * np.repeat(inv, 16, axis=1)).astype(np.float32)
    k = np.clip(np.rint(2.0 * np.abs(y.astype(np.float64))), 0, 4).astype(np.int64)      # level index = half units
    nib = np.where((y < 0) & (k > 0), 8 | k, k).astype(np.uint8)
    assert np.array_equal(q.codes, nib[:, 0::2] | (nib[:, 1::2] << 4))


def test_max_fpx_6_is_the_unrestricted_e2m1():
    """max_fpx = 6 is the E2M1 reference itself (App. B): the restricted rounding rule with all eight levels kept."""
    L = oracle.levels(GRID_E2M1)
    assert oracle.lib().orc_gmax(GRID_E2M1) == 6.0 and oracle.lib().orc_num_levels(GRID_E2M1) == 8
    assert oracle.lib().orc_num_levels(GRID_E2M1_MAX4) == 7 and oracle.lib().orc_num_levels(GRID_E2M1_MAX2) == 5
    for a in np.linspace(0, 4.0, 161):          # below the first dropped midpoint all three rules agree ...
        if a < 1.99:
            assert oracle.round_rtne(float(a), GRID_E2M1) == oracle.round_rtne(float(a), GRID_E2M1_MAX2)
        if a < 3.99:
            assert oracle.round_rtne(float(a), GRID_E2M1) == oracle.round_rtne(float(a), GRID_E2M1_MAX4)
    assert L[oracle.round_rtne(5.5, GRID_E2M1)] == 6.0 and L[oracle.round_rtne(5.5, GRID_E2M1_MAX4)] == 4.0


def test_e1m2_is_int4_with_scale_times_four():
    bits = _rand_bits(32, 64, 22, 3.0)
    for axis in (AXIS_ROW, AXIS_COL):
        for rounding in (ROUND_RTNE, ROUND_SR):
            a = oracle.quantize(bits, axis, 16, GRID_INT4, rounding, seed_rht=1, seed_sr=2)
            b = oracle.quantize(bits, axis, 16, GRID_E1M2, rounding, seed_rht=1, seed_sr=2)
            assert np.array_equal(b.scales, a.scales * np.float32(4.0))
            assert np.array_equal(oracle.dequantize(a), oracle.dequantize(b))


def test_rtne_error_bound_and_sr_error_bound():
    """|x' - Q(x')| <= s/2 for RTNE on the uniform grid, < s for SR (x' the rotated value)."""
    bits = _rand_bits(64, 64, 23)
    mask = oracle.rht_sign_mask(1)
    x = bf16_vals(bits).astype(np.float32)
    xr = np.stack([oracle.rht16_f32(x[r, 16 * b:16 * b + 16], mask) for r in range(64) for b in range(4)])
    xr = xr.reshape(64, 64).astype(np.float64)
    for rounding, bound in ((ROUND_RTNE, 0.5), (ROUND_SR, 1.0)):
        q = oracle.quantize(bits, AXIS_ROW, 16, GRID_INT4, rounding, seed_rht=1, seed_sr=9)
        s = np.repeat(q.scales.astype(np.float64), 16, axis=1)
        err = np.abs(oracle.dequantize(q) - xr)
        assert np.all(err <= bound * s * (1 + 1e-6))


def test_layout_of_row_and_col_variants():
    """A single non-zero element: where its code and scale land, for both variants (RHT off)."""
    rows, cols = 32, 48
    for (r, c) in ((0, 0), (5, 17), (31, 47), (16, 32), (15, 31)):
        x = np.zeros((rows, cols), dtype=np.float32)
        x[r, c] = -3.0
        bits = bf16_bits(x)
        q = oracle.quantize(bits, AXIS_ROW, 0, GRID_INT4)
        assert q.codes.shape == (rows, cols // 2) and q.scales.shape == (rows, cols // 16)
        expect = np.zeros_like(q.codes)
        expect[r, c // 2] = (0x9 if c % 2 == 0 else 0x90)     # -7 in two's complement = 0x9
        assert np.array_equal(q.codes, expect)
        es = np.zeros_like(q.scales)
        es[r, c // 16] = np.float32(3.0) / np.float32(7.0)
        assert np.array_equal(q.scales, es)
        qc = oracle.quantize(bits, AXIS_COL, 0, GRID_INT4)
        assert qc.codes.shape == (cols, rows // 2) and qc.scales.shape == (cols, rows // 16)
        expect = np.zeros_like(qc.codes)
        expect[c, r // 2] = (0x9 if r % 2 == 0 else 0x90)
        assert np.array_equal(qc.codes, expect)
        es = np.zeros_like(qc.scales)
        es[c, r // 16] = np.float32(3.0) / np.float32(7.0)
        assert np.array_equal(qc.scales, es)


def test_col_variant_is_row_variant_of_the_transpose_with_its_own_sr_stream():
    bits = _rand_bits(64, 48, 24)
    bt = np.ascontiguousarray(bits.T)
    for grid in (GRID_INT4, GRID_E2M1):
        a = oracle.quantize(bits, AXIS_COL, 16, grid, ROUND_RTNE, seed_rht=1)
        b = oracle.quantize(bt, AXIS_ROW, 16, grid, ROUND_RTNE, seed_rht=1)
        assert np.array_equal(a.codes, b.codes) and np.array_equal(a.scales, b.scales)
    a = oracle.quantize(bits, AXIS_COL, 16, GRID_INT4, ROUND_SR, seed_rht=1, seed_sr=2)
    b = oracle.quantize(bt, AXIS_ROW, 16, GRID_INT4, ROUND_SR, seed_rht=1, seed_sr=2)
    assert np.array_equal(a.scales, b.scales) and not np.array_equal(a.codes, b.codes)   # variant word differs


def test_rotation_happens_before_scaling_and_rounding():
    """Brute force on one block: rotate in FP64 with the matrix, then s = amax/7 and nearest integer."""
    rng = np.random.default_rng(31)
    mask = oracle.rht_sign_mask(7)
    eps = np.array([-1.0 if (mask >> i) & 1 else 1.0 for i in range(16)])
    Hp = np.diag(eps) @ oracle.hadamard_matrix(16)
    x = rng.integers(-40, 40, size=(8, 16)).astype(np.float32)      # integers: FP32 butterflies are exact
    q = oracle.quantize(bf16_bits(x), AXIS_ROW, 16, GRID_INT4, seed_rht=7, want_y=True)
    xr = x.astype(np.float64) @ Hp
    amax = np.abs(xr).max(axis=1)
    assert np.array_equal(q.scales[:, 0], (amax.astype(np.float32) / np.float32(7)))
    inv = np.float32(7) / amax.astype(np.float32)
    y = (xr.astype(np.float32) * inv[:, None]).astype(np.float32)
    assert np.array_equal(q.y, y)
    codes = np.stack([q.codes & 0xF, q.codes >> 4], -1).reshape(8, 16).astype(np.int64)
    codes = np.where(codes >= 8, codes - 16, codes)
    assert np.array_equal(codes, np.rint(y.astype(np.float64)).astype(np.int64))


def test_zero_and_tiny_blocks():
    x = np.zeros((16, 32), dtype=np.float32)
    x[3, 20] = 1e-35                                   # below 2^-100: treated as a zero block
    x[4, 2] = 2.0
    for fmt in (SCALE_FP32, SCALE_POW2):
        q = oracle.quantize(bf16_bits(x), AXIS_ROW, 16, GRID_INT4, scale_fmt=fmt, seed_rht=1)
        assert np.all(q.codes[3] == 0) and np.all(q.scales[3] == 0)
        assert np.any(q.codes[4, :8] != 0) and q.scales[4, 0] > 0 and q.scales[4, 1] == 0
        assert np.all(np.isfinite(oracle.dequantize(q)))


def test_pow2_scale_is_the_next_power_of_two_and_is_idempotent():
    bits = _rand_bits(32, 64, 25, 0.02)
    q = oracle.quantize(bits, AXIS_ROW, 0, GRID_INT4, scale_fmt=SCALE_POW2)
    f = oracle.quantize(bits, AXIS_ROW, 0, GRID_INT4, scale_fmt=SCALE_FP32)
    m, e = np.frexp(q.scales)
    assert np.all(m == 0.5)                                           # exact powers of two
    assert np.all(q.scales >= f.scales) and np.all(q.scales < 2 * f.scales)
    # q * 2^e is exactly BF16-representable, so quantizing the dequantized tensor reproduces codes and scales
    deq = oracle.dequantize(q)
    again = oracle.quantize(bf16_bits(deq), AXIS_ROW, 0, GRID_INT4, scale_fmt=SCALE_POW2)
    assert np.array_equal(bf16_vals(bf16_bits(deq)), deq)
    assert np.array_equal(again.codes, q.codes) and np.array_equal(again.scales, q.scales)


def test_1x32_blocks_with_a_power_of_two_scale():
    """The MXFP4 block layout of Sec. 2.1's footnote (1 x 32 blocks, E8M0 scale) on the uniform grid: the shared scale is
    the larger of the two halves' power-of-two scales (rounding up to a power of two is monotone), the half that owns it
    keeps its POW2 codes, and every code is round-half-even of x / s clipped to the grid (numpy's rint; no RHT, so x / s is
    an exact division by a power of two)."""
    bits = _rand_bits(32, 128, 41, 1.7)
    bits[3, 32:64] = 0                                          # an all-zero 32-block
    bits[5, 64:80] = 0                                          # a zero half beside a non-zero half
    x = bf16_vals(bits)
    for axis in (AXIS_ROW, AXIS_COL):
        xs = x if axis == AXIS_ROW else x.T
        a = oracle.quantize(bits, axis, rht_block=0, scale_fmt=SCALE_POW2)
        b = oracle.quantize(bits, axis, rht_block=0, scale_fmt=SCALE_E8M0_B32)
        pair = np.maximum(a.scales[:, 0::2], a.scales[:, 1::2])
        assert np.array_equal(b.scales[:, 0::2], pair) and np.array_equal(b.scales[:, 1::2], pair)
        nz = b.scales > 0
        m, e = np.frexp(b.scales[nz])
        assert np.all(m == 0.5)                                 # powers of two: representable in E8M0
        s = np.repeat(b.scales.astype(np.float64), 16, axis=1)
        q = np.zeros_like(xs)
        np.divide(xs, s, out=q, where=s > 0)
        q = np.clip(np.rint(q), -7, 7).astype(np.int64)
        nib = (q & 0xF).astype(np.uint8)
        assert np.array_equal(b.codes, nib[:, 0::2] | (nib[:, 1::2] << 4))
        own = np.repeat(a.scales == b.scales, 8, axis=1)        # per code byte: this half owns the shared scale
        assert np.array_equal(b.codes[own], a.codes[own])
        assert np.all(np.abs(oracle.dequantize(b) - xs) <= s / 2 + 1e-300)
    # with the RHT and SR the block indices and draws stay per 16 elements: only the scale is shared
    a = oracle.quantize(bits, AXIS_ROW, rht_block=16, scale_fmt=SCALE_E8M0_B32, rounding=ROUND_SR, seed_rht=1, seed_sr=2)
    assert np.array_equal(a.scales[:, 0::2], a.scales[:, 1::2])
    w = oracle.quantize(bits, AXIS_ROW, rht_block=64, scale_fmt=SCALE_E8M0_B32, seed_rht=1)
    p = oracle.quantize(bits, AXIS_ROW, rht_block=64, scale_fmt=SCALE_POW2, seed_rht=1)
    pair = np.maximum(p.scales[:, 0::2], p.scales[:, 1::2])
    assert np.array_equal(w.scales[:, 0::2], pair) and np.array_equal(w.scales[:, 1::2], pair)
    with pytest.raises(Exception):
        oracle.quantize(_rand_bits(16, 48, 1), AXIS_ROW, scale_fmt=SCALE_E8M0_B32)      # 48 is not a multiple of 32


def test_e4m3_helpers_round_trip():
    vals = [oracle.e4m3_value(c) for c in range(0x7F)]
    assert vals[0] == 0 and vals[1] == 2.0 ** -9 and vals[0x7E] == 448.0 and vals[0x38] == 1.0
    assert all(b > a for a, b in zip(vals, vals[1:]))
    for c in range(0x7F):
        assert oracle.e4m3_encode(vals[c]) == c
    assert oracle.e4m3_encode(1e9) == 0x7E and oracle.e4m3_encode(0.0) == 0
    for c in range(1, 0x7E):                          # midpoints go to the even code
        mid = (vals[c] + vals[c + 1]) / 2
        assert oracle.e4m3_encode(mid) == (c if c % 2 == 0 else c + 1)


def test_e4m3_tensor_scale_mode_brute_force():
    bits = _rand_bits(16, 64, 26)
    x = bf16_vals(bits)
    ts = float(np.float32(4 * np.abs(x).max() / (7 * 448)))
    q = oracle.quantize(bits, AXIS_ROW, 16, GRID_INT4, scale_fmt=SCALE_E4M3_TENSOR, seed_rht=1, tensor_scale=ts)
    assert q.scales.dtype == np.uint8
    mask = oracle.rht_sign_mask(1)
    deq = oracle.dequantize(q)
    for r in range(16):
        for b in range(4):
            xr = oracle.rht16_f32(x[r, 16 * b:16 * b + 16].astype(np.float32), mask)
            z = np.float32(np.abs(xr).max()) / np.float32(7)
            byte = oracle.e4m3_encode(float(z / np.float32(ts)))
            assert q.scales[r, b] == byte
            s = np.float32(ts) * np.float32(oracle.e4m3_value(byte))
            y = xr * (np.float32(1) / s)
            expect = np.clip(np.rint(y.astype(np.float64)), -7, 7) * float(s)
            assert np.array_equal(deq[r, 16 * b:16 * b + 16], expect)


# ------------------------------------------------------------------ GEMM on dequantized operands (Sec. 2.2)

def test_gemm_reduces_to_integer_matmul_when_scales_are_one():
    rng = np.random.default_rng(41)
    M, N, K = 24, 40, 64
    qa = rng.integers(-7, 8, size=(M, K))
    qb = rng.integers(-7, 8, size=(N, K))
    qa[:, ::16] = 7                                   # amax = 7 in every block -> scale exactly 1 (RHT off)
    qb[:, ::16] = -7
    A = oracle.quantize(bf16_bits(qa), AXIS_ROW, 0, GRID_INT4)
    B = oracle.quantize(bf16_bits(qb), AXIS_ROW, 0, GRID_INT4)
    assert np.all(A.scales == 1) and np.all(B.scales == 1)
    Cm, S = oracle.gemm(A, B)
    assert np.array_equal(Cm, (qa @ qb.T).astype(np.float64))
    assert np.array_equal(S, (np.abs(qa) @ np.abs(qb).T).astype(np.float64))
    # not symmetric in its operands: C is [M][N] with A's rows first
    assert Cm.shape == (M, N)
    c, s = oracle.gemm_sampled(A, B, [0, 3, 23], [0, 39, 7])
    assert np.array_equal(c, Cm[[0, 3, 23], [0, 39, 7]]) and np.array_equal(s, S[[0, 3, 23], [0, 39, 7]])
    c2, _ = oracle.gemm_sampled(A, B, [3], [39], 16, 48)
    assert c2[0] == float(qa[3, 16:48] @ qb[39, 16:48])


def test_gemm_one_hot_operands_pick_out_entries():
    K = 32
    a = np.zeros((16, K), dtype=np.float32)
    b = np.zeros((16, K), dtype=np.float32)
    for i in range(16):
        a[i, i] = 2.0
        b[i, (i + 1) % 16] = 3.0
    A = oracle.quantize(bf16_bits(a), AXIS_ROW, 0, GRID_INT4, scale_fmt=SCALE_POW2)
    B = oracle.quantize(bf16_bits(b), AXIS_ROW, 0, GRID_INT4, scale_fmt=SCALE_POW2)
    Cm, _ = oracle.gemm(A, B)
    # POW2 scale of amax 2 is 2/7 -> 0.5, code 4; of amax 3: 3/7 -> 0.5, code 6: values are exact
    expect = np.zeros((16, 16))
    for i in range(16):
        expect[(i + 1) % 16, i] = 6.0
    assert np.array_equal(Cm, expect)


def test_freivalds_and_closeness_to_the_unquantized_product():
    rng = np.random.default_rng(43)
    M, N, K = 48, 32, 128
    X = rng.standard_normal((M, K))
    W = rng.standard_normal((N, K)) * 0.02
    xb, wb = bf16_bits(X), bf16_bits(W)
    exact = bf16_vals(xb) @ bf16_vals(wb).T
    errs = {}
    for grid in (GRID_INT4, GRID_E2M1):
        A = oracle.quantize(xb, AXIS_ROW, 16, grid, seed_rht=1)
        B = oracle.quantize(wb, AXIS_ROW, 16, grid, seed_rht=1)
        Cm, S = oracle.gemm(A, B)
        v = rng.standard_normal(N)
        lhs = Cm @ v
        rhs = oracle.dequantize(A) @ (oracle.dequantize(B).T @ v)
        assert np.max(np.abs(lhs - rhs)) <= 1e-12 * np.max(S)
        errs[grid] = np.linalg.norm(Cm - exact) / np.linalg.norm(exact)
        assert errs[grid] < 0.25        # same rotation on both operands: only quantization error remains
    # a different rotation on the two operands breaks the identity (XH')(WH')^T = XW^T
    A = oracle.quantize(xb, AXIS_ROW, 16, GRID_INT4, seed_rht=1)
    B = oracle.quantize(wb, AXIS_ROW, 16, GRID_INT4, seed_rht=5)
    assert oracle.rht_sign_mask(1) != oracle.rht_sign_mask(5)
    Cm, _ = oracle.gemm(A, B)
    assert np.linalg.norm(Cm - exact) / np.linalg.norm(exact) > 0.5


# ------------------------------------------------------------------ tensor diagnostics (Eq. 3, Eq. 6, Eq. 7)

def test_effective_bucket_ratio_spans_one_over_k_to_one():
    """Eq. 6: B_eff = exp(entropy) / K is 1/K when one bucket holds everything and 1 for uniform use of the K = 8 buckets."""
    one = np.zeros(8)
    one[3] = 1000.0
    assert abs(oracle.diagnostics_from_sums(np.concatenate([[1, 0, 0], one, np.zeros(8)]))["b_eff"] - 1 / 8) < 1e-9
    flat = np.full(8, 125.0)
    assert abs(oracle.diagnostics_from_sums(np.concatenate([[1, 0, 0], flat, np.zeros(8)]))["b_eff"] - 1.0) < 1e-9
    two = np.zeros(8)
    two[[0, 5]] = 500.0                                     # two equally used buckets: exp(log 2) / 8
    assert abs(oracle.diagnostics_from_sums(np.concatenate([[1, 0, 0], two, np.zeros(8)]))["b_eff"] - 2 / 8) < 1e-9


@pytest.mark.parametrize("grid", [GRID_INT4, GRID_E1M2, GRID_E2M1])
def test_diagnostics_of_exactly_representable_and_of_zero_tensors(grid):
    """A tensor that lies on the grid quantizes without error: NMSE = 0, alpha = 1 (Eq. 3), zero bias in every bin; an
    all-zero tensor uses one bucket (B_eff = 1/8)."""
    rng = np.random.default_rng(5)
    L = oracle.levels(grid)
    idx = rng.integers(0, 8, size=(32, 64))
    idx[:, ::16] = 7                                        # every block holds g_max, so its scale is a power of two
    x = L[idx] * rng.choice([-1.0, 1.0], size=idx.shape) * 2.0 ** rng.integers(-3, 4, size=(32, 1))
    xb = bf16_bits(x)
    q = oracle.quantize(xb, AXIS_ROW, rht_block=0, grid=grid)
    d = oracle.diagnose(xb, q, 0, 0)
    assert d["nmse"] == 0.0 and d["alpha"] == 1.0
    assert np.all(np.nan_to_num(d["bias"]) == 0.0)
    assert np.array_equal(d["count"], np.bincount(idx.reshape(-1), minlength=8))
    z = np.zeros((16, 32), dtype=np.uint16)
    dz = oracle.diagnose(z, oracle.quantize(z, AXIS_ROW, rht_block=16, grid=grid, seed_rht=3), 16, 3)
    assert abs(dz["b_eff"] - 1 / 8) < 1e-9 and dz["count"][0] == 16 * 32


def test_diagnostics_against_a_matrix_formulation():
    """The same sums from independent ingredients: x' by an FP64 matrix product with H'_16, xq by the dequantizer; the
    residual of the projection is orthogonal to x' (Eq. 3), and quantization noise on a uniform grid with unit scale has
    variance 1/12 per element."""
    rng = np.random.default_rng(11)
    x = rng.standard_normal((48, 160)) * np.exp(rng.standard_normal((48, 1)))
    xb = bf16_bits(x)
    mask = oracle.rht_sign_mask(7)
    eps = np.array([-1.0 if (mask >> i) & 1 else 1.0 for i in range(16)])
    Hp = np.diag(eps) @ oracle.hadamard_matrix(16)
    for grid in (GRID_INT4, GRID_E2M1):
        q = oracle.quantize(xb, AXIS_ROW, rht_block=16, grid=grid, seed_rht=7)
        d = oracle.diagnose(xb, q, 16, 7)
        xp = (bf16_vals(xb).reshape(48, 10, 16) @ Hp).reshape(48, 160)
        xq = oracle.dequantize(q)
        assert np.isclose(d["sums"][0], np.sum(xp * xp), rtol=1e-6)
        assert np.isclose(d["nmse"], np.sum((xq - xp) ** 2) / np.sum(xp * xp), rtol=1e-4)
        assert np.isclose(d["alpha"], np.sum(xq * xp) / np.sum(xp * xp), rtol=1e-6)
        assert abs(np.sum((xq - d["alpha"] * xp) * xp)) < 1e-6 * np.sum(xp * xp)
    # unit-scale uniform grid: every block holds 7 (scale exactly 1), the other elements are uniform in (-7, 7)
    u = rng.uniform(-7, 7, size=(256, 256))
    u[:, ::16] = 7.0
    ub = bf16_bits(u)
    q = oracle.quantize(ub, AXIS_ROW, rht_block=0, grid=GRID_INT4)
    assert np.all(q.scales == 1.0)
    d = oracle.diagnose(ub, q, 0, 0)
    n_free = 256 * 256 * 15 / 16
    assert abs(d["sums"][1] / n_free - 1 / 12) < 0.003      # BF16 inputs are themselves on a fine grid: still 1/12
    assert np.nanmax(np.abs(d["bias"][1:7])) < 0.01         # symmetric bins: no bias (Sec. 3.1)


def test_diagnostics_with_a_wide_rht_block_equal_those_of_the_pre_rotated_tensor():
    """RHT block 64 on entries in {-1, 0, 1} (the rotated tensor is BF16-exact, 1/8 being a power of two): the sums of
    orc_diagnose must be those of the pre-rotated tensor quantized without rotation; the rotation preserves the energy."""
    rng = np.random.default_rng(64)
    x = rng.integers(-1, 2, size=(48, 256)).astype(np.float32)
    bits = bf16_bits(x)
    signs = oracle.rht_signs(5)
    rot = np.stack([np.concatenate([oracle.rht_f32(r[c:c + 64], 64, signs) for c in range(0, r.size, 64)]) for r in x])
    pre = bf16_bits(rot)
    for grid in (GRID_INT4, GRID_E2M1):
        a = oracle.diagnose(bits, oracle.quantize(bits, AXIS_ROW, rht_block=64, grid=grid, seed_rht=5), 64, 5)
        b = oracle.diagnose(pre, oracle.quantize(pre, AXIS_ROW, rht_block=0, grid=grid), 0, 5)
        assert np.array_equal(a["sums"], b["sums"]) and np.array_equal(a["count"], b["count"])
        assert a["sums"][0] == float(np.sum(x.astype(np.float64) ** 2))
