"""Pins of the per-round CPU oracle against facts the paper and the mathematics
fix (no GPU). A plausible mistake in the oracle - wrong Philox constant, wrong
sign or offset in the fixed-point rounding, swapped index in packing or in the
decode sum - fails at least one of these."""
import ctypes
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import roundpath as orp

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def identity_code(n):
    return np.arange(n + 1, dtype=np.int32), np.arange(n, dtype=np.int32), np.ones(n, np.float32)


# ------------------------------------------------------------------ Philox
def _curand_host():
    for name in ("libcurand.so.10", "/usr/local/cuda/lib64/libcurand.so.10", "libcurand.so"):
        try:
            return ctypes.CDLL(name)
        except OSError:
            continue
    return None


def test_philox_matches_curand_host_generator():
    """Independent library routine: cuRAND's HOST Philox4_32_10 generator (runs on
    the CPU). Found by observation: its block t (4 words) is the Philox block of
    counter (t // 65536, 0, t % 65536, 0) under key = (seed_lo, seed_hi)."""
    lib = _curand_host()
    if lib is None:
        pytest.skip("libcurand not found")
    for seed in (0, 1, 0x123456789ABCDEF0, 0xDEADBEEFCAFEF00D):
        gen = ctypes.c_void_p()
        assert lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) == 0
        assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
        nblk = 3 * 65536 + 17
        out = np.zeros(4 * nblk, np.uint32)
        assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p),
                                  ctypes.c_size_t(out.size)) == 0
        lib.curandDestroyGenerator(gen)
        out = out.reshape(-1, 4)
        key = [seed & 0xFFFFFFFF, seed >> 32]
        rng = np.random.default_rng(seed & 0xFFFF)
        picks = np.unique(np.concatenate([[0, 1, 65535, 65536, 65537, nblk - 1],
                                          rng.integers(0, nblk, 3000)]))
        for t in picks:
            t = int(t)
            got = orp.philox4x32_10([t // 65536, 0, t % 65536, 0], key)
            assert (got == out[t]).all(), (seed, t)


def test_philox_is_a_bijection_and_diffuses():
    """For a fixed key Philox is a permutation of the counter space: distinct
    counters give distinct blocks; flipping one counter bit flips about half of
    the 128 output bits."""
    key = [0xA4093822, 0x299F31D0]
    seen = set()
    rng = np.random.default_rng(0)
    flips = []
    for _ in range(2000):
        ctr = rng.integers(0, 2 ** 32, 4, dtype=np.uint64).astype(np.uint32)
        a = orp.philox4x32_10(ctr, key)
        seen.add(a.tobytes())
        c2 = ctr.copy()
        word, bit = rng.integers(0, 4), rng.integers(0, 32)
        c2[word] ^= np.uint32(1 << bit)
        b = orp.philox4x32_10(c2, key)
        flips.append(sum(bin(int(x) ^ int(y)).count("1") for x, y in zip(a, b)))
    assert len(seen) == 2000
    assert 60 < np.mean(flips) < 68


def test_uniform15_lane_selection_and_uniformity():
    """Eight stream positions share one block; even positions take the low 15 bits
    of their word, odd ones the high 15 bits. Each draw is in [0, 2^15) and the
    draws are uniform (chi-square on 64 bins)."""
    seed, rnd, worker = 0x0123456789ABCDEF, (7 << 32) | 5, 3
    for pos in (0, 1, 2, 7, 8, 1234567, (1 << 33) + 5):
        blk = orp.philox4x32_10([(pos >> 3) & 0xFFFFFFFF, worker, rnd & 0xFFFFFFFF, rnd >> 32],
                                [seed & 0xFFFFFFFF, seed >> 32])
        word = int(blk[(pos & 7) >> 1])
        want = (word >> 17) if pos & 1 else (word & 0x7FFF)
        assert orp.uniform15(seed, rnd, worker, pos) == want
    u = np.array([orp.uniform15(11, 0, 0, pos) for pos in range(200_000)])
    assert u.min() >= 0 and u.max() < 32768
    hist = np.bincount(u >> 9, minlength=64)
    chi2 = ((hist - len(u) / 64) ** 2 / (len(u) / 64)).sum()
    assert chi2 < 120  # 63 dof: mean 63, 120 is beyond the 99.99th percentile
    # different workers / rounds / seeds give different streams
    assert orp.uniform15(11, 0, 1, 0) != orp.uniform15(11, 0, 0, 0) or \
        orp.uniform15(11, 0, 1, 8) != orp.uniform15(11, 0, 0, 8)
    assert [orp.uniform15(11, 1, 0, t) for t in range(8)] != [orp.uniform15(11, 0, 0, t) for t in range(8)]
    assert [orp.uniform15(12, 0, 0, t) for t in range(8)] != [orp.uniform15(11, 0, 0, t) for t in range(8)]


# ------------------------------------------------------------------ quantiser, one coordinate
@pytest.mark.parametrize("b", [1, 2, 3, 4, 5, 6, 7, 8])
def test_quantizer_exactly_unbiased_by_enumeration_of_all_uniforms(b):
    """E[Q(x) | x] = x (Sec. II-B). Brute force: enumerate ALL 2^15 values of the
    uniform for one coordinate; the mean dequantised value equals x up to the
    2^-15-of-a-step resolution of the uniform, and the variance equals the
    closed form step^2 * f(1-f) <= step^2/4 (the paper's per-coordinate bound)."""
    rng = np.random.default_rng(b)
    S = np.float32(3.7)
    inv = np.float32(orp.inv_scale(S, b))
    step = (S / ((1 << (b - 1)) - 1)) if b >= 2 else 2.0 * S
    xs = np.concatenate([rng.uniform(-S, S, 6), [0.0, S, -S, S / 3, -S * 0.999]]).astype(np.float32)
    for x in xs:
        vals = np.array([orp.dequantize_one(orp.quantize_one(float(x), float(inv), b, u), float(S), b)
                         for u in range(0, 32768)], np.float64)
        assert abs(vals.mean() - float(x)) <= step * (2.0 ** -15) + 2e-6 * float(S), (b, x)
        y = (float(x) / float(S)) * (((1 << (b - 1)) - 1) if b >= 2 else 0.5)
        if b == 1:
            y += 0.5
        f = y - np.floor(y)
        assert abs(vals.var() - step ** 2 * f * (1 - f)) <= step ** 2 * 2e-4
        assert vals.var() <= step ** 2 / 4 + 1e-12
        # only the two neighbouring grid points occur
        assert len(np.unique(vals)) <= 2


def _exact_code(x, inv, b, u):
    """The quantiser's definition in exact rational arithmetic: the sum
    x*inv + offset + u rounded to the nearest integer (ties to the even one),
    then the floor of its quotient by 2^15. Written twice over: directly, and as
    one fp32 fused multiply-add into a float of [2^23, 2^24), whose spacing is 1,
    so that its rounding to nearest-even IS the rounding to an integer."""
    offset = (((1 << (b - 1)) - 1) << 15) if b >= 2 else (1 << 14)
    t = Fraction(float(x)) * Fraction(float(inv)) + offset + u
    whole = t.numerator // t.denominator
    frac = t - whole
    fixed = whole + (1 if frac > Fraction(1, 2) or (frac == Fraction(1, 2) and whole % 2 == 1) else 0)
    direct = fixed // (1 << 15)
    # the fused form: t + 2^23 < 2^24 always, and |x| <= S keeps t above -L 2^-9 > -1/4,
    # so a sum below 2^23 (where floats are 1/2 apart) still rounds to 2^23 itself
    s = t + (1 << 23)
    assert (1 << 23) - Fraction(1, 4) < s < (1 << 24)
    sw = s.numerator // s.denominator
    sf = s - sw
    mant = sw + (1 if sf > Fraction(1, 2) or (sf == Fraction(1, 2) and sw % 2 == 1) else 0)
    if s < (1 << 23):
        mant = 1 << 23
    assert (mant - (1 << 23)) // (1 << 15) == direct
    return direct


def test_quantizer_equals_exact_rational_arithmetic_on_every_case():
    """Equality, not statistics: >= 10^5 random (x, S, b, u) and hand-picked boundary
    cases (y an integer, y = +-L, x = +-S, tiny x, exact ties of the 15-bit fraction)
    against the definition evaluated with exact rationals."""
    rng = np.random.default_rng(2024)
    cases = []
    for _ in range(100_000):
        b = int(rng.integers(1, 9))
        S = np.float32(10.0 ** rng.uniform(-12, 12))
        kind = rng.integers(0, 4)
        if kind == 0:
            x = np.float32(rng.uniform(-1, 1)) * S
        elif kind == 1:   # near a level: y close to an integer
            L = max((1 << (b - 1)) - 1, 1)
            x = np.float32(rng.integers(-L, L + 1) / L) * S
            x = np.nextafter(x, np.float32(rng.choice([-np.inf, np.inf])), dtype=np.float32) if rng.random() < 0.5 else x
        elif kind == 2:   # tiny against the scale
            x = np.float32(rng.uniform(-1, 1)) * S * np.float32(2.0 ** -int(rng.integers(10, 60)))
        else:
            x = np.float32(rng.standard_normal()) * S * np.float32(0.3)
        x = np.float32(np.clip(x, -S, S))
        u = int(rng.integers(0, 32768)) if rng.random() < 0.9 else int(rng.choice([0, 1, 32766, 32767]))
        cases.append((x, S, b, u))
    # hand-picked: powers of two make x * inv an exact integer or an exact half
    for b in range(1, 9):
        L = (1 << (b - 1)) - 1 if b >= 2 else 1
        for S in (np.float32(1.0), np.float32(2.0 ** -40), np.float32(3.0), np.float32(2.0 ** 50)):
            for x in (S, -S, np.float32(0.0), np.float32(-0.0), S / 2, -S / 2, S * np.float32(2.0 ** -16),
                      -S * np.float32(2.0 ** -16), S * np.float32(2.0 ** -15), S * np.float32(3 * 2.0 ** -17),
                      -S * np.float32(3 * 2.0 ** -17), S * np.float32(1e-30), -S * np.float32(1e-30),
                      S * np.float32(1 / L) if L else S):
                for u in (0, 1, 2, 16383, 16384, 32766, 32767):
                    cases.append((np.float32(x), S, b, u))
    ties = 0
    for x, S, b, u in cases:
        inv = np.float32(orp.inv_scale(float(S), b))
        got = orp.quantize_one(float(x), float(inv), b, u)
        want = _exact_code(x, inv, b, u)
        assert got == want, (float(x), float(S), b, u, got, want)
        assert 0 <= got <= (2 * ((1 << (b - 1)) - 1) if b >= 2 else 1)
        y = Fraction(float(x)) * Fraction(float(inv))
        ties += (y * 2).denominator == 1 and y.denominator == 2
    assert ties > 50   # the exact-half cases were really exercised


def test_reciprocal_scale_is_the_correctly_rounded_quotient():
    """inv = fl(L 2^15 / S): the exact quotient lies within half a unit in the last
    place of the returned float (ties: the even neighbour)."""
    rng = np.random.default_rng(77)
    for _ in range(20_000):
        b = int(rng.integers(1, 9))
        num = (((1 << (b - 1)) - 1) << 15) if b >= 2 else (1 << 14)
        S = np.float32(2.0 ** rng.uniform(-60, 60) * rng.uniform(1, 2))
        q = np.float32(orp.inv_scale(float(S), b))
        exact = Fraction(num) / Fraction(float(S))
        lo = Fraction(float(np.nextafter(q, np.float32(0))))
        hi = Fraction(float(np.nextafter(q, np.float32(np.inf))))
        qf = Fraction(float(q))
        assert abs(exact - qf) <= (qf - lo) / 2 and abs(exact - qf) <= (hi - qf) / 2, (b, float(S))
        if abs(exact - qf) == (hi - qf) / 2 or abs(exact - qf) == (qf - lo) / 2:
            assert (int(np.float32(q).view(np.uint32)) & 1) == 0


@pytest.mark.parametrize("b", [2, 3, 5, 8])
def test_quantizer_against_the_plain_rule_of_the_paper(b):
    """Eq. rv_quant with nothing rounded: level = floor(L*x/S + u/2^15) in exact rationals
    on the floats x and S. The oracle keeps y = L*x/S to 15 fractional bits and multiplies by
    the rounded reciprocal scale, so it may differ from the unrounded rule only when
    y*2^15 + u lies within one unit (2^-15 of a level step) of a level boundary, and then by
    one level. Every disagreement is listed with the side the exact arithmetic takes; the
    float64 evaluation of the same rule is reported beside it."""
    rng = np.random.default_rng(100 + b)
    L = (1 << (b - 1)) - 1
    S = np.float32(0.0123)
    inv = np.float32(orp.inv_scale(S, b))
    N = 20000
    xs = [np.float32(rng.uniform(-float(S), float(S))) for _ in range(N)]
    us = [int(rng.integers(0, 32768)) for _ in range(N)]
    # plus inputs placed next to a boundary on purpose
    for lvl in range(-L, L):
        for du in (-2, -1, 0, 1, 2):
            u = int(rng.integers(4, 32760))
            y_units = (lvl + 1) * 32768 - u + du          # y*2^15 + u = boundary + du
            xs.append(np.float32(y_units / 32768.0 / L * float(S)))
            us.append(u)
    differ = []
    for x, u in zip(xs, us):
        code = orp.quantize_one(float(x), float(inv), b, u)
        t = Fraction(L) * Fraction(float(x)) / Fraction(float(S)) * 32768 + u
        exact = (t / 32768).numerator // (t / 32768).denominator   # floor of an exact rational
        want = exact + L
        t64 = L * float(x) / float(S) * 32768.0 + u
        want64 = int(np.floor(t64 / 32768.0)) + L
        if code != want:
            dist = abs(t - round(t / 32768) * 32768)
            differ.append((float(x), u, code, want, want64, float(dist)))
            assert abs(code - want) == 1
            assert dist <= 1, differ[-1]
    # about 2 / 32768 of random inputs fall that close to a boundary; the planted ones add a few
    assert len(differ) <= 12 + 3 * 2 * L, differ


def test_quantizer_special_cases():
    """One-hot vector: the non-zero coordinate is sent as exactly +-S (code 2L or 0);
    zero vector: scale 0 and every code the zero level; scaling the input by a
    power of two leaves the codes unchanged and scales the norm."""
    rp, ci, a = identity_code(1)
    for b in (2, 4, 8):
        L = (1 << (b - 1)) - 1
        G = np.zeros((1, 512), np.float32)
        G[0, 77] = -2.5
        codes, scales, st, _ = orp.encode_quantize(rp, ci, a, [b], 512, 5, 0, G)
        assert st == 0 and scales[0, 0] == np.float32(2.5)
        deq = orp.dequantize_worker(512, b, 512, codes, scales[0])
        assert deq[77] == np.float32(-2.5) and np.count_nonzero(deq) == 1
        G[0, 77] = 2.5
        codes, scales, st, _ = orp.encode_quantize(rp, ci, a, [b], 512, 5, 0, G)
        assert orp.dequantize_worker(512, b, 512, codes, scales[0])[77] == np.float32(2.5)
        Z = np.zeros((1, 512), np.float32)
        codes, scales, st, _ = orp.encode_quantize(rp, ci, a, [b], 512, 5, 0, Z)
        assert st == 0 and scales[0, 0] == 0
        assert (orp.dequantize_worker(512, b, 512, codes, scales[0]) == 0).all()
        # every b-bit field holds the zero level L
        bitstr = "".join(format(int(wd), "032b")[::-1] for wd in codes)
        fields = {int(bitstr[t * b:(t + 1) * b][::-1], 2) for t in range(512)}
        assert fields == {L}
    rng = np.random.default_rng(3)
    G = rng.standard_normal((1, 1024)).astype(np.float32)
    c1, s1, _, _ = orp.encode_quantize(rp, ci, a, [5], 256, 9, 4, G)
    c2, s2, _, _ = orp.encode_quantize(rp, ci, a, [5], 256, 9, 4, G * np.float32(2.0 ** -7))
    assert (c1 == c2).all() and (s2 == s1 * np.float32(2.0 ** -7)).all()


def test_nonfinite_and_tiny_buckets_are_flushed():
    rp, ci, a = identity_code(1)
    G = np.ones((1, 1024), np.float32)
    G[0, 600] = np.nan
    codes, scales, st, _ = orp.encode_quantize(rp, ci, a, [4], 512, 1, 0, G)
    assert st & orp.STATUS_NONFINITE
    assert scales[0, 1] == 0 and scales[0, 0] > 0
    G = np.full((1, 512), 1e-30, np.float32)  # squares underflow
    codes, scales, st, _ = orp.encode_quantize(rp, ci, a, [4], 512, 1, 0, G)
    assert st == 0 and scales[0, 0] == 0


@pytest.mark.parametrize("B", [128, 256, 512])
def test_bucket_norm_is_the_l2_norm(B):
    """Scale = ||x||_2 over the bucket (Eq. quant_def); the last bucket is ragged."""
    rng = np.random.default_rng(B)
    d = 3 * 512 + 200
    G = (rng.standard_normal((1, d)) * 10.0 ** rng.uniform(-3, 3, d)).astype(np.float32)
    rp, ci, a = identity_code(1)
    _, scales, st, _ = orp.encode_quantize(rp, ci, a, [4], B, 1, 0, G)
    nb = (d + B - 1) // B
    assert scales.shape == (1, nb)
    for beta in range(nb):
        ref = np.sqrt(np.sum(G[0, beta * B:(beta + 1) * B].astype(np.float64) ** 2))
        assert abs(scales[0, beta] - ref) <= 4e-7 * ref


def test_codes_never_leave_their_range_on_adversarial_inputs():
    """|x| <= S must hold for every coordinate so that level stays in [-L, L]:
    one-hot buckets, equal-magnitude buckets, huge and tiny magnitudes."""
    rp, ci, a = identity_code(1)
    rng = np.random.default_rng(5)
    for b in (1, 2, 8):
        for trial in range(40):
            G = np.zeros((1, 512), np.float32)
            kind = trial % 4
            mag = np.float32(10.0 ** rng.uniform(-15, 15))
            if kind == 0:
                G[0, rng.integers(0, 512)] = mag * rng.choice([-1, 1])
            elif kind == 1:
                G[0, :] = mag * rng.choice([-1, 1], 512)
            elif kind == 2:
                G[0, :2] = [mag, -mag * np.float32(1e-4)]
            else:
                G[0, :] = mag * rng.standard_normal(512)
            for rnd in range(3):
                _, _, st, _ = orp.encode_quantize(rp, ci, a, [b], 512, trial, rnd, G)
                assert st == 0


# ------------------------------------------------------------------ vector-level statistics
def test_unbiasedness_and_variance_bound_monte_carlo():
    """E[Q(x)] = x and E||Q(x)-x||^2 <= phi(z)||x||^2 with phi = B/(4 L^2) per
    bucket (Sec. II-B), by Monte-Carlo over rounds; the exact variance
    sum (S/L)^2 f(1-f) is matched too."""
    rng = np.random.default_rng(17)
    d, B, b = 1024, 256, 3
    L = 3
    G = rng.standard_normal((1, d)).astype(np.float32)
    rp, ci, a = identity_code(1)
    rounds = 3000
    acc = np.zeros(d)
    err2 = 0.0
    for t in range(rounds):
        codes, scales, _, _ = orp.encode_quantize(rp, ci, a, [b], B, 99, t, G)
        q = orp.dequantize_worker(d, b, B, codes, scales[0]).astype(np.float64)
        acc += q
        err2 += np.sum((q - G[0]) ** 2)
    mean = acc / rounds
    S = np.repeat(scales[0].astype(np.float64), B)
    step = S / L
    y = np.abs(G[0].astype(np.float64)) / step
    f = y - np.floor(y)
    var = step ** 2 * f * (1 - f)
    z = (mean - G[0]) / np.sqrt(np.maximum(var, 1e-30) / rounds)
    assert np.abs(z[var > 1e-12]).max() < 5.5
    assert abs(err2 / rounds - var.sum()) < 0.03 * var.sum()
    bound = sum(B / (4 * L * L) * np.sum(G[0, t * B:(t + 1) * B].astype(np.float64) ** 2)
                for t in range(d // B))
    assert err2 / rounds <= bound


# ------------------------------------------------------------------ packing / layout
def test_stream_position_is_a_block_permutation():
    pos = [orp.stream_position(m) for m in range(3 * 512)]
    for q in range(3):
        assert sorted(pos[q * 512:(q + 1) * 512]) == list(range(q * 512, (q + 1) * 512))


def test_hand_built_layout_examples():
    """Hand-derived from the wire format: offset o = 128c + 4l + e sits at stream
    position 16l + 4c + e, b bits per position, little-endian words. With b = 8 a
    one-hot +S coordinate is the byte 0xFE among 0x7F bytes."""
    rp, ci, a = identity_code(1)
    cases = {}
    with open(os.path.join(GOLDEN, "layout_examples.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if line:
                m, word, shift = (int(t) for t in line.split())
                cases[m] = (word, shift)
    assert len(cases) >= 6
    for m, (word, shift) in cases.items():
        G = np.zeros((1, 1024), np.float32)
        G[0, m] = 1.0
        codes, _, _, _ = orp.encode_quantize(rp, ci, a, [8], 512, 0, 0, G)
        expect = np.full(codes.shape, 0x7F7F7F7F, np.uint32)
        blk = m // 512
        # the other block holds an all-zero bucket: zero level everywhere as well
        expect[word] = (0x7F7F7F7F & ~(0xFF << shift)) | (0xFE << shift)
        assert (codes == expect).all(), m
        assert word // 128 == blk


def test_hand_built_layout_examples_where_a_code_straddles_two_words():
    """b = 3 and b = 5: a one-hot +-S coordinate whose field crosses a word boundary. The
    two words it touches are hand-derived (golden file); every other word must be the
    periodic background of zero-level fields, stated here by its bit rule."""
    rp, ci, a = identity_code(1)
    rows = []
    with open(os.path.join(GOLDEN, "layout_examples_odd_widths.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if line:
                t = line.split()
                rows.append((int(t[0]), int(t[1]), int(t[2]), int(t[3]), int(t[4], 16), int(t[5], 16)))
    assert len(rows) >= 4 and {r[0] for r in rows} == {3, 5}
    for b, m, sign, w0, first, second in rows:
        G = np.zeros((1, 1024), np.float32)
        G[0, m] = 0.75 * sign
        codes, scales, st, _ = orp.encode_quantize(rp, ci, a, [b], 512, 0, 0, G)
        assert st == 0 and codes.size == 2 * 16 * b
        expect = np.zeros(codes.size, np.uint32)
        for blk in range(2):
            for wd in range(16 * b):
                bits = [0 if (32 * wd + s) % b == b - 1 else 1 for s in range(32)]
                expect[blk * 16 * b + wd] = sum(v << s for s, v in enumerate(bits))
        expect[w0], expect[w0 + 1] = first, second
        assert (codes == expect).all(), (b, m, sign, [hex(int(c)) for c in codes[w0:w0 + 2]])


@pytest.mark.parametrize("b", [1, 2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("d", [1, 511, 512, 513, 1500])
def test_pack_roundtrip_and_sizes(b, d):
    """unpack(pack(codes)) reproduces every coordinate to within one quantisation
    step for every bit width and ragged length; message sizes are whole blocks."""
    rng = np.random.default_rng(b * 1000 + d)
    G = rng.standard_normal((1, d)).astype(np.float32)
    rp, ci, a = identity_code(1)
    codes, scales, st, x = orp.encode_quantize(rp, ci, a, [b], 128, 3, 1, G, want_x=True)
    assert st == 0
    assert (x[0] == G[0]).all()
    assert codes.size == ((d + 511) // 512) * 16 * b
    deq = orp.dequantize_worker(d, b, 128, codes, scales[0])
    S = np.repeat(scales[0], 128)[:d]
    step = S / ((1 << (b - 1)) - 1) if b >= 2 else 2 * S
    assert (np.abs(deq - G[0]) <= step * (1 + 1e-6)).all()


# ------------------------------------------------------------------ encode / decode
def test_encode_is_the_weighted_sum_in_partition_order():
    """f_i = sum_j a_ij g_j (Sec. II-A), checked against float64 and, for the
    order, against an explicit float32 fma chain on a case where order matters."""
    rng = np.random.default_rng(2)
    k, n, d = 5, 3, 700
    G = (rng.standard_normal((k, d)) * 10.0 ** rng.uniform(-4, 4, (k, 1))).astype(np.float32)
    rp = np.array([0, 2, 5, 6], np.int32)
    ci = np.array([0, 3, 1, 2, 4, 4], np.int32)
    a = rng.uniform(0.1, 2.0, 6).astype(np.float32)
    _, _, _, x = orp.encode_quantize(rp, ci, a, [4, 4, 4], 128, 1, 0, G, want_x=True)
    dense = np.zeros((n, k))
    for i in range(n):
        for e in range(rp[i], rp[i + 1]):
            dense[i, ci[e]] = a[e]
    ref = dense @ G.astype(np.float64)
    mag = np.abs(dense) @ np.abs(G.astype(np.float64))
    assert (np.abs(x - ref) <= 3 * 6e-8 * mag + 1e-30).all()


def test_decode_special_cases_and_linearity_in_the_mask():
    """All workers received, identity code, w = 1: g_hat = sum_i Q(g_i). Empty
    mask: g_hat = 0. Exact enumeration of all 2^n straggler patterns: the
    probability-weighted mean of the decoded vectors equals
    sum_i (1-p_i) w_i q_i (the estimator is linear in the indicators)."""
    rng = np.random.default_rng(4)
    n, d, B = 4, 1300, 256
    bits = np.array([2, 3, 4, 8], np.uint8)
    p = np.array([0.1, 0.2, 0.3, 0.4])
    w = rng.uniform(0.5, 2.0, n).astype(np.float32)
    G = rng.standard_normal((n, d)).astype(np.float32)
    rp, ci, a = identity_code(n)
    codes, scales, _, _ = orp.encode_quantize(rp, ci, a, bits, B, 8, 2, G)
    off = orp.worker_word_offsets(d, bits)
    q = np.stack([orp.dequantize_worker(d, int(bits[i]), B, codes[off[i]:off[i + 1]], scales[i])
                  for i in range(n)]).astype(np.float64)
    ones = np.ones(n, np.float32)
    ghat, _ = orp.decode(d, bits, B, ones, np.ones((1, n), np.uint8), codes, scales)
    assert np.abs(ghat[0] - q.sum(0)).max() <= 1e-5 * np.abs(q).sum(0).max()
    ghat0, _ = orp.decode(d, bits, B, w, np.zeros((1, n), np.uint8), codes, scales)
    assert (ghat0 == 0).all()
    masks = np.array(list(itertools.product([0, 1], repeat=n)), np.uint8)
    gh, _ = orp.decode(d, bits, B, w, masks, codes, scales)
    prob = np.prod(np.where(masks == 1, 1 - p, p), axis=1)
    mean = (prob[:, None] * gh.astype(np.float64)).sum(0)
    want = (((1 - p) * w.astype(np.float64))[:, None] * q).sum(0)
    assert np.abs(mean - want).max() <= 2e-6 * np.abs(want).max()
    # single survivor = that worker's scaled message
    for i in range(n):
        m1 = np.zeros((1, n), np.uint8)
        m1[0, i] = 1
        g1, _ = orp.decode(d, bits, B, w, m1, codes, scales)
        assert np.abs(g1[0] - float(w[i]) * q[i]).max() <= 1e-6 * np.abs(q[i]).max() * w[i]


def test_batched_decode_equals_single_calls_and_update_rule():
    """R realisations against one set of messages equal R separate decodes; the
    fused update is beta <- beta - lr_r * g_hat_r in order (Eq. update_param)."""
    rng = np.random.default_rng(6)
    n, d, B = 5, 900, 128
    bits = np.array([1, 2, 5, 8, 3], np.uint8)
    w = rng.uniform(0.5, 2.0, n).astype(np.float32)
    G = rng.standard_normal((n, d)).astype(np.float32)
    rp, ci, a = identity_code(n)
    codes, scales, _, _ = orp.encode_quantize(rp, ci, a, bits, B, 1, 0, G)
    masks = (rng.random((6, n)) > 0.3).astype(np.uint8)
    lr = rng.uniform(0.01, 0.1, 6).astype(np.float32)
    beta0 = rng.standard_normal(d).astype(np.float32)
    gh, beta = orp.decode(d, bits, B, w, masks, codes, scales, lr=lr, beta=beta0)
    ref = beta0.astype(np.float64).copy()
    for r in range(6):
        g1, _ = orp.decode(d, bits, B, w, masks[r:r + 1], codes, scales)
        assert (g1[0] == gh[r]).all()
        ref -= float(lr[r]) * gh[r].astype(np.float64)
    assert np.abs(beta - ref).max() <= 1e-6 * np.abs(ref).max()


def test_block_entry_points_agree_with_whole_vector_drivers():
    rng = np.random.default_rng(8)
    n, k, d, B = 3, 4, 1100, 256
    bits = np.array([3, 8, 1], np.uint8)
    rp = np.array([0, 2, 4, 6], np.int32)
    ci = np.array([0, 1, 1, 2, 0, 3], np.int32)
    a = rng.uniform(0.2, 1.0, 6).astype(np.float32)
    w = rng.uniform(0.5, 2.0, n).astype(np.float32)
    G = rng.standard_normal((k, d)).astype(np.float32)
    codes, scales, _, _ = orp.encode_quantize(rp, ci, a, bits, B, 21, 3, G)
    off = orp.worker_word_offsets(d, bits)
    mask = np.array([1, 0, 1], np.uint8)
    gh, _ = orp.decode(d, bits, B, w, mask[None], codes, scales)
    for q in range(3):
        Gblk = np.zeros((k, 512), np.float32)
        hi = min(d, (q + 1) * 512)
        Gblk[:, :hi - q * 512] = G[:, q * 512:hi]
        cb, sb, _, _ = orp.encode_block(rp, ci, a, bits, B, 21, 3, q, Gblk)
        wb = 0
        for i in range(n):
            nw = 16 * int(bits[i])
            assert (cb[wb:wb + nw] == codes[off[i] + q * nw: off[i] + (q + 1) * nw]).all()
            wb += nw
        gb = orp.decode_block(bits, B, w, mask, cb, sb)
        assert (gb[:hi - q * 512] == gh[0, q * 512:hi]).all()


def test_adam_two_track_against_torch_adam_and_float64():
    """The Adam step of the two-track variant (Sec. V-E). With g_v = g_w it is plain Adam:
    compare several steps with torch.optim.Adam (an independent library routine) and with
    the published recursion in float64; with g_v != g_w only the second moment changes."""
    import torch
    rng = np.random.default_rng(4)
    d = 1000
    lr, b1, b2, eps = 1e-2, 0.9, 0.999, 1e-8
    beta0 = rng.standard_normal(d).astype(np.float32)
    grads = [rng.standard_normal(d).astype(np.float32) * 10.0 ** rng.uniform(-3, 1) for _ in range(6)]
    beta, m, u = beta0.copy(), np.zeros(d, np.float32), np.zeros(d, np.float32)
    tp = torch.nn.Parameter(torch.from_numpy(beta0.copy()))
    opt = torch.optim.Adam([tp], lr=lr, betas=(b1, b2), eps=eps)
    b64, m64, u64 = beta0.astype(np.float64), np.zeros(d), np.zeros(d)
    for t, g in enumerate(grads, start=1):
        beta, m, u = orp.adam_two_track(g, g, lr, b1, b2, eps, t, beta, m, u)
        tp.grad = torch.from_numpy(g.copy())
        opt.step()
        m64 = b1 * m64 + (1 - b1) * g
        u64 = b2 * u64 + (1 - b2) * g.astype(np.float64) ** 2
        b64 = b64 - lr * (m64 / (1 - b1 ** t)) / (np.sqrt(u64 / (1 - b2 ** t)) + eps)
        assert np.abs(beta - tp.detach().numpy()).max() <= 2e-6 * max(1.0, np.abs(beta).max())
        assert np.abs(beta - b64).max() <= 2e-6 * max(1.0, np.abs(b64).max())
    # second track: only u (and through it the step) sees g_v
    gw, gv = grads[0], grads[1]
    z = np.zeros(d, np.float32)
    _, m1, u1 = orp.adam_two_track(gw, gv, lr, b1, b2, eps, 1, beta0, z, z)
    b1f, b2f = float(np.float32(b1)), float(np.float32(b2))   # the decay rates as fp32 holds them
    assert np.allclose(m1, (1 - b1f) * gw, rtol=1e-6, atol=0)
    assert np.allclose(u1, (1 - b2f) * gv.astype(np.float64) ** 2, rtol=1e-6, atol=0)


def test_global_norm_encoder_pins():
    """The paper's main formulation (Sec. II-B, Eq. quant_def with ||x||_2 over all d). (i) For
    d <= 512 there is one block and one bucket: codes and scale must equal the bucket-wise
    path with B = 512 bit for bit; (ii) the scale is the l2 norm of f_i (float64) to fp32
    accuracy; (iii) a zero worker is sent as zero codes with scale 0; (iv) E[Q(x)] = x by
    Monte-Carlo over rounds, error shrinking like 1/sqrt(rounds)."""
    rng = np.random.default_rng(21)
    n = k = 4
    bits = np.array([2, 3, 5, 8], np.uint8)
    rp = np.arange(n + 1, dtype=np.int32)
    ci = np.arange(n, dtype=np.int32)
    a = np.ones(n, np.float32)
    # (i)
    for d in (1, 77, 512):
        G = rng.standard_normal((k, d)).astype(np.float32)
        c1, s1, st1, _ = orp.encode_quantize_global(rp, ci, a, bits, 3, 5, G)
        c2, s2, st2, _ = orp.encode_quantize(rp, ci, a, bits, 512, 3, 5, G)
        assert st1 == 0 and st2 == 0
        assert (c1 == c2).all() and (s1.view(np.uint32) == s2[:, 0].view(np.uint32)).all()
    # (ii), (iii)
    d = 512 * 37 + 123
    G = (rng.standard_normal((k, d)) * 10.0 ** rng.uniform(-3, 2, (k, 1))).astype(np.float32)
    G[2] = 0.0
    codes, scales, st, x = orp.encode_quantize_global(rp, ci, a, bits, 3, 5, G, want_x=True)
    assert st == 0
    want = np.sqrt((x.astype(np.float64) ** 2).sum(axis=1))
    assert np.allclose(scales, want, rtol=3e-6, atol=0) and scales[2] == 0.0
    off = orp.worker_word_offsets(d, bits)
    q2 = orp.dequantize_worker(d, int(bits[2]), 512, codes[off[2]:off[3]], np.zeros(orp.num_blocks(d), np.float32))
    assert (q2 == 0).all()
    # every code inside its range: |x| <= S for each coordinate
    for i in (0, 1, 3):
        qi = orp.dequantize_worker(d, int(bits[i]), 512, codes[off[i]:off[i + 1]],
                                   np.full(orp.num_blocks(d), scales[i], np.float32))
        L = (1 << (int(bits[i]) - 1)) - 1
        assert np.abs(qi - x[i]).max() <= scales[i] / L * 1.0001
    # (iv)
    d = 700
    G = rng.standard_normal((k, d)).astype(np.float32)
    acc = np.zeros((n, d))
    rounds = 2000
    for t in range(rounds):
        codes, scales, _, x = orp.encode_quantize_global(rp, ci, a, bits, 9, t, G, want_x=True)
        off = orp.worker_word_offsets(d, bits)
        for i in range(n):
            acc[i] += orp.dequantize_worker(d, int(bits[i]), 512, codes[off[i]:off[i + 1]],
                                            np.full(orp.num_blocks(d), scales[i], np.float32))
    for i in range(n):
        L = (1 << (int(bits[i]) - 1)) - 1
        sigma = scales[i] / L / 2.0 / np.sqrt(rounds)       # per-coordinate std of the mean is at most this
        assert np.abs(acc[i] / rounds - x[i]).max() <= 6.0 * sigma


def test_grouped_bucket_encoder_pins():
    """Buckets of 1024 / 2048 / 4096 coordinates (whole groups of pack blocks), pinned from both
    ends and from outside: (i) a group of one block is the 512-bucket encoder bit for bit;
    (ii) a group that covers every block is the global-norm encoder bit for bit; (iii) every
    bucket's scale equals the float64 l2 norm of that stretch of f_i to fp32 accuracy, a zero
    stretch is sent as zero codes with scale 0, and every dequantised value lies within one
    level step of its bucket; (iv) the bucket boundaries are where they should be: changing one
    value changes the scale of its own bucket only; (v) E[Q(x)] = x by Monte-Carlo."""
    rng = np.random.default_rng(33)
    n = k = 4
    bits = np.array([2, 3, 5, 8], np.uint8)
    rp = np.arange(n + 1, dtype=np.int32)
    ci = np.arange(n, dtype=np.int32)
    a = np.ones(n, np.float32)
    d = 512 * 9 + 77                                    # 10 pack blocks, the last one ragged
    G = (rng.standard_normal((k, d)) * 10.0 ** rng.uniform(-2, 2, (k, 1))).astype(np.float32)
    # (i)
    c1, s1, st1, _ = orp.encode_quantize_grouped(rp, ci, a, bits, 512, 3, 5, G)
    c2, s2, st2, _ = orp.encode_quantize(rp, ci, a, bits, 512, 3, 5, G)
    assert st1 == 0 and st2 == 0 and (c1 == c2).all() and (s1.view(np.uint32) == s2.view(np.uint32)).all()
    # (ii)
    c1, s1, _, _ = orp.encode_quantize_grouped(rp, ci, a, bits, 512 * 16, 3, 5, G)
    c2, s2, _, _ = orp.encode_quantize_global(rp, ci, a, bits, 3, 5, G)
    assert s1.shape == (n, 1) and (c1 == c2).all() and (s1[:, 0].view(np.uint32) == s2.view(np.uint32)).all()
    # (iii)
    G[2, 2048:4096] = 0.0
    for B in (1024, 2048, 4096):
        codes, scales, st, x = orp.encode_quantize_grouped(rp, ci, a, bits, B, 3, 5, G, want_x=True)
        nb = (d + B - 1) // B
        assert st == 0 and scales.shape == (n, nb)
        xp = np.zeros((n, nb * B))
        xp[:, :d] = x
        want = np.sqrt((xp.reshape(n, nb, B) ** 2).sum(axis=2))
        assert np.allclose(scales, want, rtol=3e-6, atol=0)
        per_block = orp.expand_grouped_scales(scales, d, B)
        assert per_block.shape == (n, orp.num_blocks(d))
        off = orp.worker_word_offsets(d, bits)
        for i in range(n):
            qi = orp.dequantize_worker(d, int(bits[i]), 512, codes[off[i]:off[i + 1]], per_block[i])
            L = (1 << (int(bits[i]) - 1)) - 1
            step = np.repeat(per_block[i], 512)[:d] / L
            assert (np.abs(qi - x[i]) <= step * 1.0001).all()
        t0 = 2048 // B
        if B <= 2048:
            assert (scales[2, t0:4096 // B] == 0.0).all()
            assert (orp.dequantize_worker(d, int(bits[2]), 512, codes[off[2]:off[3]], per_block[2])[2048:4096] == 0).all()
    # (iv)
    for B in (1024, 2048):
        _, s_a, _, _ = orp.encode_quantize_grouped(rp, ci, a, bits, B, 3, 5, G)
        G2 = G.copy()
        m = 3 * 1024 + 5
        G2[1, m] += 100.0
        _, s_b, _, _ = orp.encode_quantize_grouped(rp, ci, a, bits, B, 3, 5, G2)
        changed = np.argwhere(s_a.view(np.uint32) != s_b.view(np.uint32))
        assert changed.tolist() == [[1, m // B]]
    # (v)
    d = 1500
    G = rng.standard_normal((k, d)).astype(np.float32)
    acc = np.zeros((n, d))
    rounds = 1500
    for t in range(rounds):
        codes, scales, _, x = orp.encode_quantize_grouped(rp, ci, a, bits, 1024, 9, t, G, want_x=True)
        off = orp.worker_word_offsets(d, bits)
        per_block = orp.expand_grouped_scales(scales, d, 1024)
        for i in range(n):
            acc[i] += orp.dequantize_worker(d, int(bits[i]), 512, codes[off[i]:off[i + 1]], per_block[i])
    for i in range(n):
        L = (1 << (int(bits[i]) - 1)) - 1
        sigma = np.repeat(per_block[i], 512)[:d] / L / 2.0 / np.sqrt(rounds)
        assert (np.abs(acc[i] / rounds - x[i]) <= 6.0 * sigma + 1e-12).all()


def test_global_norm_split_into_ranges_pins():
    """The global norm over a vector split into contiguous ranges of pack blocks: with every range
    but the last a power-of-two number of blocks the combined sums, and hence every code and
    scale, equal the unsplit encoder's bit for bit; the sums agree with float64; an uneven split
    gives the same sum up to the order of additions; a changed value in one range changes the
    codes of the others only through the norm."""
    rng = np.random.default_rng(71)
    n, k = 3, 4
    d = 512 * 11 + 37                     # 12 pack blocks
    rp = np.array([0, 2, 3, 5], np.int32)
    ci = np.array([0, 1, 2, 1, 3], np.int32)
    a = rng.uniform(0.2, 1.5, 5).astype(np.float32)
    bits = np.array([2, 5, 8], np.uint8)
    G = (rng.standard_normal((k, d)) * 10.0 ** rng.uniform(-2, 2, (k, 1))).astype(np.float32)
    whole_c, whole_s, st, x = orp.encode_quantize_global(rp, ci, a, bits, 13, 2, G, want_x=True)
    whole_sums = orp.global_sumsq(rp, ci, a, G)
    ref64 = (x.astype(np.float64) ** 2).sum(axis=1)
    assert np.allclose(whole_sums, ref64, rtol=2e-6)
    assert (np.sqrt(whole_sums).astype(np.float32).view(np.uint32) == whole_s.view(np.uint32)).all()
    off = orp.worker_word_offsets(d, bits)
    for per in (4, 8):                    # blocks per range: powers of two -> ranges of 4,4,4 and 8,4
        cuts = list(range(0, 12, per)) + [12]
        sums = np.stack([orp.global_sumsq(rp, ci, a, np.ascontiguousarray(G[:, b0 * 512:min(b1 * 512, d)]))
                         for b0, b1 in zip(cuts[:-1], cuts[1:])])
        comb = orp.combine_sumsq(sums)
        assert (comb.view(np.uint32) == whole_sums.view(np.uint32)).all()
        for b0, b1 in zip(cuts[:-1], cuts[1:]):
            Gr = np.ascontiguousarray(G[:, b0 * 512:min(b1 * 512, d)])
            c, s, st = orp.encode_quantize_with_norm(rp, ci, a, bits, 13, 2, Gr, comb, first_block=b0)
            assert st == 0 and (s.view(np.uint32) == whole_s.view(np.uint32)).all()
            roff = orp.worker_word_offsets(Gr.shape[1], bits)
            for i in range(n):
                b = int(bits[i])
                want = whole_c[off[i] + b0 * 16 * b: off[i] + b1 * 16 * b]
                assert (c[roff[i]:roff[i + 1]] == want).all(), (per, b0, i)
    # an uneven split (5 + 7 blocks): the same sum in another order
    sums = np.stack([orp.global_sumsq(rp, ci, a, np.ascontiguousarray(G[:, :5 * 512])),
                     orp.global_sumsq(rp, ci, a, np.ascontiguousarray(G[:, 5 * 512:]))])
    comb = orp.combine_sumsq(sums)
    assert np.allclose(comb, ref64, rtol=2e-6)
    # the order is the pairwise tree: (r0 + r1) + (r2 + r3), a last range without partner + 0;
    # values chosen so that left-to-right and right-to-left sums give another float
    e = 2.0 ** -24
    v = np.array([[e], [1.0], [e], [e]], np.float32)
    assert orp.combine_sumsq(v)[0] == np.float32(1.0 + 2.0 ** -23)        # left to right: 1.0
    v = np.array([[e], [e], [1.0]], np.float32)
    assert orp.combine_sumsq(v)[0] == np.float32(1.0 + 2.0 ** -23)        # right to left: 1.0
    assert orp.combine_sumsq(v[:1])[0] == np.float32(e)
