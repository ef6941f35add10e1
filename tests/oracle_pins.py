"""Pins for the CPU oracle: facts the paper and plain mathematics fix, checked with exact
rational arithmetic (fractions.Fraction) or closed forms, never with the oracle itself.

Every function asserts; the mutation tests call the same functions against deliberately
broken builds of the oracle and expect at least one of them to fail.
"""
from __future__ import annotations

import math
from fractions import Fraction

import numpy as np

from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import synth

FB = synth.STANDIN_FORMATBOOK


def bf16_value(bits: int) -> Fraction:
    """Exact value of a finite bf16 bit pattern."""
    s, e, m = bits >> 15, (bits >> 7) & 0xFF, bits & 0x7F
    assert e != 0xFF
    mag = Fraction(m, 128) * Fraction(2) ** (-126) if e == 0 else (1 + Fraction(m, 128)) * Fraction(2) ** (e - 127)
    return -mag if s else mag


def f32_value(x) -> Fraction:
    return Fraction(float(x))


def floor_log2(a: Fraction) -> int:
    assert a > 0
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    assert Fraction(2) ** e <= a < Fraction(2) ** (e + 1)
    return e


def unpack_codes(row: np.ndarray) -> np.ndarray:
    out = np.empty(row.shape[-1] * 2, dtype=np.uint8)
    out[0::2] = row & 15
    out[1::2] = row >> 4
    return out


def rand_block_bits(rng, B, scale_exp_range=(-20, 20), zero_frac=0.1):
    """Random bf16 block as bit patterns: mixed magnitudes, some zeros, both signs."""
    e = rng.integers(*scale_exp_range)
    vals = rng.standard_t(3, size=B) * 2.0 ** e
    vals[rng.random(B) < zero_frac] = 0.0
    return synth.f32_to_bf16_bits(vals.astype(np.float32))


# ---------------------------------------------------------------- sizes / metadata (Table 1)

def pin_effective_bits(golden_path):
    for line in open(golden_path):
        if line.startswith("#") or not line.strip():
            continue
        B, printed = line.split()
        B, printed = int(B), float(printed)
        C = 4 * B
        x = synth.f32_to_bf16_bits(np.linspace(-3, 3, 2 * C, dtype=np.float32).reshape(2, C))
        q = orc.quantize(x, FB, orc.Config(block_size=B))
        # 4-bit codes + 10 bits of metadata (5-bit dialect id, 5-bit exponent) per block
        bits = (q.codes.size * 8 + (q.meta.size) * 10) / x.size
        assert q.codes.shape == (2, C // 2) and q.meta.shape == (2, C // B)
        assert abs(bits - (4 + 10 / B)) < 1e-12
        assert abs(bits - printed) < 0.006       # the table prints two decimals
        assert int(q.did.max()) < 32 and int(q.did.min()) >= 0


# ---------------------------------------------------------------- normalisation (Sec. 3.1)

def pin_scale_is_floor_log2(seed=0, n=300):
    rng = np.random.default_rng(seed)
    for _ in range(n):
        bits = rand_block_bits(rng, 32, (-100, 100))
        q = orc.quantize(bits.reshape(1, 32), FB)
        vals = [abs(bf16_value(int(b))) for b in bits]
        amax = max(vals)
        e = int(q.exponent[0, 0])
        if amax == 0:
            assert e == -124
            continue
        assert e == max(-124, floor_log2(amax))
        if floor_log2(amax) >= -124:
            vmax = amax * Fraction(2) ** (3 - e)
            assert 8 <= vmax < 16          # "maximum in [8,16)"
        assert int(q.meta[0, 0] & 0xFF) == e + 124   # E8M0 code of 2^(e-3)


def pin_exponent_clamp():
    cfg = orc.Config(exp_min=-15, exp_max=16)
    big = synth.f32_to_bf16_bits(np.full(32, 2.0 ** 40, dtype=np.float32))
    small = synth.f32_to_bf16_bits(np.full(32, 2.0 ** -40, dtype=np.float32))
    qb = orc.quantize(big.reshape(1, 32), FB, cfg)
    qs = orc.quantize(small.reshape(1, 32), FB, cfg)
    assert int(qb.exponent[0, 0]) == 16 and int(qs.exponent[0, 0]) == -15
    # clamped from above: every element saturates at the largest magnitude of the dialect
    d = int(qb.did[0, 0])
    y = orc.dequantize(qb, FB)
    assert np.all(y == float(FB[d, 7]) * 2.0 ** 13)
    assert np.all(orc.dequantize(qs, FB) == 0.0)


def pin_zero_block():
    """All-zero block (silent in the paper): exponent = exp_min, every dialect of the lowest
    dynamic range ties so the lowest id wins, sign bits of -0 are kept, decode gives +-0."""
    bits = np.zeros(32, dtype=np.uint16)
    bits[[3, 17]] = 0x8000
    for cfg in (orc.Config(), orc.Config(exp_min=-15, exp_max=16)):
        q = orc.quantize(bits.reshape(1, 32), FB, cfg)
        assert int(q.exponent[0, 0]) == cfg.exp_min
        assert int(q.did[0, 0]) == min(d for d in range(32) if int(FB[d, 7]) == 8)
        codes = unpack_codes(q.codes[0])
        assert np.array_equal(codes, np.where(bits == 0x8000, 8, 0))
        y = orc.dequantize(q, FB)[0]
        assert np.all(y == 0) and np.array_equal(np.signbit(y), bits == 0x8000)


# ---------------------------------------------------------------- rounding (Sec. 3.2)

def pin_rounding_is_nearest(seed=1, n=200):
    """Every code is a nearest magnitude of the chosen dialect (exact rationals); exact
    half-way cases go to the larger magnitude."""
    rng = np.random.default_rng(seed)
    for it in range(n):
        B = 32 if it % 2 == 0 else 16
        bits = rand_block_bits(rng, B)
        q = orc.quantize(bits.reshape(1, B), FB, orc.Config(block_size=B))
        d, e = int(q.did[0, 0]), int(q.exponent[0, 0])
        codes = unpack_codes(q.codes[0])
        for b, c in zip(bits, codes):
            v = abs(bf16_value(int(b))) * Fraction(2) ** (3 - e)
            chosen = int(FB[d, c & 7])
            dist = abs(v - chosen)
            for m in FB[d]:
                assert dist <= abs(v - int(m))
                if abs(v - int(m)) == dist:
                    assert int(m) <= chosen
            assert (c >> 3) == (int(b) >> 15)        # sign bit copied, also for zeros


def pin_uniform_dialect_closed_form():
    """For the uniform dialect {0,2,...,14} nearest-with-ties-up is floor((v+1)/2), capped at 7."""
    d = next(i for i in range(32) if list(FB[i]) == [0, 2, 4, 6, 8, 10, 12, 14])
    # all bf16 magnitudes v in [0,15): block = that value + one element pinning the scale (v=14 -> e=0, 14*2^-3)
    pats = [p for p in range(0x0000, 0x7F80) if bf16_value(p) * 8 < 15]
    pats = pats[:: max(1, len(pats) // 4000)] + [synth.f32_to_bf16_bits(np.array([k / 16], np.float32))[0] for k in range(0, 30)]
    setter = synth.f32_to_bf16_bits(np.array([14 / 8], np.float32))[0]
    for p in pats:
        p = int(p)
        blk = np.zeros(32, dtype=np.uint16)
        blk[0], blk[5] = setter, p
        q = orc.quantize(blk.reshape(1, 32), FB, cluster_id=np.zeros(1, np.int32),
                         cluster_mask=np.array([1 << d], np.uint32))
        assert int(q.did[0, 0]) == d and int(q.exponent[0, 0]) == 0
        v = bf16_value(p) * 8
        want = min(7, math.floor((v + 1) / 2))
        assert int(unpack_codes(q.codes[0])[5] & 7) == want


def pin_representable_values_roundtrip():
    """Every representable value of every dialect, both signs, several exponents, decodes to itself."""
    for d in range(32):
        top = int(FB[d, 7])
        for e in (-124, -60, -3, 0, 5, 100, 127):
            for j in range(8):
                for sgn in (1.0, -1.0):
                    mag = int(FB[d, j])
                    vals = np.zeros(32, dtype=np.float64)
                    vals[31] = math.ldexp(top, e - 3)       # fixes the block exponent and dynamic range
                    vals[7] = sgn * math.ldexp(mag, e - 3)
                    bits = synth.f32_to_bf16_bits(vals.astype(np.float32))
                    assert np.all(synth.bf16_bits_to_f32(bits).astype(np.float64) == vals)
                    q = orc.quantize(bits.reshape(1, 32), FB, cluster_id=np.zeros(1, np.int32),
                                     cluster_mask=np.array([1 << d], np.uint32))
                    assert int(q.did[0, 0]) == d and int(q.exponent[0, 0]) == e
                    y = orc.dequantize(q, FB)[0]
                    assert y[7] == vals[7] and y[31] == vals[31] and np.all(y[:7] == 0)
                    assert np.signbit(y[7]) == (sgn < 0)


def pin_single_nonzero_block_truncates(patterns=None):
    """A block with one nonzero element x: two-stage selection picks a dialect whose largest
    magnitude is floor(v), so xhat keeps the leading 4 significant bits of x (truncation);
    checked for bf16 bit patterns against exact rational arithmetic."""
    if patterns is None:
        patterns = range(0, 0x10000)
    pats = np.array([p for p in patterns if ((p >> 7) & 0xFF) != 0xFF], dtype=np.uint16)
    x = np.zeros((len(pats), 32), dtype=np.uint16)
    pos = np.arange(len(pats)) % 32
    x[np.arange(len(pats)), pos] = pats
    q = orc.quantize(x, FB)
    y = orc.dequantize(q, FB)
    for i, p in enumerate(pats):
        p = int(p)
        a = abs(bf16_value(p))
        got = f32_value(y[i, pos[i]])
        if a == 0:
            assert got == 0 and int(q.exponent[i, 0]) == -124
        else:
            e = max(-124, floor_log2(a))
            v = a * Fraction(2) ** (3 - e)
            want = math.floor(v) * Fraction(2) ** (e - 3) if v >= 8 else None
            assert int(q.exponent[i, 0]) == e
            if want is not None:
                assert abs(got) == want, (hex(p), got, want)
                assert int(FB[int(q.did[i, 0]), 7]) == math.floor(v)
            else:   # below the clamp: nearest value of a dialect whose top is 8
                assert int(FB[int(q.did[i, 0]), 7]) == 8
                dd = FB[int(q.did[i, 0])]
                assert abs(abs(got) * Fraction(2) ** (3 - e) - v) == min(abs(int(m) - v) for m in dd)
        assert bool(np.signbit(y[i, pos[i]])) == bool(p >> 15)
        assert np.count_nonzero(y[i]) <= 1


# ---------------------------------------------------------------- approximate error and selection (Sec. 3.2)

def _group_max_v(bits, e, B, G):
    v = [abs(bf16_value(int(b))) * Fraction(2) ** (3 - e) for b in bits]
    gs = B // G
    return v, [max(v[g * gs:(g + 1) * gs]) for g in range(G)]


def pin_error_terms_and_argmin(seed=2, n=150):
    """err_q4[d] = sum over the G contiguous group maxima of |bin midpoint - nearest magnitude|
    (exact, in quarter units); it stays within G/4 of the true absolute error of the group
    maxima; the chosen dialect is the lowest-id minimiser inside the stage-1 group."""
    rng = np.random.default_rng(seed)
    for it in range(n):
        B, G = [(32, 8), (16, 8), (32, 32), (16, 16)][it % 4]
        cfg = orc.Config(block_size=B, num_groups=G)
        bits = rand_block_bits(rng, B)
        if it % 7 == 0:                       # few distinct values => ties between dialects
            bits[:] = bits[rng.integers(0, 2, size=B)]
        q = orc.quantize(bits.reshape(1, B), FB, cfg, want_errors=True)
        d_star, e = int(q.did[0, 0]), int(q.exponent[0, 0])
        v, gm = _group_max_v(bits, e, B, G)
        vmax = max(v)
        bucket = max(8, math.floor(vmax)) if vmax < 16 else 15
        cands = [d for d in range(32) if int(FB[d, 7]) == bucket]
        err = q.err_q4[0, 0]
        assert [d for d in range(32) if err[d] >= 0] == cands
        for d in cands:
            total, exact = Fraction(0), Fraction(0)
            for m in gm:
                k = min(31, math.floor(2 * m))
                mid = Fraction(2 * k + 1, 4)
                t = min(abs(mid - int(f)) for f in FB[d])
                # closed form of the midpoint error: |2k+1-4r|/4 with r the nearest magnitude
                r = min((int(f) for f in FB[d]), key=lambda f: abs(mid - f))
                assert t == Fraction(abs(2 * k + 1 - 4 * r), 4)
                true = min(abs(m - int(f)) for f in FB[d])
                assert abs(t - true) <= Fraction(1, 4)
                total += t
                exact += true
            assert Fraction(int(err[d]), 4) == total
            assert abs(total - exact) <= Fraction(G, 4)
        best = min(int(err[d]) for d in cands)
        assert int(err[d_star]) == best and d_star == min(d for d in cands if int(err[d]) == best)
        # the block maximum always lands on the top magnitude of the chosen dialect
        if 8 <= vmax < 16:
            codes = unpack_codes(q.codes[0])
            imax = max(range(B), key=lambda i: v[i])
            assert int(codes[imax] & 7) == 7


def pin_groups_are_contiguous():
    """Two blocks with the same multiset of values but different grouping must see different
    group maxima: contiguous groups of B/G elements."""
    cfg = orc.Config()
    base = np.full(32, 0.25, dtype=np.float32)
    a = base.copy(); a[0:4] = [15, 9.5, 9.5, 9.5]          # all large values in ONE contiguous group
    b = base.copy(); b[[0, 4, 8, 12]] = [15, 9.5, 9.5, 9.5]  # spread over four groups
    qa = orc.quantize(synth.f32_to_bf16_bits(a).reshape(1, 32), FB, cfg, want_errors=True)
    qb = orc.quantize(synth.f32_to_bf16_bits(b).reshape(1, 32), FB, cfg, want_errors=True)
    for d in range(25, 32):    # dialects with top magnitude 15
        def term(u, d=d):
            k = math.floor(2 * u)
            return min(abs(Fraction(2 * k + 1, 4) - int(f)) for f in FB[d])
        ea = term(Fraction(15)) + 7 * term(Fraction(1, 4))
        eb = term(Fraction(15)) + 3 * term(Fraction(19, 2)) + 4 * term(Fraction(1, 4))
        assert Fraction(int(qa.err_q4[0, 0, d]), 4) == ea
        assert Fraction(int(qb.err_q4[0, 0, d]), 4) == eb


def pin_select_all_mode(seed=3, n=60):
    rng = np.random.default_rng(seed)
    cfg = orc.Config(select_mode=1)
    for _ in range(n):
        bits = rand_block_bits(rng, 32)
        q = orc.quantize(bits.reshape(1, 32), FB, cfg, want_errors=True)
        err = q.err_q4[0, 0]
        assert np.all(err >= 0)
        assert int(q.did[0, 0]) == int(np.argmin(err))      # numpy argmin returns the first minimum


# ---------------------------------------------------------------- SeDA (Sec. 3.4)

def pin_seda_choice_inside_mask(seed=4, n=120):
    rng = np.random.default_rng(seed)
    w = synth.Workload("t", T=8, C=64, seed=9, kind=1, n_outlier=0, outlier_gain=1.0,
                       seda=True, n_clusters=4, cluster_seed=5)
    cid, masks = synth.clusters(w)
    for m in masks:
        assert bin(int(m)).count("1") == 8
        assert sorted(int(FB[d, 7]) for d in range(32) if (int(m) >> d) & 1) == list(range(8, 16))
    for it in range(n):
        bits = rand_block_bits(rng, 32)
        if it % 3 == 0:
            mask = int(masks[it % 4])           # paper-structured: one dialect per bucket
        else:
            mask = int(rng.integers(1, 2 ** 32))
        q = orc.quantize(bits.reshape(1, 32), FB, cluster_id=np.zeros(1, np.int32),
                         cluster_mask=np.array([mask], np.uint32), want_errors=True)
        d, e = int(q.did[0, 0]), int(q.exponent[0, 0])
        assert (mask >> d) & 1
        v, _ = _group_max_v(bits, e, 32, 8)
        bucket = max(8, math.floor(max(v)))
        inter = [dd for dd in range(32) if (mask >> dd) & 1 and int(FB[dd, 7]) == bucket]
        err = q.err_q4[0, 0]
        cands = inter if inter else [dd for dd in range(32) if (mask >> dd) & 1]
        assert [dd for dd in range(32) if err[dd] >= 0] == cands
        if it % 3 == 0:
            assert cands == [d]                 # exactly one candidate remains after stage 1
        assert int(err[d]) == min(int(err[dd]) for dd in cands)
    # cluster id -1 means unconstrained
    bits = rand_block_bits(rng, 32)
    qa = orc.quantize(bits.reshape(1, 32), FB)
    qb = orc.quantize(bits.reshape(1, 32), FB, cluster_id=np.array([-1], np.int32),
                      cluster_mask=np.array([1], np.uint32))
    assert np.array_equal(qa.codes, qb.codes) and np.array_equal(qa.meta, qb.meta)


def _round_to_f32(q):
    """The binary32 number nearest to the rational q (ties to even), by integer arithmetic: returns a Fraction.
    (Overflow is out of range for the pins that use it.)"""
    from fractions import Fraction
    if q == 0:
        return Fraction(0)
    sign, a = (-1 if q < 0 else 1), abs(q)
    e = a.numerator.bit_length() - a.denominator.bit_length()      # a in [2^(e-1), 2^(e+1))
    if Fraction(2) ** e > a:
        e -= 1                                                     # now 2^e <= a < 2^(e+1)
    e = max(e, -126)                                               # subnormals share the spacing of 2^-126
    ulp = Fraction(2) ** (e - 23)
    n = a / ulp
    k = n.numerator // n.denominator
    rem = n - k
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and k % 2 == 1):
        k += 1
    return sign * k * ulp


def pin_affine_producer(seed=21, n=400):
    """y = x * g + bias (App. D.2 fusion with the preceding operation; LayerNorm tail / modulation): g is the
    float32 nearest to 1 + gain, y the float32 nearest to the EXACT x * g + bias (one rounding), checked in
    rationals; identity for gain 1 / bias 0 (or gain 0 with plus_one), signed zeros included."""
    from fractions import Fraction
    rng = np.random.default_rng(seed)
    bf = lambda a: synth.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))
    val = lambda bits: Fraction(float(synth.bf16_bits_to_f32(np.asarray(bits, dtype=np.uint16).reshape(1))[0]))
    C = 8
    for it in range(n):
        k = rng.integers(-20, 20)
        x = bf(rng.standard_normal((2, C)) * np.exp2(float(k)))
        gain = bf(rng.standard_normal(C) * np.exp2(float(rng.integers(-30, 3))))
        # biases near -x*g make the sum cancel, where a second rounding would show
        bias = bf(-synth.bf16_bits_to_f32(x[0]) * (1 + synth.bf16_bits_to_f32(gain)) * (1 + rng.standard_normal(C) * 2.0 ** -9))
        if it % 7 == 0:
            bias = bf(rng.standard_normal(C) * np.exp2(float(rng.integers(-20, 20))))
        for plus_one in (False, True):
            y = orc.affine_f32(x, gain, bias, plus_one)
            for t in range(2):
                for c in range(C):
                    g = _round_to_f32(1 + val(gain[c])) if plus_one else val(gain[c])
                    want = _round_to_f32(val(x[t, c]) * g + val(bias[c]))
                    assert Fraction(float(y[t, c])) == want, (it, t, c, plus_one)
    # identity, bit for bit (signed zeros: -0 * 1 + 0 = +0 is the IEEE sum, so bias -0 keeps the sign)
    x = bf(np.array([[1.5, -2.0, 0.0, -0.0, 3e-39, -1e38, 7.0, 0.25]], dtype=np.float32))
    one, zero, nzero = bf(np.ones(8)), bf(np.zeros(8)), bf(np.full(8, -0.0))
    for g, p1 in ((one, False), (zero, True)):
        y = orc.affine_f32(x, g, nzero, p1)
        assert np.array_equal(y.view(np.uint32), synth.bf16_bits_to_f32(x).view(np.uint32))
    y = orc.affine_f32(x, one, zero, False)
    assert np.signbit(y[0, 3]) == False and y[0, 3] == 0.0        # -0 + 0 = +0
    # a row stride, and a gain that 1 + gain cannot hold in float32 (2^-30): g rounds to exactly 1
    wide = np.zeros((2, 16), dtype=np.uint16)
    wide[:, :8] = bf(rng.standard_normal((2, 8)))
    tiny = bf(np.full(8, 2.0 ** -30))
    y = orc.affine_f32(wide[:, :8], tiny, zero, True)
    assert np.array_equal(y, synth.bf16_bits_to_f32(wide[:, :8]))
    y = orc.affine_f32(wide[:, :8], tiny, zero, False)
    assert np.array_equal(y, synth.bf16_bits_to_f32(wide[:, :8]) * np.float32(2.0 ** -30))


def _sqrt_to_f32(q):
    """The binary32 number nearest to sqrt(q) for a positive rational q (ties cannot occur: the midpoint of two
    neighbouring floats has 25 significant bits, its square at most 50, so it is never the exact root of a
    49-bit argument unless representable).  Candidate from the double square root, verified by squaring
    the midpoints to its neighbours in exact rationals."""
    from fractions import Fraction
    assert q > 0
    c = np.float32(math.sqrt(float(q)))
    for _ in range(4):
        lo, hi = np.nextafter(c, np.float32(0)), np.nextafter(c, np.float32(np.inf))
        mlo = (Fraction(float(lo)) + Fraction(float(c))) / 2
        mhi = (Fraction(float(c)) + Fraction(float(hi))) / 2
        if mlo * mlo <= q <= mhi * mhi:
            assert mlo * mlo != q and mhi * mhi != q
            return Fraction(float(c))
        c = lo if q < mlo * mlo else hi
    raise AssertionError("square root candidate did not settle")


def _layernorm_rational(xv, gv, bv, plus_one, eps):
    """The stated LayerNorm order in exact rationals, every operation rounded to binary32 by _round_to_f32."""
    from fractions import Fraction
    R = _round_to_f32
    C = len(xv)
    nblk = C // 32

    def total(bs):
        acc = Fraction(0)
        for b0 in range(0, nblk, 32):
            v = [bs[b0 + i] if b0 + i < nblk else Fraction(0) for i in range(32)]
            for off in (16, 8, 4, 2, 1):
                v = [R(v[i] + v[i ^ off]) for i in range(32)]
            acc = R(acc + v[0])
        return acc

    bs = []
    for b in range(nblk):
        s_ = xv[b * 32]
        for i in range(1, 32):
            s_ = R(s_ + xv[b * 32 + i])
        bs.append(s_)
    mean = R(total(bs) / C)
    d = [R(x - mean) for x in xv]
    bs = []
    for b in range(nblk):
        q = Fraction(0)
        for i in range(32):
            q = R(d[b * 32 + i] * d[b * 32 + i] + q)
        bs.append(q)
    var = R(total(bs) / C)
    rstd = R(1 / _sqrt_to_f32(R(var + eps)))
    out = []
    for c in range(C):
        g = R(1 + gv[c]) if plus_one else gv[c]
        out.append(R(R(d[c] * rstd) * g + bv[c]))
    return out, mean, var


def pin_layernorm_producer(seed=22):
    """LayerNorm + modulation (App. D.2 fusion with the preceding operation): the float32 result equals the stated
    order of operations carried out in exact rationals with one rounding per operation (square root checked by
    squaring); it stays within a few units in the last place of the exact LayerNorm; a row of equal values
    normalises to the bias; the row stride is honoured."""
    from fractions import Fraction
    rng = np.random.default_rng(seed)
    bf = lambda a: synth.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))
    val = lambda bits: [Fraction(float(v)) for v in synth.bf16_bits_to_f32(np.asarray(bits, dtype=np.uint16))]
    eps = float(np.float32(1e-6))
    # 1, 3, 33, 65 blocks: short last segments.  "wide": magnitudes spread over 2^-12 .. 2^12 inside a block, so that
    # the additions round, the mean has 24 significant bits and the squares are not representable - with a single
    # block (C = 32) mean and variance are the block's own sums divided by a power of two, nothing hides a rounding
    for C, plus_one, wide in [(32, False, False), (32, True, True), (64, False, True), (96, True, False), (1056, False, True),
                              (2080, True, False)]:
        x = bf(rng.standard_t(3, size=(2, C)) * np.exp2(float(rng.integers(-6, 6))) + rng.standard_normal())
        if wide:
            x = bf(rng.standard_normal((2, C)) * np.exp2(rng.integers(-12, 13, size=(2, C)).astype(np.float64)))
        gain = bf(rng.standard_normal(C) * 0.5)
        bias = bf(rng.standard_normal(C))
        y, stats = orc.layernorm_f32(x, gain, bias, plus_one, eps, want_stats=True)
        for t in range(2):
            want, mean, var = _layernorm_rational(val(x[t]), val(gain), val(bias), plus_one, Fraction(eps))
            assert Fraction(float(stats[t, 0])) == mean and Fraction(float(stats[t, 1])) == var, (C, t)
            got = [Fraction(float(v)) for v in y[t]]
            assert got == want, (C, t, next(i for i in range(C) if got[i] != want[i]))
            # against the exact LayerNorm: mean and variance in rationals, the root in double precision
            xv = val(x[t])
            m = sum(xv) / C
            v = sum((a - m) ** 2 for a in xv) / C
            assert abs(mean - m) <= Fraction(1, 2 ** 18) * max(abs(a) for a in xv)
            assert abs(var - v) <= Fraction(1, 2 ** 17) * v
            r = 1.0 / math.sqrt(float(v) + eps)
            for c in range(0, C, 7):
                g = float(val(gain[c:c + 1])[0]) + (1.0 if plus_one else 0.0)
                exact = float(xv[c] - m) * r * g + float(val(bias[c:c + 1])[0])
                assert abs(float(y[t, c]) - exact) <= 3e-5 * (1.0 + abs(exact)), (C, t, c)
    # a row of equal values: d = 0 everywhere, y = bias bit for bit (fma(+-0, g, b) = b)
    x = bf(np.full((1, 64), 3.0))
    gain, bias = bf(rng.standard_normal(64)), bf(rng.standard_normal(64) + 2.0)
    y = orc.layernorm_f32(x, gain, bias, True, eps)
    assert np.array_equal(y[0], synth.bf16_bits_to_f32(bias))
    # row stride
    wide = bf(rng.standard_normal((3, 128)))
    gain, bias = bf(np.ones(64)), bf(np.zeros(64))
    a = orc.layernorm_f32(wide[:, :64], gain, bias, False, eps)
    b = orc.layernorm_f32(np.ascontiguousarray(wide[:, :64]), gain, bias, False, eps)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def pin_f32_input(seed=9, n=30):
    """fp32 input: every block equals the block-wise definition on the exact values (pinned above
    through quantize_block_f64), values that happen to be bf16 give the bf16 result, and a value
    between two bf16 neighbours is NOT rounded to bf16 first (its bin comes from the fp32 mantissa)."""
    rng = np.random.default_rng(seed)
    for it in range(n):
        x = (rng.standard_normal((3, 64)) * np.exp2(rng.integers(-30, 30, size=(3, 1)))).astype(np.float32)
        x[0, 5] = -0.0
        if it % 5 == 0:
            x[1, :32] = 0.0
        q = orc.quantize_f32(x, FB)
        for t in range(3):
            for blk in range(2):
                code, did, e, _ = orc.quantize_block_f64(x[t, blk * 32:blk * 32 + 32].astype(np.float64), FB)
                assert np.array_equal(unpack_codes(q.codes[t, blk * 16:(blk + 1) * 16]), code)
                assert int(q.meta[t, blk]) == (e + 124) | (did << 8)
        bits = synth.f32_to_bf16_bits(x)
        xb = synth.bf16_bits_to_f32(bits)
        qa, qb = orc.quantize_f32(xb, FB), orc.quantize(bits, FB)
        assert np.array_equal(qa.codes, qb.codes) and np.array_equal(qa.meta, qb.meta)
    # SeDA tables restrict the fp32 path exactly as the bf16 path (Sec. 3.4): on bf16-representable values
    # the two agree with the same masks (the bf16 path's SeDA behaviour is pinned on its own), every
    # choice lies inside the token's mask, and a one-dialect mask forces that dialect
    for it in range(10):
        x = (rng.standard_normal((6, 64)) * np.exp2(rng.integers(-20, 20, size=(6, 1)))).astype(np.float32)
        bits = synth.f32_to_bf16_bits(x)
        xb = synth.bf16_bits_to_f32(bits)
        masks = rng.integers(1, 2 ** 32, size=3, dtype=np.uint64).astype(np.uint32)
        masks[2] = np.uint32(1) << np.uint32(rng.integers(0, 32))
        cid = np.array([0, 1, 2, -1, 2, 0], dtype=np.int32)
        qa = orc.quantize_f32(xb, FB, cluster_id=cid, cluster_mask=masks)
        qb = orc.quantize(bits, FB, cluster_id=cid, cluster_mask=masks)
        assert np.array_equal(qa.codes, qb.codes) and np.array_equal(qa.meta, qb.meta)
        qf = orc.quantize_f32(x, FB, cluster_id=cid, cluster_mask=masks)
        did = qf.meta >> 8
        for t in range(6):
            if cid[t] >= 0:
                assert all((int(masks[cid[t]]) >> int(d)) & 1 for d in did[t])
        assert all(int(d) == int(masks[2]).bit_length() - 1 for d in did[2]) and all(int(d) == int(masks[2]).bit_length() - 1 for d in did[4])
        free = orc.quantize_f32(x, FB)
        assert np.array_equal(free.meta[3], qf.meta[3]) and np.array_equal(free.codes[3], qf.codes[3])
    # 8.0 sets the scale (e = 3, v = x); 2.4990234375 = 2.5 - 2^-10 lies below the 2|3 boundary of
    # dialect d0..: as fp32 its bin is floor(4.998) = 4, while its bf16 rounding 2.5 has bin 5
    x = np.zeros((1, 32), np.float32)
    x[0, 0], x[0, 1] = 8.0, 2.4990234375
    q = orc.quantize_f32(x, FB)
    did = int(q.meta[0, 0]) >> 8
    codes = unpack_codes(q.codes[0])
    assert int(FB[did, codes[1] & 7]) == 2
    qb = orc.quantize(synth.f32_to_bf16_bits(x), FB)
    assert int(FB[int(qb.meta[0, 0]) >> 8, unpack_codes(qb.codes[0])[1] & 7]) == 3


def _e4m3_value(b: int) -> Fraction:
    """FP8 e4m3 from its definition: 1 sign, 4 exponent bits (bias 7), 3 mantissa bits; exponent 0 = subnormal."""
    s, ex, mant = b >> 7, (b >> 3) & 15, b & 7
    v = Fraction(mant, 8) * Fraction(2) ** -6 if ex == 0 else (1 + Fraction(mant, 8)) * Fraction(2) ** (ex - 7)
    return -v if s else v


def pin_mxfp8_view(seed=10):
    """App. D.2: the e4m3 byte times the E8M0 block scale is exactly the decoded FB4 value, for every
    dialect, index, sign and scale; the scale byte is the E8M0 code of 2^(e-3)."""
    rng = np.random.default_rng(seed)
    codes = rng.integers(0, 256, size=(40, 32), dtype=np.uint8)        # 40 x 64 elements: every nibble value
    did = np.arange(80).reshape(40, 2) % 32
    sb = rng.integers(0, 252, size=(40, 2))
    sb[0], sb[1] = [0, 1], [250, 251]
    meta = (sb | (did << 8)).astype(np.uint16)
    q = orc.Quantized(codes, meta)
    y = orc.dequantize(q, FB)
    for layout in (0, 1):
        e, sc = orc.to_mxfp8(q, FB, layout)
        for t in range(40):
            for c in range(64):
                k = int(sc[orc.mxfp8_scale_offset(t, c // 32, 2, layout)])
                assert k == int(sb[t, c // 32])                          # E8M0 code = scale byte
                want = f32_value(y[t, c])
                got = _e4m3_value(int(e[t, c])) * Fraction(2) ** (k - 127)
                assert got == want
                assert (int(e[t, c]) >> 7) == int(np.signbit(y[t, c]))   # signed zeros keep their sign
                assert (int(e[t, c]) & 0x7F) != 0x7F                     # never the NaN pattern


def pin_mxfp8_scale_layout():
    """The tiled scale layout: 512-byte tiles of 128 rows x 4 columns, column tiles of a row band
    contiguous; inside a tile rows 32 apart are 4 bytes apart, neighbouring rows 16 bytes, neighbouring
    columns 1 byte; every scale has its own byte; padding holds 0x7f."""
    off = orc.mxfp8_scale_offset
    n_col = 10                                               # 3 column tiles (padded to 12)
    assert off(0, 0, n_col, 1) == 0 and off(0, 4, n_col, 1) == 512 and off(0, 8, n_col, 1) == 1024
    assert off(128, 0, n_col, 1) == 3 * 512
    assert off(1, 0, n_col, 1) - off(0, 0, n_col, 1) == 16
    assert off(32, 0, n_col, 1) - off(0, 0, n_col, 1) == 4 and off(96, 0, n_col, 1) == 12
    assert off(0, 3, n_col, 1) == 3 and off(31, 3, n_col, 1) == 31 * 16 + 3 and off(127, 3, n_col, 1) == 511
    T = 300
    seen = {off(r, c, n_col, 1) for r in range(T) for c in range(n_col)}
    assert len(seen) == T * n_col and max(seen) < 3 * 3 * 512
    assert [off(r, c, n_col, 0) for r in (0, 1) for c in (0, 9)] == [0, 9, 10, 19]
    meta = np.full((T, n_col), 130 | (3 << 8), dtype=np.uint16)
    q = orc.Quantized(np.zeros((T, n_col * 16), np.uint8), meta)
    _, sc = orc.to_mxfp8(q, FB, 1)
    assert len(sc) == 3 * 3 * 512
    real = np.zeros(len(sc), bool)
    real[list(seen)] = True
    assert np.all(sc[real] == 130) and np.all(sc[~real] == 0x7F)


def pin_weight_quantization(seed=11, n=25):
    """Exhaustive selection (Sec. 3.3 / App. C): the chosen dialect attains the minimum of the exact
    (rational) squared error over all 32 dialects, lowest id among exact ties; its elements are rounded
    to the nearest magnitude; its error never exceeds that of the online (LUT, two-stage) choice."""
    rng = np.random.default_rng(seed)
    for it in range(n):
        B = 32 if it % 3 else 16
        cfg = orc.Config(block_size=B, num_groups=8)
        bits = rand_block_bits(rng, B, (-6, 6) if it % 2 else (-20, 20))
        if it == 4:
            bits[:] = 0
        q, sse = orc.quantize_weights(bits.reshape(1, B), FB, cfg, want_sse=True)
        did, e = int(q.did[0, 0]), int(q.exponent[0, 0])
        vals = [abs(bf16_value(int(b))) * Fraction(2) ** (3 - e) for b in bits]
        exact = []
        for d in range(32):
            mags = [int(m) for m in FB[d]]
            exact.append(sum(min((v - m) ** 2 for m in mags) for v in vals))
        assert exact[did] == min(exact) and did == exact.index(min(exact))
        for d in range(32):
            assert abs(float(exact[d]) - sse[0, 0, d]) <= 1e-12 * max(1.0, float(exact[d]))
        codes = unpack_codes(q.codes[0])
        for i, v in enumerate(vals):
            m = int(FB[did, codes[i] & 7])
            assert all(abs(v - m) <= abs(v - int(mm)) for mm in FB[did])
            assert (codes[i] >> 3) == (int(bits[i]) >> 15)
        qa = orc.quantize(bits.reshape(1, B), FB, cfg)
        assert int(qa.exponent[0, 0]) == e
        assert exact[did] <= exact[int(qa.did[0, 0])]


def _meta_with_dialects(rows):
    """meta records (scale byte 124) for rows of dialect ids"""
    return np.array([[124 | (d << 8) for d in r] for r in rows], dtype=np.uint16)


def pin_subformatbook_hand_counted():
    """Sec. 3.4 sub-formatbook construction on cases counted by hand.  Stand-in formatbook: buckets
    (largest magnitude 8..15) hold dialects {0,1} {2,3} {4,5,6} {7,8,9} {10..13} {14..18} {19..24} {25..31}."""
    assert [int(FB[d, 7]) for d in (0, 1, 2, 3, 4, 6, 7, 9, 10, 13, 14, 18, 19, 24, 25, 31)] == \
        [8, 8, 9, 9, 10, 10, 11, 11, 12, 12, 13, 13, 14, 14, 15, 15]
    meta = _meta_with_dialects([
        [1, 1, 0, 5, 5, 6, 31, 30],      # token 0
        [1, 3, 3, 2, 6, 6, 26, 30],      # token 1
        [0, 0, 0, 0, 0, 0, 0, 0],        # token 2 (anchor of cluster 1)
        [12, 12, 11, 11, 13, 17, 17, 20],  # token 3 (no anchor: must not count)
    ])
    # cluster 0 = tokens 0 and 1: bucket 8: d1 x3 vs d0 x1 -> 1; bucket 9: d3 x2 vs d2 x1 -> 3;
    # bucket 10: d5 x2, d6 x3 -> 6; bucket 15: d30 x2, d31, d26 -> 30; buckets 11,12,13,14 empty -> 7,10,14,19
    want0 = sum(1 << d for d in (1, 3, 6, 7, 10, 14, 19, 30))
    # cluster 1 = token 2: only d0 occurs; every other bucket takes its lowest id
    want1 = sum(1 << d for d in (0, 2, 4, 7, 10, 14, 19, 25))
    # cluster 2 has no anchors at all: lowest id everywhere
    got = orc.build_subformatbook(meta, [0, 2, 1], [0, 1, 0], 3, FB)
    assert [int(m) for m in got] == [want0, want1, want1]
    # an anchor listed twice counts twice: token 0 twice + token 1 -> bucket 10: d5 x4 vs d6 x4... d5=2*2=4, d6=1*2+2=4: tie -> 5
    got = orc.build_subformatbook(meta, [0, 0, 1], [0, 0, 0], 1, FB)
    assert int(got[0]) == sum(1 << d for d in (1, 3, 5, 7, 10, 14, 19, 30))
    # anchors outside the tensor or outside the clusters are ignored
    got = orc.build_subformatbook(meta, [0, 1, 7, -1, 3], [0, 0, 0, 0, 5], 1, FB)
    assert int(got[0]) == want0
    # a custom stage-1 table with two buckets {0..15} {16..31}: one pick per bucket
    s1 = np.array([0x0000FFFF] * 16 + [0xFFFF0000] * 16, dtype=np.uint32)
    got = orc.build_subformatbook(meta, [3], [0], 1, FB, stage1=s1)
    assert int(got[0]) == (1 << 11) | (1 << 17)          # d11 x2 = d12 x2 -> lowest; d17 x2 vs d20 x1


def pin_subformatbook_one_dialect_per_bucket_and_closed_loop(seed=8):
    """An 8-dialect sub-formatbook has one dialect per dynamic range (Sec. 3.4); tokens that were
    quantized under a sub-formatbook M give M back on every bucket their blocks fell into."""
    w = synth.Workload("t", T=96, C=256, seed=seed, kind=1, n_outlier=2, outlier_gain=50.0,
                       seda=True, n_clusters=3, cluster_seed=seed + 1)
    bits = synth.activation(w)
    cid, masks = synth.clusters(w)
    free = orc.quantize(bits, FB)
    tok = np.arange(w.T, dtype=np.int32)
    built = orc.build_subformatbook(free.meta, tok, cid, 3, FB)
    for m in built:
        assert sorted(int(FB[d, 7]) for d in range(32) if (int(m) >> d) & 1) == list(range(8, 16))
    # most frequent: no other member of the bucket was chosen more often
    for c in range(3):
        cnt = np.bincount(free.did[cid == c].ravel(), minlength=32)
        for d in range(32):
            if (int(built[c]) >> d) & 1:
                rivals = [dd for dd in range(32) if int(FB[dd, 7]) == int(FB[d, 7])]
                assert cnt[d] == max(cnt[dd] for dd in rivals)
                assert d == min(dd for dd in rivals if cnt[dd] == cnt[d])
    # closed loop
    con = orc.quantize(bits, FB, cluster_id=cid, cluster_mask=masks)
    again = orc.build_subformatbook(con.meta, tok, cid, 3, FB)
    for c in range(3):
        used_buckets = {int(FB[d, 7]) for d in np.unique(con.did[cid == c])}
        for d in range(32):
            if int(FB[d, 7]) in used_buckets:
                assert ((int(again[c]) >> d) & 1) == ((int(masks[c]) >> d) & 1)


# ---------------------------------------------------------------- decomposition (Sec. 3.3)

def pin_salient_is_per_tile_argmax(seed=5):
    rng = np.random.default_rng(seed)
    for T, tile in [(40, 20), (47, 20), (5, 20), (64, 1), (33, 7)]:
        s = rng.random(T).astype(np.float32)
        s[rng.integers(0, T, size=T // 3)] = s[0]          # ties
        idx = orc.select_salient(s, tile)
        assert len(idx) == -(-T // tile)
        for k, t0 in enumerate(range(0, T, tile)):
            assert int(idx[k]) == t0 + int(np.argmax(s[t0:t0 + tile]))   # numpy: first maximum
        assert np.all(np.diff(idx) > 0)
    # the last token of the sequence as the unique maximum of its tile: a full last tile, a ragged one,
    # and a last tile that holds that token alone
    for T, tile, want in [(40, 20, [0, 39]), (47, 20, [0, 20, 46]), (41, 20, [0, 20, 40]), (7, 7, [6]), (3, 20, [2])]:
        s = np.full(T, 0.125, dtype=np.float32)
        s[T - 1] = 0.875
        assert [int(i) for i in orc.select_salient(s, tile)] == want
    # ... and as one of two equal maxima of the ragged last tile: the lower index wins
    s = np.full(47, 0.125, dtype=np.float32)
    s[[43, 46]] = 0.875
    assert [int(i) for i in orc.select_salient(s, 20)] == [0, 20, 43]


def pin_salient_topk(seed=12):
    """Global reading of the salient set: the k largest scores, ties to the lowest index, ascending."""
    rng = np.random.default_rng(seed)
    s = np.array([0.5, 0.9, 0.1, 0.9, 0.9, 0.2, 0.5], dtype=np.float32)
    assert list(orc.select_salient_topk(s, 0)) == []
    assert list(orc.select_salient_topk(s, 1)) == [1]
    assert list(orc.select_salient_topk(s, 2)) == [1, 3]                 # tie at 0.9: lowest indices first
    assert list(orc.select_salient_topk(s, 4)) == [0, 1, 3, 4]           # tie at 0.5: index 0 before 6
    assert list(orc.select_salient_topk(s, 7)) == list(range(7))
    for T, k in [(50, 3), (333, 17), (1000, 50), (64, 64)]:
        s = rng.random(T).astype(np.float32)
        s[rng.integers(0, T, size=T // 4)] = s[1]                         # many ties
        got = orc.select_salient_topk(s, k)
        order = np.argsort(-s.astype(np.float64), kind="stable")          # stable: ties keep index order
        assert np.array_equal(got, np.sort(order[:k]))
        assert np.all(np.diff(got) > 0)


def pin_decomposition(seed=6, n=40):
    """Act = Q(Act) + Delta exactly; Q(Act) + Q(Delta) is never farther from Act than Q(Act)
    in any element; the residual codes decode to the sign of Delta."""
    rng = np.random.default_rng(seed)
    for it in range(n):
        T, C = 4, 64
        x = np.stack([rand_block_bits(rng, C, (-30, 30)) for _ in range(T)])
        sal = np.array([1, 3], dtype=np.int32)
        q = orc.quantize(x, FB, salient_idx=sal)
        q_plain = orc.quantize(x, FB)
        assert np.array_equal(q.codes, q_plain.codes) and np.array_equal(q.meta, q_plain.meta)
        main = orc.dequantize(q_plain, FB)
        full = orc.dequantize(q, FB)
        assert np.array_equal(full[[0, 2]], main[[0, 2]])
        for s, t in enumerate(sal):
            # residual block quantized like any other block, from the exact difference
            for blk in range(C // 32):
                sl = slice(blk * 32, blk * 32 + 32)
                delta = [bf16_value(int(b)) - f32_value(m) for b, m in zip(x[t, sl], main[t, sl])]
                assert all(Fraction(float(np.float32(float(dl)))) == dl for dl in delta)   # exact in fp32
                code, did, e, _ = orc.quantize_block_f64(np.array([float(dl) for dl in delta]), FB)
                assert np.array_equal(unpack_codes(q.res_codes[s, blk * 16:(blk + 1) * 16]), code)
                assert int(q.res_meta[s, blk]) == (e + 124) | (did << 8)
            rcodes = unpack_codes(q.res_codes[s])
            for c in range(C):
                xv = bf16_value(int(x[t, c]))
                # decoded sum = Q(Act) + Q(Delta), the residual decoded by the same formula
                rm = int(q.res_meta[s, c // 32])
                rmag = int(FB[rm >> 8, rcodes[c] & 7]) * Fraction(2) ** ((rm & 0xFF) - 127)
                rval = -rmag if rcodes[c] & 8 else rmag
                assert f32_value(full[t, c]) == f32_value(main[t, c]) + rval
                e0 = abs(xv - f32_value(main[t, c]))
                e1 = abs(xv - f32_value(full[t, c]))
                assert e1 <= e0
                rq = f32_value(full[t, c]) - f32_value(main[t, c])       # decoded residual (sum is exact)
                dl = xv - f32_value(main[t, c])
                assert rq == 0 or (rq > 0) == (dl > 0)


def pin_residual_uses_the_seda_mask(seed=14):
    """App. C: with SeDA and decomposition together, the residual is constrained to the cluster's
    sub-formatbook like the original values; its block equals the block-wise definition under that mask."""
    rng = np.random.default_rng(seed)
    w = synth.Workload("t", T=6, C=128, seed=15, kind=1, n_outlier=1, outlier_gain=50.0, seda=True, n_clusters=2,
                       cluster_seed=16)
    bits = synth.activation(w)
    cid, masks = synth.clusters(w)
    masks = masks.copy()
    masks[1] = 0x00F00F03                     # an arbitrary mask as well
    sal = np.array([0, 2, 5], dtype=np.int32)
    q = orc.quantize(bits, FB, cluster_id=cid, cluster_mask=masks, salient_idx=sal)
    main = orc.dequantize(orc.Quantized(q.codes, q.meta), FB)
    for s_, t in enumerate(sal):
        allowed = int(masks[cid[t]])
        for blk in range(4):
            rdid = int(q.res_meta[s_, blk]) >> 8
            assert (allowed >> rdid) & 1
            sl = slice(blk * 32, blk * 32 + 32)
            delta = np.array([float(bf16_value(int(b)) - f32_value(m)) for b, m in zip(bits[t, sl], main[t, sl])])
            code, did, e, _ = orc.quantize_block_f64(delta, FB, allowed=allowed)
            assert did == rdid and int(q.res_meta[s_, blk]) & 0xFF == e + 124
            assert np.array_equal(unpack_codes(q.res_codes[s_, blk * 16:(blk + 1) * 16]), code)


def pin_dequantize_formula(seed=7):
    rng = np.random.default_rng(seed)
    codes = rng.integers(0, 256, size=(3, 32), dtype=np.uint8)
    did = rng.integers(0, 32, size=(3, 2))
    sb = np.array([[0, 1], [121, 124], [250, 251]])
    meta = (sb | (did << 8)).astype(np.uint16)
    y = orc.dequantize(orc.Quantized(codes, meta), FB)
    yb = orc.dequantize(orc.Quantized(codes, meta), FB, out_dtype="bf16")
    for t in range(3):
        cc = unpack_codes(codes[t])
        for c in range(64):
            m = int(FB[did[t, c // 32], cc[c] & 7])
            want = math.ldexp(m, int(sb[t, c // 32]) - 127)       # F * 2^(e-3), e = byte - 124
            want = -want if cc[c] & 8 else want
            assert float(y[t, c]) == want and bool(np.signbit(y[t, c])) == bool(cc[c] & 8)
            assert float(synth.bf16_bits_to_f32(yb[t:t + 1, c])[0]) == want   # 4-bit magnitudes are exact in bf16


def pin_dequantize_f16(seed=13):
    """Half-precision decode = the fp32 decode rounded to IEEE half (numpy's conversion as the independent
    rounding: nearest even, overflow to infinity, gradual underflow), residual rows included."""
    rng = np.random.default_rng(seed)
    codes = rng.integers(0, 256, size=(6, 32), dtype=np.uint8)
    did = rng.integers(0, 32, size=(6, 2))
    sb = np.array([[0, 90], [100, 103], [110, 121], [124, 130], [139, 140], [141, 251]])   # under- and overflow
    meta = (sb | (did << 8)).astype(np.uint16)
    q = orc.Quantized(codes, meta, salient_idx=np.array([2, 3], np.int32),
                      res_codes=rng.integers(0, 256, size=(2, 32), dtype=np.uint8),
                      res_meta=(np.array([[103, 113], [118, 123]]) | (did[:2] << 8)).astype(np.uint16))
    y32 = orc.dequantize(q, FB)
    assert np.count_nonzero(y32.view(np.uint32) & 0xFFFF) > 20      # sums that are not bf16 values
    with np.errstate(over="ignore"):
        want = y32.astype(np.float16).view(np.uint16)
    got = orc.dequantize(q, FB, out_dtype="f16")
    assert np.array_equal(got, want)
    assert np.isinf(want.view(np.float16)).any() and (want.view(np.float16) == 0).any()


def _round_to_bf16_bits(q) -> int:
    """bf16 bit pattern nearest to the rational q (round to nearest, ties to even), by integer arithmetic.
    Normal range only (the pins that use it stay inside it)."""
    sign, a = (1 if q < 0 else 0), abs(Fraction(q))
    if a == 0:
        return sign << 15
    e = floor_log2(a)
    assert -126 <= e <= 126
    n = a / Fraction(2) ** (e - 7)                  # in [128, 256): 8 significant bits wanted
    k = n.numerator // n.denominator
    rem = n - k
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and k % 2 == 1):
        k += 1
    if k == 256:
        k, e = 128, e + 1
    return (sign << 15) | ((e + 127) << 7) | (k - 128)


def pin_dequantize_bf16_rounds_sums_to_nearest_even(seed=17):
    """bf16 decode of a salient row = Q(Act) + Q(Delta) rounded to nearest, ties to even.  A decoded FB4
    value alone has 4 significant bits and is a bf16 number; the sum of two at different scales is not.
    Expected bits come from the exact rational sum rounded by integer arithmetic written here."""
    # hand-made: dialect 0 = {0 1 2 3 4 5 6 8}; main = 8 * 2^5 = 256 (index 7, scale byte 132), residual scale
    # byte 127 = 2^0.  256 + 1 = 257 and 256 + 3 = 259 are exact ties of the 8-bit grid (spacing 2 above 256):
    # 257 -> 256 (even mantissa), 259 -> 260; 256 + 2 = 258 is representable; 256 - 1 = 255 is representable
    # (spacing 1 below 256); 256 + 5 = 261 -> tie -> 260; 256 + 6 = 262 stays; -256 - 3 -> -260.
    assert [int(m) for m in FB[0]] == [0, 1, 2, 3, 4, 5, 6, 8]
    n = 32
    main_codes = np.full(n, 7, dtype=np.uint8)
    res_idx = np.array([1, 3, 2, 1 | 8, 5, 6, 3 | 8, 0] * 4, dtype=np.uint8)
    main_codes[6::8] = 7 | 8                                     # element 6 of every eight: -256
    pack = lambda c: (c[0::2] | (c[1::2] << 4)).astype(np.uint8).reshape(1, -1)
    q = orc.Quantized(pack(main_codes), np.array([[132 | (0 << 8)]], np.uint16),
                      salient_idx=np.array([0], np.int32), res_codes=pack(res_idx),
                      res_meta=np.array([[127 | (0 << 8)]], np.uint16))
    got = orc.dequantize(q, FB, out_dtype="bf16")[0]
    want_vals = [256, 260, 258, 255, 260, 262, -260, 256]
    for i in range(n):
        assert float(synth.bf16_bits_to_f32(got[i:i + 1])[0]) == want_vals[i % 8], (i, hex(int(got[i])))
    # random codes, metadata and residuals at nearby scales: sums of up to 15 significant bits
    rng = np.random.default_rng(seed)
    T, C = 4, 64
    codes = rng.integers(0, 256, size=(T, C // 2), dtype=np.uint8)
    did = rng.integers(0, 32, size=(T, 2))
    sb = rng.integers(100, 150, size=(T, 2))
    meta = (sb | (did << 8)).astype(np.uint16)
    sal = np.array([1, 2], np.int32)
    rcodes = rng.integers(0, 256, size=(2, C // 2), dtype=np.uint8)
    rdid = rng.integers(0, 32, size=(2, 2))
    rsb = sb[sal] - rng.integers(5, 12, size=(2, 2))
    rmeta = (rsb | (rdid << 8)).astype(np.uint16)
    q = orc.Quantized(codes, meta, salient_idx=sal, res_codes=rcodes, res_meta=rmeta)
    got = orc.dequantize(q, FB, out_dtype="bf16")
    inexact = 0
    for t in range(T):
        cc = unpack_codes(codes[t])
        for c in range(C):
            mag = int(FB[did[t, c // 32], cc[c] & 7]) * Fraction(2) ** (int(sb[t, c // 32]) - 127)
            val = -mag if cc[c] & 8 else mag
            if t in (1, 2):
                s_ = t - 1
                rc = unpack_codes(rcodes[s_])
                rmag = int(FB[rdid[s_, c // 32], rc[c] & 7]) * Fraction(2) ** (int(rsb[s_, c // 32]) - 127)
                val += -rmag if rc[c] & 8 else rmag
            if val == 0:
                assert int(got[t, c]) & 0x7FFF == 0
                continue
            want = _round_to_bf16_bits(val)
            assert int(got[t, c]) == want, (t, c, hex(int(got[t, c])), hex(want))
            inexact += bf16_value(want) != val
    assert inexact > 30, inexact                                  # the rounding was exercised


def pin_decomposition_with_clamped_exponent(seed=18, n=30):
    """Residual pass under the 5-bit exponent range (e in [-15, 16]): Delta is the difference between the input
    and the decoded, possibly saturated, value; where that difference needs more than 24 significant bits it
    is rounded to binary32 first.  Every residual block must equal the block-wise definition on those values,
    and blocks with a saturated element must occur."""
    rng = np.random.default_rng(seed)
    cfg = orc.Config(exp_min=-15, exp_max=16)
    saturated = rounded = 0
    for it in range(n):
        x = np.stack([rand_block_bits(rng, 64, (8, 44) if it % 2 == 0 else (-44, -8), zero_frac=0.05) for _ in range(3)])
        if it % 3 == 0:
            x[1, 5] = synth.f32_to_bf16_bits(np.array([1.9921875 * 2.0 ** 50], np.float32))[0]   # 8 bits at 2^50
        sal = np.array([0, 1, 2], dtype=np.int32)
        q = orc.quantize(x, FB, cfg, salient_idx=sal)
        main = orc.dequantize(orc.Quantized(q.codes, q.meta), FB)
        for t in range(3):
            for blk in range(2):
                sl = slice(blk * 32, blk * 32 + 32)
                e = int(q.meta[t, blk] & 0xFF) - 124
                assert -15 <= e <= 16
                delta = []
                for b, m in zip(x[t, sl], main[t, sl]):
                    xv = bf16_value(int(b))
                    assert abs(f32_value(m)) <= 15 * Fraction(2) ** (e - 3)
                    saturated += abs(xv) >= 16 * Fraction(2) ** (e - 3)
                    exact = xv - f32_value(m)
                    r = _round_to_f32(exact)
                    rounded += r != exact
                    delta.append(float(r))
                code, did, re_, _ = orc.quantize_block_f64(np.array(delta), FB, cfg)
                assert np.array_equal(unpack_codes(q.res_codes[t, blk * 16:(blk + 1) * 16]), code)
                assert int(q.res_meta[t, blk]) == (re_ + 124) | (did << 8)
                # the sign of a saturated element's residual is the sign of the element
                for b, dl in zip(x[t, sl], delta):
                    if abs(bf16_value(int(b))) >= 16 * Fraction(2) ** (e - 3):
                        assert (dl < 0) == bool(int(b) >> 15) and dl != 0
    assert saturated > 100 and rounded > 0


def pin_mse():
    x = synth.f32_to_bf16_bits(np.array([[1.0, 2.0, -3.0, 0.5]], np.float32))
    r = np.array([[1.5, 2.0, -1.0, 0.5]], np.float32)
    assert orc.mse(x, r) == (0.25 + 4.0) / 4


ALL_PINS = [
    pin_scale_is_floor_log2, pin_exponent_clamp, pin_zero_block, pin_rounding_is_nearest, pin_uniform_dialect_closed_form,
    pin_representable_values_roundtrip, pin_error_terms_and_argmin, pin_groups_are_contiguous,
    pin_select_all_mode, pin_seda_choice_inside_mask, pin_salient_is_per_tile_argmax, pin_salient_topk, pin_decomposition, pin_residual_uses_the_seda_mask,
    pin_dequantize_formula, pin_dequantize_f16, pin_dequantize_bf16_rounds_sums_to_nearest_even,
    pin_decomposition_with_clamped_exponent, pin_mse, pin_f32_input, pin_affine_producer, pin_layernorm_producer, pin_mxfp8_view, pin_mxfp8_scale_layout, pin_weight_quantization,
    pin_subformatbook_hand_counted,
    pin_subformatbook_one_dialect_per_bucket_and_closed_loop,
]
