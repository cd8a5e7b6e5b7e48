"""Pins of the differential-KV oracle (Sec. 5.1, Eq. 7) against things other than itself."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import attention as OA
from oracle import residual as OR
from paper_2605_22566_b200 import workloads as W


def bits_of(x):
    """bf16 bit pattern of a value that is exactly representable (checked)."""
    b = np.array([x], dtype=np.float32).view(np.uint32)[0]
    assert b & 0xFFFF == 0, x
    return np.uint16(b >> 16)


def frac_of(bits):
    """Exact rational value of a bf16 bit pattern, from the format's definition."""
    b = int(bits)
    sign = -1 if b >> 15 else 1
    e = (b >> 7) & 0xFF
    m = b & 0x7F
    assert 0 < e < 255
    return sign * Fraction(128 + m, 128) * Fraction(2) ** (e - 127)


def rne_bf16_from_fraction(x):
    """Round an exact rational to bf16 (nearest, ties to even) by brute force over its two neighbours."""
    if x == 0:
        return np.uint16(0)
    sign = 0x8000 if x < 0 else 0
    a = abs(x)
    e = 0
    while Fraction(2) ** (e + 1) <= a:
        e += 1
    while Fraction(2) ** e > a:
        e -= 1
    scaled = a / Fraction(2) ** e * 128  # in [128, 256)
    lo = int(scaled)
    rem = scaled - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (lo & 1)):
        lo += 1
    if lo == 256:
        lo, e = 128, e + 1
    return np.uint16(sign | ((e + 127) << 7) | (lo - 128))


def one_entry(base, delta):
    """Reconstruct a 1 x 32 tensor whose entry 5 has a residual."""
    b = np.full((1, 32), bits_of(base), dtype=np.uint16)
    bitmap = np.array([[1 << 5]], dtype=np.uint32)
    out = OR.reconstruct(b, bitmap, np.array([bits_of(delta)], dtype=np.uint16), np.array([0, 1], dtype=np.int32))
    assert np.array_equal(np.delete(out[0], 5), np.delete(b[0], 5))  # the other entries are the base
    return out[0, 5]


def test_hand_worked_sums_and_ties():
    # bf16 has 8 significant bits: around 1.0 the spacing is 2^-7
    assert one_entry(1.0, 0.5) == bits_of(1.5)
    assert one_entry(1.0, 2.0 ** -7) == bits_of(1.0 + 2.0 ** -7)
    assert one_entry(1.0, 2.0 ** -8) == bits_of(1.0)                    # tie, even significand below
    assert one_entry(1.0 + 2.0 ** -7, 2.0 ** -8) == bits_of(1.0 + 2.0 ** -6)  # tie, even significand above
    assert one_entry(1.0, 2.0 ** -8 + 2.0 ** -15) == bits_of(1.0 + 2.0 ** -7)  # just above the tie
    assert one_entry(1.0, -(2.0 ** -9)) == bits_of(1.0)                  # tie below 1 (spacing 2^-8): even is 1.0
    assert one_entry(-3.0, 1.0) == bits_of(-2.0)
    assert one_entry(0.75, -0.75) == np.uint16(0)                        # exact cancellation: +0


def test_empty_residual_is_identity_and_negated_base_gives_zero():
    rng = np.random.default_rng(1)
    base = W.fill_bits(123, 0, 6 * 64).reshape(6, 64)
    none = OR.reconstruct(base, np.zeros((6, 2), np.uint32), np.zeros(0, np.uint16), np.zeros(7, np.int32))
    assert np.array_equal(none, base)
    full = np.full((6, 2), 0xFFFFFFFF, dtype=np.uint32)
    neg = (base ^ np.uint16(0x8000)).reshape(-1)
    z = OR.reconstruct(base, full, neg, (np.arange(7) * 64).astype(np.int32))
    assert np.all(z == 0)


def test_against_exact_rational_arithmetic_on_random_entries():
    bitmap, vals, row_ptr = W.residual_stream(7, W.KIND_DK, 0, 3, 1, 12, 64, 0.3)
    base = W.fill_bits(99, 0, 12 * 64).reshape(12, 64)
    out = OR.reconstruct(base, bitmap, vals, row_ptr)
    k = 0
    checked = 0
    for r in range(12):
        for d in range(64):
            if (int(bitmap[r, d >> 5]) >> (d & 31)) & 1:
                want = rne_bf16_from_fraction(frac_of(base[r, d]) + frac_of(vals[k]))
                assert out[r, d] == want, (r, d)
                k += 1
                checked += 1
            else:
                assert out[r, d] == base[r, d]
    assert k == len(vals) == row_ptr[-1] and checked > 150


def test_sparse_format_against_a_dense_difference_built_independently():
    # the dense delta is generated first; the sparse triple is derived from it with a plain loop
    rng = np.random.default_rng(5)
    rows, D = 9, 96
    dense = np.zeros((rows, D), dtype=np.uint16)
    mask = rng.random((rows, D)) < 0.27
    dense[mask] = W.f32_to_bf16_bits((rng.standard_normal(mask.sum()) * 0.1).astype(np.float32))
    mask &= (dense & 0x7FFF) != 0
    bitmap = np.zeros((rows, D // 32), dtype=np.uint32)
    vals, row_ptr = [], [0]
    for r in range(rows):
        for d in range(D):
            if mask[r, d]:
                bitmap[r, d // 32] |= np.uint32(1 << (d % 32))
                vals.append(dense[r, d])
        row_ptr.append(len(vals))
    base = W.fill_bits(5, 0, rows * D).reshape(rows, D)
    out = OR.reconstruct(base, bitmap, np.array(vals, dtype=np.uint16), np.array(row_ptr, dtype=np.int32))
    want = W.f32_to_bf16_bits(W.bf16_bits_to_f32(base) + W.bf16_bits_to_f32(dense))  # fp32 sum is exact here, one rounding
    assert np.array_equal(out[mask], want[mask])
    assert np.array_equal(out[~mask], base[~mask])


def test_generator_density_and_format():
    bitmap, vals, row_ptr = W.residual_stream(11, W.KIND_DV, 2, 40, 3, 256, 128, 0.25)
    nnz = int(row_ptr[-1])
    assert nnz == len(vals) and abs(nnz / (256 * 128) - 0.25) < 0.01
    assert np.all((vals & 0x7FFF) != 0)
    pop = np.array([bin(int(w)).count("1") for w in bitmap.reshape(-1)]).reshape(256, 4).sum(axis=1)
    assert np.array_equal(np.cumsum(pop), row_ptr[1:])
    other = W.residual_stream(11, W.KIND_DV, 2, 40, 4, 256, 128, 0.25)  # another prefix: another residual
    assert not np.array_equal(other[0], bitmap)


def test_attention_over_reconstructed_state_equals_attention_over_base_plus_delta():
    """Eq. 7 inside the attention definition: the context-aware state is what the query attends over."""
    Hkv, D, n = 2, 64, 37
    kb = W.fill_bits(1, 0, n * Hkv * D).reshape(n * Hkv, D)
    vb = W.fill_bits(2, 0, n * Hkv * D).reshape(n * Hkv, D)
    rk = W.residual_stream(3, W.KIND_DK, 0, 0, 1, n * Hkv, D, 0.25)
    rv = W.residual_stream(3, W.KIND_DV, 0, 0, 1, n * Hkv, D, 0.30)
    K = OR.bf16_to_f64(OR.reconstruct(kb, *rk)).reshape(n, Hkv, D)
    V = OR.bf16_to_f64(OR.reconstruct(vb, *rv)).reshape(n, Hkv, D)
    _, dk = OR.densify(*rk, D)
    _, dv = OR.densify(*rv, D)
    K2 = (OR.bf16_to_f64(kb) + OR.bf16_to_f64(dk)).reshape(n, Hkv, D)
    V2 = (OR.bf16_to_f64(vb) + OR.bf16_to_f64(dv)).reshape(n, Hkv, D)
    q = OR.bf16_to_f64(W.fill_bits(4, 0, D))
    for h in range(Hkv):
        o1, l1 = OA.attend(q, K[:, h], V[:, h], 0.125)
        o2, l2 = OA.attend(q, K2[:, h], V2[:, h], 0.125)
        # the only difference is the single bf16 rounding of the reconstructed entries (2^-9 relative)
        assert np.max(np.abs(o1 - o2)) < 2e-2 and abs(l1 - l2) < 2e-2
        assert np.max(np.abs(o1 - o2)) > 0  # and it is there: the state really is stored in bf16


def _states(rows=10, D=64, seed=21):
    """A base and a prefix-conditioned state: the base plus a sparse large change plus a dense tiny one."""
    base = W.fill_bits(seed, 0, rows * D).reshape(rows, D)
    big = W.residual_stream(seed, W.KIND_DK, 0, 1, 1, rows, D, 0.25, sigma=0.25)
    tiny = W.residual_stream(seed, W.KIND_DV, 0, 1, 2, rows, D, 0.6, sigma=2.0 ** -12)
    full = OR.reconstruct(OR.reconstruct(base, *big), *tiny)
    return base, full


def test_encode_hand_worked_and_degenerate_cases():
    b = np.full((1, 32), bits_of(1.0), dtype=np.uint16)
    f = b.copy()
    f[0, 3] = bits_of(1.5)       # difference 0.5
    f[0, 7] = bits_of(1.0 + 2.0 ** -7)  # difference 2^-7
    f[0, 9] = bits_of(0.5)       # difference -0.5
    bm, vals, rp = OR.encode(b, f, 2.0 ** -6)
    assert bm.tolist() == [[(1 << 3) | (1 << 9)]] and vals.tolist() == [bits_of(0.5), bits_of(-0.5)] and rp.tolist() == [0, 2]
    bm, vals, rp = OR.encode(b, f, 0.0)
    assert bm.tolist() == [[(1 << 3) | (1 << 7) | (1 << 9)]] and rp.tolist() == [0, 3]
    bm, vals, rp = OR.encode(b, f, 0.5)   # a magnitude equal to the threshold is dropped
    assert int(rp[-1]) == 0 and not bm.any()
    bm, vals, rp = OR.encode(b, b, 0.0)   # identical states: nothing to store
    assert int(rp[-1]) == 0


def test_encode_keeps_what_exceeds_the_threshold_checked_with_rationals():
    base, full = _states()
    tau = 2.0 ** -8
    bm, vals, rp = OR.encode(base, full, tau)
    has, delta = OR.densify(bm, vals, rp, base.shape[1])
    for r in range(base.shape[0]):
        for d in range(base.shape[1]):
            want = rne_bf16_from_fraction(frac_of(full[r, d]) - frac_of(base[r, d])) if full[r, d] != base[r, d] else np.uint16(0)
            mag = abs(frac_of(want)) if (int(want) & 0x7FFF) else Fraction(0)
            assert has[r, d] == (mag > Fraction(tau)), (r, d)
            if has[r, d]:
                assert delta[r, d] == want
    assert 0.15 < has.mean() < 0.35  # the large changes survive, the tiny ones do not


def test_encode_then_reconstruct_is_within_threshold_of_the_full_state():
    base, full = _states(rows=16, D=128, seed=33)
    prev_nnz = None
    for tau in (0.0, 2.0 ** -10, 2.0 ** -6, 1.0):
        res = OR.encode(base, full, tau)
        back = OR.reconstruct(base, *res)
        err = np.abs(OR.bf16_to_f64(back) - OR.bf16_to_f64(full))
        ulp = np.abs(OR.bf16_to_f64(full)) * 2.0 ** -8 + np.abs(OR.bf16_to_f64(full) - OR.bf16_to_f64(base)) * 2.0 ** -8
        assert np.all(err <= tau * (1 + 2.0 ** -8) + ulp)
        nnz = int(res[2][-1])
        assert prev_nnz is None or nnz <= prev_nnz  # a larger threshold never stores more
        prev_nnz = nnz
