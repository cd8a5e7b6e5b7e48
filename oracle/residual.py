"""Differential KV: reconstruction of a prefix-conditioned KV state from a base and a sparse residual.

TEST INFRASTRUCTURE ONLY (see the package docstring).

Sec. 5.1, Eq. 7: for an operation v under a prefix path P,
    KV(P, v) = KV_base(v) + dKV(P, v),
where KV_base(v) is computed once from the operation alone and dKV(P, v) holds only the entries the
prefix changed (the section reports more than 75 % of key entries and more than 70 % of value
entries below a small threshold).  The oracle is that sum written out, entry by entry.

Readings the paper leaves open:
  * storage format of the residual (none is given): a bitmap of the entries that carry a value,
    the values packed in (row, column) order, and the exclusive prefix sum of the rows' counts;
  * precision: base, residual values and the reconstructed state are bf16 like the KV cache; an
    entry with a residual becomes the exact sum rounded once to bf16 (round to nearest, ties to
    even); an entry without one is the base, bit for bit.

Pins (tests/test_oracle_residual.py): hand-worked bf16 sums including ties in both directions, an
empty residual (identity), a residual equal to minus the base (exact zeros), reconstruction from a
dense difference built independently of the sparse format, exact rational arithmetic on random
entries, and attention over the reconstructed state against attention over base + dense delta; for
`encode` (the residual from the two states, thresholded): hand-worked differences including one equal
to the threshold, the kept set and the stored values against exact rational arithmetic, and the bound
|reconstruct(encode) - full| <= threshold + rounding with a stored count that falls as the threshold rises.
"""
from __future__ import annotations

import numpy as np


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact value of bf16 bit patterns (the upper half of an IEEE binary32)."""
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16_rne(x: np.ndarray) -> np.ndarray:
    """fp64 -> bf16 bit patterns with a single rounding, nearest, ties to even (normal range, finite).

    A bf16 has 8 significant bits: x = m * 2^e with 0.5 <= |m| < 1 is rounded to rint(m * 256) * 2^(e-8);
    numpy's rint rounds halves to even.  The result is exactly representable in binary32, so its bit
    pattern can be read off after a (then exact) conversion.
    """
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)
    r = np.ldexp(np.rint(m * 256.0), e - 8)
    b = r.astype(np.float32).view(np.uint32)
    assert np.all((b & np.uint32(0xFFFF)) == 0), "rounded value must fit bf16"
    return (b >> np.uint32(16)).astype(np.uint16)


def densify(bitmap: np.ndarray, values: np.ndarray, row_ptr: np.ndarray, head_dim: int):
    """(has[rows, D] bool, delta[rows, D] uint16 bf16 bits, 0 where absent) from the bitmap format.

    Bit j of word w of a row marks column 32 * w + j; the values follow in (row, column) order, which
    is the order boolean indexing of a row-major array visits; row_ptr must be the exclusive prefix
    sum of the rows' bit counts.
    """
    rows = bitmap.shape[0]
    bits = (bitmap.astype(np.uint32)[:, :, None] >> np.arange(32, dtype=np.uint32)) & np.uint32(1)
    has = bits.reshape(rows, head_dim).astype(bool)
    counts = np.concatenate([[0], np.cumsum(has.sum(axis=1))])
    assert np.array_equal(counts, np.asarray(row_ptr, dtype=np.int64)), "row_ptr must count the bits of every row"
    assert len(values) == counts[-1]
    delta = np.zeros((rows, head_dim), dtype=np.uint16)
    delta[has] = values
    return has, delta


def reconstruct(base_bits: np.ndarray, bitmap: np.ndarray, values: np.ndarray, row_ptr: np.ndarray) -> np.ndarray:
    """Eq. 7 for one tensor: base_bits uint16[rows, D] -> uint16[rows, D]."""
    rows, D = base_bits.shape
    has, delta = densify(bitmap, values, row_ptr, D)
    # exact in fp64: both addends have 8-bit significands and their exponents differ by far less than 44
    total = bf16_to_f64(base_bits) + bf16_to_f64(delta)
    return np.where(has, f64_to_bf16_rne(total), base_bits).astype(np.uint16)


def encode(base_bits: np.ndarray, full_bits: np.ndarray, threshold: float):
    """The residual of Eq. 7 from the two states it relates: dKV = KV(P, v) - KV_base(v), kept sparse.

    base_bits, full_bits: uint16[rows, D] (bf16).  Sec. 5.1 drops the entries of the difference that
    fall below a small threshold and stores the rest.  Readings: the difference of an entry is the
    exact difference rounded once to bf16 (the precision it is stored in); it is kept when the
    magnitude of that stored value exceeds `threshold` (so threshold 0 keeps every non-zero
    difference).  Returns (bitmap uint32[rows, D // 32], values uint16[nnz], row_ptr int32[rows + 1])
    in the format `reconstruct` reads.
    """
    rows, D = base_bits.shape
    diff = f64_to_bf16_rne(bf16_to_f64(full_bits) - bf16_to_f64(base_bits))  # the subtraction is exact in fp64
    keep = np.abs(bf16_to_f64(diff)) > float(threshold)
    bitmap = np.zeros((rows, D // 32), dtype=np.uint32)
    values = []
    row_ptr = [0]
    for r in range(rows):
        for d in range(D):
            if keep[r, d]:
                bitmap[r, d >> 5] |= np.uint32(1 << (d & 31))
                values.append(diff[r, d])
        row_ptr.append(len(values))
    return bitmap, np.array(values, dtype=np.uint16), np.array(row_ptr, dtype=np.int32)
