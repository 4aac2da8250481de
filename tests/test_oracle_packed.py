"""The packed-triangle container of the oracle (oracle/packed.py), pinned by what its definition fixes:
a one-to-one index map onto [0, elements), rows in order without gaps, 16-byte groups, and pack / unpack
being inverse to each other on triangular matrices (brute force, one entry at a time, on small sizes)."""
import numpy as np
import pytest

from oracle import packed as pk
from oracle import values as ov

SIZES = [1, 2, 3, 4, 5, 6, 7, 8, 9, 12, 13, 16, 17, 31, 64]
ORIENT = [pk.LOWER_TRI, pk.UPPER_TRI]


def in_triangle(prop, i, j):
    return i >= j if prop in (pk.LOWER_TRI, pk.STRICT_LOWER, pk.UNIT_LOWER) else i <= j


@pytest.mark.parametrize("prop", ORIENT)
@pytest.mark.parametrize("n", SIZES)
def test_index_map_is_one_to_one_and_covers_the_triangle(n, prop):
    total = pk.elements(n, prop)
    seen = {}
    n4 = 4 * ((n + 3) // 4)
    for i in range(n):
        for j in range(n4):
            at = pk.index(n, prop, i, j)
            if j < n and in_triangle(prop, i, j):
                assert at >= 0, f"entry ({i}, {j}) of the triangle is not stored"
            if at >= 0:
                assert 0 <= at < total and at not in seen
                seen[at] = (i, j)
    assert len(seen) == total                                  # onto: no position of the container is unused
    # row-major: positions grow along a row and from row to row
    order = [seen[at] for at in range(total)]
    assert order == sorted(order)


@pytest.mark.parametrize("prop", ORIENT)
@pytest.mark.parametrize("n", SIZES)
def test_rows_are_whole_16_byte_groups_and_follow_without_gaps(n, prop):
    at = 0
    for i in range(n):
        first, end = pk.row_range(n, prop, i)
        assert first % 4 == 0 and (end - first) % 4 == 0 and end - first >= 4
        assert pk.row_offset(n, prop, i) == at and at % 4 == 0
        # what is stored beyond the triangle: fewer than four entries next to the diagonal, fewer than four past the edge
        inside = sum(1 for j in range(first, min(end, n)) if in_triangle(prop, i, j))
        assert inside == (i + 1 if prop == pk.LOWER_TRI else n - i)
        assert (end - first) - inside <= 6
        at += end - first
    assert pk.elements(n, prop) == at
    assert n * (n + 1) // 2 <= at <= n * (n + 1) // 2 + 6 * n   # the triangle plus at most a few entries per row
    assert at <= 4 * ((n + 3) // 4) * n                          # never more than the dense rows rounded up to 16 bytes


@pytest.mark.parametrize("prop", [pk.LOWER_TRI, pk.UPPER_TRI, pk.STRICT_LOWER, pk.UNIT_UPPER])
@pytest.mark.parametrize("n", [1, 3, 4, 5, 8, 13, 64])
def test_pack_places_every_entry_where_the_index_map_says_and_unpack_inverts_it(n, prop):
    rng = np.random.default_rng(n * 10 + prop)
    a = rng.standard_normal((n, n)).astype(np.float32)
    lower = prop in (pk.LOWER_TRI, pk.STRICT_LOWER, pk.UNIT_LOWER)
    a = np.tril(a) if lower else np.triu(a)
    if prop in (pk.STRICT_LOWER,):
        np.fill_diagonal(a, 0.0)
    if prop in (pk.UNIT_UPPER,):
        np.fill_diagonal(a, 1.0)
    p = pk.pack(a, prop)
    assert p.dtype == np.float32 and p.shape == (pk.elements(n, prop),)
    n4 = 4 * ((n + 3) // 4)
    for i in range(n):
        for j in range(n4):
            at = pk.index(n, prop, i, j)
            if at >= 0:
                assert p[at] == (a[i, j] if j < n else 0.0)      # padding next to the diagonal holds the stored zeros of a
    assert np.array_equal(pk.unpack(p, n, prop), a)
    # an all-ones triangle: exactly n(n+1)/2 ones arrive, everything else in the container is zero
    ones = (np.tril if lower else np.triu)(np.ones((n, n), dtype=np.float32))
    assert pk.pack(ones, prop).sum() == n * (n + 1) // 2


def test_only_triangles_can_be_packed():
    for prop in (pk.GENERAL, pk.IDENTITY, pk.DIAGONAL, pk.SYMMETRIC):
        assert not pk.packable(prop)
        with pytest.raises(ValueError):
            pk.elements(8, prop)
    with pytest.raises(ValueError):
        pk.unpack(np.zeros(5, dtype=np.float32), 4, pk.LOWER_TRI)


def test_a_packed_operand_stands_for_its_dense_matrix_in_the_value_oracle():
    # L * B with L handed over packed: unpacking gives back the dense operand bit for bit, so the value is the dense one
    rng = np.random.default_rng(5)
    n = 12
    l = np.tril(rng.standard_normal((n, n))).astype(np.float32)
    b = rng.standard_normal((n, 7)).astype(np.float32)
    descs = [(n, n, ov.LOWER_TRI), (n, 7, ov.GENERAL)]
    x_dense, _ = ov.evaluate([l, b], descs)
    x_packed, _ = ov.evaluate([pk.unpack(pk.pack(l, pk.LOWER_TRI), n, pk.LOWER_TRI), b], descs)
    assert np.array_equal(x_dense, x_packed)
    assert np.allclose(x_dense, l.astype(np.float64) @ b.astype(np.float64), rtol=0, atol=1e-12)
