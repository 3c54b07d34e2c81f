"""The two facts the table form of the server's sum (Algorithm 3, server side) rests on, checked on the
host with numpy: the multiplication that gathers four workers' bits of a coordinate into a table
offset, and the bound on the magnitudes' exponents under which adding per-group partial sums gives
the bits of the worker-by-worker binary64 sum."""
import numpy as np
import pytest

GATHER_MUL = 0x10204080        # 2^28 + 2^21 + 2^14 + 2^7


def table_offset(x, c):
    return ((((x & (0x01010101 << c)) & 0xFFFFFFFF) * (GATHER_MUL >> c)) & 0xFFFFFFFF) >> 25


def test_gather_multiplication_yields_eight_times_the_four_bits():
    """x holds one byte per worker (byte k = worker k's eight sign bits); for every coordinate c and every
    combination of the four workers' bits at c, whatever the other 28 bits are, the offset is
    8 * (bit of worker 0 + 2 * bit of worker 1 + 4 * ... )."""
    rng = np.random.default_rng(0)
    for c in range(8):
        for m in range(16):
            for _ in range(50):
                x = int(rng.integers(0, 1 << 32))
                for k in range(4):
                    x &= ~(1 << (8 * k + c))
                    x |= ((m >> k) & 1) << (8 * k + c)
                assert table_offset(x, c) == 8 * m, (c, m, hex(x))


def sequential(signs, s):
    acc = np.float64(0.0)
    for sg, v in zip(signs, s):
        acc = np.float64(acc + (np.float64(v) if sg else -np.float64(v)))
    return acc


def grouped(signs, s):
    acc = np.float64(0.0)
    for g in range(0, len(s), 4):
        part = np.float64(0.0)
        for sg, v in zip(signs[g:g + 4], s[g:g + 4]):
            part = np.float64(part + (np.float64(v) if sg else -np.float64(v)))
        acc = np.float64(acc + part)
    return acc


@pytest.mark.parametrize("W", [5, 8, 16, 33, 64])
def test_grouped_sum_equals_sequential_sum_inside_the_exponent_bound(W):
    """Magnitudes (binary32, full 24-bit significands) whose exponents differ by at most
    29 - ceil(log2 W): every partial sum is an integer below 2^53 in units of the smallest magnitude's
    last place, so both orders give the same binary64 bits, zeros and subnormals included."""
    rng = np.random.default_rng(W)
    limit = 29 - int(np.ceil(np.log2(W)))
    for trial in range(300):
        e0 = int(rng.integers(-126, 100 - limit))
        exps = rng.integers(e0, e0 + limit + 1, size=W)
        exps[rng.integers(0, W)] = e0
        exps[rng.integers(0, W)] = e0 + limit                       # the full spread is present
        mant = rng.integers(1 << 23, 1 << 24, size=W).astype(np.float64)
        s = (mant * np.exp2(exps.astype(np.float64) - 23)).astype(np.float32)
        if trial % 7 == 0:
            s[rng.integers(0, W)] = 0.0
        if trial % 11 == 0 and e0 == -126:
            s[rng.integers(0, W)] = np.float32(1e-42)                # a subnormal shares the smallest normals' exponent
        signs = rng.integers(0, 2, size=W)
        a, b = sequential(signs, s), grouped(signs, s)
        assert a.tobytes() == b.tobytes(), (trial, s, signs)


def test_grouped_sum_can_differ_outside_the_bound():
    """Exponents further apart than the bound allows: worker by worker each 2^-53 is absorbed by 1.0 (a
    tie, rounded to even); grouped, the two of them first add up to 2^-52, which 1.0 does not absorb.
    This is why a chunk that fails the check is added worker by worker."""
    s = np.array([0, 0, 0, 1.0, 2.0 ** -53, 2.0 ** -53, 0, 0], np.float32)
    signs = [1] * 8
    assert sequential(signs, s) == 1.0
    assert grouped(signs, s) == 1.0 + 2.0 ** -52
