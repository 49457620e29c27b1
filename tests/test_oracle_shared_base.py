"""Pins of the oracle's shared-base storage format (paper Section 2.2, "Overhead of Storing Samples")."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "shared_base_example.txt")


def dataset_from_codes(c1, c2, bits):
    """A one-plane-pair dataset from explicit codes (rows x features), through the oracle's packer (pinned elsewhere)."""
    c1, c2 = np.asarray(c1, np.uint8), np.asarray(c2, np.uint8)
    m, n = c1.shape
    p1 = np.stack([oracle.pack_codes(c1[k], bits) for k in range(m)])
    p2 = np.stack([oracle.pack_codes(c2[k], bits) for k in range(m)])
    return oracle.Dataset(p1, p2, m, n, bits, oracle.UNIFORM, np.zeros(n, np.float32), np.ones(n, np.float32), None)


def up_bits(plane, n):
    """Independent reading of a one-bit plane: numpy's own little-endian bit unpacking."""
    return np.unpackbits(plane, axis=1, bitorder="little")[:, :n]


def test_hand_example():
    rec = {}
    for line in open(GOLDEN):
        if line.strip() and not line.startswith("#"):
            key, *vals = line.split()
            rec[key] = vals
    bits, n = int(rec["bits"][0]), int(rec["n"][0])
    c1, c2 = [int(v) for v in rec["codes1"]], [int(v) for v in rec["codes2"]]
    base, up1, up2 = oracle.shared_base_encode(dataset_from_codes([c1], [c2], bits))
    for got, key in ((base, "base_bytes"), (up1, "up1_bytes"), (up2, "up2_bytes")):
        want = [int(v, 16) for v in rec[key]]
        assert list(got[0, : len(want)]) == want and not got[0, len(want):].any()
    p1, p2 = oracle.shared_base_decode(base, up1, up2, n, bits)
    assert list(oracle.unpack_codes(p1[0], n, bits)) == c1 and list(oracle.unpack_codes(p2[0], n, bits)) == c2


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_every_pair_of_neighbouring_codes_round_trips(bits):
    """All (lower level, up bit of sample 1, up bit of sample 2): the base is the smaller code, decoding gives the
    two codes back; codes two levels apart are not two samples of one value and are refused."""
    s = (1 << bits) - 1
    pairs = [(l + u1, l + u2) for l in range(s) for u1 in (0, 1) for u2 in (0, 1)]
    c1 = np.array([[p[0] for p in pairs]], np.uint8)
    c2 = np.array([[p[1] for p in pairs]], np.uint8)
    ds = dataset_from_codes(c1, c2, bits)
    base, up1, up2 = oracle.shared_base_encode(ds)
    n = len(pairs)
    assert (oracle.unpack_codes(base[0], n, bits) == np.minimum(c1, c2)[0]).all()
    assert (up_bits(up1, n)[0] == (c1 - np.minimum(c1, c2))[0]).all() and (up_bits(up2, n)[0] == (c2 - np.minimum(c1, c2))[0]).all()
    p1, p2 = oracle.shared_base_decode(base, up1, up2, n, bits)
    assert (p1 == ds.plane1).all() and (p2 == ds.plane2).all()
    with pytest.raises(oracle.OracleError):
        oracle.shared_base_encode(dataset_from_codes([[0, 2]], [[2, 2]], bits))


@pytest.mark.parametrize("m,n,bits,seed", [(40, 64, 4, 0), (33, 61, 4, 1), (20, 1000, 8, 2), (17, 2050, 2, 3), (25, 37, 3, 4), (3, 1, 2, 5)])
def test_quantized_samples_round_trip(m, n, bits, seed):
    """Two stochastic roundings of one value differ by at most one level, so every quantized dataset encodes; an
    independent numpy reading of the three planes reproduces the codes; the format takes bits + 2 bits per value."""
    rng = np.random.default_rng(seed)
    A = rng.uniform(-1, 1, (m, n)).astype(np.float32)
    A[:, n // 2] = 0.5                                     # a constant feature
    ds = oracle.quantize(A, bits, seed=seed + 10)
    base, up1, up2 = oracle.shared_base_encode(ds)
    c1, c2 = oracle.unpack_plane(ds.plane1, n, bits), oracle.unpack_plane(ds.plane2, n, bits)
    cb_ = oracle.unpack_plane(base, n, bits)
    assert (cb_ == np.minimum(c1, c2)).all()
    assert (cb_ + up_bits(up1, n) == c1).all() and (cb_ + up_bits(up2, n) == c2).all()
    p1, p2 = oracle.shared_base_decode(base, up1, up2, n, bits)
    assert (p1 == ds.plane1).all() and (p2 == ds.plane2).all()
    # padding is zero, strides are what the layout says
    assert base.shape[1] == oracle.row_bytes(n, bits) and up1.shape[1] == oracle.up_row_bytes(n) == (((n + 7) // 8 + 15) // 16) * 16
    assert not up_bits(up1, up1.shape[1] * 8)[:, n:].any() and not up_bits(up2, up2.shape[1] * 8)[:, n:].any()


def test_bits_per_value():
    """bits + 2 instead of 2 * bits per value (container widths: 2, 4, 4, 8): 10 vs 16 at 8 bits, 6 vs 8 at 4 bits."""
    n = 1024
    for bits, cb in ((2, 2), (3, 4), (4, 4), (8, 8)):
        two_planes = 2 * oracle.row_bytes(n, bits) * 8 / n
        shared = (oracle.row_bytes(n, bits) + 2 * oracle.up_row_bytes(n)) * 8 / n
        assert two_planes == 2 * cb and shared == cb + 2
