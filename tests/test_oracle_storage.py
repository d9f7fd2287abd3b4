"""Pins for the oracle's storage helpers: packing, fp16 decode and the boundary gate (Eq. 4)."""
import numpy as np


def test_half_decode_matches_numpy_exhaustively(qo):
    h = np.arange(65536, dtype=np.uint16)
    want = h.view(np.float16).astype(np.float32)
    got = np.array([qo.half_to_float(int(v)) for v in h], dtype=np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))


def test_int4_pack_layout_and_roundtrip(qo):
    codes = np.array([-8, 7, -1, 0, 3, -5, 1, 2], np.int32)
    packed = qo.pack(4, codes)
    # even element in the low nibble, two's complement
    assert list(packed) == [0x78, 0x0f, 0xb3, 0x21]
    assert np.array_equal(qo.unpack(4, packed, 8), codes)
    every = np.arange(256, dtype=np.uint8)
    un = qo.unpack(4, every, 512)
    assert un.min() == -8 and un.max() == 7
    assert np.array_equal(qo.pack(4, un), every)
    lo = (every & 0xf).astype(np.int32); hi = (every >> 4).astype(np.int32)
    assert np.array_equal(un[0::2], np.where(lo > 7, lo - 16, lo))
    assert np.array_equal(un[1::2], np.where(hi > 7, hi - 16, hi))


def test_int8_pack_roundtrip(qo):
    every = np.arange(256, dtype=np.uint8)
    un = qo.unpack(8, every, 256)
    assert np.array_equal(un, every.view(np.int8).astype(np.int32))
    assert np.array_equal(qo.pack(8, un), every)


def test_gate_and_clamp_exhaustive(qo):
    for (qmin, qmax, span) in ((-8, 7, 15), (-7, 7, 15), (-128, 127, 255)):
        for w in range(qmin, qmax + 1):
            for step in range(-span, span + 1):
                g = qo.applied_step(w, step, qmin, qmax, 0)
                c = qo.applied_step(w, step, qmin, qmax, 1)
                inside = qmin <= w + step <= qmax
                assert g == (step if inside else 0)            # Eq. 4: masked, weight unchanged
                assert qmin <= w + g <= qmax
                assert w + c == min(qmax, max(qmin, w + step))  # saturating variant
                if inside:
                    assert g == c == step


def test_half_encode_matches_numpy_and_roundtrips(qo):
    """binary16 rounding (nearest even) on every representable value, every midpoint between neighbours,
    random doubles over the whole range, subnormals, overflow and signed zero."""
    all_bits = np.arange(1 << 16, dtype=np.uint16)
    vals = all_bits.view(np.float16).astype(np.float64)
    finite = np.isfinite(vals)
    assert np.array_equal(qo.to_half(vals[finite]), all_bits[finite])            # round trip
    pos = np.sort(vals[finite & (vals >= 0)])
    mids = (pos[:-1] + pos[1:]) / 2.0                                            # ties go to the even neighbour
    rng = np.random.default_rng(0)
    rnd = np.concatenate([rng.standard_normal(200_000) * 10.0 ** rng.integers(-9, 5, 200_000), mids, -mids,
                          [65519.9, 65520.0, 1e9, -1e9, 2.0 ** -25, 2.0 ** -25 * 1.0000001, 0.0, -0.0]])
    with np.errstate(over="ignore"):
        want = rnd.astype(np.float16).view(np.uint16)
    assert np.array_equal(qo.to_half(rnd), want)
