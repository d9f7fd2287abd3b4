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
