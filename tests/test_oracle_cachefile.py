"""Pins for oracle/cachefile.py (CPU only)."""
import struct

import numpy as np
import pytest

from oracle import cachefile as cf


def test_fnv1a64_published_vectors():
    """Test vectors of the FNV-1a 64-bit hash from its authors' reference list."""
    assert cf.fnv1a64(b"") == 0xCBF29CE484222325
    assert cf.fnv1a64(b"a") == 0xAF63DC4C8601EC8C
    assert cf.fnv1a64(b"foobar") == 0x85944171F73967E8


def _tiny():
    layers = [dict(op=0, C=3, K=4, R=3, S=3, stride=1, pad=1, groups=1, H=5, W=6, in0=-1, in1=-1, act=1, has_bias=1,
                   w_off=0, b_off=512),
              dict(op=1, C=4, K=4, R=2, S=2, stride=2, pad=0, groups=1, H=5, W=6, in0=0, in1=-1, act=0, has_bias=0,
                   w_off=0, b_off=0)]
    raw = bytes(range(256)) * 3                     # 768 bytes
    cached = bytes(reversed(range(256))) * 2        # 512 bytes
    return layers, [(4, 1, 1), None], [2, 0], 3, raw, cached


def test_layout_written_out_by_hand():
    """Every field of a two-layer file at the offset the format gives it."""
    layers, choices, queues, n_little, raw, cached = _tiny()
    data = cf.encode(layers, choices, queues, n_little, raw, cached)
    assert len(data) == 4096 + 4096 + 4096 and len(data) % 4096 == 0
    assert data[0:8] == b"NNV12WC\0"
    assert struct.unpack_from("<II", data, 8) == (1, 2)
    assert struct.unpack_from("<QQQQ", data, 16) == (768, 512, 4096, 8192)
    assert struct.unpack_from("<II", data, 48) == (3, 0)
    tables = data[64:64 + 2 * 88]
    assert struct.unpack_from("<Q", data, 56)[0] == cf.fnv1a64(tables)
    assert struct.unpack_from("<14i", tables, 0) == (0, 3, 4, 3, 3, 1, 1, 1, 5, 6, -1, -1, 1, 1)
    assert struct.unpack_from("<QQ", tables, 56) == (0, 512)
    assert struct.unpack_from("<14i", tables, 72)[:3] == (1, 4, 4)
    assert struct.unpack_from("<4i", tables, 144) == (4, 1, 1, 2)
    assert struct.unpack_from("<4i", tables, 160) == (-1, -1, 0, -1)            # pool layer
    assert data[64 + 176:4096] == bytes(4096 - 240)                              # zero padding
    assert data[4096:4096 + 768] == raw and data[4096 + 768:8192] == bytes(4096 - 768)
    assert data[8192:8192 + 512] == cached and data[8192 + 512:] == bytes(4096 - 512)


def test_round_trip_and_no_cached_blob():
    layers, choices, queues, n_little, raw, cached = _tiny()
    got = cf.decode(cf.encode(layers, choices, queues, n_little, raw, cached))
    assert got["layers"] == layers and got["choices"] == choices and got["queue_of"] == [2, -1]
    assert got["n_little"] == 3 and got["raw"] == raw and got["cached"] == cached
    data = cf.encode(layers, [(1, 1, 0), None], None, 0, raw, b"")
    assert len(data) == 8192
    got = cf.decode(data)
    assert got["cached"] == b"" and got["queue_of"] == [-1, -1] and got["n_little"] == 0


def test_corruption_is_detected():
    layers, choices, queues, n_little, raw, cached = _tiny()
    data = bytearray(cf.encode(layers, choices, queues, n_little, raw, cached))
    for pos in (0, 8, 70, 64 + 150):                      # magic, version, a layer field, a plan field
        bad = bytearray(data)
        bad[pos] ^= 0x40
        with pytest.raises(ValueError):
            cf.decode(bytes(bad))
    with pytest.raises(ValueError):
        cf.decode(bytes(data[:-1]))
    with pytest.raises(ValueError):
        cf.decode(bytes(data[:40]))
    rng = np.random.default_rng(3)
    blob = rng.integers(0, 256, 5000, dtype=np.uint8).tobytes()
    assert cf.decode(cf.encode(layers, choices, queues, n_little, blob, b""))["raw"] == blob
