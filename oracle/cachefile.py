"""CPU oracle: the on-disk model file (raw weights, cached post-transform weights, kernel plan).

TEST INFRASTRUCTURE ONLY -- never imported by the product path.

The paper keeps two things in storage between runs: the kernel scheduling plan the decision stage
produced, and the post-transformed weights that let a cold inference skip the transformation at
the price of a larger read (its Sections 3 and 3.1.2; Table 4 lists the storage overhead).  It
prints no file layout, so the layout is this library's own definition, written out here byte by
byte with `struct` and nothing else.  All integers little-endian.

    header, 64 bytes
        0   8s   magic  b"NNV12WC\\0"
        8   u32  version = 1
       12   u32  n_layers
       16   u64  w_bytes      bytes of the raw weight blob
       24   u64  c_bytes      bytes of the cached (post-transform) blob, 0 = none
       32   u64  raw_off      file offset of the raw blob    = round_up(64 + 88 * n_layers, 4096)
       40   u64  cached_off   file offset of the cached blob = raw_off + round_up(w_bytes, 4096)
       48   u32  n_little     preparation queues of the stored schedule, 0 = no schedule
       52   u32  0
       56   u64  FNV-1a (64 bit) of the two tables below
    layer table, 72 bytes per layer
        14 x i32  op C K R S stride pad groups H W in0 in1 act has_bias,  2 x u64  w_off b_off
    plan table, 16 bytes per layer
        4 x i32   variant math cached queue        (-1 -1 0 -1 for pool layers)
    zero padding up to raw_off, the raw blob, zero padding up to cached_off, the cached blob,
    zero padding up to a multiple of 4096.
"""
import struct

MAGIC = b"NNV12WC\0"
VERSION = 1
HEADER = struct.Struct("<8sIIQQQQIIQ")
LAYER = struct.Struct("<14i2Q")
PLAN = struct.Struct("<4i")
LAYER_FIELDS = ("op", "C", "K", "R", "S", "stride", "pad", "groups", "H", "W", "in0", "in1", "act", "has_bias",
                "w_off", "b_off")
PAGE = 4096


def fnv1a64(data):
    """Fowler-Noll-Vo hash, variant 1a, 64 bit: h = offset basis; for each byte: h ^= byte; h *= prime."""
    h = 0xCBF29CE484222325
    for b in data:
        h ^= b
        h = (h * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
    return h


def _round_up(v, a):
    return (v + a - 1) // a * a


def encode(layers, choices, queue_of, n_little, raw_blob, cached_blob):
    """Bytes of the file.  layers: dicts with LAYER_FIELDS; choices: (variant, math, cached) or None per
    layer; queue_of: int per layer or None; blobs: bytes-like."""
    n = len(layers)
    tables = b"".join(LAYER.pack(*[int(L[f]) for f in LAYER_FIELDS]) for L in layers)
    for i in range(n):
        c = choices[i]
        q = -1 if (queue_of is None or c is None) else int(queue_of[i])
        tables += PLAN.pack(-1, -1, 0, -1) if c is None else PLAN.pack(int(c[0]), int(c[1]), int(c[2]), q)
    raw_blob, cached_blob = bytes(raw_blob), bytes(cached_blob or b"")
    raw_off = _round_up(HEADER.size + len(tables), PAGE)
    cached_off = raw_off + _round_up(len(raw_blob), PAGE)
    head = HEADER.pack(MAGIC, VERSION, n, len(raw_blob), len(cached_blob), raw_off, cached_off, int(n_little), 0,
                       fnv1a64(tables))
    out = bytearray(cached_off + _round_up(len(cached_blob), PAGE))
    out[:len(head)] = head
    out[len(head):len(head) + len(tables)] = tables
    out[raw_off:raw_off + len(raw_blob)] = raw_blob
    out[cached_off:cached_off + len(cached_blob)] = cached_blob
    return bytes(out)


def decode(data):
    """Inverse of encode; raises ValueError on a bad magic, version, size or table hash."""
    if len(data) < HEADER.size:
        raise ValueError("file shorter than its header")
    magic, ver, n, w_bytes, c_bytes, raw_off, cached_off, n_little, zero, h = HEADER.unpack_from(data, 0)
    if magic != MAGIC or ver != VERSION:
        raise ValueError("not a version-1 model file")
    tlen = n * (LAYER.size + PLAN.size)
    if raw_off != _round_up(HEADER.size + tlen, PAGE) or cached_off != raw_off + _round_up(w_bytes, PAGE) or \
            len(data) != cached_off + _round_up(c_bytes, PAGE):
        raise ValueError("inconsistent offsets or file size")
    tables = data[HEADER.size:HEADER.size + tlen]
    if fnv1a64(tables) != h:
        raise ValueError("table hash mismatch")
    layers, choices, queue_of = [], [], []
    for i in range(n):
        layers.append(dict(zip(LAYER_FIELDS, LAYER.unpack_from(tables, i * LAYER.size))))
    for i in range(n):
        v, m, c, q = PLAN.unpack_from(tables, n * LAYER.size + i * PLAN.size)
        choices.append(None if v < 0 else (v, m, c))
        queue_of.append(q)
    return dict(layers=layers, choices=choices, queue_of=queue_of, n_little=n_little,
                raw=bytes(data[raw_off:raw_off + w_bytes]), cached=bytes(data[cached_off:cached_off + c_bytes]))
