"""CPU-only: the library's model file against the oracle's byte-by-byte definition, both ways."""
import os

import numpy as np
import pytest

import workloads as wl
from oracle import cachefile as ocf
from paper_2206_07446_b200 import binding as nb


def _setup(layers, seed=0):
    ws, bs = wl.make_weights(layers, seed=seed)
    blob, w_off, b_off = wl.weight_blob(layers, ws, bs)
    plan = nb.Plan(layers, w_off, b_off)
    descs = [dict(L, w_off=w_off[i], b_off=b_off[i]) for i, L in enumerate(layers)]
    return plan, descs, np.ascontiguousarray(blob)


def _choices(plan, layers, cached):
    out = []
    for i, L in enumerate(layers):
        if L["op"] != wl.OP_CONV:
            out.append(None)
            continue
        el = nb.nnv_eligible(plan, i)
        v = nb.VAR_DEPTHWISE if nb.VAR_DEPTHWISE in el else (nb.VAR_WINO_F2 if nb.VAR_WINO_F2 in el else nb.VAR_IM2COL)
        m = nb.MATH_FP32 if v == nb.VAR_DEPTHWISE else nb.MATH_TF32
        out.append((v, m, 1 if (cached and v != nb.VAR_DEPTHWISE) else 0))
    return out


@pytest.mark.parametrize("cached", [0, 1])
def test_written_file_is_the_oracles_bytes(tmp_path, cached):
    layers = wl.tiny_net()
    plan, descs, blob = _setup(layers, seed=1)
    choices = _choices(plan, layers, cached)
    offs, ctotal = nb.nnv_cached_layout(plan, choices)
    rng = np.random.default_rng(5)
    cblob = rng.integers(0, 256, max(ctotal, 1), dtype=np.uint8) if cached else None
    queues = [(i % 3) if c is not None else 0 for i, c in enumerate(choices)]
    path = str(tmp_path / "model.nnv")
    nb.nnv_cache_write(path, plan, choices, queues, 2, blob, blob.size, cblob, ctotal if cached else 0)
    data = open(path, "rb").read()
    want = ocf.encode(descs, choices, queues, 2, blob.tobytes(), cblob.tobytes()[:ctotal] if cached else b"")
    assert data == want
    got = ocf.decode(data)
    assert got["choices"] == choices and got["raw"] == blob.tobytes() and got["n_little"] == 2

    cf = nb.CacheFile(path)
    assert (cf.n_layers, cf.w_bytes, cf.c_bytes, cf.n_little, cf.file_bytes) == \
        (len(layers), blob.size, ctotal if cached else 0, 2, len(data))
    ls, cs, qs = cf.read_plan()
    assert ls == descs and cs == choices
    assert qs == [q if c is not None else -1 for q, c in zip(queues, choices)]
    w = np.zeros(cf.w_bytes, np.uint8)
    c = np.zeros(max(cf.c_bytes, 1), np.uint8)
    cf.read_blobs(w, c if cached else None)
    assert np.array_equal(w, blob)
    if cached:
        assert np.array_equal(c[:ctotal], cblob[:ctotal])
    cf.drop_pages()
    cf.close()


def test_library_reads_a_file_the_oracle_wrote(tmp_path):
    layers = wl.cfg1()
    plan, descs, blob = _setup(layers)
    path = str(tmp_path / "o.nnv")
    open(path, "wb").write(ocf.encode(descs, [(nb.VAR_IM2COL, nb.MATH_TF32, 0)], None, 0, blob.tobytes(), b""))
    cf = nb.CacheFile(path)
    ls, cs, qs = cf.read_plan()
    assert ls == descs and cs == [(nb.VAR_IM2COL, nb.MATH_TF32, 0)] and qs == [-1] and cf.n_little == 0
    w = np.zeros(cf.w_bytes, np.uint8)
    cf.read_blobs(w)
    assert np.array_equal(w, blob)


def test_damaged_files_are_refused(tmp_path):
    layers = wl.cfg1()
    plan, descs, blob = _setup(layers)
    good = ocf.encode(descs, [(nb.VAR_IM2COL, nb.MATH_TF32, 0)], None, 0, blob.tobytes(), b"")
    for name, data in [("magic", b"X" + good[1:]), ("version", good[:8] + b"\x02" + good[9:]),
                       ("table", good[:70] + bytes([good[70] ^ 1]) + good[71:]), ("short", good[:-4096]),
                       ("tiny", good[:20])]:
        path = str(tmp_path / (name + ".nnv"))
        open(path, "wb").write(data)
        with pytest.raises(nb.NnvError) as e:
            nb.CacheFile(path)
        assert e.value.status == 1, name                          # NNV_ERR_INVALID_ARG
    with pytest.raises(nb.NnvError) as e:
        nb.CacheFile(str(tmp_path / "missing.nnv"))
    assert e.value.status == 3                                    # NNV_ERR_STATE
    with pytest.raises(nb.NnvError):                              # a choice the layer cannot run
        nb.nnv_cache_write(str(tmp_path / "bad.nnv"), plan, [(nb.VAR_DEPTHWISE, 0, 0)], None, 0, blob, blob.size, None, 0)


def test_cold_run_refuses_a_file_written_for_another_model(tmp_path):
    """Same layer count, fitting offsets, different shapes: nnv_cold_run_file must refuse before any device work
    (the pointers below are never dereferenced: the comparison of the descriptors comes first)."""
    layers = wl.tiny_net()
    plan, descs, blob = _setup(layers, seed=1)
    choices = _choices(plan, layers, 0)
    path = str(tmp_path / "a.nnv")
    nb.nnv_cache_write(path, plan, choices, None, 0, blob, blob.size, None, 0)
    other = [dict(L) for L in layers]
    conv = next(i for i, L in enumerate(other) if L["op"] == wl.OP_CONV)
    other[conv]["act"] = (other[conv]["act"] + 1) % 3          # the same byte layout, another network
    plan2, _, _ = _setup(other, seed=1)
    cache = nb.CacheFile(path)
    stage = np.zeros(blob.size, np.uint8)
    io = np.zeros(1 << 16, np.float32)
    with pytest.raises(nb.NnvError) as e:
        nb.nnv_cold_run_file(plan2, choices, cache, stage, stage.size, None, 0, io, io, 256, 1 << 30, 1, 2, 3, 1)
    assert e.value.status == 1 and "differs from the plan" in str(e.value)
    cache.close()
