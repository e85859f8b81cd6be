"""Host-side save / load of the compact index (no GPU): the library writes and reads back arrays produced by the
oracle's encoder, so the round trip also shows that the library's structural check accepts the oracle's reading of the
format; damaged and inconsistent files are refused."""
import os

import numpy as np
import pytest
import torch

import oracle as O
import paper_2601_17702_b200 as S


def _host_layer(c):
    return S.CompactLayer(torch.from_numpy(c["row_ptr"].astype(np.int64)), torch.from_numpy(c["blk_ptr"].astype(np.int32)),
                          torch.from_numpy(c["blk_first"].astype(np.int32)), torch.from_numpy(c["blk_desc"].astype(np.int64)),
                          torch.from_numpy(c["payload"].astype(np.int32)))


def _layers(seed, D=50, n_layers=3):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n_layers):
        lists = [np.sort(rng.choice(5000, size=int(rng.choice([0, 1, 5, 32, 33, 90])), replace=False)) for _ in range(D)]
        rp = np.cumsum([0] + [len(l) for l in lists]).astype(np.uint64)
        out.append(_host_layer(O.compact_encode(rp, np.concatenate(lists).astype(np.int32))))
    return out


def test_round_trip(tmp_path):
    layers = _layers(1)
    path = str(tmp_path / "index.s3c")
    S.s3_compact_save(path, layers, 50)
    n_layers, d_sae, nb, nw = S.s3_compact_file_info(path)
    assert (n_layers, d_sae) == (3, 50)
    assert nb == [c.blk_first.numel() for c in layers] and nw == [c.payload.numel() for c in layers]
    back, d = S.s3_compact_load(path)
    assert d == 50
    for a, b in zip(layers, back):
        for name in S.COMPACT_FIELDS:
            assert torch.equal(getattr(a, name), getattr(b, name)), name


def test_empty_index_round_trip(tmp_path):
    c = O.compact_encode(np.zeros(9, np.uint64), np.zeros(0, np.int32))
    path = str(tmp_path / "empty.s3c")
    S.s3_compact_save(path, [_host_layer(c)], 8)
    back, _ = S.s3_compact_load(path)
    assert back[0].blk_first.numel() == 0 and back[0].payload.tolist() == [0]


def test_damaged_files_are_refused(tmp_path):
    layers = _layers(2, n_layers=1)
    path = str(tmp_path / "index.s3c")
    S.s3_compact_save(path, layers, 50)
    raw = bytearray(open(path, "rb").read())
    flipped = bytearray(raw)
    flipped[len(raw) - 40] ^= 0x10                      # one bit inside the payload
    bad = str(tmp_path / "flipped.s3c")
    open(bad, "wb").write(flipped)
    with pytest.raises(S.S3Error, match="checksum"):
        S.s3_compact_load(bad)
    open(bad, "wb").write(raw[: len(raw) // 2])         # cut short
    with pytest.raises(S.S3Error):
        S.s3_compact_load(bad)
    open(bad, "wb").write(b"not an index" + bytes(100))
    with pytest.raises(S.S3Error, match="not a compact index"):
        S.s3_compact_file_info(bad)
    with pytest.raises(S.S3Error):
        S.s3_compact_file_info(str(tmp_path / "missing.s3c"))


def test_inconsistent_arrays_are_refused_on_save(tmp_path):
    path = str(tmp_path / "x.s3c")
    good = _layers(3, n_layers=1)[0]

    def variant(**kw):
        f = {n: getattr(good, n).clone() for n in S.COMPACT_FIELDS}
        for n, fn in kw.items():
            fn(f[n])
        return S.CompactLayer(*[f[n] for n in S.COMPACT_FIELDS])

    def bump(i, v):
        def fn(t):
            t[i] += v
        return fn

    cases = [variant(payload=bump(-1, 1)),                 # closing word not zero
             variant(blk_desc=bump(-1, 1 << 20)),          # payload offset far outside
             variant(blk_desc=bump(0, 40)),                # width beyond 31
             variant(blk_ptr=bump(-1, 1)),                 # block count disagrees with the list lengths
             variant(row_ptr=bump(3, 10**6))]              # row_ptr not monotone afterwards / block counts off
    for c in cases:
        with pytest.raises(S.S3Error):
            S.s3_compact_save(path, [c], 50)
    assert not os.path.exists(path)
