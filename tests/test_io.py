"""Dump / load of an MXFP4 pair (io.py): the bytes come back as they went in, and a damaged file is refused."""
import os
import struct

import numpy as np
import pytest
import torch

import oracle
from paper_2503_13565_b200 import io as mxio
from paper_2503_13565_b200 import synth


def test_round_trip_of_a_cast_matrix(tmp_path):
    w = synth.bits_of(synth.weight(3, 1, 203, 1440))
    codes, scales, _ = oracle.quantize(w)
    path = str(tmp_path / "w.mxq")
    mxio.save_mxfp4(path, codes, scales)
    assert os.path.getsize(path) == 32 + codes.size + scales.size
    c2, s2 = mxio.load_mxfp4(path)
    assert c2.dtype == np.uint8 and np.array_equal(c2, codes) and np.array_equal(s2, scales)
    # torch tensors in, torch tensors out
    mxio.save_mxfp4(path, torch.from_numpy(codes), torch.from_numpy(scales))
    c3, s3 = mxio.load_mxfp4(path, device="cpu")
    assert torch.equal(c3, torch.from_numpy(codes)) and torch.equal(s3, torch.from_numpy(scales))
    # the header is what the module says: magic, version 1, reserved 0, N, K
    with open(path, "rb") as f:
        assert struct.unpack("<8sIIQQ", f.read(32)) == (b"MXQ4PAIR", 1, 0, 203, 1440)


def test_arrays_that_are_not_a_pair_are_refused(tmp_path):
    path = str(tmp_path / "x.mxq")
    with pytest.raises(ValueError):
        mxio.save_mxfp4(path, np.zeros((4, 16), np.uint8), np.zeros((4, 2), np.uint8))    # K = 32: one scale byte per row
    with pytest.raises(ValueError):
        mxio.save_mxfp4(path, np.zeros((4, 24), np.uint8), np.zeros((4, 1), np.uint8))    # K = 48
    with pytest.raises(TypeError):
        mxio.save_mxfp4(path, np.zeros((4, 16), np.int8), np.zeros((4, 1), np.uint8))


def test_damaged_files_are_refused(tmp_path):
    path = str(tmp_path / "w.mxq")
    codes, scales = np.arange(4 * 32, dtype=np.uint8).reshape(4, 32), np.full((4, 2), 127, np.uint8)
    mxio.save_mxfp4(path, codes, scales)
    raw = open(path, "rb").read()
    for damaged in (raw[:20], raw[:-1], raw + b"\0", b"MXQ4PAIX" + raw[8:], raw[:8] + struct.pack("<I", 2) + raw[12:],
                    raw[:16] + struct.pack("<QQ", 4, 48) + raw[32:]):
        with open(path, "wb") as f:
            f.write(damaged)
        with pytest.raises(ValueError):
            mxio.load_mxfp4(path)
