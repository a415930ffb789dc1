"""Dump and load of a quantised matrix: the MXFP4 pair of Sec. III-D-3 (packed E2M1 codes [N][K/2], E8M0 scale bytes
[N][K/32]) as one little-endian file, so that a model cast once need not be cast again at load time and so that
separate processes (the oracle, a test) can exchange the same bytes.

Layout: 32-byte header -- magic ``MXQ4PAIR`` (8 bytes), format version (u32), reserved (u32, zero), N (u64), K (u64) --
then N*K/2 code bytes, then N*K/32 scale bytes, both exactly as the library's canonical arrays.  No arithmetic here.
"""
from __future__ import annotations

import struct

import numpy as np

MAGIC = b"MXQ4PAIR"
VERSION = 1
_HEADER = struct.Struct("<8sIIQQ")


def save_mxfp4(path: str, codes, scales) -> None:
    """codes [N][K/2] uint8, scales [N][K/32] uint8 (numpy arrays or torch tensors, on any device)."""
    c = _as_numpy(codes)
    s = _as_numpy(scales)
    if c.ndim != 2 or s.ndim != 2 or c.dtype != np.uint8 or s.dtype != np.uint8:
        raise TypeError("codes and scales must be 2-D uint8 arrays")
    n, half_k = c.shape
    k = 2 * half_k
    if k % 32 != 0 or s.shape != (n, k // 32):
        raise ValueError("codes %s and scales %s are not the MXFP4 pair of one [N][K] matrix with K %% 32 == 0" % (c.shape, s.shape))
    with open(path, "wb") as f:
        f.write(_HEADER.pack(MAGIC, VERSION, 0, n, k))
        f.write(np.ascontiguousarray(c).tobytes())
        f.write(np.ascontiguousarray(s).tobytes())


def load_mxfp4(path: str, device=None):
    """Returns (codes, scales): numpy arrays, or torch tensors on ``device`` if one is given."""
    with open(path, "rb") as f:
        head = f.read(_HEADER.size)
        if len(head) != _HEADER.size:
            raise ValueError("%s: shorter than its header" % path)
        magic, version, reserved, n, k = _HEADER.unpack(head)
        if magic != MAGIC:
            raise ValueError("%s: not an MXFP4 pair file" % path)
        if version != VERSION or reserved != 0:
            raise ValueError("%s: format version %d is not supported" % (path, version))
        if n < 1 or k < 32 or k % 32 != 0:
            raise ValueError("%s: impossible shape %d x %d" % (path, n, k))
        body = f.read()
    want = n * (k // 2) + n * (k // 32)
    if len(body) != want:
        raise ValueError("%s: %d bytes after the header, %d expected for %d x %d" % (path, len(body), want, n, k))
    codes = np.frombuffer(body, np.uint8, n * (k // 2)).reshape(n, k // 2).copy()
    scales = np.frombuffer(body, np.uint8, n * (k // 32), offset=n * (k // 2)).reshape(n, k // 32).copy()
    if device is None:
        return codes, scales
    import torch
    return torch.from_numpy(codes).to(device), torch.from_numpy(scales).to(device)


def _as_numpy(a) -> np.ndarray:
    if isinstance(a, np.ndarray):
        return a
    return a.detach().cpu().numpy()
