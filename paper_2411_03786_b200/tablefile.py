"""Save and load a model bigram table (and its extension) so the one-off build can be reused.

File layout (little endian): 8-byte magic ``NGTAB001``, a 4-byte header length, a JSON header
(V, d, k_tab, w_ext, sha256 of the payload, free-form ``meta``), then ``tab[V, k_tab]`` int32 and,
if ``w_ext > 0``, ``ext[V, k_tab, w_ext]`` int32.
"""
from __future__ import annotations

import hashlib
import json
import struct

import numpy as np

MAGIC = b"NGTAB001"


def save_table(path: str, tab: np.ndarray, ext: np.ndarray | None = None, d: int = 0, meta: dict | None = None) -> None:
    tab = np.ascontiguousarray(tab, dtype="<i4")
    V, k_tab = tab.shape
    payload = tab.tobytes()
    w_ext = 0
    if ext is not None:
        ext = np.ascontiguousarray(ext, dtype="<i4")
        assert ext.shape[:2] == (V, k_tab)
        w_ext = int(ext.shape[2])
        payload += ext.tobytes()
    header = json.dumps({"V": int(V), "d": int(d), "k_tab": int(k_tab), "w_ext": w_ext,
                         "sha256": hashlib.sha256(payload).hexdigest(), "meta": meta or {}}).encode()
    with open(path, "wb") as f:
        f.write(MAGIC + struct.pack("<I", len(header)) + header + payload)


def load_table(path: str):
    """Returns ``(tab, ext or None, header dict)``; raises ValueError on a damaged or foreign file."""
    with open(path, "rb") as f:
        blob = f.read()
    if blob[:8] != MAGIC:
        raise ValueError(f"{path}: not a model table file")
    (hlen,) = struct.unpack("<I", blob[8:12])
    header = json.loads(blob[12:12 + hlen])
    payload = blob[12 + hlen:]
    V, k, w = header["V"], header["k_tab"], header["w_ext"]
    if len(payload) != 4 * V * k * (1 + w) or hashlib.sha256(payload).hexdigest() != header["sha256"]:
        raise ValueError(f"{path}: payload does not match its header")
    tab = np.frombuffer(payload, dtype="<i4", count=V * k).reshape(V, k).astype(np.int32)
    ext = None
    if w:
        ext = np.frombuffer(payload, dtype="<i4", offset=4 * V * k).reshape(V, k, w).astype(np.int32)
    if tab.min() < 0 or tab.max() >= V:
        raise ValueError(f"{path}: token id out of range")
    return tab, ext, header
