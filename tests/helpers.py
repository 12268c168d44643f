"""Test helpers: the scale-factor atom layout written out from its definition in
include/fp4root.h, and host<->device shuttles.  No arithmetic of the method lives here."""
import numpy as np


def sf_offsets(rows: int, kblocks: int) -> np.ndarray:
    """Byte offset of the scale of (row r, block kb) in the 128-row x 4-block atom layout."""
    r = np.arange(rows, dtype=np.int64)[:, None]
    kb = np.arange(kblocks, dtype=np.int64)[None, :]
    return ((r // 128) * (kblocks // 4) + kb // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + kb % 4


def sf_to_atoms(plain: np.ndarray) -> np.ndarray:
    rows, kblocks = plain.shape
    out = np.zeros(rows * kblocks, np.uint8)
    out[sf_offsets(rows, kblocks).ravel()] = plain.ravel()
    return out


def sf_from_atoms(atoms: np.ndarray, rows: int, kblocks: int) -> np.ndarray:
    return np.asarray(atoms).ravel()[sf_offsets(rows, kblocks)]


def mismatch_report(a: np.ndarray, b: np.ndarray) -> str:
    bad = np.argwhere(a != b)
    return f"{len(bad)} of {a.size} differ; first at {bad[:5].tolist()}"


def nibbles(codes: np.ndarray) -> np.ndarray:
    rows, half = codes.shape
    return np.stack([codes & 0xF, codes >> 4], -1).reshape(rows, half * 2)
