"""Test-side helpers: an independent bit packer/unpacker built on numpy.packbits (the layout the C ABI
states: element k -> word k // 32, bit k % 32, bit 1 <-> +1), used to compare packed GPU outputs with
the oracle's unpacked +-1 values.  Not used by the library or by the oracle."""
import numpy as np


def np_pack_pm1(x: np.ndarray, ld_w: int | None = None) -> np.ndarray:
    """Pack the last axis of a +-1 (or real) array: bit = (x >= 0).  Returns uint32 [..., ld_w]."""
    bits = (np.asarray(x) >= 0).astype(np.uint8)
    k = bits.shape[-1]
    kw = (k + 31) // 32
    ld = kw if ld_w is None else ld_w
    pad = ld * 32 - k
    bits = np.concatenate([bits, np.zeros(bits.shape[:-1] + (pad,), np.uint8)], axis=-1)
    by = np.packbits(bits, axis=-1, bitorder="little")
    return np.ascontiguousarray(by).view(np.uint32).reshape(bits.shape[:-1] + (ld,))


def np_unpack_pm1(words: np.ndarray, k: int) -> np.ndarray:
    """Inverse of np_pack_pm1 on the first k bits of the last axis: returns int8 +-1."""
    w = np.ascontiguousarray(words).view(np.uint32)
    by = w.view(np.uint8).reshape(w.shape[:-1] + (w.shape[-1] * 4,))
    bits = np.unpackbits(by, axis=-1, bitorder="little")[..., :k]
    return (2 * bits.astype(np.int8) - 1).astype(np.int8)


def padding_is_zero(words: np.ndarray, k: int) -> bool:
    w = np.ascontiguousarray(words).view(np.uint32)
    by = w.view(np.uint8).reshape(w.shape[:-1] + (w.shape[-1] * 4,))
    bits = np.unpackbits(by, axis=-1, bitorder="little")
    return not bits[..., k:].any()
