"""Comparison helpers shared by the tests (no method arithmetic here)."""
import numpy as np


def bf16_ordinal(bits: np.ndarray) -> np.ndarray:
    """Map bf16 bit patterns to integers that are monotone in the value:
    sign-magnitude -> two's-complement-like ordering, with +0 and -0 both 0."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.int32)
    mag = b & 0x7FFF
    return np.where((b & 0x8000) != 0, -mag, mag)


def bf16_isnan(bits: np.ndarray) -> np.ndarray:
    b = np.asarray(bits, dtype=np.uint16)
    return ((b & 0x7F80) == 0x7F80) & ((b & 0x007F) != 0)


def ordinal_distance(a_bits: np.ndarray, b_bits: np.ndarray) -> np.ndarray:
    """|ordinal(a) - ordinal(b)| with NaN positions required to match (distance
    0 where both are NaN, a huge value where only one is)."""
    a = np.asarray(a_bits, dtype=np.uint16)
    b = np.asarray(b_bits, dtype=np.uint16)
    d = np.abs(bf16_ordinal(a) - bf16_ordinal(b))
    na, nb = bf16_isnan(a), bf16_isnan(b)
    d = np.where(na & nb, 0, d)
    d = np.where(na ^ nb, 1 << 20, d)
    return d


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widening through numpy (used to express expected values, not to compute the method)."""
    b = np.asarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def e4m3_ordinal(bits: np.ndarray) -> np.ndarray:
    """Monotone integer order of FP8-E4M3 bit patterns (+0 and -0 both 0)."""
    b = np.asarray(bits, dtype=np.uint8).astype(np.int32)
    mag = b & 0x7F
    return np.where((b & 0x80) != 0, -mag, mag)


def e4m3_isnan(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint8) & 0x7F) == 0x7F


def e4m3_ordinal_distance(a_bits: np.ndarray, b_bits: np.ndarray) -> np.ndarray:
    a = np.asarray(a_bits, dtype=np.uint8)
    b = np.asarray(b_bits, dtype=np.uint8)
    d = np.abs(e4m3_ordinal(a) - e4m3_ordinal(b))
    na, nb = e4m3_isnan(a), e4m3_isnan(b)
    d = np.where(na & nb, 0, d)
    d = np.where(na ^ nb, 1 << 20, d)
    return d
