"""bfloat16 <-> float32 conversions used to prepare inputs (round to nearest even)."""
import numpy as np


def f32_to_bf16_bits(a):
    """uint16 bit patterns of `a` rounded to bfloat16 (RNE); finite inputs only."""
    b = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    r = b + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits):
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_bf16(a):
    """float32 array whose values are exactly representable in bfloat16."""
    a = np.asarray(a)
    return bf16_bits_to_f32(f32_to_bf16_bits(a)).reshape(a.shape)
