"""A second, independent decoder of the canonical block format (numpy only).

It exists to cross-check the C oracle: it reads the bytes with numpy views,
decodes to float64 and multiplies with ``@``.  It shares no code with the
oracle or with the CUDA library.
"""
import numpy as np


BB = {4: 18, 5: 22, 6: 26, 8: 34}


def _codes(fmt, b):
    """b: uint8 [blocks, block bytes] -> int64 codes [blocks, 32]."""
    if fmt == 8:
        return b[:, 2:].copy().view(np.int8).astype(np.int64)
    nib = b[:, -16:]
    q = np.empty((b.shape[0], 32), dtype=np.int64)
    q[:, 0::2] = nib & 0x0F
    q[:, 1::2] = nib >> 4
    if fmt == 5:
        bits = np.unpackbits(b[:, 2:6], axis=1, bitorder="little")          # bit i of the 32-bit word
        q += bits.astype(np.int64) << 4
    elif fmt == 6:
        hb = b[:, 2:10].astype(np.int64)                                     # byte i // 4, field i % 4
        q += np.stack([(hb >> (2 * f)) & 3 for f in range(4)], axis=2).reshape(-1, 32) << 4
    return q - {4: 8, 5: 16, 6: 32}[fmt]


def decode(fmt, blocks, N, K):
    nb = K // 32
    b = np.asarray(blocks, dtype=np.uint8).reshape(N * nb, BB[fmt])
    d = b[:, :2].copy().view("<u2").view(np.float16).astype(np.float64)  # [N*nb, 1]
    return (d * _codes(fmt, b)).reshape(N, K)


def codes(fmt, blocks, N, K):
    nb = K // 32
    b = np.asarray(blocks, dtype=np.uint8).reshape(N * nb, BB[fmt])
    return _codes(fmt, b).reshape(N, K)


def scales_bits(fmt, blocks, N, K):
    nb = K // 32
    bb = BB[fmt]
    b = np.asarray(blocks, dtype=np.uint8).reshape(N * nb, bb)
    return b[:, :2].copy().view("<u2").reshape(N, nb)
