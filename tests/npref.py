"""A second, independent decoder of the canonical block format (numpy only).

It exists to cross-check the C oracle: it reads the bytes with numpy views,
decodes to float64 and multiplies with ``@``.  It shares no code with the
oracle or with the CUDA library.
"""
import numpy as np


def decode(fmt, blocks, N, K):
    nb = K // 32
    bb = 18 if fmt == 4 else 34
    b = np.asarray(blocks, dtype=np.uint8).reshape(N * nb, bb)
    d = b[:, :2].copy().view("<u2").view(np.float16).astype(np.float64)  # [N*nb, 1]
    if fmt == 4:
        lo = (b[:, 2:] & 0x0F).astype(np.int64)
        hi = (b[:, 2:] >> 4).astype(np.int64)
        q = np.empty((N * nb, 32), dtype=np.int64)
        q[:, 0::2] = lo
        q[:, 1::2] = hi
        q -= 8
    else:
        q = b[:, 2:].copy().view(np.int8).astype(np.int64)
    return (d * q).reshape(N, K)


def codes(fmt, blocks, N, K):
    nb = K // 32
    bb = 18 if fmt == 4 else 34
    b = np.asarray(blocks, dtype=np.uint8).reshape(N * nb, bb)
    if fmt == 4:
        q = np.empty((N * nb, 32), dtype=np.int64)
        q[:, 0::2] = b[:, 2:] & 0x0F
        q[:, 1::2] = b[:, 2:] >> 4
        q -= 8
    else:
        q = b[:, 2:].copy().view(np.int8).astype(np.int64)
    return q.reshape(N, K)


def scales_bits(fmt, blocks, N, K):
    nb = K // 32
    bb = 18 if fmt == 4 else 34
    b = np.asarray(blocks, dtype=np.uint8).reshape(N * nb, bb)
    return b[:, :2].copy().view("<u2").reshape(N, nb)
