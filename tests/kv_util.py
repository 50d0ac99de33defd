"""Byte layout of the blocked KV cache (include/resq_kv.h), for the tests: placing records that the oracle
quantized into a cache image and reading records back out of one.  Layout only -- no arithmetic of the method."""
import numpy as np

BLOCK, BLOCK_BYTES = 32, 5632
OFF = {"k": (0, 512, 2304), "v": (2816, 3328, 5120)}  # 8-bit codes, packed 4-bit codes, (s8, z8, s4, z4)


def empty_image(n_seqs, n_kv_heads, capacity, fill=0):
    return np.full((n_seqs, n_kv_heads, capacity // BLOCK, BLOCK_BYTES), fill, np.uint8)


def put(image, which, b, h, pos, c8, c4, meta):
    """Writes one record (c8 uint8 [16], c4 uint8 [56], meta fp32 [4]) at (sequence b, head h, position pos)."""
    o8, o4, om = OFF[which]
    blk, p = image[b, h, pos // BLOCK], pos % BLOCK
    blk[o8 + 16 * p: o8 + 16 * p + 16] = c8
    blk[o4 + 56 * p: o4 + 56 * p + 56] = c4
    blk[om + 16 * p: om + 16 * p + 16] = np.asarray(meta, np.float32).view(np.uint8)


def get(image, which, b, h, pos):
    o8, o4, om = OFF[which]
    blk, p = image[b, h, pos // BLOCK], pos % BLOCK
    return (blk[o8 + 16 * p: o8 + 16 * p + 16].copy(), blk[o4 + 56 * p: o4 + 56 * p + 56].copy(),
            blk[om + 16 * p: om + 16 * p + 16].copy().view(np.float32))
