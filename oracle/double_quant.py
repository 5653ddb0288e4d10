"""Double quantisation of the block constants (Limitations; App. F): the plain definition.

TEST INFRASTRUCTURE ONLY, like the rest of this package.

The paper names the technique (quantising the block constants themselves, after Dettmers et al.)
and states the one thing that signed normalisation changes: one extra bit per block for the
sign, so that the second quantiser only sees magnitudes.  It does not use the technique and
fixes no format.  The reading implemented here, in fp32 throughout:

    a_b      = |m_b|                                   magnitude of block b's constant
    s_b      = 1 if m_b < 0 else 0                     sign bit (bit b mod 8 of byte b div 8)
    g_k      = max over the 256 constants of group k of a_b   (the last group may be shorter)
    t_k      = g_k / 255                                (fp32 division)
    q_b      = min(255, round-half-even(a_b / t_k))     (fp32 division; 0 when t_k = 0)
    m^_b     = (-1)^{s_b} * (t_k * q_b)                 (fp32 product)

i.e. 8-bit uniform quantisation of the magnitudes against the group's maximum.  The weights'
codes are not touched: they were formed with the exact m_b, only the decoder's constant changes.

Parity pins (tests/test_oracle_pins.py): a hand-made group with exact arithmetic, the error
bound |m^ - m| <= g/510 (+ rounding), exact signs, group boundaries, zero groups, and agreement
with the fp64 formula round(255 a / g) up to ties.
"""
from __future__ import annotations

import numpy as np

GROUP = 256


def compress(m, signed: bool):
    """m: fp32 block constants -> (q uint8[B], g float32[ceil(B/256)], sign uint8[ceil(B/8)] or None)."""
    m = np.ascontiguousarray(m, np.float32).reshape(-1)
    B = m.size
    a = np.abs(m)
    G = (B + GROUP - 1) // GROUP
    g = np.zeros(G, np.float32)
    q = np.zeros(B, np.uint8)
    for k in range(G):
        blk = a[k * GROUP:(k + 1) * GROUP]
        g[k] = blk.max()
        t = np.float32(g[k]) / np.float32(255.0)
        if t == 0:
            continue
        r = np.rint((blk / t).astype(np.float32))            # numpy's rint rounds halves to even
        q[k * GROUP:(k + 1) * GROUP] = np.minimum(r, 255).astype(np.uint8)
    sign = None
    if signed:
        bits = (m < 0).astype(np.uint8)
        bits = np.concatenate([bits, np.zeros(-B % 8, np.uint8)])
        sign = (bits.reshape(-1, 8) << np.arange(8, dtype=np.uint8)).sum(1).astype(np.uint8)
    return q, g, sign


def expand(q, g, sign, n_blocks: int):
    """-> fp32 reconstructed block constants m^."""
    q = np.asarray(q, np.uint8)[:n_blocks]
    t = (np.asarray(g, np.float32) / np.float32(255.0)).astype(np.float32)
    out = (np.repeat(t, GROUP)[:n_blocks] * q.astype(np.float32)).astype(np.float32)
    if sign is not None:
        bits = (np.repeat(np.asarray(sign, np.uint8), 8)[:n_blocks] >> (np.arange(n_blocks) % 8).astype(np.uint8)) & 1
        out = np.where(bits == 1, -out, out).astype(np.float32)
    return out
