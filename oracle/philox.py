"""Philox4x32-10 counter-based generator and the uniform convention of the
decode step (oracle side; test infrastructure only).

The acceptance rule draws r ~ U[0,1] per verified position (Algorithm "S2D2
SampleBlock", the accept test) and one more uniform for the residual resample.
Reading used here: counter = (absolute position, sequence stream id, step index,
stream), key = (seed, 0); stream 0 = accept test, 1 = residual resample,
2 = draft sampling.  u = ((x0 >> 8) + 0.5) * 2^-24, which lies strictly inside
(0, 1) and is exact in fp32 and fp64.
"""
from __future__ import annotations

M0 = 0xD2511F53
M1 = 0xCD9E8D57
W0 = 0x9E3779B9
W1 = 0xBB67AE85
MASK32 = 0xFFFFFFFF

STREAM_ACCEPT = 0
STREAM_RESAMPLE = 1
STREAM_DRAFT = 2


def philox4x32_10(counter, key):
    """Ten rounds of Philox-4x32 (Salmon et al., 2011). Python ints in, 4 ints out."""
    c0, c1, c2, c3 = (int(c) & MASK32 for c in counter)
    k0, k1 = (int(k) & MASK32 for k in key)
    for r in range(10):
        p0 = M0 * c0
        p1 = M1 * c2
        hi0, lo0 = p0 >> 32, p0 & MASK32
        hi1, lo1 = p1 >> 32, p1 & MASK32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & MASK32, lo1, (hi0 ^ c3 ^ k1) & MASK32, lo0
        k0 = (k0 + W0) & MASK32
        k1 = (k1 + W1) & MASK32
    return c0, c1, c2, c3


def uniform(seed: int, position: int, seq_stream: int, step: int, stream: int) -> float:
    x0 = philox4x32_10((position, seq_stream, step, stream), (seed, 0))[0]
    return ((x0 >> 8) + 0.5) * (2.0 ** -24)
