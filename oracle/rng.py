"""Counter-based random numbers for sampled decoding. TEST INFRASTRUCTURE ONLY.

Philox-4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as
1, 2, 3", SC 2011), written from the published definition: a 128-bit counter and a 64-bit key
go through ten rounds of two 32x32 -> 64-bit multiplications and xors, the key being bumped
by the Weyl constants between rounds. Pinned to the published known-answer vectors
(tests/golden/philox4x32_10_kat.txt).

The decode loop draws one uniform per (sequence, step): counter = (step, sequence, 0, 0),
key = the 64-bit seed; the uniform is the top 24 bits of the first output word times 2^-24,
which float32 and float64 both hold exactly.
"""

PHILOX_M0, PHILOX_M1 = 0xD2511F53, 0xCD9E8D57
PHILOX_W0, PHILOX_W1 = 0x9E3779B9, 0xBB67AE85
_MASK = 0xFFFFFFFF


def philox4x32_10(counter, key):
    """counter: four 32-bit words, key: two 32-bit words -> four 32-bit words."""
    c = [int(x) & _MASK for x in counter]
    k = [int(x) & _MASK for x in key]
    for rnd in range(10):
        if rnd:
            k = [(k[0] + PHILOX_W0) & _MASK, (k[1] + PHILOX_W1) & _MASK]
        p0, p1 = PHILOX_M0 * c[0], PHILOX_M1 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & _MASK, (p0 >> 32) ^ c[3] ^ k[1], p0 & _MASK]
    return c


def step_uniform(seed: int, sequence: int, step: int) -> float:
    """The uniform in [0, 1) that decides the sampled token of `sequence` at `step` (step 0 is
    the token drawn after the prompt)."""
    key = (seed & _MASK, (seed >> 32) & _MASK)
    word = philox4x32_10((step, sequence, 0, 0), key)[0]
    return (word >> 8) * 2.0 ** -24
