"""Counter-based integer generator and the integer-only delay draws.

TEST INFRASTRUCTURE (see the package header).  Everything here is exact
Python-integer arithmetic, so results are bit-reproducible.

The paper fixes no generator: it samples "uniformly at random xi from D_c"
(Algorithm 3) and injects random compute / network delays (Section 3.3.2,
Section 5 "System delay").  The convention used here:

* mixing function = the SplitMix64 output function (Steele, Lea, Flood 2014);
* a stream key is derived from (seed, stream id, client), a draw from
  (key, counter); the golden-ratio increment separates the inputs;
* a sample index takes the high 32 bits of a draw, times N, shifted by 32;
* an Exp(mean) delay is floor(-ln(u) * mean_ticks) with -ln(u) from an
  integer log2 (leading bit + 32 fraction bits by repeated squaring) times
  a fixed-point ln 2; at least one tick;
* a Uniform[lo, hi] delay is lo + floor(u32 * (hi - lo + 1) / 2^32).
"""

MASK64 = (1 << 64) - 1
GAMMA = 0x9E3779B97F4A7C15
STREAM_SAMPLE, STREAM_COMPUTE, STREAM_NETWORK, STREAM_SETUP = 0, 1, 2, 3
TICKS_PER_UNIT = 1 << 20
LN2_Q32 = 2977044471  # floor(ln(2) * 2^32)


def mix64(z: int) -> int:
    z &= MASK64
    z ^= z >> 30
    z = (z * 0xBF58476D1CE4E5B9) & MASK64
    z ^= z >> 27
    z = (z * 0x94D049BB133111EB) & MASK64
    z ^= z >> 31
    return z


def stream_key(seed: int, stream: int, client: int) -> int:
    k = mix64((seed + GAMMA * (stream + 1)) & MASK64)
    return mix64((k + GAMMA * (client + 1)) & MASK64)


def draw(key: int, counter: int) -> int:
    return mix64((key + GAMMA * (counter + 1)) & MASK64)


def sample_index(r: int, n: int) -> int:
    """Uniform index in [0, n) from a 64-bit draw (n < 2^32)."""
    return ((r >> 32) * n) >> 32


def neg_log2_q32(r: int) -> int:
    """-log2(x / 2^64) in Q32 fixed point, x = r (1 if r == 0); result >= 1."""
    x = r if r != 0 else 1
    e = x.bit_length() - 1
    m = x << (63 - e)                 # Q1.63, in [1, 2)
    f = 0
    for _ in range(32):
        p = m * m                     # Q2.126, in [1, 4)
        if p >> 127:
            f = (f << 1) | 1
            m = p >> 64
        else:
            f = f << 1
            m = p >> 63
    return ((64 - e) << 32) - f


def exp_ticks(r: int, mean_ticks: int) -> int:
    t = (neg_log2_q32(r) * LN2_Q32 * mean_ticks) >> 64
    return t if t >= 1 else 1


def uniform_ticks(r: int, lo_ticks: int, hi_ticks: int) -> int:
    t = lo_ticks + (((r >> 32) * (hi_ticks - lo_ticks + 1)) >> 32)
    return t if t >= 1 else 1


def to_ticks(units: float) -> int:
    """Time units -> integer ticks, rounding half up."""
    import math
    return int(math.floor(units * TICKS_PER_UNIT + 0.5))


def to_q16(factor: float) -> int:
    import math
    return int(math.floor(factor * 65536.0 + 0.5))
