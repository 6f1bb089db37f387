"""Writes tests/golden/rng_vectors.txt from the CPU checker alone (run by hand:
python tests/golden/make_golden.py).  The library's host generator must
reproduce every line."""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import rng  # noqa: E402

CASES = [(0, 0, 0, 0), (0, 0, 0, 1), (0, 1, 0, 0), (0, 2, 5, 29), (7, 1, 15, 9299),
         (2021, 0, 1023, 439), (2 ** 64 - 1, 2, 63, 2 ** 32), (42, 1, 3, 2 ** 50 + 1)]

with open(os.path.join(HERE, "rng_vectors.txt"), "w") as f:
    f.write("# seed stream client counter draw(hex) mean_ticks exp_ticks -- from oracle/rng.py\n")
    for seed, st, c, k in CASES:
        r = rng.draw(rng.stream_key(seed, st, c), k)
        mean = rng.to_ticks(1.0 if st != 2 else 0.5)
        f.write(f"{seed} {st} {c} {k} {r:016x} {mean} {rng.exp_ticks(r, mean)}\n")
