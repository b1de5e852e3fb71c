"""Seeded synthetic inputs shared by the tests and the benchmark.

Only input generation lives here (lists of p, lists of ranks); none of the schedule
arithmetic.  The generator is splitmix64 (Steele, Lea, Flood, "Fast splittable pseudorandom
number generators", OOPSLA 2014): state += 0x9E3779B97F4A7C15, then two xor-shift-multiply
steps and a final xor-shift.
"""
from __future__ import annotations

_M64 = (1 << 64) - 1

P_SINGLE = 2**20 + 1          # the non-power-of-two single-p workload (q = 21)
P_EXPAND = 100003             # round-table expansion workload (q = 17)
N_EXPAND = 1000
P_LARGE = 2**30 - 1           # chunked large-p workload (q = 30)
LARGE_CHUNKS = 8
SEED_BATCH = 220510072
SEED_SPOT = 220510073


class SplitMix64:
    def __init__(self, seed: int):
        self.state = seed & _M64

    def next(self) -> int:
        self.state = (self.state + 0x9E3779B97F4A7C15) & _M64
        z = self.state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
        return z ^ (z >> 31)


def small_sweep() -> list[int]:
    """Every p in 2..1024 (the exhaustive small sweep)."""
    return list(range(2, 1025))


def batch_p_list(count: int = 4096, seed: int = SEED_BATCH, lo_exp: int = 10, hi_exp: int = 20) -> list[int]:
    """`count` values of p, octave-uniform in [2^lo_exp, 2^hi_exp): per draw an exponent
    e = lo_exp + next() % (hi_exp - lo_exp), then p = 2^e + next() % 2^e.  Duplicates allowed.
    (Integer reading of "log-uniform in [2^10, 2^20]".)"""
    g = SplitMix64(seed)
    out = []
    for _ in range(count):
        e = lo_exp + g.next() % (hi_exp - lo_exp)
        out.append((1 << e) + g.next() % (1 << e))
    return out


def spot_ranks(p: int, count: int, seed: int = SEED_SPOT) -> list[int]:
    """`count` ranks r = next() % p for spot checks at very large p."""
    g = SplitMix64(seed)
    return [g.next() % p for _ in range(count)]


def large_chunks(p: int = P_LARGE, chunks: int = LARGE_CHUNKS) -> list[tuple[int, int]]:
    """Rank ranges [c*2^27, min((c+1)*2^27, p)) for the chunked large-p workload."""
    step = 1 << 27
    return [(c * step, min((c + 1) * step, p)) for c in range(chunks) if c * step < p]
