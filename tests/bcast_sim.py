"""Brute-force simulation of the n-block broadcast in the 1-ported, bidirectional model.

Independent of the oracle and of the CUDA library: it is handed the expanded round tables
(one (send block, receive block, to, from) record per processor and round, Algorithm 6) and
checks the conditions the paper states for a correct, round-optimal broadcast:

  a) a processor only sends a block it already holds (Section 2, conditions a/b),
  b) every non-root processor receives every block exactly once,
  c) what r sends in a round is what its to-processor receives in that round, and the to/from
     processors are the circulant neighbours r +- skips[k], k = (j + x) mod q,
  d) all processors are complete after exactly n-1+q rounds and not one round earlier.

The skips are recomputed here from the closed form skips[k] = ceil(p / 2^(q-k)) (nested
ceil-halving composes), not taken from the code under test.
"""
import numpy as np


def ceil_log2(p):
    q = 0
    while (1 << q) < p:
        q += 1
    return q


def closed_form_skips(p):
    q = ceil_log2(p)
    return [-((-p) >> (q - k)) for k in range(q + 1)]


def reroot(table, root):
    """Round table for broadcasting from `root`: processor r plays virtual rank (r-root) mod p and
    its neighbours are shifted back by +root (Section 2: renumber by subtracting the root)."""
    p = table.shape[0]
    virt = (np.arange(p) - root) % p
    t = table[virt].copy()
    t[:, :, 2] = (t[:, :, 2] + root) % p
    t[:, :, 3] = (t[:, :, 3] + root) % p
    return t


def simulate(p, n, table, root=0):
    """Return None if `table` (int32 [p][n-1+q][4]) is a correct round-optimal broadcast of n
    blocks from `root`, else a string describing the first violation."""
    q = ceil_log2(p)
    rounds = n - 1 + q
    if table.shape != (p, rounds, 4):
        return "table shape %r != %r" % (table.shape, (p, rounds, 4))
    if p == 1:
        return None
    sk = closed_form_skips(p)
    x = (q - (n - 1 + q) % q) % q
    ranks = np.arange(p)
    have = np.zeros((p, n), dtype=bool)
    have[root, :] = True
    got = np.zeros((p, n), dtype=np.int64)
    for j in range(rounds):
        k = (j + x) % q
        sb, rb, to, fr = (table[:, j, c].astype(np.int64) for c in range(4))
        if not np.array_equal(to, (ranks + sk[k]) % p):
            return "round %d: to-processor is not r+skips[%d]" % (j, k)
        if not np.array_equal(fr, (ranks - sk[k]) % p):
            return "round %d: from-processor is not r-skips[%d]" % (j, k)
        if (sb >= n).any() or (rb >= n).any() or (sb < -1).any() or (rb < -1).any():
            return "round %d: block out of range" % j
        if not np.array_equal(rb[to], sb):
            return "round %d: send of r differs from receive of its to-processor" % j
        snd = sb >= 0
        if not have[ranks[snd], sb[snd]].all():
            bad = ranks[snd][~have[ranks[snd], sb[snd]]][0]
            return "round %d: processor %d sends block %d it does not hold" % (j, bad, sb[bad])
        if j == rounds - 1 and have.all():
            return "complete before the last round"
        rcv = rb >= 0
        np.add.at(got, (ranks[rcv], rb[rcv]), 1)
        have[ranks[rcv], rb[rcv]] = True
    nonroot = ranks != root
    if not have.all():
        return "not complete after n-1+q rounds"
    if not (got[nonroot] == 1).all():
        return "a non-root processor received a block %s times" % (
            "0" if (got[nonroot] == 0).any() else ">1")
    return None


def simulate_allgather(p, n, pack, unpack):
    """Brute-force run of the irregular allgather (Algorithm 9) on block numbers: pack[r] and
    unpack[r] are processor r's int32 [n-1+q][p] tables (block of buffer j sent / received per
    round).  Processor j owns all n blocks of buffer j.  Returns None if in every round every
    sent block is held by its sender and is the one the to-processor unpacks for the same buffer,
    every processor gets every block of every foreign buffer exactly once, and all are complete
    after n-1+q rounds; else a description of the first violation."""
    q = ceil_log2(p)
    rounds = n - 1 + q
    if p == 1:
        return None
    sk = closed_form_skips(p)
    x = (q - (n - 1 + q) % q) % q
    have = np.zeros((p, p, n), dtype=bool)          # [processor][buffer][block]
    for j in range(p):
        have[j, j, :] = True
    got = np.zeros((p, p, n), dtype=np.int64)
    procs = np.arange(p)
    bufs = np.arange(p)
    for jr in range(rounds):
        k = (jr + x) % q
        to = (procs + sk[k]) % p
        sb = np.stack([pack[r][jr] for r in range(p)]).astype(np.int64)      # [proc][buffer]
        rb = np.stack([unpack[r][jr] for r in range(p)]).astype(np.int64)
        if (sb >= n).any() or (rb >= n).any() or (sb < -1).any() or (rb < -1).any():
            return "round %d: block out of range" % jr
        if not np.array_equal(rb[to], sb):
            return "round %d: a packed block is not what the to-processor unpacks" % jr
        snd = sb >= 0
        pr, bf = np.nonzero(snd)
        if not have[pr, bf, sb[snd]].all():
            return "round %d: a processor packs a block it does not hold" % jr
        rcv = rb >= 0
        pr, bf = np.nonzero(rcv)
        np.add.at(got, (pr, bf, rb[rcv]), 1)
        have[pr, bf, rb[rcv]] = True
    if not have.all():
        return "not complete after n-1+q rounds"
    foreign = procs[:, None] != bufs[None, :]
    if not (got[foreign] == 1).all():
        return "a block of a foreign buffer was received %s than once" % (
            "fewer" if (got[foreign] == 0).any() else "more")
    return None
