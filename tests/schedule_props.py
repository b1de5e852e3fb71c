"""Property checker for schedule tables, written with Python sets from the sentences that
follow Theorem 1 of arXiv 2205.10072 (and from Algorithms 5 and 9).  Independent of the oracle
and of the CUDA library: it recomputes the skips from their closed form and the baseblocks from
the list construction described after Algorithm 2.

What a correct schedule of processor r (q rounds, root 0) looks like:

  receive row   in the home round h (skips[h] <= r < skips[h+1]) the entry is the baseblock of r,
                a block of the current phase; every other entry is negative, entry + q being a
                block of the previous phase; these q-1 blocks differ from each other and from the
                baseblock.  The root has no baseblock and no home round: q different negative
                entries.
  send row      the root sends block k in round k.  Any other processor sends, in round k,
                either a previous-phase block (negative entry) that it holds at that point --
                its own baseblock of the previous phase, or one that it received in an earlier
                round of the row -- or, in a round after its home round, its baseblock.
  pairing       what r sends in round k is what processor (r + skips[k]) mod p receives in
                round k (Algorithm 5, Algorithm 9's lookup).

count_violations returns the number of rows of a range that break each of the three.
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


def baseblock_list(p):
    """Baseblocks of processors 0..p-1 (entry 0, the root, is None): processor skips[k] has
    baseblock k, and the processors after it up to skips[k+1]-1 repeat the list from 1 on."""
    sk = closed_form_skips(p)
    q = len(sk) - 1
    bb = [None] * p
    for k in range(q):
        lo, hi = sk[k], sk[k + 1]
        if lo < p:
            bb[lo] = k
        for x in range(lo + 1, min(hi, p)):
            bb[x] = bb[x - lo]
    return bb


def home_round(sk, r):
    for k in range(len(sk) - 1):
        if sk[k] <= r < sk[k + 1]:
            return k
    return None


def recv_row_ok(q, bb, h, row):
    others = [int(row[k]) for k in range(q) if k != h]
    if h is not None and int(row[h]) != bb:
        return False
    if any(e >= 0 or e + q < 0 for e in others):
        return False
    blocks = {e + q for e in others}
    if len(blocks) != len(others):
        return False
    return bb not in blocks


def send_row_ok(q, r, bb, h, send_row, recv_row):
    if r == 0:
        return all(int(send_row[k]) == k for k in range(q))
    held_previous = {bb}                      # previous-phase blocks the processor can pass on
    for k in range(q):
        e = int(send_row[k])
        after_home = h is not None and k > h
        if not (after_home and e == bb):
            if e >= 0 or e + q < 0:
                return False
            if recv_row is not None and e + q not in held_previous:
                return False
        if recv_row is not None and k != h:
            got = int(recv_row[k])
            if -q <= got < 0:
                held_previous.add(got + q)
    return True


def count_violations(p, r_begin, r_end, recv, send):
    """recv, send: int8 arrays [r_end - r_begin][q] (rows of the range) or None."""
    sk = closed_form_skips(p)
    q = len(sk) - 1
    bbs = baseblock_list(p)
    bad_recv = bad_send = bad_pair = 0
    for j in range(r_end - r_begin):
        r = r_begin + j
        bb, h = bbs[r], home_round(sk, r)
        if recv is not None and not recv_row_ok(q, bb, h, recv[j]):
            bad_recv += 1
        if send is not None and not send_row_ok(q, r, bb, h, send[j],
                                                recv[j] if recv is not None else None):
            bad_send += 1
        if recv is not None and send is not None:
            for k in range(q):
                t = (r + sk[k]) % p
                if r_begin <= t < r_end and int(recv[t - r_begin][k]) != int(send[j][k]):
                    bad_pair += 1
                    break
    return bad_recv, bad_send, bad_pair
