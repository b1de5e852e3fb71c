"""Reader for the schedules printed in the paper (Tables 1-5), stored under tests/golden/."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")

TABLES = ["table1_p20", "table2_p33", "table3_p32", "table4_p31", "table5_p9_left"]
SECOND_P9 = "table5_p9_right"


def load(name):
    p, sk, bb, recv, send = None, None, None, {}, {}
    with open(os.path.join(GOLDEN, name + ".txt")) as f:
        for ln in f:
            if ln.startswith("#") or not ln.strip():
                continue
            t = ln.split()
            if t[0] == "p":
                p = int(t[1])
            elif t[0] == "skips":
                sk = [int(v) for v in t[1:]]
            elif t[0] == "baseblock":
                bb = [int(v) for v in t[1:]]
            elif t[0] == "recv":
                recv[int(t[1])] = [int(v) for v in t[2:]]
            elif t[0] == "send":
                send[int(t[1])] = [int(v) for v in t[2:]]
    q = len(sk) - 1
    # printed tables are round-major; the library and the oracle are rank-major [p][q]
    recv = np.array([recv[k] for k in range(q)], dtype=np.int8).T.copy()
    send = np.array([send[k] for k in range(q)], dtype=np.int8).T.copy()
    return {"p": p, "q": q, "skips": sk, "baseblock": bb, "recv": recv, "send": send}
