"""The parity harness itself must catch planted faults (paper Sec. 5.8 lists the mutation kinds:
substitution, deletion, duplication, adjacent swap, same-length tail resplit)."""
import random

import numpy as np

import workloads as wl
from gpu_util import cpu_vocab


def _equal(a, b):
    return a.size == b.size and np.array_equal(a, b)


def test_planted_faults_are_caught():
    cfg = wl.CONFIGS["C1"]
    text = wl.request(cfg)
    ids, po = cpu_vocab("C1").encode(text, 0)
    rng = random.Random(0)
    for _ in range(200):
        k = rng.randrange(1, ids.size - 2)
        sub = ids.copy(); sub[k] = (sub[k] + 1) % 4352
        dele = np.delete(ids, k)
        dup = np.insert(ids, k, ids[k])
        swap = ids.copy()
        if swap[k] == swap[k + 1]:
            continue
        swap[k], swap[k + 1] = swap[k + 1], swap[k]
        for mutated in (sub, dele, dup, swap):
            assert not _equal(mutated, ids)
    # same-length tail resplit: move one piece boundary by one byte; lengths stay equal, offsets differ
    for _ in range(50):
        k = rng.randrange(1, po.size - 2)
        if po[k] + 1 >= po[k + 1]:
            continue
        moved = po.copy(); moved[k] += 1
        assert moved.size == po.size and not _equal(moved, po)
