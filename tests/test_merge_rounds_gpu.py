"""GPU parity of the merge rounds (paper Sec. 4.2) on vocabularies built to stress them: small alphabets with
dense, deep merge trees (long runs of identical pairs, guards that block for many rounds), pieces of every
length class (<= 32 bytes, 33..64, 65..128, 129..256, in shared memory up to 4,096 tokens, beyond that in
global scratch) and enough unsettled short pieces for the thread-per-piece path.  Ids must equal the oracle's."""
import random

import numpy as np
import pytest

import oracle
from gpu_util import gpu_encode, same

pytestmark = pytest.mark.gpu


def _dense_vocab(rng, n_merges, alphabet):
    toks, seen, merges = list(alphabet), set(), []
    while len(merges) < n_merges:
        a = rng.choice(toks[-40:] if rng.random() < 0.3 else toks)       # a bias towards recent results: deep trees
        b = rng.choice(toks[-40:] if rng.random() < 0.3 else toks)
        if (a, b) in seen:
            continue
        seen.add((a, b))
        merges.append((a, b, 256 + len(merges)))
        toks.append(256 + len(merges) - 1)
    return np.array(merges, dtype=np.int32)


@pytest.mark.parametrize("seed", range(12))
def test_dense_vocabularies_all_length_classes(seed):
    import paper_2607_29678_b200 as tt
    rng = random.Random(1000 + seed)
    alphabet = [b"ab", b"abc", b"abcdefgh", b"abcdefghijklmnopqrstuvwxyz", b"ab \t", b" \t", b"aA", b"0123456789ab"][seed % 8]
    merges = _dense_vocab(rng, [5, 50, 300, 2000, 8000][seed % 5], alphabet)
    pattern = seed % 2
    gv, cv = tt.Vocab(merges, None, pattern), oracle.Vocab(merges, None)
    texts = [bytes(rng.choice(alphabet) for _ in range(n)) for n in (2, 31, 32, 33, 64, 65, 128, 129, 256, 257, 4096, 4097, 20000)]
    texts.append(b" ".join(bytes(rng.choice(alphabet) for _ in range(rng.randrange(1, 40))) for _ in range(9000)))
    texts.append(b"\n".join(bytes([rng.choice(alphabet)]) * rng.randrange(1, 600) for _ in range(50)))
    texts.append(b" ".join(bytes(rng.choice(alphabet) for _ in range(rng.randrange(30, 260))) for _ in range(200)))
    unit = bytes(rng.choice(alphabet) for _ in range(rng.randrange(1, 5)))
    texts.append(unit * 2500)
    for s in texts:
        text = np.frombuffer(s, dtype=np.uint8)
        ids, status = gpu_encode(gv, text, offset=rng.randrange(16))
        want, _ = cv.encode(text, pattern, nthreads=8)
        assert status == 0 and same(ids, want), (seed, len(s), s[:60])


def test_no_merges_and_one_merge():
    """Degenerate vocabularies: without merges every byte is a token; with one merge only that pair combines."""
    import paper_2607_29678_b200 as tt
    text = np.frombuffer(("aab aaaa b " * 300 + "a" * 5000).encode(), dtype=np.uint8)
    for merges in (np.zeros((0, 3), dtype=np.int32), np.array([[ord("a"), ord("a"), 256]], dtype=np.int32)):
        gv, cv = tt.Vocab(merges, None, 0), oracle.Vocab(merges, None)
        ids, status = gpu_encode(gv, text)
        want, _ = cv.encode(text, 0)
        assert status == 0 and same(ids, want)
    assert int((ids == 256).sum()) > 2500
