"""The parity harness itself must catch planted faults (paper Sec. 5.8 lists the mutation kinds: substitution,
deletion, duplication, adjacent swap, same-length tail resplit).

What is under test here is the comparison the parity tests apply (``gpu_util.same``) and the shadow
verifier's comparison (``tt_verifier_submit`` with a reference callback): a correct output is mutated ON THE
HOST in each of the five ways and both must reject every mutant.  The GPU test mutates what the CUDA path
returned (ids from tt_encode, piece offsets from tt_pretokenize); the CPU test does the same with the
oracle's output so that the helper is exercised without a device too."""
import random

import numpy as np
import pytest

import workloads as wl
from gpu_util import cpu_vocab, same


def _tail_resplit(cv, ids):
    """A same-length re-split of the tail: two adjacent tokens (X)(Y) are replaced by two other vocabulary
    entries (X')(Y') that spell the same bytes with the cut moved -- the id count, the decoded text and
    every earlier id stay the same.  Returns the mutant, or None if no such spot exists near the end."""
    entries = {}
    for t in range(256 + cv.n_merges):
        entries.setdefault(cv.token_bytes(t), t)
    for k in range(ids.size - 2, max(ids.size - 400, 0), -1):
        b = cv.token_bytes(int(ids[k])) + cv.token_bytes(int(ids[k + 1]))
        for cut in range(1, len(b)):
            l, r = entries.get(b[:cut]), entries.get(b[cut:])
            if l is not None and r is not None and (l, r) != (int(ids[k]), int(ids[k + 1])):
                out = ids.copy(); out[k] = l; out[k + 1] = r
                return out
    return None


def _mutants(cv, ids, rng, vocab_size):
    """(kind, mutated sequence) for the five kinds, at random positions."""
    for _ in range(60):
        k = rng.randrange(1, ids.size - 2)
        sub = ids.copy(); sub[k] = (sub[k] + 1 + rng.randrange(vocab_size - 1)) % vocab_size
        yield "substitute", sub
        yield "delete", np.delete(ids, k)
        yield "duplicate", np.insert(ids, k, ids[k])
        if ids[k] != ids[k + 1]:
            swap = ids.copy(); swap[k], swap[k + 1] = swap[k + 1], swap[k]
            yield "swap", swap
    rs = _tail_resplit(cv, ids)
    assert rs is not None and rs.size == ids.size and cv.decode(rs[-400:]) == cv.decode(ids[-400:])
    yield "tail resplit", rs


def _check_planted_faults(ids, pieces, text):
    import paper_2607_29678_b200 as tt
    cfg = wl.CONFIGS["C1"]
    cv = cpu_vocab("C1")
    want, want_po = cv.encode(text, cfg.pattern_id)
    assert same(ids, want) and same(pieces, want_po[:-1])          # the unmutated output passes
    rng = random.Random(0)
    muts = list(_mutants(cv, ids, rng, 256 + cfg.n_merges))
    assert {k for k, _ in muts} == {"substitute", "delete", "duplicate", "swap", "tail resplit"}
    for kind, m in muts:
        assert not same(m, want), kind
    # piece level: a same-length resplit moves one boundary by a byte (count unchanged); deletions and duplicates too
    n_piece_mut = 0
    for _ in range(60):
        k = rng.randrange(1, pieces.size - 2)
        if pieces[k] + 1 < pieces[k + 1]:
            moved = pieces.copy(); moved[k] += 1
            assert moved.size == pieces.size and not same(moved, want_po[:-1])
            n_piece_mut += 1
        assert not same(np.delete(pieces, k), want_po[:-1]) and not same(np.insert(pieces, k, pieces[k]), want_po[:-1])
    assert n_piece_mut > 10
    # a wrong dtype or shape is not "equal" either
    assert not same(ids.astype(np.float64), want) and not same(ids.reshape(1, -1), want)
    # the shadow verifier rejects the same mutants: reference engine = the oracle, full sampling
    ver = tt.Verifier(lambda t: cv.encode(t, cfg.pattern_id)[0], sample_rate=1.0, queue_cap=len(muts) + 8)
    raw = text.tobytes()
    assert ver.submit(raw, ids) == 1
    for _, m in muts:
        assert ver.submit(raw, m.astype(np.int32)) == 1
    ver.drain()
    st = ver.stats()
    assert st["checked"] == len(muts) + 1 and st["mismatches"] == len(muts) and st["dropped"] == 0
    ver.close()


def test_planted_faults_in_oracle_output_are_caught():
    cfg = wl.CONFIGS["C1"]
    text = wl.request(cfg)
    ids, po = cpu_vocab("C1").encode(text, cfg.pattern_id)
    _check_planted_faults(ids.copy(), po[:-1].copy(), text)


@pytest.mark.gpu
def test_planted_faults_in_gpu_output_are_caught():
    from gpu_util import gpu_encode, gpu_pretok, gpu_vocab
    cfg = wl.CONFIGS["C1"]
    text = wl.request(cfg)
    ids, status = gpu_encode(gpu_vocab("C1"), text)
    assert status == 0
    pieces, status = gpu_pretok(gpu_vocab("C1"), text)
    assert status == 0
    _check_planted_faults(ids, pieces, text)
