"""Pins for the oracle's byte-level BPE and the end-to-end encode (paper Sec. 4.2)."""
import json
import os
import random

import numpy as np
import pytest

import oracle
import workloads as wl
from patterns import PATTERNS

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "bpe_examples.jsonl")


def _vocab_from_pairs(pairs):
    pairs = np.asarray(pairs, dtype=np.int32).reshape(-1, 2)
    merges = np.concatenate([pairs, 256 + np.arange(len(pairs), dtype=np.int32)[:, None]], axis=1)
    return oracle.Vocab(merges)


def test_hand_worked_examples():
    n = 0
    with open(GOLDEN, encoding="utf-8") as f:
        for line in f:
            d = json.loads(line)
            if "piece" not in d:
                continue
            v = _vocab_from_pairs(d["merges"])
            for variant in (0, 1, 2):
                assert list(v.bpe(d["piece"], variant)) == d["ids"], (d, variant)
            n += 1
    assert n >= 10


def _random_wellformed_pairs(rng, n_merges, alphabet):
    """Random merge table whose operands are base ids or results of lower ranks."""
    ids = list(alphabet)
    seen, pairs = set(), []
    while len(pairs) < n_merges:
        p = (rng.choice(ids), rng.choice(ids))
        if p in seen:
            continue
        seen.add(p)
        pairs.append(p)
        ids.append(256 + len(pairs) - 1)
    return pairs


def _rounds(pairs, piece):
    """The schedule the paper licenses (Sec. 4.2): per round take the minimum rank present and merge
    all leftmost non-overlapping occurrences of that pair.  Must equal iterated single merges."""
    rank = {p: i for i, p in enumerate(pairs)}
    t = list(piece)
    while True:
        present = [rank[(a, b)] for a, b in zip(t, t[1:]) if (a, b) in rank]
        if not present:
            return t
        m = min(present)
        pr, out, i = pairs[m], [], 0
        while i < len(t):
            if i + 1 < len(t) and (t[i], t[i + 1]) == pr:
                out.append(256 + m)
                i += 2
            else:
                out.append(t[i])
                i += 1
        t = out


def test_round_schedule_equals_definition_and_heap_equals_rescan():
    rng = random.Random(3)
    for trial in range(300):
        alphabet = [97 + k for k in range(rng.randrange(1, 4))]
        pairs = _random_wellformed_pairs(rng, rng.randrange(1, 12), alphabet)
        v = _vocab_from_pairs(pairs)
        for _ in range(20):
            piece = bytes(rng.choice(alphabet) for _ in range(rng.randrange(1, 24)))
            a = list(v.bpe(piece, 0))
            assert a == list(v.bpe(piece, 1))
            assert a == _rounds(pairs, piece)
            assert v.decode(a) == piece


def test_long_piece_heap_equals_rescan():
    cfg = wl.CONFIGS["C1"]
    merges, _ = wl.load_vocab(cfg)
    v = oracle.Vocab(merges)
    text = wl.request(cfg, n_chars=3000).tobytes()
    assert list(v.bpe(text, 0)) == list(v.bpe(text, 1))
    blanks = b" " * 5000
    assert list(v.bpe(blanks, 0)) == list(v.bpe(blanks, 1))


def _token_table(v):
    return [v.token_bytes(i) for i in range(256 + v.n_merges)]


@pytest.mark.parametrize("name", ["C1", "C2"])
def test_equals_independent_bpe_library(name):
    """Same ranks + same pattern string given to tiktoken (an independent byte-pair encoder) must
    give the same IDs."""
    tiktoken = pytest.importorskip("tiktoken")
    cfg = wl.CONFIGS[name]
    merges, _ = wl.load_vocab(cfg)
    v = oracle.Vocab(merges)
    toks = _token_table(v)
    assert len(set(toks)) == len(toks)
    enc = tiktoken.Encoding("pin", pat_str=PATTERNS[cfg.pattern_id], mergeable_ranks={b: i for i, b in enumerate(toks)},
                            special_tokens={})
    text = wl.request(cfg, n_chars=min(cfg.n_chars, 30000))
    ids, _ = v.encode(text, cfg.pattern_id)
    assert list(ids) == enc.encode(text.tobytes().decode("utf-8"), disallowed_special=())


def test_equals_independent_bpe_library_pattern1():
    tiktoken = pytest.importorskip("tiktoken")
    cfg = wl.CONFIGS["C4"]
    merges, _ = wl.load_vocab(cfg)
    merges = merges[:20000]
    v = oracle.Vocab(merges)
    toks = _token_table(v)
    enc = tiktoken.Encoding("pin1", pat_str=PATTERNS[1], mergeable_ranks={b: i for i, b in enumerate(toks)}, special_tokens={})
    text = wl.request(wl.CONFIGS["C2"], n_chars=20000)
    ids, _ = v.encode(text, 1)
    assert list(ids) == enc.encode(text.tobytes().decode("utf-8"), disallowed_special=())


@pytest.mark.parametrize("name", ["C1", "C2", "C4"])
def test_end_to_end_invariants(name):
    cfg = wl.CONFIGS[name]
    merges, _ = wl.load_vocab(cfg)
    v = oracle.Vocab(merges)
    text = wl.request(cfg, n_chars=min(cfg.n_chars, 60000))
    ids, po = v.encode(text, cfg.pattern_id)
    assert v.decode(ids) == text.tobytes()
    assert ids.min() >= 0 and ids.max() < 256 + cfg.n_merges
    assert len(ids) <= text.size and po[0] == 0 and po[-1] == text.size
    assert list(po[:-1]) == list(oracle.pretokenize(text, cfg.pattern_id))
    ids_mt, _ = v.encode(text, cfg.pattern_id, nthreads=3)
    assert list(ids_mt) == list(ids)


def test_batch_equals_documents_alone():
    cfg = wl.CONFIGS["C5"]
    merges, _ = wl.load_vocab(cfg)
    v = oracle.Vocab(merges)
    text, off = wl.batch(cfg, n_docs=5, scale=0.01)
    ids, ioff = v.encode_batch(text, off, cfg.pattern_id, nthreads=2)
    for d in range(5):
        alone, _ = v.encode(text[off[d]:off[d + 1]], cfg.pattern_id)
        assert list(ids[ioff[d]:ioff[d + 1]]) == list(alone)
    assert ioff[-1] == len(ids)


def test_non_identity_byte_map_and_result_ids():
    rng = random.Random(9)
    perm = list(range(256))
    rng.shuffle(perm)
    byte_map = np.array([1000 + p for p in perm], dtype=np.int32)
    merges = np.array([[byte_map[97], byte_map[98], 5], [5, byte_map[99], 7]], dtype=np.int32)
    v = oracle.Vocab(merges, byte_map)
    assert list(v.bpe(b"abcab", 0)) == [7, 5]
    assert v.decode([7, 5]) == b"abcab"


# ---- whole-piece rule (ignore_merges) -------------------------------------------------------------
IGNORE_GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "ignore_merges_examples.jsonl")


def test_ignore_merges_hand_worked_examples():
    n = 0
    with open(IGNORE_GOLDEN, encoding="utf-8") as f:
        for line in f:
            d = json.loads(line)
            if "piece" not in d:
                continue
            pairs = np.asarray(d["merges"], dtype=np.int32)
            merges = np.concatenate([pairs, 256 + np.arange(len(pairs), dtype=np.int32)[:, None]], axis=1)
            assert list(oracle.Vocab(merges).bpe(d["piece"], 2)) == d["plain"], d
            assert list(oracle.Vocab(merges, ignore_merges=True).bpe(d["piece"], 2)) == d["ignore"], d
            n += 1
    assert n >= 8


def test_ignore_merges_against_a_dictionary_of_entry_strings():
    """Independent restatement on a stored vocabulary: entry strings are built here by concatenation, the first
    entry that spells given bytes is kept in a dict, and every piece of a text is looked up in it before
    falling back to the merge loop (which the pins above cover).  Also: the rule changes nothing for pieces
    that are no entry, and ids always spell the text."""
    cfg = wl.CONFIGS["C1"]
    merges, byte_map = wl.load_vocab(cfg)
    spell = {int(byte_map[b]): bytes([b]) for b in range(256)}
    first = {bytes([b]): int(byte_map[b]) for b in range(256)}
    for left, right, result in merges.tolist():
        spell[result] = spell[left] + spell[right]
        first.setdefault(spell[result], result)
    plain, ign = oracle.Vocab(merges, byte_map), oracle.Vocab(merges, byte_map, ignore_merges=True)
    text = wl.request(cfg).tobytes()
    pieces = oracle.pieces(text, cfg.pattern_id)
    ids, _ = ign.encode(text, cfg.pattern_id)
    want, changed = [], 0
    for p in pieces:
        if p in first:
            want.append(first[p])
            changed += list(plain.bpe(p, 2)) != [first[p]]
        else:
            want.extend(plain.bpe(p, 2).tolist())
    assert ids.tolist() == want
    assert ign.decode(ids) == text
    # every entry that is one piece under the pattern encodes to the first entry with its spelling
    rng = random.Random(5)
    entries = [s for s in first if len(s) >= 2]
    for s in rng.sample(entries, 400):
        if len(oracle.pieces(s, cfg.pattern_id)) == 1:
            assert ign.encode(s, cfg.pattern_id)[0].tolist() == [first[s]]
