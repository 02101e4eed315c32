"""Pins for the oracle's added-token literal pass (leftmost-longest, paper Sec. 4.3/4.4)."""
import random
import re

import numpy as np

import oracle
import workloads as wl

# hand-worked: (text, literals, expected segments as (start, end, literal index or -1))
WORKED = [
    ("a<|x|>b", ["<|x|>"], [(0, 1, -1), (1, 6, 0), (6, 7, -1)]),
    ("<|x|><|x|>", ["<|x|>"], [(0, 5, 0), (5, 10, 0)]),
    ("abcd", ["ab", "abc"], [(0, 3, 1), (3, 4, -1)]),                   # the longer literal at the same position
    ("xabc", ["xab", "abc"], [(0, 3, 0), (3, 4, -1)]),                  # the leftmost wins, its overlap is lost
    ("aaaaa", ["aa"], [(0, 2, 0), (2, 4, 0), (4, 5, -1)]),              # non-overlapping, left to right
    ("aaaa", ["aaa", "aa"], [(0, 3, 0), (3, 4, -1)]),
    ("ab", ["b", "ab", "a"], [(0, 2, 1)]),
    ("", ["x"], []),
    ("xyz", [], [(0, 3, -1)]),
    ("é<s>é", ["<s>"], [(0, 2, -1), (2, 5, 0), (5, 7, -1)]),
]


def test_hand_worked_literal_splits():
    for text, lits, want in WORKED:
        assert oracle.split_added(text.encode(), lits) == want, (text, lits)


def test_literal_split_equals_longest_first_regex_alternation():
    """Independent engine: a leftmost-first alternation of the escaped literals, longest first, finds the same
    occurrences (at one position the first alternative that matches is then the longest)."""
    rng = random.Random(3)
    for trial in range(300):
        alpha = rng.choice(["ab", "abc<|>", "a<"])
        lits = list({"".join(rng.choice(alpha) for _ in range(rng.randrange(1, 5))) for _ in range(rng.randrange(1, 6))})
        text = "".join(rng.choice(alpha) for _ in range(rng.randrange(0, 60)))
        rx = re.compile("|".join(re.escape(x) for x in sorted(lits, key=len, reverse=True)))
        want = [(m.start(), m.end(), lits.index(m.group())) for m in rx.finditer(text)]
        got = [s for s in oracle.split_added(text.encode(), lits) if s[2] >= 0]
        assert got == want, (text, lits)
        # the segments tile the text
        segs = oracle.split_added(text.encode(), lits)
        assert [s[0] for s in segs] == [0] * bool(segs) + [s[1] for s in segs[:-1]] and (not segs or segs[-1][1] == len(text))


def test_encode_added_segments_are_independent_texts():
    cfg = wl.CONFIGS["C1"]
    merges, byte_map = wl.load_vocab(cfg)
    v = oracle.Vocab(merges, byte_map)
    lits, lit_ids = ["<|user|>", "<|assistant|>", "<|end|>"], [900001, 900002, 900003]
    text = b"<|user|>\nHello there, it's 12345!<|end|><|assistant|>Sure thing.\n<|end|>"
    ids = oracle.encode_added(v, text, 0, lits, lit_ids)
    want = [900001] + v.encode(b"\nHello there, it's 12345!", 0)[0].tolist() + [900003, 900002] + \
        v.encode(b"Sure thing.\n", 0)[0].tolist() + [900003]
    assert ids.tolist() == want
    # without literals it is the plain encoding
    assert np.array_equal(oracle.encode_added(v, text, 0, [], []), v.encode(text, 0)[0])
