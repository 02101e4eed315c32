"""Pins for the oracle's pre-tokenizer (paper Sec. 4.1: leftmost-first alternation with
backtracking, each match beginning at the previous match's end).

The oracle is a hand-written sequential matcher; here it is compared with a genuine backtracking
regex engine on exhaustive small alphabets and random strings, with worked examples, and with
structural invariants."""
import itertools
import json
import os
import random

import numpy as np
import pytest

import oracle
from patterns import PATTERNS, engine_starts

regex = pytest.importorskip("regex")
R = [regex.compile(p) for p in PATTERNS]
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "pretok_examples.jsonl")


def _engine_chunk(args):
    """Worker: piece starts of the regex engine for the documents [lo, hi) of an exhaustive set, as offsets into
    the concatenation (the same layout oracle.pretokenize_batch returns)."""
    pat, text, off, lo, hi = args
    r = regex.compile(PATTERNS[pat])
    out = []
    raw = text.tobytes()
    for d in range(lo, hi):
        b = int(off[d])
        out.extend(b + x for x in engine_starts(r, raw[b:int(off[d + 1])].decode("utf-8")))
    return np.asarray(out, dtype=np.int64)


def _exhaustive(pat, alphabet, maxlen):
    """Every string of 1..maxlen symbols: the oracle (one batch call, each string matched alone) against the
    backtracking engine (worker processes).  Returns the first few strings on which they differ."""
    import multiprocessing as mp
    import workloads as wl
    text, off = wl.exhaustive(alphabet, maxlen)
    n = off.size - 1
    got = oracle.pretokenize_batch(text, off, pat, nthreads=min(8, os.cpu_count() or 1))
    nproc = min(8, os.cpu_count() or 1)
    step = max(1, (n + 4 * nproc - 1) // (4 * nproc))
    jobs = [(pat, text, off, lo, min(n, lo + step)) for lo in range(0, n, step)]
    if n < 50_000 or nproc == 1:
        parts = [_engine_chunk(j) for j in jobs]
    else:
        with mp.get_context("fork").Pool(nproc) as pool:
            parts = pool.map(_engine_chunk, jobs)
    want = np.concatenate(parts)
    if got.size == want.size and np.array_equal(got, want):
        return []
    bad = sorted(set(got.tolist()) ^ set(want.tolist()))[:6]
    which = sorted({int(np.searchsorted(off, b, side="right") - 1) for b in bad})
    return [text[off[d]:off[d + 1]].tobytes().decode("utf-8") for d in which]


def test_exhaustive_generator_and_batch_call_are_what_they_claim():
    """The exhaustive sets come from a generator and the oracle is called once per set: the generator must
    produce itertools.product order, and the batch call must equal the per-string call."""
    import workloads as wl
    alphabet = "aé中 \n'"
    text, off = wl.exhaustive(alphabet, 4)
    docs = ["".join(t).encode("utf-8") for ln in range(1, 5) for t in itertools.product(alphabet, repeat=ln)]
    assert off.size - 1 == len(docs) and text.tobytes() == b"".join(docs)
    assert [text[off[i]:off[i + 1]].tobytes() for i in (0, 5, 41, len(docs) - 1)] == [docs[i] for i in (0, 5, 41, len(docs) - 1)]
    for pat in (0, 1, 2, 3):
        want = np.concatenate([oracle.pretokenize(d, pat) + off[i] for i, d in enumerate(docs)])
        assert np.array_equal(oracle.pretokenize_batch(text, off, pat, nthreads=3), want)


# The sets and lengths are the ones on which the run-local closed forms were validated when the path was
# surveyed (pattern 0: three sets; pattern 1: five sets), plus the earlier sets of this suite.
@pytest.mark.parametrize("alphabet,maxlen", [
    ("asl1 \t\n\r!'", 7),              # letters, digit, blank, tab, LF, CR, punctuation, apostrophe
    ("rRevl't !", 7),                  # every contraction spelling
    ("eé中²́ 　\u00a0\n's", 6),   # multi-byte letters, No digit, mark, ideographic space, no-break space
    ("a1 \r\n\u00a0!", 6),             # CR, LF, no-break space
])
def test_pattern0_equals_backtracking_engine(alphabet, maxlen):
    assert _exhaustive(0, alphabet, maxlen) == []


@pytest.mark.parametrize("alphabet,maxlen", [
    ("a\u0301's/\n !", 7),         # marks with contraction and tail chains (8 symbols: a, U+0301, ', s, /, LF, SP, !)
    ("Aal's1 \n/", 7),
    ("Aá's !/\n", 7),
    ("Aa中́'s !/\n", 6),
    ("AaBb中́1 \t", 6),
    ("ǅaʰA'l \r", 6),         # titlecase, modifier letter
])
def test_pattern1_equals_backtracking_engine(alphabet, maxlen):
    assert _exhaustive(1, alphabet, maxlen) == []


@pytest.mark.parametrize("alphabet,maxlen", [("a12 \t\n!'", 6), ("1²٣ a.", 7)])
def test_pattern2_single_digit_variant_equals_backtracking_engine(alphabet, maxlen):
    assert _exhaustive(2, alphabet, maxlen) == []
    assert [p.decode() for p in oracle.pieces("ab1234 56", 2)] == ["ab", "1", "2", "3", "4", " ", "5", "6"]


def _agreeing_codepoints():
    """Code points whose class agrees between the oracle's frozen table and the regex engine's own
    (possibly newer) Unicode tables; random strings are drawn only from these."""
    t = oracle.class_table()
    pools = []
    probes = [(r"\p{Ll}", oracle.K_LL), (r"[\p{Lu}\p{Lt}]", oracle.K_LU), (r"[\p{Lm}\p{Lo}]", oracle.K_LB),
              (r"\p{N}", oracle.K_N), (r"\s", oracle.K_W), (r"\p{M}", oracle.K_M)]
    rng = random.Random(5)
    sample = [rng.randrange(0x20, 0x30000) for _ in range(6000)] + list(range(0x20, 0x250))
    sample = [c for c in sample if not (0xD800 <= c <= 0xDFFF)]
    for c in sample:
        ch = chr(c)
        code = oracle.K_O
        for pat, k in probes:
            if regex.fullmatch(pat, ch):
                code = k
                break
        if code == t[c]:
            pools.append(c)
    return pools


def test_random_unicode_strings_equal_engine():
    pool = _agreeing_codepoints()
    assert len(pool) > 5000
    rng = random.Random(11)
    special = list(" \t\n\r'/!.,") + ["'s", "'re", "'LL", "\r\n", "  "]
    for pat in (0, 1, 2):
        for _ in range(3000):
            n = rng.randrange(1, 40)
            s = "".join(rng.choice(special) if rng.random() < 0.5 else chr(rng.choice(pool)) for _ in range(n))
            assert engine_starts(R[pat], s) == list(oracle.pretokenize(s, pat)), repr(s)


def test_worked_examples():
    n = 0
    with open(GOLDEN, encoding="utf-8") as f:
        for line in f:
            d = json.loads(line)
            if "text" not in d:
                continue
            for pat, key in ((0, "p0"), (1, "p1")):
                got = [p.decode("utf-8") for p in oracle.pieces(d["text"], pat)]
                assert got == d[key], (d["text"], key, got)
            n += 1
    assert n >= 30


def test_pieces_partition_the_input():
    import workloads as wl
    for name in ("C1", "C2"):
        cfg = wl.CONFIGS[name]
        text = wl.request(cfg, n_chars=20000)
        for pat in (0, 1):
            st = oracle.pretokenize(text, pat)
            assert st[0] == 0 and np.all(np.diff(st) > 0) and st[-1] < text.size
            # every start is a code-point boundary
            assert np.all((text[st] & 0xC0) != 0x80)
            assert b"".join(oracle.pieces(text, pat)) == text.tobytes()


def test_document_cut_is_idempotent():
    """Cutting the text at a piece boundary and matching both halves alone gives the same pieces
    (a match never looks behind its own start)."""
    import workloads as wl
    text = wl.request(wl.CONFIGS["C2"], n_chars=5000)
    for pat in (0, 1):
        st = oracle.pretokenize(text, pat)
        for k in (len(st) // 3, len(st) // 2):
            cut = int(st[k])
            tail = oracle.pretokenize(text[cut:], pat) + cut
            assert list(tail) == list(st[k:])


def test_class_table_spot_values_and_engine_agreement():
    t = oracle.class_table()
    assert t[0x20] == oracle.K_W and t[0x3000] == oracle.K_W and t[0x85] == oracle.K_W and t[0xA0] == oracle.K_W
    assert t[0x1C] == oracle.K_O            # str.isspace() says True, White_Space says no
    assert t[0xE9] == oracle.K_LL and t[0x4E2D] == oracle.K_LB and t[0x0301] == oracle.K_M
    assert t[0xB2] == oracle.K_N and t[0x01C5] == oracle.K_LU and t[0x2160] == oracle.K_N
    assert t[ord("A")] == oracle.K_LU and t[ord("z")] == oracle.K_LL and t[ord("7")] == oracle.K_N
    assert t[ord("'")] == oracle.K_O and t[ord("/")] == oracle.K_O and t[0x1F600] == oracle.K_O
    assert int((t == oracle.K_W).sum()) == 25
    # the regex engine's \s is exactly the whitespace class
    ws = [c for c in range(0x3100) if regex.fullmatch(r"\s", chr(c))]
    assert ws == [c for c in range(0x3100) if t[c] == oracle.K_W]
    # Against the engine's (newer) tables over U+0020..U+2FFF: every disagreement must be a code
    # point that is unassigned in the frozen 15.0.0 database, except U+0295, whose General_Category
    # changed after 15.0.
    import unicodedata
    differ = []
    for c in range(0x20, 0x3000):
        ch = chr(c)
        want = (oracle.K_LL if regex.fullmatch(r"\p{Ll}", ch) else oracle.K_LU if regex.fullmatch(r"[\p{Lu}\p{Lt}]", ch)
                else oracle.K_LB if regex.fullmatch(r"[\p{Lm}\p{Lo}]", ch) else oracle.K_N if regex.fullmatch(r"\p{N}", ch)
                else oracle.K_W if regex.fullmatch(r"\s", ch) else oracle.K_M if regex.fullmatch(r"\p{M}", ch) else oracle.K_O)
        if t[c] != want:
            differ.append(c)
    assert len(differ) < 60
    for c in differ:
        assert c == 0x295 or unicodedata.category(chr(c)) == "Cn", hex(c)


@pytest.mark.parametrize("data,ok", [
    (b"", True), (b"abc", True), ("é中😀".encode(), True),
    (b"\x80", False), (b"\xc3", False), (b"\xc0\xaf", False), (b"\xe0\x80\xaf", False),
    (b"\xed\xa0\x80", False), (b"\xf4\x90\x80\x80", False), (b"\xf0\x8f\xbf\xbf", False),
    (b"a\xe4\xb8", False), (b"\xf5\x80\x80\x80", False), (b"\xef\xbf\xbf", True), (b"\xf4\x8f\xbf\xbf", True),
])
def test_strict_utf8(data, ok):
    assert (oracle.utf8_check(data) >= 0) == ok
    if not ok:
        with pytest.raises(oracle.InvalidUtf8):
            oracle.pretokenize(data, 0)


def test_pattern3_three_splitter_composition_equals_engine():
    """Pattern 3 against the regex engine doing the three stages one after the other (isolated matches, gaps
    kept, each piece re-split by the next stage): exhaustive small alphabets and random Unicode strings."""
    from patterns import SPLIT3_A, SPLIT3_B, engine_starts_split3
    ra, rb = regex.compile(SPLIT3_A), regex.compile(SPLIT3_B)
    n = 0
    for alphabet, maxlen in [("a1中 ", 6), ("1中x' \n", 5), ("12 !中文a", 5)]:
        for ln in range(1, maxlen + 1):
            for tup in itertools.product(alphabet, repeat=ln):
                s = "".join(tup)
                assert engine_starts_split3(ra, rb, R[0], s) == list(oracle.pretokenize(s, 3)), repr(s)
                n += 1
    assert n > 20000
    pool = _agreeing_codepoints()
    rng = random.Random(12)
    special = list(" \t\n\r'/!.,0123456789中文") + ["'s", "\r\n", "  ", "1234567"]
    for _ in range(3000):
        k = rng.randrange(1, 40)
        s = "".join(rng.choice(special) if rng.random() < 0.5 else chr(rng.choice(pool)) for _ in range(k))
        assert engine_starts_split3(ra, rb, R[0], s) == list(oracle.pretokenize(s, 3)), repr(s)
    # the composition is not pattern 0: context is cut at the stage boundaries
    assert [p.decode() for p in oracle.pieces("x  12", 3)] == ["x", "  ", "12"]
    assert [p.decode() for p in oracle.pieces("x  12", 0)] == ["x", " ", " ", "12"]
