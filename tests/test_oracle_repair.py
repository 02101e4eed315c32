"""Pins for the oracle's incremental repair (paper Sec. 3.3): the result of every append equals a full
tokenization, the stable boundaries really cut the dependence on the left context, and the boundary
condition is needed (a matched run of records alone can splice wrongly)."""
import random

import numpy as np
import pytest

import oracle
import workloads as wl
from oracle import repair


def _stream(rng, text: bytes, n_cuts: int):
    """Cuts valid UTF-8 into consecutive appends at random character boundaries."""
    cuts = set()
    while len(cuts) < n_cuts:
        c = rng.randrange(1, len(text))
        while c < len(text) and (text[c] & 0xC0) == 0x80:
            c += 1
        if c < len(text):
            cuts.add(c)
    cuts = [0] + sorted(cuts) + [len(text)]
    return [text[a:b] for a, b in zip(cuts[:-1], cuts[1:])]


@pytest.mark.parametrize("pattern", [0, 1, 2, 3])
def test_stable_boundaries_cut_left_context(pattern):
    """At every stable boundary p of a text T the pieces of T from p on are the pieces of T[p:]: the text to
    the left has no influence (checked by tokenizing the suffix alone), and p itself begins a piece."""
    rng = random.Random(pattern)
    n_checked = 0
    for trial in range(6):
        text = wl.generate(wl.KIND_MIX_UNI if trial % 2 else wl.KIND_TRANSCRIPT_ADV, 500 + trial, 3000).tobytes()[:6000]
        text = text.decode("utf-8", errors="ignore").encode("utf-8")
        starts = oracle.pretokenize(text, pattern).tolist()
        start_set = set(starts)
        bounds = [p for p in range(1, len(text)) if repair.is_stable_boundary(text, p)]
        assert len(bounds) > 100
        for p in bounds:
            assert p in start_set
        for p in rng.sample(bounds, 60):
            suffix = (oracle.pretokenize(text[p:], pattern) + p).tolist()
            assert suffix == [s for s in starts if s >= p], (pattern, p, text[max(0, p - 10):p + 10])
            n_checked += 1
    assert n_checked >= 300


@pytest.mark.parametrize("name,window", [("C1", 512), ("C1", 24), ("C2", 64)])
def test_append_streams_equal_full_tokenization(name, window):
    cfg = wl.CONFIGS[name]
    merges, byte_map = wl.load_vocab(cfg)
    vocab = oracle.Vocab(merges, byte_map)
    rng = random.Random(window)
    text = wl.generate(cfg.kind, 4242 + window, 12000).tobytes()
    text = text + "é中 1234567890123 x's's's tail   \n\n  end".encode() * 3
    sess = repair.Session(vocab, cfg.pattern_id, window=window)
    done = b""
    first_window = 0
    parts = _stream(rng, text, 40)
    for part in parts:
        info = sess.append(part)
        done += part
        want, _ = vocab.encode(done, cfg.pattern_id)
        assert sess.ids == want.tolist(), (len(done), info)
        assert sess.off[-1] == len(done) and sess.text == done
        byte_off, _ = vocab.spans(done, want)
        assert sess.off == byte_off.tolist()
        first_window += info["attempts"] == 1 and info["window_chars"] == window
    if window == 512:
        assert first_window >= 0.8 * len(parts)        # natural text splices on the first window (the first
                                                       # appends are shorter than the window: full tokenization)


def test_matched_run_without_a_stable_boundary_can_be_wrong():
    """Digits in groups of three, single-digit tokens except one merged pair: cached and fresh records agree over
    a long run of digit tokens although the fresh window groups the digits with another phase.  Without
    condition (3) the splice takes fresh records that are not those of the full text; with it the session
    widens the window and stays exact (paper Sec. 3.3: context-dependent digit grouping defeats a matched run)."""
    merges = np.array([[ord("7"), ord("8"), 256]], dtype=np.int32)
    vocab = oracle.Vocab(merges)
    a, b = b"x " + b"123456" * 7, b"789"
    full, _ = vocab.encode(a + b, 0)
    bad = repair.Session(vocab, 0, window=20)
    bad.append(a)
    bad.append(b, check_boundary=False)
    assert bad.ids != full.tolist()                     # the unchecked splice is wrong
    good = repair.Session(vocab, 0, window=20)
    good.append(a)
    info = good.append(b)
    assert good.ids == full.tolist() and info["attempts"] > 1
