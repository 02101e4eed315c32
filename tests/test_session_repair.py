"""GPU sessions (incremental repair on append, paper Sec. 3.3) against the oracle's protocol and against a full
tokenization: after every append the stored IDs and byte offsets are those of the whole text, and the
window that was accepted, the matched run and the splice point are the ones the oracle's protocol finds."""
import random

import numpy as np
import pytest

import oracle
import workloads as wl
from oracle import repair
from gpu_util import cpu_vocab, gpu_vocab, same

pytestmark = pytest.mark.gpu


def _parts(rng, text: bytes, n_cuts: int):
    cuts = set()
    while len(cuts) < n_cuts:
        c = rng.randrange(1, len(text))
        while c < len(text) and (text[c] & 0xC0) == 0x80:
            c += 1
        if c < len(text):
            cuts.add(c)
    cuts = [0] + sorted(cuts) + [len(text)]
    return [text[a:b] for a, b in zip(cuts[:-1], cuts[1:])]


@pytest.mark.parametrize("name,window,pattern", [("C1", 512, None), ("C1", 24, None), ("C2", 64, None), ("C4", 200, None), ("C2", 48, 3), ("C2", 100, 2)])
def test_append_stream_matches_oracle_protocol_and_full_tokenization(name, window, pattern):
    import paper_2607_29678_b200 as tt
    cfg = wl.CONFIGS[name]
    pat = cfg.pattern_id if pattern is None else pattern
    gv, cv = gpu_vocab(name, pattern=pat), cpu_vocab(name)
    rng = random.Random(1000 + window)
    text = wl.generate(cfg.kind, 99 + window, 9000).tobytes()
    text = text + "é中 1234567890123 x's's's tail   \n\n  end GPU加速 done".encode() * 3
    sess = tt.Session(gv, len(text) + 16, window_chars=window)
    ref = repair.Session(cv, pat, window=window)
    done = b""
    for part in _parts(rng, text, 30):
        info = sess.append(part)
        want_info = ref.append(part)
        done += part
        ids, off, nbytes = sess.records()
        full, _ = cv.encode(done, pat)
        assert nbytes == len(done) and info["status"] == 0 and info["n_tokens"] == full.size
        assert same(ids.cpu().numpy(), full)
        assert off.cpu().numpy().tolist() == ref.off
        for key in ("attempts", "window_chars", "window_start", "run_tokens", "splice_byte"):
            assert info[key] == want_info[key], (key, info, want_info, len(done))


def test_digit_run_without_stable_boundary_is_not_spliced():
    """The counterexample of the oracle's pins on the GPU: single-digit tokens, one merged pair, a window that
    groups the digits with another phase.  The session must widen and stay exact."""
    import paper_2607_29678_b200 as tt
    merges = np.array([[ord("7"), ord("8"), 256]], dtype=np.int32)
    gv, cv = tt.Vocab(merges, None, 0), oracle.Vocab(merges)
    a, b = b"x " + b"123456" * 7, b"789"
    sess = tt.Session(gv, 1024, window_chars=20)
    sess.append(a)
    info = sess.append(b)
    ids, off, _ = sess.records()
    full, _ = cv.encode(a + b, 0)
    assert same(ids.cpu().numpy(), full) and info["attempts"] > 1


def test_rejected_append_leaves_the_session_unchanged():
    import paper_2607_29678_b200 as tt
    gv, cv = gpu_vocab("C1"), cpu_vocab("C1")
    sess = tt.Session(gv, 4096, window_chars=32)
    good = "The quick brown fox jumps over the lazy dog. ".encode() * 20
    sess.append(good)
    with pytest.raises(tt.TokTierError) as err:
        sess.append(b"broken \xff\xfe bytes")
    assert err.value.code == tt.TT_ERR_INVALID_UTF8
    with pytest.raises(tt.TokTierError) as err:
        sess.append(b"x" * 8000)
    assert err.value.code == tt.TT_ERR_TOO_LARGE
    sess.append(b" And on it goes.")
    ids, _, nbytes = sess.records()
    full, _ = cv.encode(good + b" And on it goes.", 0)
    assert nbytes == len(good) + 16 and same(ids.cpu().numpy(), full)
