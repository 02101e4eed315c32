"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element, at the
level of piece boundaries and at the level of token IDs (paper Sec. 4.1: both levels are needed,
because ID agreement can hide a boundary fault).  Bit-exact is the only tolerance."""
import itertools
import random

import numpy as np
import pytest

import oracle
import workloads as wl
from gpu_util import cpu_vocab, first_difference, gpu_encode, gpu_encode_batch, gpu_pretok, gpu_vocab, same

pytestmark = pytest.mark.gpu

TILE = 4096


def _expect_pieces(text, pattern):
    return oracle.pretokenize(text, pattern)


@pytest.mark.parametrize("name,n_chars", [("C1", None), ("C2", None), ("C3", None), ("C4", 400_000)])
def test_piece_offsets_match_oracle(name, n_chars):
    cfg = wl.CONFIGS[name]
    text = wl.request(cfg, n_chars=n_chars)
    got, status = gpu_pretok(gpu_vocab(name), text)
    assert status == 0
    want = _expect_pieces(text, cfg.pattern_id)
    assert same(got, want)


@pytest.mark.parametrize("name,n_chars", [("C1", None), ("C2", None), ("C3", None), ("C4", 400_000)])
def test_token_ids_match_oracle(name, n_chars):
    cfg = wl.CONFIGS[name]
    text = wl.request(cfg, n_chars=n_chars)
    ids, status = gpu_encode(gpu_vocab(name), text)
    assert status == 0
    want, _ = cpu_vocab(name).encode(text, cfg.pattern_id, nthreads=4)
    assert same(ids, want)


@pytest.mark.parametrize("pattern", [0, 1])
@pytest.mark.parametrize("offset", [0, 1, 7, 15])
def test_misaligned_text_pointer(pattern, offset):
    name = "C2" if pattern == 0 else "C4"
    text = wl.generate(wl.KIND_MIX_UNI, 77 + offset, 30_000)
    got, status = gpu_pretok(gpu_vocab(name), text, offset=offset)
    assert status == 0 and same(got, _expect_pieces(text, pattern))
    ids, status = gpu_encode(gpu_vocab(name), text, offset=offset)
    want, _ = cpu_vocab(name).encode(text, pattern)
    assert status == 0 and same(ids, want)


def _alphabet_docs(alphabet, maxlen):
    docs = []
    for ln in range(1, maxlen + 1):
        for tup in itertools.product(alphabet, repeat=ln):
            docs.append("".join(tup).encode("utf-8"))
    return docs


def _batch_pieces_check_arrays(name, pattern, text, off):
    """One tt_pretokenize call over a batch of documents against the oracle matching every document alone."""
    got, status = gpu_pretok(gpu_vocab(name), text, doc_off=off)
    assert status == 0
    want = oracle.pretokenize_batch(text, off, pattern, nthreads=8)
    if not same(got, want):
        bad = np.setxor1d(got, want)[:5]
        which = sorted({int(np.searchsorted(off, b, side="right") - 1) for b in bad})
        raise AssertionError(f"piece mismatch in documents {[text[off[w]:off[w + 1]].tobytes() for w in which]}")


def _batch_pieces_check(name, pattern, docs):
    text = np.frombuffer(b"".join(docs), dtype=np.uint8)
    off = np.zeros(len(docs) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(d) for d in docs])
    _batch_pieces_check_arrays(name, pattern, text, off)


# Exhaustive sets: every string of 1..maxlen symbols, each as its own document of ONE batch call (up to 19 million
# documents).  Alphabets and lengths are those on which the run-local rules were validated when the path was
# surveyed, plus the sets this suite had before.
@pytest.mark.parametrize("alphabet,maxlen", [
    ("asl1 \t\n\r!'", 7), ("rRevl't !", 7), ("eé中²\u0301 \u3000\u00a0\n's", 6), ("a1 \r\n\u00a0!", 6), ("as1 \t\n!'", 6)])
def test_exhaustive_small_alphabets_pattern0(alphabet, maxlen):
    _batch_pieces_check_arrays("C1", 0, *wl.exhaustive(alphabet, maxlen))


@pytest.mark.parametrize("alphabet,maxlen", [
    ("a\u0301's/\n !", 8), ("Aal's1 \n/", 7), ("Aá's !/\n", 7), ("Aa中\u0301's !/\n", 6), ("AaBb中\u03011 \t", 6),
    ("ǅaʰA'l \r", 6)])
def test_exhaustive_small_alphabets_pattern1(alphabet, maxlen):
    _batch_pieces_check_arrays("C4", 1, *wl.exhaustive(alphabet, maxlen))


SEAM_CONSTRUCTS = ["don't", "x's's's", " \n \n  x", "1234567", "é中😀²", "!!!\n\n\nabc", "a   b", "\r\n\r\n", "'re're",
                   "A中B", "HelloWORLDab", "!\n/\n/x", "x́\ny", " 　 z", "12'll3", "a\n\n\n\n\n\n\n\n\n\n\n\n\n\n\n\n\n\nb"]


@pytest.mark.parametrize("pattern", [0, 1])
def test_constructs_at_every_tile_seam_position(pattern):
    """Each construct is placed so that every one of its bytes falls on a tile boundary once."""
    name = "C2" if pattern == 0 else "C4"
    rng = random.Random(pattern)
    for cons in SEAM_CONSTRUCTS:
        cb = cons.encode("utf-8")
        docs = []
        for k in range(-4, len(cb) + 5):
            pad = TILE - k
            filler = wl.generate(wl.KIND_MIX, rng.randrange(1 << 30), TILE)[:max(pad, 0)].tobytes()
            docs.append(filler + cb + b" tail text 123\n")
        _batch_pieces_check(name, pattern, docs)


@pytest.mark.parametrize("pattern", [0, 1])
def test_long_runs_across_tiles(pattern):
    name = "C2" if pattern == 0 else "C4"
    rng = random.Random(100 + pattern)
    docs = []
    for _ in range(60):
        parts = []
        for _ in range(rng.randrange(1, 5)):
            k = rng.randrange(8)
            if k == 0:
                parts.append("7" * rng.randrange(1, 13000))
            elif k == 1:
                parts.append(rng.choice(["", "!", "a", "\n", "!\n"]) + " " * rng.randrange(1, 13000) + rng.choice(["", "x", "\n", "!", "1"]))
            elif k == 2:
                parts.append(rng.choice(["!", "a", ""]) + "\n" * rng.randrange(1, 9000) + rng.choice(["", " ", "  x", "/"]))
            elif k == 3:
                parts.append(rng.choice([";\n", "", "a"]) + rng.choice(["/", "'", "=", "-"]) * rng.randrange(1, 9000))
            elif k == 4:
                parts.append("٣" * rng.randrange(1, 5000))
            elif k == 5:
                parts.append(rng.choice(["!", "a"]) + "\r\n" * rng.randrange(1, 3000) + "\t " * rng.randrange(0, 3000) + "z")
            elif k == 6:
                parts.append("中" * rng.randrange(1, 3000) + "ABC" + "é" * rng.randrange(1, 3000))
            else:
                parts.append(" " * rng.randrange(1, 5000) + "\n" * rng.randrange(1, 5000) + " " * rng.randrange(1, 5000))
        docs.append("".join(parts).encode("utf-8"))
    _batch_pieces_check(name, pattern, docs)


@pytest.mark.parametrize("pattern", [0, 1, 2])
def test_long_runs_in_single_requests(pattern):
    """Runs that fill whole tiles, each text a request of its own (no document mask: the walks may step over whole
    slots of digits or blanks and look ahead in the raw text): digit runs with a non-ASCII digit, a letter or nothing
    in them, blank runs with tabs, form feeds, no-break and ideographic spaces, with and without a CR/LF at the far
    end, at every alignment to the 16-byte slots."""
    name = "C4" if pattern == 1 else "C2"
    gv, cv = gpu_vocab(name, pattern=pattern), cpu_vocab(name)
    rng = random.Random(300 + pattern)
    for trial in range(48):
        parts = [rng.choice(["", "x", "ab ", "é", "12 "]) + "y" * rng.randrange(0, 40)]
        for _ in range(rng.randrange(1, 4)):
            k = rng.randrange(6)
            n = rng.choice([rng.randrange(1, 300), rng.randrange(1000, 9000), rng.randrange(15000, 30000)])
            if k == 0:
                parts.append("7" * n)
            elif k == 1:                                          # a digit run with one foreign character somewhere
                cut = rng.randrange(0, n + 1)
                parts.append("3" * cut + rng.choice(["٣", "²", "a", ".", " "]) + "8" * (n - cut))
            elif k == 2:
                parts.append(rng.choice(["", "!", "a", "\n"]) + " " * n + rng.choice(["", "x", "\n", "\r\n!", "1", "\u00a0\n"]))
            elif k == 3:                                          # blanks of several kinds, a CR/LF somewhere or nowhere
                blanks = "".join(rng.choice([" ", " ", " ", "\t", "\x0c", "\x0b"]) for _ in range(min(n, 4000))) + " " * max(n - 4000, 0)
                cut = rng.randrange(0, len(blanks) + 1)
                parts.append(blanks[:cut] + rng.choice(["", "\n", "\r", "\u3000", "\u00a0", "\u2028"]) + blanks[cut:] + rng.choice(["", "z", "\n"]))
            elif k == 4:
                parts.append(" " * rng.randrange(1, 40) + "word" + "\t" * n)
            else:
                parts.append("0" * n + " " * rng.randrange(1, 5000) + "9" * rng.randrange(1, 5000))
        text = np.frombuffer("".join(parts).encode("utf-8"), dtype=np.uint8)
        want_ids, want = cv.encode(text, pattern, nthreads=4)
        got, status = gpu_pretok(gv, text)
        assert status == 0 and same(got, want[:-1]), (trial, first_difference(got, want[:-1]))
        ids, status = gpu_encode(gv, text)
        assert status == 0 and same(ids, want_ids), trial


def test_bulk_text_short_pieces_of_every_length():
    """More than 4 MB in one call (the kernels for bulk text), made of random-letter words of every length from 2 to
    40 under a small vocabulary, so that nearly every word needs merging: all the length classes of the short-piece
    lists, their boundaries, and the warp-per-piece list are filled, some of them with a single length only."""
    rng = np.random.default_rng(77)
    gv, cv = gpu_vocab("C1"), cpu_vocab("C1")
    pattern = wl.CONFIGS["C1"].pattern_id
    for lengths in (range(2, 41), (6, 7), (10, 11, 16, 17), (32, 33), (3,)):
        lengths = list(lengths)
        words = []
        total = 0
        while total < 4_400_000:
            n = lengths[int(rng.integers(0, len(lengths)))]
            w = (97 + rng.integers(0, 26, n)).astype(np.uint8)
            words.append(w); words.append(np.frombuffer(b" ", dtype=np.uint8))
            total += n + 1
        text = np.concatenate(words)
        doc_off = np.array([0, text.size // 3, text.size], dtype=np.int64)
        while text[doc_off[1]] != 32:                            # cut between words
            doc_off[1] += 1
        ids, ioff, status = gpu_encode_batch(gv, text, doc_off)
        want, woff = cv.encode_batch(text, doc_off, pattern, nthreads=8)
        assert status == 0 and same(ioff, woff) and same(ids, want), (lengths[:4], first_difference(ids, want))
        one, status = gpu_encode(gv, text)                       # the same text as one request of more than 4 MB
        assert status == 0 and same(one, cv.encode(text, pattern, nthreads=8)[0])


def test_batch_ids_match_documents_alone():
    cfg = wl.CONFIGS["C5"]
    text, off = wl.batch(cfg, n_docs=12, scale=0.02)
    off = np.concatenate([off[:5], [off[4]], off[5:]]).astype(np.int64)   # an empty document in the middle
    ids, ioff, status = gpu_encode_batch(gpu_vocab("C5"), text, off)
    assert status == 0
    want, woff = cpu_vocab("C5").encode_batch(text, off, cfg.pattern_id, nthreads=4)
    assert same(ioff, woff)
    assert same(ids, want)


def test_adversarial_long_pieces_ids():
    """64 KB blanks/tabs, 20,000 digits and 50 KB of one punctuation character (pattern 1 vocabulary)."""
    cfg = wl.CONFIGS["C4"]
    v, cv = gpu_vocab("C4"), cpu_vocab("C4")
    for piece in (b"x" + b" " * 65536 + b"y", b"\n" + b"\t" * 65536, b"9" * 20000, b";\n" + b"/" * 51200 + b"a",
                  b"'" * 51200, b"=" * 51200 + b"\n", ("中" * 3000).encode(), b" \t" * 32768):
        text = np.frombuffer(piece, dtype=np.uint8)
        ids, status = gpu_encode(v, text)
        want, _ = cv.encode(text, cfg.pattern_id)
        assert status == 0 and same(ids, want), piece[:20]


def test_edge_cases_and_status_codes():
    import paper_2607_29678_b200 as tt
    v = gpu_vocab("C1")
    ids, status = gpu_encode(v, np.zeros(0, dtype=np.uint8))
    assert status == 0 and ids.size == 0
    for one in (b"a", b" ", b"\n", b"7", b"'", "中".encode(), "😀".encode(), b"\x00"):
        ids, status = gpu_encode(v, np.frombuffer(one, dtype=np.uint8))
        want, _ = cpu_vocab("C1").encode(one, 0)
        assert status == 0 and same(ids, want)
    for bad in (b"abc\x80def", b"\xc3", b"ab\xe4\xb8", b"\xc0\xaf", b"\xed\xa0\x80", b"\xf4\x90\x80\x80", b"x" * 5000 + b"\xff"):
        ids, status = gpu_encode(v, np.frombuffer(bad, dtype=np.uint8))
        assert status == tt.TT_ERR_INVALID_UTF8 and ids.size == 0
    text = wl.request(wl.CONFIGS["C1"])
    ids, status = gpu_encode(v, text, ids_cap=10)
    assert status == tt.TT_ERR_CAPACITY and ids.size == 0
    # the handle is still usable after errors
    ids, status = gpu_encode(v, text)
    want, _ = cpu_vocab("C1").encode(text, 0)
    assert status == 0 and same(ids, want)


def test_pretokenize_capacity_rule():
    """tt_pretokenize writes n_pieces starts and one closing entry: a capacity of len + 1 is accepted, len is
    refused on the host; an empty text is accepted with no output buffer at all."""
    import torch
    import paper_2607_29678_b200 as tt
    from gpu_util import to_dev
    v = gpu_vocab("C1")
    text = np.frombuffer(b"a b c d", dtype=np.uint8)            # 7 bytes
    d = to_dev(text)
    bufs = v.alloc(text.size)
    npc = torch.zeros(1, dtype=torch.int64, device="cuda")
    po = torch.full((text.size + 1,), -1, dtype=torch.int32, device="cuda")
    v.pretokenize(d, po, npc, bufs)
    torch.cuda.synchronize()
    n = int(npc.item())
    want = oracle.pretokenize(text, 0)
    assert same(po[:n].cpu().numpy(), want) and int(po[n].item()) == text.size
    with pytest.raises(tt.TokTierError) as err:
        v.pretokenize(d, po[:text.size], npc, bufs)
    assert err.value.code == tt.TT_ERR_ARG
    empty = torch.zeros(0, dtype=torch.uint8, device="cuda")
    v.pretokenize(empty, torch.zeros(0, dtype=torch.int32, device="cuda"), npc, bufs)
    torch.cuda.synchronize()
    assert int(npc.item()) == 0 and int(bufs["status"].item()) == 0


def test_whole_piece_table_holds_exactly_the_self_encoding_entries():
    """tt_vocab_table_entries against the oracle: an entry of 2..24 bytes belongs to the whole-piece table exactly if
    the oracle's BPE of its own bytes is that one entry (the library decides this with its merge kernel at load)."""
    for name in ("C1", "C2"):
        cv = cpu_vocab(name)
        want = 0
        for r in range(cv.n_merges):
            t = cv.token_bytes(256 + r)
            if 2 <= len(t) <= 24:
                ids = cv.bpe(t, 0)
                want += int(ids.size == 1 and ids[0] == 256 + r)
        assert gpu_vocab(name).table_entries() == want


@pytest.mark.parametrize("pattern", [0, 1])
def test_every_ascii_code_in_random_strings(pattern):
    """Strings over all 128 ASCII codes (control characters included), many of them aligned so that whole 16-byte
    chunks are ASCII: the table-free classification of such chunks against the oracle's class table, through the
    piece boundaries and the ids."""
    rng = random.Random(900 + pattern)
    name = "C2" if pattern == 0 else "C4"
    docs = []
    for _ in range(3000):
        n = rng.choice([1, 5, 16, 17, 31, 32, 48, 100, 333])
        docs.append(bytes(rng.randrange(128) for _ in range(n)))
    docs.append(bytes(range(128)) * 3)
    text = np.frombuffer(b"".join(docs), dtype=np.uint8)
    off = np.zeros(len(docs) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(d) for d in docs])
    _batch_pieces_check_arrays(name, pattern, text, off)
    ids, ioff, status = gpu_encode_batch(gpu_vocab(name), text, off)
    want, woff = cpu_vocab(name).encode_batch(text, off, pattern, nthreads=8)
    assert status == 0 and same(ioff, woff) and same(ids, want)
    one, status = gpu_encode(gpu_vocab(name), text, offset=5)
    want1, _ = cpu_vocab(name).encode(text, pattern, nthreads=8)
    assert status == 0 and same(one, want1)


def test_host_wrapper_and_non_identity_ids():
    import paper_2607_29678_b200 as tt
    rng = random.Random(4)
    perm = list(range(256))
    rng.shuffle(perm)
    byte_map = np.array([5000 + p for p in perm], dtype=np.int32)
    base, _ = wl.load_vocab(wl.CONFIGS["C1"])
    remap = {i: int(byte_map[i]) for i in range(256)}
    remap.update({256 + r: 100_000 + 3 * r for r in range(base.shape[0])})
    merges = np.array([[remap[a], remap[b], remap[c]] for a, b, c in base.tolist()], dtype=np.int32)
    gv = tt.Vocab(merges, byte_map, 0)
    cv = oracle.Vocab(merges, byte_map)
    text = wl.request(wl.CONFIGS["C1"])
    want, _ = cv.encode(text, 0)
    assert same(gv.encode_host(text), want)
    ids, status = gpu_encode(gv, text)
    assert status == 0 and same(ids, want)


def test_result_does_not_depend_on_schedule():
    """Same input, repeated calls and a reused workspace: identical output every time."""
    import torch
    cfg = wl.CONFIGS["C2"]
    v = gpu_vocab("C2")
    text = wl.request(cfg)
    from gpu_util import to_dev
    d = to_dev(text)
    bufs = v.alloc(text.size)
    outs = []
    for _ in range(3):
        v.encode(d, bufs)
        torch.cuda.synchronize()
        outs.append(bufs["ids"][:int(bufs["count"].item())].cpu().numpy().copy())
    assert same(outs[0], outs[1]) and same(outs[0], outs[2])


def test_full_size_c4_ids_and_pieces():
    """The whole 3,000,000-char adversarial request of config C4 (pattern 1, 199,744 merges)."""
    cfg = wl.CONFIGS["C4"]
    text = wl.request(cfg)
    got, status = gpu_pretok(gpu_vocab("C4"), text)
    assert status == 0 and same(got, _expect_pieces(text, 1))
    ids, status = gpu_encode(gpu_vocab("C4"), text)
    want, _ = cpu_vocab("C4").encode(text, 1, nthreads=8)
    assert status == 0 and same(ids, want)


def test_full_size_c5_batch_every_document():
    """One tt_encode_batch call over the full 256-request batch of config C5, in the configuration the
    benchmark times: the ids and the token offsets of every document against the oracle encoding each
    document alone, element by element."""
    cfg = wl.CONFIGS["C5"]
    text, off = wl.batch(cfg)
    assert off.size - 1 == 256
    ids, ioff, status = gpu_encode_batch(gpu_vocab("C5"), text, off)
    assert status == 0
    want, woff = cpu_vocab("C5").encode_batch(text, off, cfg.pattern_id, nthreads=16)
    assert same(ioff, woff), first_difference(ioff, woff)
    assert same(ids, want), first_difference(ids, want)
    # decode(encode(x)) == x on one document, through the vocabulary's byte strings
    d = 64
    assert cpu_vocab("C5").decode(ids[ioff[d]:ioff[d] + 2000]) == text[off[d]:off[d + 1]].tobytes()[:len(cpu_vocab("C5").decode(ids[ioff[d]:ioff[d] + 2000]))]


def _random_wellformed_merges(rng, n_merges, alphabet):
    ids = list(alphabet)
    seen, rows = set(), []
    while len(rows) < n_merges:
        p = (rng.choice(ids), rng.choice(ids))
        if p in seen:
            continue
        seen.add(p)
        rows.append((p[0], p[1], 256 + len(rows)))
        ids.append(256 + len(rows) - 1)
    return np.array(rows, dtype=np.int32)


@pytest.mark.parametrize("seed,n_merges,alpha", [(1, 6, "ab"), (2, 40, "abc"), (3, 300, "abcd"), (4, 2000, "ab"), (5, 25, "a")])
def test_merge_kernels_on_random_tables(seed, n_merges, alpha):
    """Random well-formed merge tables over tiny alphabets (dense in repeated pairs and equal-token runs)
    and letter-only documents of every length class: <= 32 bytes (registers), <= 64 and <= 256 (warp),
    longer (CTA, shared memory and global scratch).  Each document is one piece under pattern 0."""
    import paper_2607_29678_b200 as tt
    rng = random.Random(seed)
    merges = _random_wellformed_merges(rng, n_merges, [ord(c) for c in alpha])
    gv = tt.Vocab(merges, None, 0)
    cv = oracle.Vocab(merges)
    lens = list(range(1, 70)) + [100, 128, 129, 200, 255, 256, 257, 300, 511, 1000, 2047, 2048, 2049, 4095, 4096, 4097, 5000, 9000, 20000]
    docs = [bytes(rng.choice(alpha.encode()) for _ in range(n)) for n in lens for _ in range(3)]
    text = np.frombuffer(b"".join(docs), dtype=np.uint8)
    off = np.zeros(len(docs) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(d) for d in docs])
    ids, ioff, status = gpu_encode_batch(gv, text, off)
    assert status == 0
    for k, d in enumerate(docs):
        want = cv.bpe(d, 2)
        got = ids[ioff[k]:ioff[k + 1]]
        assert same(got, want), (len(d), d[:40])


def test_single_digit_pattern_variant():
    """TT_PATTERN_CL100K_N1: pieces on exhaustive strings with digits, ids on config C2's text."""
    import paper_2607_29678_b200 as tt
    cfg = wl.CONFIGS["C2"]
    merges, byte_map = wl.load_vocab(cfg)
    gv = tt.Vocab(merges, byte_map, tt.TT_PATTERN_CL100K_N1)
    docs = _alphabet_docs("a12 \t\n!'", 5) + _alphabet_docs("1²٣ a.", 5)
    text = np.frombuffer(b"".join(docs), dtype=np.uint8)
    off = np.zeros(len(docs) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(d) for d in docs])
    got, status = gpu_pretok(gv, text, doc_off=off)
    want = np.concatenate([oracle.pretokenize(d, 2) + off[i] for i, d in enumerate(docs)])
    assert status == 0 and same(got, want)
    big = wl.request(cfg)
    ids, status = gpu_encode(gv, big)
    want_ids, _ = cpu_vocab("C2").encode(big, 2, nthreads=4)
    assert status == 0 and same(ids, want_ids)


@pytest.mark.parametrize("pattern", [0, 1, 2])
def test_random_unicode_documents(pattern):
    """Documents of random code points from every plane (plus the ASCII constructs the rules care about),
    each encoded as its own document of one batch call: piece boundaries against the oracle."""
    import paper_2607_29678_b200 as tt
    rng = random.Random(2024 + pattern)
    merges, byte_map = wl.load_vocab(wl.CONFIGS["C1"])
    gv = tt.Vocab(merges, byte_map, pattern)
    special = list(" \t\n\r'/!.,1aZ") + ["'s", "'re", "'LL", "\r\n", "  ", "\n\n", "12345", "́", "　", " "]
    ranges = [(0x20, 0x7F), (0xA0, 0x250), (0x300, 0x370), (0x370, 0x530), (0x600, 0x700), (0x900, 0xA00), (0x2000, 0x2070),
              (0x3000, 0x3100), (0x4E00, 0x4F00), (0xAC00, 0xAD00), (0xFF00, 0xFFF0), (0x1D400, 0x1D500), (0x1F300, 0x1F700)]
    docs = []
    for _ in range(6000):
        n = rng.randrange(1, 60)
        parts = []
        for _ in range(n):
            if rng.random() < 0.45:
                parts.append(rng.choice(special))
            else:
                lo, hi = rng.choice(ranges)
                parts.append(chr(rng.randrange(lo, hi)))
        docs.append("".join(parts).encode("utf-8"))
    text = np.frombuffer(b"".join(docs), dtype=np.uint8)
    off = np.zeros(len(docs) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(d) for d in docs])
    got, status = gpu_pretok(gv, text, doc_off=off)
    assert status == 0
    want = np.concatenate([oracle.pretokenize(d, pattern) + off[i] for i, d in enumerate(docs)])
    if not same(got, want):
        bad = sorted(set(got.tolist()) ^ set(want.tolist()))[:3]
        which = [int(np.searchsorted(off, b, side="right") - 1) for b in bad]
        raise AssertionError(f"piece mismatch in documents {[docs[w] for w in which]}")


def test_cjk_latin_mixtures_in_long_documents():
    """Pattern 1 on caseless-script text with glued upper/lower-case words, marks and contraction chains,
    in documents far longer than a tile: the case-boundary decisions taken from the class masks, the
    sparse matcher behind them and its search for the document end (long pieces next to unresolved
    constructs, documents that end inside such pieces).  Piece boundaries and IDs against the oracle."""
    rng = random.Random(4242)
    atoms = ["中", "文", "使用", "手机", "A", "B", "GPU", "App", "iPhone", "a", "word", "'", "'s", "'T", " ", "  ", "，", "。",
             "!", "!!", "/", "\n", "1", "2024", "́", "é", "É", "ǅ", "ʰ", "\t", "x's's's"]
    w = [10, 10, 5, 5, 5, 3, 3, 2, 2, 3, 2, 1, 1, 1, 2, 1, 2, 1, 0.5, 0.5, 0.5, 0.5, 1, 0.5, 0.2, 1, 1, 0.3, 0.3, 0.3, 0.2]
    long_runs = ["中", " ", "A", "a", "9", "\n", "=", "文B", " \t"]
    docs = []
    for _ in range(40):
        parts = []
        for _ in range(rng.randrange(200, 4000)):
            if rng.random() < 0.004:
                parts.append(rng.choice(long_runs) * rng.randrange(40, 6000))
            else:
                parts.append(rng.choices(atoms, w)[0])
        docs.append("".join(parts).encode("utf-8"))
    _batch_pieces_check("C4", 1, docs)
    text = np.frombuffer(b"".join(docs), dtype=np.uint8)
    off = np.zeros(len(docs) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(d) for d in docs])
    ids, ioff, status = gpu_encode_batch(gpu_vocab("C4"), text, off)
    want, woff = cpu_vocab("C4").encode_batch(text, off, 1, nthreads=8)
    assert status == 0 and same(ioff, woff) and same(ids, want)


@pytest.mark.parametrize("kind", ["marks", "thai"])
@pytest.mark.parametrize("pattern", [0, 1])
def test_mark_dense_text_without_blanks(kind, pattern):
    """Text whose words are glued and carry a combining mark every second or third letter, and Thai-like text
    (caseless consonants with vowel signs and tone marks, a blank only between phrases): under pattern 1 nearly every
    piece holds unresolved constructs, so the sparse sequential path decides most of the text.  Pieces and ids
    against the oracle: one 1,000,000-char text, a misaligned copy of a part of it, and a batch of documents."""
    name = "C2" if pattern == 0 else "C4"
    k = wl.KIND_MARKS if kind == "marks" else wl.KIND_THAI
    text = wl.generate(k, 11, 1_000_000)
    got, status = gpu_pretok(gpu_vocab(name), text)
    assert status == 0 and same(got, _expect_pieces(text, pattern))
    ids, status = gpu_encode(gpu_vocab(name), text)
    want, _ = cpu_vocab(name).encode(text, pattern, nthreads=16)
    assert status == 0 and same(ids, want)
    part = text[:200_000]
    while (part[-1] & 0xC0) == 0x80 or part[-1] >= 0xC0:            # end on a character boundary
        part = part[:-1]
    ids, status = gpu_encode(gpu_vocab(name), part, offset=9)
    want, _ = cpu_vocab(name).encode(part, pattern, nthreads=8)
    assert status == 0 and same(ids, want)
    docs = [wl.generate(k, 100 + d, 200 + 97 * d).tobytes() for d in range(60)]
    _batch_pieces_check(name, pattern, docs)
    btext = np.frombuffer(b"".join(docs), dtype=np.uint8)
    off = np.zeros(len(docs) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(d) for d in docs])
    ids, ioff, status = gpu_encode_batch(gpu_vocab(name), btext, off)
    want, woff = cpu_vocab(name).encode_batch(btext, off, pattern, nthreads=8)
    assert status == 0 and same(ioff, woff) and same(ids, want)


@pytest.mark.parametrize("pattern", [0, 1])
def test_unresolved_constructs_before_long_plain_runs(pattern):
    """A mark, a caseless letter before an upper-case one, or a chain of contraction suffixes, followed at once (or after
    a few characters) by hundreds to thousands of bytes of one plain class (blanks, tabs, line feeds, one punctuation
    character, digits, slashes, apostrophes) and then by a tail that the rules have to place: whatever the construct
    turns out to be must not reach the pieces far inside or behind the run.  Piece boundaries and ids per document."""
    name = "C2" if pattern == 0 else "C4"
    rng = random.Random(5150 + pattern)
    heads = ["x\u0301", "!\u0301", "\u0301", "中A", "x's's's", "a'", "É\u0301'", "1\u0301", " \u0301", "word", "'s", "A\u0301B"]
    mids = ["", " ", "!", "\n", "a", "'", "/"]
    runs = [" ", "\t", " \t", "\n", "\r\n", "=", "*", "'", "/", "9", "!\n", " \n", "\u3000"]
    tails = ["abc", "A", "\u0301x", "\n", "'s", " x", "  x", "1", "!", "/a", "", "aB", "中"]
    docs = []
    for _ in range(700):
        n = rng.choice([230, 260, 500, 2049, 2300, 4500, 9000])
        run = rng.choice(runs)
        docs.append((rng.choice(["", "lead in. ", "xy\n"]) + rng.choice(heads) + rng.choice(mids) + run * (n // len(run)) + rng.choice(tails)
                     + rng.choice(["", " end", "\n"])).encode("utf-8"))
    _batch_pieces_check(name, pattern, docs)
    text = np.frombuffer(b"".join(docs), dtype=np.uint8)
    off = np.zeros(len(docs) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(d) for d in docs])
    ids, ioff, status = gpu_encode_batch(gpu_vocab(name), text, off)
    want, woff = cpu_vocab(name).encode_batch(text, off, pattern, nthreads=8)
    assert status == 0 and same(ioff, woff) and same(ids, want)
    # and as one text: the documents glued together, so that a run can follow whatever the document before left
    got, status = gpu_pretok(gpu_vocab(name), text)
    assert status == 0 and same(got, _expect_pieces(text, pattern))


def test_bulk_text_of_pieces_outside_the_vocabulary():
    """Megabytes of random words (Latin and CJK, 2..80 bytes) that are no vocabulary entries: every CTA
    handles many tiles and its piece queues fill and empty many times (thread-per-piece and warp-per-piece
    merges in bulk).  IDs against the oracle."""
    rng = random.Random(777)
    parts, size = [], 0
    while size < 6_000_000:
        k = rng.random()
        if k < 0.45:
            w = " " + "".join(rng.choice("abcdefghijklmnopqrstuvwxyzABCDE") for _ in range(rng.randrange(1, 70)))
        elif k < 0.9:
            w = "，" + "".join(chr(rng.randrange(0x4E00, 0x9FA5)) for _ in range(rng.randrange(1, 26)))
        elif k < 0.95:
            w = " the quick brown fox\n"
        else:
            w = str(rng.randrange(10 ** rng.randrange(1, 40)))
        parts.append(w)
        size += len(w)
    text = np.frombuffer("".join(parts).encode("utf-8"), dtype=np.uint8)
    for name in ("C4", "C3"):
        cfg = wl.CONFIGS[name]
        ids, status = gpu_encode(gpu_vocab(name), text)
        want, _ = cpu_vocab(name).encode(text, cfg.pattern_id, nthreads=16)
        assert status == 0 and same(ids, want), name


@pytest.mark.parametrize("pattern", [0, 1])
def test_whitespace_lookahead_past_the_tile_single_document(pattern):
    """A blank run that begins near the end of a 2 KiB tile and runs past the kernel's look-ahead window, as
    ONE document (no boundary mask): the raw-byte look-ahead for a later CR/LF, its give-up cases (non-ASCII
    whitespace, non-ASCII non-whitespace, very long runs) and the end of the text."""
    name = "C2" if pattern == 0 else "C4"
    rng = random.Random(31 + pattern)
    tails = ["x", "\n", "\r\n", "é", "　\n", "　x", " ", "", "1", "!", "\t\n", "\x0b\x0c z"]
    for case in range(120):
        lead_len = 2048 * rng.randrange(1, 4) - rng.randrange(0, 40)
        filler = wl.generate(wl.KIND_MIX, rng.randrange(1 << 30), lead_len)[:lead_len].tobytes()
        filler = filler[:len(filler) - 1].decode("utf-8", errors="ignore").encode("utf-8")
        run = rng.choice([" ", "\t", " \t"]) * rng.choice([1, 5, 17, 40, 130, 300, 700])
        doc = filler + b"a\n" + run.encode() + rng.choice(tails).encode("utf-8") + rng.choice([b"", b" tail\n"])
        text = np.frombuffer(doc, dtype=np.uint8)
        got, status = gpu_pretok(gpu_vocab(name), text)
        assert status == 0 and same(got, _expect_pieces(text, pattern)), (case, doc[-60:])


def test_ignore_merges_whole_piece_rule():
    """TT_VOCAB_IGNORE_MERGES (paper Sec. 4.2): the hand-worked examples, random merge tables over tiny
    alphabets (where many pieces are entries that the merge loop would encode differently, including entries
    longer than 24 bytes) and a stored vocabulary on its config's text; IDs against the oracle with the same
    rule, and the rule must actually change some results."""
    import json
    import os
    import paper_2607_29678_b200 as tt
    with open(os.path.join(os.path.dirname(__file__), "golden", "ignore_merges_examples.jsonl"), encoding="utf-8") as f:
        for line in f:
            d = json.loads(line)
            if "piece" not in d:
                continue
            pairs = np.asarray(d["merges"], dtype=np.int32)
            merges = np.concatenate([pairs, 256 + np.arange(len(pairs), dtype=np.int32)[:, None]], axis=1)
            text = np.frombuffer(d["piece"].encode(), dtype=np.uint8)
            for ign, key in ((False, "plain"), (True, "ignore")):
                ids, status = gpu_encode(tt.Vocab(merges, None, 0, ignore_merges=ign), text)
                assert status == 0 and ids.tolist() == d[key], (d, key)
    differs = 0
    refused = 0
    for seed, n_merges, alpha in [(11, 60, "ab"), (12, 400, "abc"), (13, 3000, "ab"), (14, 150, "ab")]:
        rng = random.Random(seed)
        merges = _random_wellformed_merges(rng, n_merges, [ord(c) for c in alpha])
        cv, plain = oracle.Vocab(merges, ignore_merges=True), oracle.Vocab(merges)
        entries = {cv.token_bytes(int(r)) for r in merges[:, 2]}
        if max(len(e) for e in entries) > 4096:                                  # beyond the documented limit: refused
            with pytest.raises(tt.TokTierError) as err:
                tt.Vocab(merges, None, 0, ignore_merges=True)
            assert err.value.code == tt.TT_ERR_BAD_VOCAB
            refused += 1
            continue
        gv = tt.Vocab(merges, None, 0, ignore_merges=True)
        docs = [bytes(rng.choice(alpha.encode()) for _ in range(n)) for n in list(range(1, 70)) * 3 + [100, 300, 5000]]
        docs += rng.sample(sorted(entries), min(len(entries), 300))              # entries themselves, of any length
        text = np.frombuffer(b"".join(docs), dtype=np.uint8)
        off = np.zeros(len(docs) + 1, dtype=np.int64)
        off[1:] = np.cumsum([len(d) for d in docs])
        ids, ioff, status = gpu_encode_batch(gv, text, off)
        assert status == 0
        for k, d in enumerate(docs):
            want = cv.bpe(d, 2)
            assert same(ids[ioff[k]:ioff[k + 1]], want), (seed, len(d), d[:40])
            differs += not same(want, plain.bpe(d, 2))
        assert max(len(e) for e in entries) > 24
    assert differs > 20 and refused == 1
    cfg = wl.CONFIGS["C2"]
    merges, byte_map = wl.load_vocab(cfg)
    text = wl.request(cfg)
    ids, status = gpu_encode(tt.Vocab(merges, byte_map, cfg.pattern_id, ignore_merges=True), text)
    want, _ = oracle.Vocab(merges, byte_map, ignore_merges=True).encode(text, cfg.pattern_id, nthreads=4)
    assert status == 0 and same(ids, want)


def test_three_splitter_composition():
    """TT_PATTERN_SPLIT3 (paper Sec. 4.1: three splitters in sequence): piece boundaries and IDs against the
    oracle's pattern 3 -- exhaustive small alphabets and random Unicode documents in one batch, long digit and
    caseless runs across tiles, a CJK-heavy request as one document."""
    import paper_2607_29678_b200 as tt
    merges, byte_map = wl.load_vocab(wl.CONFIGS["C2"])
    gv = tt.Vocab(merges, byte_map, tt.TT_PATTERN_SPLIT3)
    cv = cpu_vocab("C2")
    rng = random.Random(33)
    docs = _alphabet_docs("a1中 ", 6) + _alphabet_docs("1中x' \n", 5) + _alphabet_docs("12 !文a\t", 5)
    for _ in range(300):
        parts = []
        for _ in range(rng.randrange(1, 6)):
            k = rng.randrange(6)
            if k == 0:
                parts.append("7" * rng.randrange(1, 9000))
            elif k == 1:
                parts.append("中" * rng.randrange(1, 3000))
            elif k == 2:
                parts.append(" " * rng.randrange(1, 3000) + rng.choice(["1", "中", "x", ""]))
            elif k == 3:
                parts.append(rng.choice(["abc", "x's", "!!", "\n\n", "٣٣٣٣"]) * rng.randrange(1, 50))
            elif k == 4:
                parts.append("".join(rng.choice("ab12中文 \n'!") for _ in range(rng.randrange(1, 200))))
            else:
                parts.append("12中34文56 x")
        docs.append("".join(parts).encode("utf-8"))
    text = np.frombuffer(b"".join(docs), dtype=np.uint8)
    off = np.zeros(len(docs) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(d) for d in docs])
    got, status = gpu_pretok(gv, text, doc_off=off)
    want = np.concatenate([oracle.pretokenize(d, 3) + off[i] for i, d in enumerate(docs)])
    assert status == 0
    if not same(got, want):
        bad = sorted(set(got.tolist()) ^ set(want.tolist()))[:3]
        which = [int(np.searchsorted(off, b, side="right") - 1) for b in bad]
        raise AssertionError(f"piece mismatch in documents {[docs[w][:80] for w in which]}")
    ids, ioff, status = gpu_encode_batch(gv, text, off)
    want_ids, woff = cv.encode_batch(text, off, 3, nthreads=8)
    assert status == 0 and same(ioff, woff) and same(ids, want_ids)
    big = wl.generate(wl.KIND_TRANSCRIPT_ADV, 77, 300_000)
    ids, status = gpu_encode(gv, big, offset=3)
    want_ids, _ = cv.encode(big, 3, nthreads=8)
    assert status == 0 and same(ids, want_ids)


def test_host_entry_point_with_pinned_buffers():
    """tt_encode_host on page-locked caller buffers: no staging, ids written by the kernel into the caller's buffer."""
    import torch
    cfg = wl.CONFIGS["C2"]
    text = wl.request(cfg)
    gv, cv = gpu_vocab("C2"), cpu_vocab("C2")
    want, _ = cv.encode(text, cfg.pattern_id, nthreads=4)
    pinned_text = torch.from_numpy(text.copy()).pin_memory()
    pinned_ids = torch.full((text.size + 1,), -7, dtype=torch.int32).pin_memory()
    for _ in range(2):
        n = gv.encode_host_into(pinned_text, pinned_ids)
        assert n == want.size and same(pinned_ids[:n].numpy(), want)
    out = np.empty(text.size, dtype=np.int32)                     # pinned in, pageable out
    n = gv.encode_host_into(pinned_text, out)
    assert n == want.size and same(out[:n], want)
    n = gv.encode_host_into(text, pinned_ids)                     # pageable in, pinned out
    assert n == want.size and same(pinned_ids[:n].numpy(), want)
    # more than 4 MB of pinned text takes the kernels for bulk text
    big_cfg = wl.CONFIGS["C3"]
    big = np.concatenate([wl.request(big_cfg, sample=s) for s in range(5)])
    gb, cb = gpu_vocab("C3"), cpu_vocab("C3")
    want_big, _ = cb.encode(big, big_cfg.pattern_id, nthreads=8)
    pinned_big = torch.from_numpy(big).pin_memory()
    ids_big = torch.empty(big.size, dtype=torch.int32).pin_memory()
    n = gb.encode_host_into(pinned_big, ids_big)
    assert n == want_big.size and same(ids_big[:n].numpy(), want_big)
    small = torch.empty(10, dtype=torch.int32).pin_memory()       # too small: capacity error, nothing written past it
    import paper_2607_29678_b200 as tt
    with pytest.raises(tt.TokTierError) as err:
        gv.encode_host_into(pinned_text, small)
    assert err.value.code == tt.TT_ERR_CAPACITY


def test_host_entry_point_pinned_views_all_patterns():
    """Pinned caller buffers as views into a larger pinned allocation: several byte alignments, a text that ends
    exactly at the end of the allocation and one that starts at its first byte, every pattern, CJK and adversarial
    runs, changing contents of the same buffer, invalid UTF-8."""
    import torch
    import paper_2607_29678_b200 as tt
    merges, byte_map = wl.load_vocab(wl.CONFIGS["C4"])
    cv = cpu_vocab("C4")
    body = wl.generate(wl.KIND_TRANSCRIPT_ADV, 4242, 150_000)

    def cut(n):                                                   # the largest length <= n that ends on a character boundary
        while n < body.size and (body[n] & 0xC0) == 0x80:
            n -= 1
        return n

    pinned = torch.empty(body.size + 64, dtype=torch.uint8).pin_memory()
    ids = torch.empty(body.size + 64, dtype=torch.int32).pin_memory()
    for pattern in (0, 1, 2, 3):
        gv = tt.Vocab(merges, byte_map, pattern)
        for off in (0, 1, 5, 15, 16, 33):
            n_text = cut(body.size - 7) if off == 5 else body.size
            view = pinned[off:off + n_text]
            view.copy_(torch.from_numpy(body[:n_text].copy()))
            want, _ = cv.encode(body[:n_text], pattern, nthreads=8)
            n = gv.encode_host_into(view, ids)
            assert n == want.size and same(ids[:n].numpy(), want), (pattern, off)
        # the text ends with the allocation; then a short text at its very start
        n_tail = cut(5000)
        tail = pinned[pinned.numel() - n_tail:]
        tail.copy_(torch.from_numpy(body[:n_tail].copy()))
        want, _ = cv.encode(body[:n_tail], pattern, nthreads=2)
        n = gv.encode_host_into(tail, ids)
        assert n == want.size and same(ids[:n].numpy(), want)
        head = pinned[:3]
        head.copy_(torch.from_numpy(np.frombuffer(b"a b", dtype=np.uint8).copy()))
        want, _ = cv.encode(np.frombuffer(b"a b", dtype=np.uint8), pattern)
        n = gv.encode_host_into(head, ids)
        assert n == want.size and same(ids[:n].numpy(), want)
    # invalid UTF-8 in pinned text is reported, not tokenized
    gv = tt.Vocab(merges, byte_map, 0)
    bad = pinned[:cut(1000)]
    bad.copy_(torch.from_numpy(body[:cut(1000)].copy()))
    bad[500] = 0xFF
    with pytest.raises(tt.TokTierError) as err:
        gv.encode_host_into(bad, ids)
    assert err.value.code == tt.TT_ERR_INVALID_UTF8


def test_repeated_calls_on_the_same_buffers():
    """The same buffers used for call after call: the results must follow the current contents of the text
    buffer, another length in the same buffers must work, and many buffer sets in rotation too."""
    import torch
    cfg = wl.CONFIGS["C2"]
    gv, cv = gpu_vocab("C2"), cpu_vocab("C2")
    texts = [wl.request(cfg, sample=s) for s in range(3)]
    n = min(t.size for t in texts) - 8
    texts = [np.frombuffer(t[:n].tobytes().decode("utf-8", errors="ignore").encode("utf-8"), dtype=np.uint8) for t in texts]
    n = min(t.size for t in texts)
    texts = [t[:n] if (t[n - 1] < 0x80) else t[:n] for t in texts]
    want = [cv.encode(t, cfg.pattern_id, nthreads=4)[0] for t in texts]
    dev = torch.zeros(n + 64, dtype=torch.uint8, device="cuda")
    bufs = gv.alloc(n)
    for rep in range(3):
        for t, w in zip(texts, want):
            if t.size != n:
                continue
            dev[:n].copy_(torch.from_numpy(t.copy()))
            gv.encode(dev[:n], bufs)
            torch.cuda.synchronize()
            k = int(bufs["count"].item())
            assert int(bufs["status"].item()) == 0 and same(bufs["ids"][:k].cpu().numpy(), w)
    # same buffers, other length
    half = texts[0][: n // 2]
    half = np.frombuffer(half.tobytes().decode("utf-8", errors="ignore").encode("utf-8"), dtype=np.uint8)
    dev[:half.size].copy_(torch.from_numpy(half.copy()))
    for _ in range(3):
        gv.encode(dev[:half.size], bufs)
        torch.cuda.synchronize()
        k = int(bufs["count"].item())
        assert same(bufs["ids"][:k].cpu().numpy(), cv.encode(half, cfg.pattern_id)[0])
    # many argument sets, each used three times in rotation
    sets = [(torch.from_numpy(texts[0].copy()).cuda(), gv.alloc(n)) for _ in range(20)]
    for rep in range(3):
        for d, b in sets:
            gv.encode(d, b)
        torch.cuda.synchronize()
        for d, b in sets:
            k = int(b["count"].item())
            assert same(b["ids"][:k].cpu().numpy(), want[0])


@pytest.mark.parametrize("pattern", [0, 1])
def test_apostrophe_chains(pattern):
    """Contraction suffixes in chains (x's's, 'it's', he'll've, quotes around words): pattern 1 decides them along
    the chain of apostrophes, pattern 0 treats every suffix as a piece of its own.  Random strings of such atoms
    as one text (several alignments) and as a batch of documents; long chains beyond the resolver's bound."""
    rng = random.Random(31 + pattern)
    gv, cv = gpu_vocab("C4", pattern=pattern), cpu_vocab("C4")
    atoms = ["'", "'s", "'t", "'re", "'ve", "'ll", "'LL", "'S", "'d", "'m", "a", "x", "It", "word", "中", "é", "É", "Ab", "AB",
             " ", "  ", "\n", "1", ",", ".", "''", "\"", "́", "he", "don", "I"]
    docs = []
    for k in range(600):
        docs.append("".join(rng.choice(atoms) for _ in range(rng.randrange(0, rng.choice([5, 60, 600])))).encode())
    for k in range(1, 24):
        for unit in ("'s", "'re", "x's", "'ll", "a'"):
            docs.append(("x" + unit * k + "y").encode())
    text = np.frombuffer(b"".join(docs), dtype=np.uint8)
    off = np.zeros(len(docs) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(d) for d in docs])
    ids, ioff, status = gpu_encode_batch(gv, text, off)
    want, woff = cv.encode_batch(text, off, pattern, nthreads=8)
    assert status == 0 and same(ioff, woff) and same(ids, want)
    want1, _ = cv.encode(text, pattern, nthreads=8)
    for offset in (0, 7, 13):
        ids1, status1 = gpu_encode(gv, text, offset=offset)
        assert status1 == 0 and same(ids1, want1)
