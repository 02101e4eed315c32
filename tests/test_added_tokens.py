"""GPU added-token literal pass (tt_encode_added) against the oracle: leftmost-longest extraction, segments
between literals tokenized as texts of their own."""
import random

import numpy as np
import pytest

import oracle
import workloads as wl
from gpu_util import to_dev, same

pytestmark = pytest.mark.gpu


def _gpu_encode_added(v, text: np.ndarray, offset: int = 0):
    import torch
    d = to_dev(text, offset)
    bufs = v.alloc(max(text.size, 1))
    v.encode_added(d, bufs, length=text.size)
    torch.cuda.synchronize()
    return bufs["ids"][:int(bufs["count"].item())].cpu().numpy(), int(bufs["status"].item())


@pytest.mark.parametrize("name", ["C1", "C4"])
def test_special_tokens_in_transcripts(name):
    """Role markers of the synthetic transcripts as added tokens, plus literals that are ordinary words,
    prefixes of one another and non-ASCII; misaligned text pointer included."""
    import paper_2607_29678_b200 as tt
    cfg = wl.CONFIGS[name]
    merges, byte_map = wl.load_vocab(cfg)
    cv = oracle.Vocab(merges, byte_map)
    gv = tt.Vocab(merges, byte_map, cfg.pattern_id)
    lits = ["<|user|>", "<|assistant|>", "<|tool|>", "<|", "the", "there", "é中", "\n\n", "```python", "```", "    "]
    ids = [500000 + k for k in range(len(lits))]
    gv.add_literals(lits, ids)
    text = wl.generate(wl.KIND_TRANSCRIPT_ADV if name == "C4" else wl.KIND_TRANSCRIPT, 321, 120_000)
    text = np.concatenate([text, np.frombuffer("<|user|><|user|>é中é中<|<|assistant|>there the".encode(), dtype=np.uint8)])
    for offset in (0, 5):
        got, status = _gpu_encode_added(gv, text, offset)
        want = oracle.encode_added(cv, text, cfg.pattern_id, lits, ids)
        assert status == 0 and same(got, want)
    assert (want >= 500000).sum() > 100


def test_overlapping_literal_chains_and_edges():
    import paper_2607_29678_b200 as tt
    merges, byte_map = wl.load_vocab(wl.CONFIGS["C1"])
    cv = oracle.Vocab(merges, byte_map)
    rng = random.Random(9)
    for trial in range(40):
        alpha = rng.choice(["ab", "abc<|>", "a<", "a é"])
        lits = sorted({"".join(rng.choice(alpha) for _ in range(rng.randrange(1, 6))) for _ in range(rng.randrange(1, 7))})
        lits = [x for x in lits if x.strip() or len(x) > 1] or ["ab"]
        ids = [700000 + k for k in range(len(lits))]
        gv = tt.Vocab(merges, byte_map, 0)
        gv.add_literals(lits, ids)
        for n in (0, 1, 2, 7, 60, 3000, 70000):
            s = "".join(rng.choice(alpha) for _ in range(n))
            if rng.random() < 0.3 and n > 10:
                s = s[:n // 2] + "a" * 5000 + s[n // 2:]          # a long chain of overlapping candidates
            text = np.frombuffer(s.encode(), dtype=np.uint8)
            got, status = _gpu_encode_added(gv, text)
            want = oracle.encode_added(cv, text, 0, lits, ids)
            assert status == 0 and same(got, want), (lits, s[:80])
    # without registered literals the call is tt_encode
    gv = tt.Vocab(merges, byte_map, 0)
    text = wl.request(wl.CONFIGS["C1"])
    got, status = _gpu_encode_added(gv, text)
    assert status == 0 and same(got, cv.encode(text, 0)[0])
    # argument checks
    with pytest.raises(tt.TokTierError):
        gv.add_literals(["x", "x"], [1, 2])
    gv.add_literals(["x"], [1])
    with pytest.raises(tt.TokTierError):
        gv.add_literals(["y"], [2])


def test_literals_with_the_three_splitter_pattern():
    """The literal pass in front of TT_PATTERN_SPLIT3: literal boundaries, the cuts of the first two splitter
    stages and pattern 0 on every span must compose."""
    import paper_2607_29678_b200 as tt
    merges, byte_map = wl.load_vocab(wl.CONFIGS["C2"])
    cv = oracle.Vocab(merges, byte_map)
    gv = tt.Vocab(merges, byte_map, tt.TT_PATTERN_SPLIT3)
    lits = ["<|sep|>", "123", "中文", "  "]
    ids = [800000 + k for k in range(len(lits))]
    gv.add_literals(lits, ids)
    rng = random.Random(21)
    parts = []
    for _ in range(4000):
        parts.append(rng.choice(["word ", "12345", "123", "中文字", "中文", "<|sep|>", "  ", " ", "x1中 ", "\n", "9 9", "it's"]))
    text = np.frombuffer("".join(parts).encode("utf-8"), dtype=np.uint8)
    got, status = _gpu_encode_added(gv, text)
    want = oracle.encode_added(cv, text, 3, lits, ids)
    assert status == 0 and same(got, want)


def test_spans_of_added_tokens():
    """Span export over the output of tt_encode_added: a literal's record covers the literal's bytes."""
    import torch
    import paper_2607_29678_b200 as tt
    merges, byte_map = wl.load_vocab(wl.CONFIGS["C1"])
    cv = oracle.Vocab(merges, byte_map)
    gv = tt.Vocab(merges, byte_map, 0)
    lits = ["<|user|>", "<|assistant|>", "é中", "\n\n"]
    ids = [600000 + k for k in range(len(lits))]
    gv.add_literals(lits, ids)
    body = wl.generate(wl.KIND_TRANSCRIPT, 77, 30_000)
    text = np.concatenate([body, np.frombuffer("<|user|>é中é中 x<|assistant|>".encode(), dtype=np.uint8)])
    d_text = torch.from_numpy(text).cuda()
    bufs = gv.alloc(text.size)
    gv.encode_added(d_text, bufs)
    n = int(bufs["count"].item())
    byte_off = torch.empty(bufs["ids"].numel() + 1, dtype=torch.int32, device="cuda")
    char_off = torch.empty_like(byte_off)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    gv.spans(bufs["ids"], bufs["count"], text.size, byte_off, char_off, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    got_ids = bufs["ids"][:n].cpu().numpy()
    bo, co = byte_off[:n + 1].cpu().numpy(), char_off[:n + 1].cpu().numpy()
    # expected offsets from the token byte strings (vocabulary entries and literals alike)
    lit_bytes = {i: s.encode("utf-8") for i, s in zip(ids, lits)}
    pos = cpos = 0
    data = text.tobytes()
    for k, t in enumerate(got_ids.tolist()):
        s = lit_bytes[t] if t in lit_bytes else cv.token_bytes(t)
        assert bo[k] == pos and co[k] == cpos and data[pos:pos + len(s)] == s
        pos += len(s)
        cpos += sum((b & 0xC0) != 0x80 for b in s)
    assert bo[n] == pos == text.size and co[n] == cpos
    assert sum(t in lit_bytes for t in got_ids.tolist()) > 20
