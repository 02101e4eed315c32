"""The seeded input generator: determinism, exact sizes, validity and the shapes the configs name."""
import re

import numpy as np

import workloads as wl


def test_deterministic_and_exact_char_count():
    for kind in range(4):
        a = wl.generate(kind, 42, 12345)
        b = wl.generate(kind, 42, 12345)
        assert np.array_equal(a, b)
        assert wl.count_chars(a) == 12345
        assert len(a.tobytes().decode("utf-8")) == 12345
        assert not np.array_equal(a, wl.generate(kind, 43, 12345))


def test_config_shapes():
    s1 = wl.request(wl.CONFIGS["C1"]).tobytes().decode()
    assert len(s1) == 4000 and s1.isascii() and "\r" not in s1
    s2 = wl.request(wl.CONFIGS["C2"]).tobytes().decode()
    frac = sum(ord(c) > 127 for c in s2) / len(s2)
    assert 0.03 < frac < 0.08
    crlf = s2.count("\r\n") / s2.count("\n")
    assert 0.05 < crlf < 0.16
    assert any(0x4E00 <= ord(c) < 0xA000 for c in s2) and any(ord(c) > 0xFFFF for c in s2)
    s4 = wl.request(wl.CONFIGS["C4"]).tobytes().decode()
    assert len(s4) == 3_000_000
    assert re.search(r"[ \t]{65536}", s4) and re.search(r"\d{20000}", s4) and re.search(r"([^\w\s])\1{51199}", s4)
    cjk = sum(0x4E00 <= ord(c) < 0xA000 for c in s4) / len(s4)
    assert 0.05 < cjk < 0.2


def test_batch_lengths_and_offsets():
    cfg = wl.CONFIGS["C5"]
    lens = wl.batch_lengths(1, 256, cfg.n_chars, 1.0, 10_000, 3_000_000)
    assert lens.min() >= 10_000 and lens.max() <= 3_000_000
    assert 200_000 < np.median(lens) < 550_000
    text, off = wl.batch(cfg, n_docs=4, scale=0.01)
    assert off[0] == 0 and off[-1] == text.size and np.all(np.diff(off) > 0)
    for d in range(4):
        text[off[d]:off[d + 1]].tobytes().decode("utf-8")


def test_vocab_files_are_well_formed():
    for name, cfg in wl.CONFIGS.items():
        merges, byte_map = wl.load_vocab(cfg)
        assert merges.shape == (cfg.n_merges, 3)
        assert np.array_equal(byte_map, np.arange(256))
        rank = np.arange(cfg.n_merges)
        assert np.all(merges[:, 0] < 256 + rank) and np.all(merges[:, 1] < 256 + rank) and merges.min() >= 0
        keys = merges[:, 0].astype(np.int64) << 32 | merges[:, 1]
        assert np.unique(keys).size == cfg.n_merges
