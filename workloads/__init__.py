"""Seeded synthetic workloads (inputs only; no tokenizer arithmetic lives here).

The five configurations mirror the benchmark's configs: a 4,000-char mixed request (C1), a
100,000-char request with ~5 % non-ASCII and CRLF lines (C2), a 1,000,000-char agent transcript (C3),
a 3,000,000-char transcript with CJK and adversarial long runs (C4), and a batch of 256 transcripts
with lognormal lengths (C5).  Vocabulary files (merge lists) are stored under ``workloads/vocabs``;
they are written by ``oracle/train_vocabs.py`` and are plain inputs to both the oracle and the CUDA
path.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "_gen.so")
_lib = None

BASE_SEED = 0x260729678

KIND_MIX, KIND_MIX_UNI, KIND_TRANSCRIPT, KIND_TRANSCRIPT_ADV, KIND_MARKS, KIND_THAI = 0, 1, 2, 3, 4, 5


def build(force: bool = False) -> str:
    """Compile the generator (plain C, gcc)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.wl_generate.restype = ctypes.c_size_t
        lib.wl_generate.argtypes = [ctypes.c_int, ctypes.c_uint64, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_size_t]
        lib.wl_batch_lengths.restype = None
        lib.wl_batch_lengths.argtypes = [ctypes.c_uint64, ctypes.c_size_t, ctypes.c_double, ctypes.c_double,
                                         ctypes.c_double, ctypes.c_double, ctypes.c_void_p]
        lib.wl_count_chars.restype = ctypes.c_size_t
        lib.wl_count_chars.argtypes = [ctypes.c_void_p, ctypes.c_size_t]
        lib.wl_exhaustive.restype = ctypes.c_size_t
        lib.wl_exhaustive.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t,
                                      ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        _lib = lib
    return _lib


def generate(kind: int, seed: int, n_chars: int) -> np.ndarray:
    """Return a uint8 array holding valid UTF-8 with exactly ``n_chars`` code points."""
    lib = _load()
    buf = np.empty(4 * n_chars + 16, dtype=np.uint8)
    n = lib.wl_generate(kind, seed & 0xFFFFFFFFFFFFFFFF, n_chars, buf.ctypes.data, buf.size)
    if n_chars and n == 0:
        raise RuntimeError("generator output did not fit")
    return buf[:n].copy()


def count_chars(text: np.ndarray) -> int:
    text = np.ascontiguousarray(text, dtype=np.uint8)
    return int(_load().wl_count_chars(text.ctypes.data, text.size))


def exhaustive(alphabet, maxlen: int):
    """Every string of 1..maxlen symbols over ``alphabet`` (a str: one symbol per character), shortest first,
    in the order of ``itertools.product``: returns (concatenated uint8 text, int64 byte offsets[n + 1])."""
    lib = _load()
    syms = [ch.encode("utf-8") for ch in alphabet]
    blob = np.frombuffer(b"".join(syms), dtype=np.uint8).copy()
    soff = np.zeros(len(syms) + 1, dtype=np.uint32)
    soff[1:] = np.cumsum([len(x) for x in syms])
    need = ctypes.c_size_t(0)
    n = lib.wl_exhaustive(blob.ctypes.data, soff.ctypes.data, len(syms), maxlen, None, 0, None, 0, ctypes.byref(need))
    text = np.empty(need.value + 16, dtype=np.uint8)
    off = np.empty(n + 1, dtype=np.int64)
    got = lib.wl_exhaustive(blob.ctypes.data, soff.ctypes.data, len(syms), maxlen, text.ctypes.data, text.size,
                            off.ctypes.data, off.size + 1, None)
    if got != n:
        raise RuntimeError("exhaustive generator: buffers too small")
    return text[:need.value], off


def batch_lengths(seed: int, n: int, median: float, sigma: float, lo: float, hi: float) -> np.ndarray:
    out = np.empty(n, dtype=np.uint64)
    _load().wl_batch_lengths(seed & 0xFFFFFFFFFFFFFFFF, n, median, sigma, lo, hi, out.ctypes.data)
    return out.astype(np.int64)


@dataclass(frozen=True)
class Config:
    name: str
    kind: int
    n_chars: int          # per request (batch: median)
    pattern_id: int       # 0 = cl100k-style, 1 = o200k-style
    n_merges: int
    corpus_chars: int
    n_docs: int = 1

    @property
    def index(self) -> int:
        return int(self.name[1:])

    @property
    def vocab_file(self) -> str:
        return os.path.join(_HERE, "vocabs", f"p{self.pattern_id}_m{self.n_merges}.npz")


CONFIGS = {
    "C1": Config("C1", KIND_MIX, 4_000, 0, 4_096, 2_000_000),
    "C2": Config("C2", KIND_MIX_UNI, 100_000, 0, 32_000, 20_000_000),
    "C3": Config("C3", KIND_TRANSCRIPT, 1_000_000, 0, 100_000, 100_000_000),
    "C4": Config("C4", KIND_TRANSCRIPT_ADV, 3_000_000, 1, 199_744, 100_000_000),
    "C5": Config("C5", KIND_TRANSCRIPT, 350_000, 0, 100_000, 100_000_000, n_docs=256),
}


def request_seed(cfg: Config, sample: int = 0) -> int:
    return BASE_SEED + cfg.index + 1000 * sample


def corpus_seed(cfg: Config) -> int:
    return (BASE_SEED ^ 0xC0FFEE) + 7919 * cfg.index


def request(cfg: Config, sample: int = 0, n_chars: int | None = None) -> np.ndarray:
    """One request text of the configuration (``sample`` picks a distinct seeded input)."""
    return generate(cfg.kind, request_seed(cfg, sample), cfg.n_chars if n_chars is None else n_chars)


def corpus(cfg: Config, n_chars: int | None = None) -> np.ndarray:
    """Training corpus for the configuration's vocabulary (distinct seed from every request)."""
    return generate(cfg.kind, corpus_seed(cfg), cfg.corpus_chars if n_chars is None else n_chars)


def batch(cfg: Config, sample: int = 0, n_docs: int | None = None, scale: float = 1.0):
    """Batch of independent requests: returns (concatenated uint8 text, int64 byte offsets[n_docs+1]).

    Lengths are lognormal(median n_chars, sigma 1.0) clipped to [10,000, 3,000,000] chars; ``scale``
    shrinks every length (tests use it to keep the oracle fast)."""
    n = cfg.n_docs if n_docs is None else n_docs
    lens = batch_lengths(request_seed(cfg, sample) ^ 0xBA7C4, n, cfg.n_chars, 1.0, 10_000, 3_000_000)
    docs = []
    for i, L in enumerate(lens):
        L = max(1, int(L * scale))
        docs.append(generate(cfg.kind, request_seed(cfg, sample) + 0x10000 * (i + 1), L))
    off = np.zeros(n + 1, dtype=np.int64)
    off[1:] = np.cumsum([d.size for d in docs])
    return (np.concatenate(docs) if docs else np.empty(0, np.uint8)), off


def load_vocab(cfg_or_path):
    """Load a stored merge list: returns (merges int32[n,3] as (left,right,result), byte_map int32[256])."""
    path = cfg_or_path if isinstance(cfg_or_path, str) else cfg_or_path.vocab_file
    z = np.load(path)
    pairs = z["pairs"].astype(np.int32)
    n = pairs.shape[0]
    merges = np.empty((n, 3), dtype=np.int32)
    merges[:, :2] = pairs
    merges[:, 2] = 256 + np.arange(n, dtype=np.int32)
    byte_map = z["byte_map"].astype(np.int32) if "byte_map" in z.files else np.arange(256, dtype=np.int32)
    return merges, byte_map
