"""CPU oracle for exact tokenization -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the bench's ``cpu_baseline`` / ``--impl reference`` legs may
import this package.  It is a thin ctypes wrapper around ``tt_oracle.cpp`` (plain sequential C++,
compiled with g++) plus the Unicode class table, which is taken from the interpreter's Unicode
database (``unicodedata``, version 15.0.0) and handed to the C++ side as a flat array.

Character classes (paper Sec. 4.1: letter, number, whitespace, other; the case-aware pattern also
needs letter case and marks): 0 other, 1 Ll, 2 Lu|Lt, 3 Lm|Lo, 4 N*, 5 whitespace (the 25
White_Space code points, i.e. what ``\\s`` matches in a Unicode regex engine), 6 M*.
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import subprocess
import unicodedata

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tt_oracle.cpp")
_LIB = os.path.join(_HERE, "_oracle.so")

K_O, K_LL, K_LU, K_LB, K_N, K_W, K_M = range(7)

UNICODE_VERSION = "15.0.0"
# SHA-256 of the 0x110000-entry class table built from Unicode 15.0.0; a different interpreter
# database changes the meaning of the patterns and must not pass silently (paper Sec. 5.2 reports
# exactly such a 15.0-vs-16.0 skew).
CLASS_TABLE_SHA256 = "c0eb98c163479363b5a49126d463f1898c330d4706dd72bc033205514b8a8bcf"

_WHITE_SPACE = [0x09, 0x0A, 0x0B, 0x0C, 0x0D, 0x20, 0x85, 0xA0, 0x1680, *range(0x2000, 0x200B), 0x2028, 0x2029,
                0x202F, 0x205F, 0x3000]

_lib = None
_table = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread", "-o", _LIB, _SRC])
    return _LIB


def class_table() -> np.ndarray:
    """uint8[0x110000] class code per code point."""
    global _table
    if _table is None:
        if unicodedata.unidata_version != UNICODE_VERSION:
            raise RuntimeError(f"oracle class table is frozen to Unicode {UNICODE_VERSION}, "
                               f"interpreter has {unicodedata.unidata_version}")
        t = np.zeros(0x110000, dtype=np.uint8)
        cat = unicodedata.category
        for cp in range(0x110000):
            c = cat(chr(cp))
            if c[0] == "L":
                t[cp] = K_LL if c == "Ll" else K_LU if c in ("Lu", "Lt") else K_LB
            elif c[0] == "N":
                t[cp] = K_N
            elif c[0] == "M":
                t[cp] = K_M
        for cp in _WHITE_SPACE:
            t[cp] = K_W
        if hashlib.sha256(t.tobytes()).hexdigest() != CLASS_TABLE_SHA256:
            raise RuntimeError("oracle class table does not match its frozen SHA-256")
        _table = t
    return _table


def class_table_sha256() -> str:
    return hashlib.sha256(class_table().tobytes()).hexdigest()


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        c = ctypes
        lib.orc_set_class_table.argtypes = [c.c_void_p]
        lib.orc_utf8_check.restype = c.c_int64
        lib.orc_utf8_check.argtypes = [c.c_void_p, c.c_size_t]
        lib.orc_pretok.restype = c.c_int64
        lib.orc_pretok.argtypes = [c.c_int, c.c_void_p, c.c_size_t, c.c_void_p, c.c_size_t]
        lib.orc_pretok_batch.restype = c.c_int64
        lib.orc_pretok_batch.argtypes = [c.c_int, c.c_void_p, c.c_void_p, c.c_size_t, c.c_int, c.c_void_p, c.c_size_t]
        lib.orc_vocab_new.restype = c.c_void_p
        lib.orc_vocab_new.argtypes = [c.c_void_p, c.c_size_t, c.c_void_p]
        lib.orc_vocab_free.argtypes = [c.c_void_p]
        lib.orc_vocab_set_ignore_merges.restype = None
        lib.orc_vocab_set_ignore_merges.argtypes = [c.c_void_p, c.c_int]
        lib.orc_token_bytes.restype = c.c_size_t
        lib.orc_token_bytes.argtypes = [c.c_void_p, c.c_int32, c.c_void_p, c.c_size_t]
        lib.orc_token_lens.restype = None
        lib.orc_token_lens.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p]
        lib.orc_bpe.restype = c.c_int64
        lib.orc_bpe.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t, c.c_int, c.c_void_p, c.c_size_t]
        lib.orc_encode.restype = c.c_int64
        lib.orc_encode.argtypes = [c.c_void_p, c.c_int, c.c_void_p, c.c_size_t, c.c_int, c.c_void_p, c.c_size_t,
                                   c.c_void_p, c.c_void_p]
        lib.orc_encode_batch.restype = c.c_int64
        lib.orc_encode_batch.argtypes = [c.c_void_p, c.c_int, c.c_void_p, c.c_void_p, c.c_size_t, c.c_int,
                                         c.c_void_p, c.c_size_t, c.c_void_p]
        lib.orc_train.restype = c.c_int64
        lib.orc_train.argtypes = [c.c_int, c.c_void_p, c.c_size_t, c.c_size_t, c.c_void_p, c.c_void_p]
        lib.orc_set_class_table(class_table().ctypes.data)
        _lib = lib
    return _lib


def _as_u8(text) -> np.ndarray:
    if isinstance(text, str):
        text = text.encode("utf-8")
    if isinstance(text, (bytes, bytearray)):
        return np.frombuffer(bytes(text), dtype=np.uint8)
    return np.ascontiguousarray(text, dtype=np.uint8)


class InvalidUtf8(ValueError):
    pass


def utf8_check(text) -> int:
    """Number of code points, or -1 if the bytes are not strict UTF-8."""
    a = _as_u8(text)
    return int(_load().orc_utf8_check(a.ctypes.data, a.size))


def pretokenize(text, pattern: int) -> np.ndarray:
    """Piece start byte offsets (int64[P]) of the sequential leftmost-first match."""
    a = _as_u8(text)
    out = np.empty(a.size + 1, dtype=np.int64)
    n = int(_load().orc_pretok(pattern, a.ctypes.data, a.size, out.ctypes.data, out.size))
    if n < 0:
        raise InvalidUtf8("invalid UTF-8")
    return out[:n].copy()


def pretokenize_batch(text, doc_off, pattern: int, nthreads: int = 1) -> np.ndarray:
    """Piece start byte offsets (int64[P], offsets into the concatenation) of a batch of documents, each
    matched as if it were alone; the same function as ``pretokenize``, called once per document."""
    a = _as_u8(text)
    doc_off = np.ascontiguousarray(doc_off, dtype=np.int64)
    out = np.empty(a.size + 1, dtype=np.int64)
    n = int(_load().orc_pretok_batch(pattern, a.ctypes.data, doc_off.ctypes.data, doc_off.size - 1, nthreads,
                                     out.ctypes.data, out.size))
    if n < 0:
        raise InvalidUtf8(f"invalid UTF-8 in document {-n - 1}")
    return out[:n].copy()


def pieces(text, pattern: int) -> list[bytes]:
    a = _as_u8(text)
    st = list(pretokenize(a, pattern)) + [a.size]
    b = a.tobytes()
    return [b[st[i]:st[i + 1]] for i in range(len(st) - 1)]


class Vocab:
    """Merge table: merges int32[n,3] rows (left, right, result); rank = row index.
    ``ignore_merges`` (paper Sec. 4.2): a piece that is a vocabulary entry as a whole is that one token."""

    def __init__(self, merges, byte_map=None, ignore_merges: bool = False):
        self.merges = np.ascontiguousarray(merges, dtype=np.int32).reshape(-1, 3)
        self.byte_map = np.ascontiguousarray(np.arange(256) if byte_map is None else byte_map, dtype=np.int32)
        self._h = _load().orc_vocab_new(self.merges.ctypes.data, self.merges.shape[0], self.byte_map.ctypes.data)
        self.ignore_merges = bool(ignore_merges)
        if ignore_merges:
            _load().orc_vocab_set_ignore_merges(self._h, 1)

    def __del__(self):
        try:
            if self._h:
                _load().orc_vocab_free(self._h)
                self._h = None
        except Exception:
            pass

    @property
    def n_merges(self) -> int:
        return self.merges.shape[0]

    def token_bytes(self, tid: int) -> bytes:
        buf = np.empty(1 << 17, dtype=np.uint8)
        n = int(_load().orc_token_bytes(self._h, int(tid), buf.ctypes.data, buf.size))
        return buf[:n].tobytes()

    def decode(self, ids) -> bytes:
        return b"".join(self.token_bytes(int(i)) for i in ids)

    def spans(self, text, ids):
        """Span export (paper App. E.3): byte_off[i] = sum of the byte lengths of tokens 0..i-1;
        char_off[i] = number of non-continuation bytes of the TEXT before byte_off[i].
        Returns (byte_off int64[T+1], char_off int64[T+1])."""
        a = _as_u8(text)
        ids = np.ascontiguousarray(ids, dtype=np.int32)
        lens = np.zeros(ids.size, dtype=np.int64)
        _load().orc_token_lens(self._h, ids.ctypes.data, ids.size, lens.ctypes.data)
        byte_off = np.zeros(ids.size + 1, dtype=np.int64)
        byte_off[1:] = np.cumsum(lens)
        if byte_off[-1] != a.size or (ids.size and lens.min() <= 0):
            raise ValueError("ids do not spell the text")
        starts_before = np.zeros(a.size + 1, dtype=np.int64)
        starts_before[1:] = np.cumsum((a & 0xC0) != 0x80)
        return byte_off, starts_before[byte_off]

    def bpe(self, piece, variant: int = 0) -> np.ndarray:
        """BPE of one piece; variant 0 = rescan definition, 1 = heap, 2 = chosen by length."""
        a = _as_u8(piece)
        out = np.empty(max(a.size, 1), dtype=np.int32)
        n = int(_load().orc_bpe(self._h, a.ctypes.data, a.size, variant, out.ctypes.data, out.size))
        return out[:n].copy()

    def encode(self, text, pattern: int, nthreads: int = 1):
        """Returns (ids int32[T], piece_off int64[P+1])."""
        a = _as_u8(text)
        ids = np.empty(max(a.size, 1), dtype=np.int32)
        po = np.empty(a.size + 1, dtype=np.int64)
        npieces = ctypes.c_int64(0)
        n = int(_load().orc_encode(self._h, pattern, a.ctypes.data, a.size, nthreads, ids.ctypes.data, ids.size,
                                   po.ctypes.data, ctypes.byref(npieces)))
        if n < 0:
            raise InvalidUtf8("invalid UTF-8")
        return ids[:n].copy(), po[:npieces.value + 1].copy()

    def encode_batch(self, text, doc_off, pattern: int, nthreads: int = 1):
        """Returns (ids int32[T], ids_off int64[n_docs+1]); each document encoded as if alone."""
        a = _as_u8(text)
        doc_off = np.ascontiguousarray(doc_off, dtype=np.int64)
        nd = doc_off.size - 1
        ids = np.empty(max(a.size, 1), dtype=np.int32)
        ioff = np.zeros(nd + 1, dtype=np.int64)
        n = int(_load().orc_encode_batch(self._h, pattern, a.ctypes.data, doc_off.ctypes.data, nd, nthreads,
                                         ids.ctypes.data, ids.size, ioff.ctypes.data))
        if n < 0:
            raise InvalidUtf8(f"invalid UTF-8 in document {-n - 1}")
        return ids[:n].copy(), ioff


def train(corpus, pattern: int, n_merges: int):
    """BPE trainer: returns (pairs int32[m,2], n_distinct_pieces)."""
    a = _as_u8(corpus)
    pairs = np.zeros((n_merges, 2), dtype=np.int32)
    nd = ctypes.c_int64(0)
    m = int(_load().orc_train(pattern, a.ctypes.data, a.size, n_merges, pairs.ctypes.data, ctypes.byref(nd)))
    if m < 0:
        raise InvalidUtf8("invalid UTF-8 in corpus")
    return pairs[:m].copy(), int(nd.value)


def split_added(text, literals) -> list[tuple[int, int, int]]:
    """Added-token literal pass (paper Sec. 4.3/4.4: a leftmost-longest literal pass extracts the added and special
    tokens before the tokenizer family handles the remaining segments).  Scans left to right; at each byte
    position the longest literal that matches there is taken and the scan continues behind it; positions
    inside a taken literal start nothing.  Returns the segments in order as (start, end, k): k = index of the
    literal, or -1 for the text between literals (empty segments are not returned)."""
    data = _as_u8(text).tobytes()
    lits = [bytes(x) if not isinstance(x, str) else x.encode("utf-8") for x in literals]
    out, p, seg = [], 0, 0
    while p < len(data):
        best = -1
        for k, lit in enumerate(lits):
            if lit and data.startswith(lit, p) and (best < 0 or len(lit) > len(lits[best])):
                best = k
        if best < 0:
            p += 1
            continue
        if p > seg:
            out.append((seg, p, -1))
        out.append((p, p + len(lits[best]), best))
        p += len(lits[best])
        seg = p
    if len(data) > seg:
        out.append((seg, len(data), -1))
    return out


def encode_added(vocab: "Vocab", text, pattern: int, literals, literal_ids) -> np.ndarray:
    """IDs of a text with added tokens: every literal found by split_added becomes its id, every segment between
    literals is encoded as if it were a text of its own."""
    data = _as_u8(text)
    ids = []
    for a, b, k in split_added(data, literals):
        if k >= 0:
            ids.append(int(literal_ids[k]))
        else:
            ids.extend(vocab.encode(data[a:b], pattern)[0].tolist())
    return np.asarray(ids, dtype=np.int32)
