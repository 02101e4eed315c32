"""B200-native exact tokenizer: thin Python binding over the C ABI in include/toktier.h.

Argument marshalling only -- every step of the path runs in the CUDA kernels of libtoktier.so.
PyTorch supplies device memory and streams.  There is no CPU fallback: if the library is missing
or no CUDA device is present, the calls raise.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtoktier.so")

TT_OK, TT_ERR_ARG, TT_ERR_BAD_VOCAB, TT_ERR_CUDA, TT_ERR_INVALID_UTF8, TT_ERR_CAPACITY, TT_ERR_INTERNAL_TIMEOUT, TT_ERR_TOO_LARGE, TT_ERR_BAD_IDS = range(9)
TT_STATIC_MAX_LEN = 262144
TT_PATTERN_CL100K, TT_PATTERN_O200K, TT_PATTERN_CL100K_N1, TT_PATTERN_SPLIT3 = 0, 1, 2, 3
TT_VOCAB_IGNORE_MERGES = 1

EXPORTS = ["tt_vocab_load", "tt_vocab_load_ex", "tt_vocab_free", "tt_vocab_table_entries", "tt_workspace_bytes", "tt_encode", "tt_encode_batch",
           "tt_pretokenize", "tt_encode_timed", "tt_encode_host", "tt_encode_static", "tt_spans", "tt_spans_workspace_bytes", "tt_class_table", "tt_strerror",
           "tt_session_create", "tt_session_free", "tt_session_set_window", "tt_session_append", "tt_session_view", "tt_session_copy", "tt_vocab_add_literals", "tt_encode_added",
           "tt_pair_info_host", "tt_verifier_create", "tt_verifier_submit", "tt_verifier_drain", "tt_verifier_get_stats", "tt_verifier_quarantined", "tt_verifier_free"]

_lib = None
REFERENCE_FN = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_size_t,
                                ctypes.POINTER(ctypes.c_int64))


class TokTierError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} (code {code})")


def lib() -> ctypes.CDLL:
    """Loads libtoktier.so (built in-tree by paper_2607_29678_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not built; run `python -m paper_2607_29678_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        c = ctypes
        L.tt_vocab_load.restype = c.c_int
        L.tt_vocab_load.argtypes = [c.c_void_p, c.c_size_t, c.c_void_p, c.c_int, c.POINTER(c.c_void_p)]
        L.tt_vocab_load_ex.restype = c.c_int
        L.tt_vocab_load_ex.argtypes = [c.c_void_p, c.c_size_t, c.c_void_p, c.c_int, c.c_uint, c.POINTER(c.c_void_p)]
        L.tt_vocab_free.restype = None
        L.tt_vocab_free.argtypes = [c.c_void_p]
        L.tt_vocab_table_entries.restype = c.c_size_t
        L.tt_vocab_table_entries.argtypes = [c.c_void_p]
        L.tt_workspace_bytes.restype = c.c_size_t
        L.tt_workspace_bytes.argtypes = [c.c_void_p, c.c_size_t, c.c_size_t]
        L.tt_encode.restype = c.c_int
        L.tt_encode.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p,
                                c.c_void_p, c.c_void_p, c.c_size_t]
        L.tt_encode_batch.restype = c.c_int
        L.tt_encode_batch.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p, c.c_size_t, c.c_void_p, c.c_void_p,
                                      c.c_size_t, c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t]
        L.tt_pretokenize.restype = c.c_int
        L.tt_pretokenize.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p, c.c_size_t, c.c_void_p, c.c_void_p,
                                     c.c_size_t, c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t]
        L.tt_encode_timed.restype = c.c_int
        L.tt_encode_timed.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p,
                                      c.c_void_p, c.c_void_p, c.c_size_t, c.POINTER(c.c_float)]
        L.tt_encode_static.restype = c.c_int
        L.tt_encode_static.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p,
                                       c.c_void_p]
        L.tt_spans_workspace_bytes.restype = c.c_size_t
        L.tt_spans_workspace_bytes.argtypes = [c.c_void_p, c.c_size_t]
        L.tt_spans.restype = c.c_int
        L.tt_spans.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t, c.c_size_t, c.c_void_p, c.c_void_p, c.c_void_p,
                               c.c_void_p, c.c_void_p, c.c_size_t]
        L.tt_encode_host.restype = c.c_int
        L.tt_encode_host.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p, c.c_size_t, c.POINTER(c.c_int64)]
        L.tt_class_table.restype = c.c_size_t
        L.tt_class_table.argtypes = [c.c_void_p, c.c_size_t]
        L.tt_strerror.restype = c.c_char_p
        L.tt_strerror.argtypes = [c.c_int]
        L.tt_session_create.restype = c.c_int
        L.tt_session_create.argtypes = [c.c_void_p, c.c_size_t, c.POINTER(c.c_void_p)]
        L.tt_session_free.restype = None
        L.tt_session_free.argtypes = [c.c_void_p]
        L.tt_session_set_window.restype = c.c_int
        L.tt_session_set_window.argtypes = [c.c_void_p, c.c_uint32]
        L.tt_session_append.restype = c.c_int
        L.tt_session_append.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p, c.c_void_p]
        L.tt_session_view.restype = c.c_int
        L.tt_session_view.argtypes = [c.c_void_p, c.POINTER(c.c_void_p), c.POINTER(c.c_void_p), c.POINTER(c.c_void_p), c.POINTER(c.c_size_t)]
        L.tt_vocab_add_literals.restype = c.c_int
        L.tt_vocab_add_literals.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t]
        L.tt_encode_added.restype = c.c_int
        L.tt_encode_added.argtypes = L.tt_encode.argtypes
        L.tt_verifier_create.restype = c.c_int
        L.tt_verifier_create.argtypes = [REFERENCE_FN, c.c_void_p, c.c_double, c.c_size_t, c.c_uint64, c.POINTER(c.c_void_p)]
        L.tt_verifier_submit.restype = c.c_int
        L.tt_verifier_submit.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p, c.c_size_t]
        L.tt_verifier_drain.restype = None
        L.tt_verifier_drain.argtypes = [c.c_void_p]
        L.tt_verifier_get_stats.restype = None
        L.tt_verifier_get_stats.argtypes = [c.c_void_p, c.c_void_p]
        L.tt_verifier_quarantined.restype = c.c_int
        L.tt_verifier_quarantined.argtypes = [c.c_void_p, c.c_size_t, c.POINTER(c.c_uint64), c.POINTER(c.c_uint64), c.POINTER(c.c_int64)]
        L.tt_verifier_free.restype = None
        L.tt_verifier_free.argtypes = [c.c_void_p]
        L.tt_session_copy.restype = c.c_int
        L.tt_session_copy.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p, c.c_void_p, c.c_void_p]
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().tt_strerror(int(code)).decode()


def class_table() -> np.ndarray:
    """uint8[0x110000]: the class code the kernels assign to every code point."""
    out = np.empty(0x110000, dtype=np.uint8)
    lib().tt_class_table(out.ctypes.data, out.size)
    return out


def pair_info_host(merges, byte_map, left, right) -> np.ndarray:
    """tt_pair_info_host: int64[n, 3] (rank, cl, cr; -1 = none) of the pairs (left[i], right[i]); runs on the host."""
    m = np.ascontiguousarray(merges, dtype=np.int32)
    bm = np.ascontiguousarray(np.arange(256) if byte_map is None else byte_map, dtype=np.int32)
    l = np.ascontiguousarray(left, dtype=np.int32)
    r = np.ascontiguousarray(right, dtype=np.int32)
    out = np.empty((l.size, 3), dtype=np.int64)
    L = lib()
    L.tt_pair_info_host.restype = ctypes.c_int
    L.tt_pair_info_host.argtypes = [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                    ctypes.c_size_t, ctypes.c_void_p]
    _check(L.tt_pair_info_host(m.ctypes.data, m.shape[0], bm.ctypes.data, l.ctypes.data, r.ctypes.data, l.size,
                               out.ctypes.data), "tt_pair_info_host")
    return out


def _check(rc: int, where: str):
    if rc != TT_OK:
        raise TokTierError(rc, where)


def _stream_ptr(stream) -> int:
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


class Vocab:
    """tt_vocab_load(_ex) / tt_vocab_free.  merges: int32[n,3] rows (left, right, result); rank = row.
    ignore_merges: a piece that is a vocabulary entry as a whole becomes that one token (TT_VOCAB_IGNORE_MERGES)."""

    def __init__(self, merges, byte_map=None, pattern_id: int = TT_PATTERN_CL100K, ignore_merges: bool = False):
        m = np.ascontiguousarray(merges, dtype=np.int32).reshape(-1, 3)
        bm = np.ascontiguousarray(np.arange(256) if byte_map is None else byte_map, dtype=np.int32)
        if bm.size != 256:
            raise ValueError("byte_map needs 256 entries")
        self.n_merges = m.shape[0]
        self.pattern_id = pattern_id
        h = ctypes.c_void_p()
        flags = TT_VOCAB_IGNORE_MERGES if ignore_merges else 0
        _check(lib().tt_vocab_load_ex(m.ctypes.data, m.shape[0], bm.ctypes.data, pattern_id, flags, ctypes.byref(h)), "tt_vocab_load_ex")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib().tt_vocab_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def table_entries(self) -> int:
        """tt_vocab_table_entries: vocabulary entries that one probe of the whole-piece table settles."""
        return int(lib().tt_vocab_table_entries(self._h))

    # -- sizes -------------------------------------------------------------------------------
    def workspace_bytes(self, max_len: int, max_docs: int = 1) -> int:
        return int(lib().tt_workspace_bytes(self._h, max_len, max_docs))

    def alloc(self, max_len: int, max_docs: int = 1, device="cuda"):
        """Device buffers for calls over at most max_len bytes: dict(ids, count, status, ids_off, workspace)."""
        import torch
        return dict(
            ids=torch.empty(max(max_len, 1), dtype=torch.int32, device=device),
            count=torch.zeros(1, dtype=torch.int64, device=device),
            status=torch.zeros(1, dtype=torch.int32, device=device),
            ids_off=torch.zeros(max_docs + 1, dtype=torch.int64, device=device),
            workspace=torch.empty(self.workspace_bytes(max_len, max_docs), dtype=torch.uint8, device=device),
        )

    # -- device entry points (asynchronous on the stream) ---------------------------------------
    def encode(self, text, bufs, stream=None, length: int | None = None):
        """tt_encode: text = uint8 CUDA tensor.  Results land in bufs['ids'], bufs['count'], bufs['status']."""
        n = int(text.numel() if length is None else length)
        ws = bufs["workspace"]
        _check(lib().tt_encode(self._h, text.data_ptr(), n, _stream_ptr(stream), bufs["ids"].data_ptr(),
                               bufs["ids"].numel(), bufs["count"].data_ptr(), bufs["status"].data_ptr(),
                               ws.data_ptr(), ws.numel()), "tt_encode")

    def add_literals(self, literals, ids):
        """tt_vocab_add_literals: added / special tokens (bytes or str) with their ids; once per vocabulary."""
        lits = [x.encode("utf-8") if isinstance(x, str) else bytes(x) for x in literals]
        blob = np.frombuffer(b"".join(lits) or b"\0", dtype=np.uint8).copy()
        off = np.zeros(len(lits) + 1, dtype=np.uint32)
        off[1:] = np.cumsum([len(x) for x in lits])
        idv = np.ascontiguousarray(ids, dtype=np.int32)
        _check(lib().tt_vocab_add_literals(self._h, blob.ctypes.data, off.ctypes.data, idv.ctypes.data, len(lits)),
               "tt_vocab_add_literals")

    def encode_added(self, text, bufs, stream=None, length: int | None = None):
        """tt_encode_added: tt_encode behind the leftmost-longest added-token pass."""
        n = int(text.numel() if length is None else length)
        ws = bufs["workspace"]
        _check(lib().tt_encode_added(self._h, text.data_ptr(), n, _stream_ptr(stream), bufs["ids"].data_ptr(),
                                     bufs["ids"].numel(), bufs["count"].data_ptr(), bufs["status"].data_ptr(),
                                     ws.data_ptr(), ws.numel()), "tt_encode_added")

    KERNEL_NAMES = ("front", "merge", "scatter")

    def encode_timed(self, text, bufs, stream=None) -> dict:
        """tt_encode_timed: like encode, synchronises, returns {kernel name: milliseconds}."""
        ws = bufs["workspace"]
        ms = (ctypes.c_float * 3)()
        _check(lib().tt_encode_timed(self._h, text.data_ptr(), int(text.numel()), _stream_ptr(stream),
                                     bufs["ids"].data_ptr(), bufs["ids"].numel(), bufs["count"].data_ptr(),
                                     bufs["status"].data_ptr(), ws.data_ptr(), ws.numel(), ms), "tt_encode_timed")
        return dict(zip(self.KERNEL_NAMES, [float(x) for x in ms]))

    def encode_batch(self, text, doc_off, bufs, stream=None):
        """tt_encode_batch: doc_off = int64 CUDA tensor [n_docs+1].  Results in bufs['ids'], bufs['ids_off'], bufs['status']."""
        ws = bufs["workspace"]
        n_docs = int(doc_off.numel()) - 1
        _check(lib().tt_encode_batch(self._h, text.data_ptr(), int(text.numel()), doc_off.data_ptr(), n_docs,
                                     _stream_ptr(stream), bufs["ids"].data_ptr(), bufs["ids"].numel(),
                                     bufs["ids_off"].data_ptr(), bufs["status"].data_ptr(), ws.data_ptr(), ws.numel()),
               "tt_encode_batch")

    def pretokenize(self, text, piece_off, n_pieces, bufs, doc_off=None, stream=None):
        """tt_pretokenize: piece_off = int32 CUDA tensor [>= len+1], n_pieces = int64 CUDA tensor [1]."""
        ws = bufs["workspace"]
        n_docs = 1 if doc_off is None else int(doc_off.numel()) - 1
        _check(lib().tt_pretokenize(self._h, text.data_ptr(), int(text.numel()), 0 if doc_off is None else doc_off.data_ptr(),
                                    n_docs, _stream_ptr(stream), piece_off.data_ptr(), piece_off.numel(),
                                    n_pieces.data_ptr(), bufs["status"].data_ptr(), ws.data_ptr(), ws.numel()),
               "tt_pretokenize")

    def encode_static(self, text, ids, count, status, stream=None, length: int | None = None):
        """tt_encode_static: encode without a workspace, for callers that may not allocate device memory
        (the library's own fixed scratch array is used; at most TT_STATIC_MAX_LEN bytes of text).
        text / ids / count / status are the caller's CUDA tensors (uint8, int32, int64[1], int32[1]).
        Calls on one device share the scratch, so do not let two of them overlap on the GPU."""
        n = int(text.numel() if length is None else length)
        _check(lib().tt_encode_static(self._h, text.data_ptr(), n, _stream_ptr(stream), ids.data_ptr(), ids.numel(),
                                      count.data_ptr(), status.data_ptr()), "tt_encode_static")

    def spans(self, ids, count, text_len: int, byte_off, char_off, status, workspace=None, stream=None):
        """tt_spans: byte / character offsets of the tokens in `ids` (int32 CUDA tensor) whose number is in
        `count` (int64 CUDA tensor [1]).  byte_off / char_off: int32 CUDA tensors [ids.numel() + 1]."""
        import torch
        if workspace is None:
            workspace = torch.empty(int(lib().tt_spans_workspace_bytes(self._h, ids.numel())), dtype=torch.uint8, device=ids.device)
        _check(lib().tt_spans(self._h, ids.data_ptr(), count.data_ptr(), ids.numel(), int(text_len), _stream_ptr(stream),
                              byte_off.data_ptr(), char_off.data_ptr(), status.data_ptr(), workspace.data_ptr(),
                              workspace.numel()), "tt_spans")
        return workspace

    # -- host convenience --------------------------------------------------------------------------
    def encode_host(self, data) -> np.ndarray:
        """tt_encode_host: bytes / uint8 array in host memory -> int32 ids in host memory."""
        a = np.frombuffer(data, dtype=np.uint8) if isinstance(data, (bytes, bytearray)) else np.ascontiguousarray(data, dtype=np.uint8)
        out = np.empty(max(a.size, 1), dtype=np.int32)
        cnt = ctypes.c_int64(0)
        _check(lib().tt_encode_host(self._h, a.ctypes.data, a.size, out.ctypes.data, out.size, ctypes.byref(cnt)),
               "tt_encode_host")
        return out[:cnt.value]

    def encode_host_into(self, text, ids_out) -> int:
        """tt_encode_host on caller buffers: `text` a uint8 host tensor / array, `ids_out` an int32 host tensor /
        array that receives the ids; returns the count.  Pinned tensors are used without staging."""
        tp = text.data_ptr() if hasattr(text, "data_ptr") else text.ctypes.data
        tn = text.numel() if hasattr(text, "numel") else text.size
        op = ids_out.data_ptr() if hasattr(ids_out, "data_ptr") else ids_out.ctypes.data
        on = ids_out.numel() if hasattr(ids_out, "numel") else ids_out.size
        cnt = ctypes.c_int64(0)
        _check(lib().tt_encode_host(self._h, tp, tn, op, on, ctypes.byref(cnt)), "tt_encode_host")
        return cnt.value


class AppendInfo(ctypes.Structure):
    """tt_append_info."""
    _fields_ = [("attempts", ctypes.c_int32), ("status", ctypes.c_int32), ("window_chars", ctypes.c_int64),
                ("window_start", ctypes.c_int64), ("run_tokens", ctypes.c_int64), ("splice_byte", ctypes.c_int64),
                ("n_tokens", ctypes.c_int64)]


class Session:
    """tt_session_*: a stored text with its token records on the device, updated by incremental repair."""

    def __init__(self, vocab: Vocab, max_bytes: int, window_chars: int | None = None):
        self.vocab = vocab                      # keeps the vocabulary alive
        h = ctypes.c_void_p()
        _check(lib().tt_session_create(vocab._h, max_bytes, ctypes.byref(h)), "tt_session_create")
        self._h = h
        if window_chars is not None:
            _check(lib().tt_session_set_window(self._h, window_chars), "tt_session_set_window")

    def close(self):
        if getattr(self, "_h", None):
            lib().tt_session_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def append(self, data, stream=None) -> dict:
        """tt_session_append (host bytes in); returns the tt_append_info fields."""
        a = np.frombuffer(bytes(data), dtype=np.uint8) if isinstance(data, (bytes, bytearray, str)) else np.ascontiguousarray(data, dtype=np.uint8)
        info = AppendInfo()
        _check(lib().tt_session_append(self._h, a.ctypes.data if a.size else None, a.size, _stream_ptr(stream), ctypes.byref(info)),
               "tt_session_append")
        return {k: getattr(info, k) for k, _ in AppendInfo._fields_}

    def records(self, stream=None):
        """tt_session_copy into fresh tensors: (ids int32[T], off int32[T + 1], stored bytes)."""
        import torch
        n = ctypes.c_size_t()
        _check(lib().tt_session_view(self._h, None, None, None, ctypes.byref(n)), "tt_session_view")
        ids = torch.empty(max(n.value, 1), dtype=torch.int32, device="cuda")
        off = torch.empty(n.value + 1, dtype=torch.int32, device="cuda")
        count = torch.zeros(1, dtype=torch.int64, device="cuda")
        _check(lib().tt_session_copy(self._h, ids.data_ptr(), n.value, off.data_ptr(), count.data_ptr(), _stream_ptr(stream)),
               "tt_session_copy")
        torch.cuda.synchronize()
        k = int(count.item())
        return ids[:k], off[:k + 1], n.value


class VerifierStats(ctypes.Structure):
    _fields_ = [(k, ctypes.c_uint64) for k in ("submitted", "sampled", "checked", "mismatches", "dropped")]


class Verifier:
    """tt_verifier_*: shadow verification of emitted sequences against a reference engine.
    reference(text: bytes) -> sequence of ids (a Python callable; it runs on the verifier's thread)."""

    def __init__(self, reference, sample_rate: float = 0.05, queue_cap: int = 64, seed: int = 0):
        def _cb(user, text, n, ids_out, cap, count_out):
            try:
                ids = np.asarray(reference(ctypes.string_at(text, n)), dtype=np.int32)
                if ids.size > cap:
                    return 1
                ctypes.memmove(ids_out, ids.ctypes.data, 4 * ids.size)
                count_out[0] = ids.size
                return 0
            except Exception:
                return 1
        self._cb = REFERENCE_FN(_cb)              # keeps the callback alive
        h = ctypes.c_void_p()
        _check(lib().tt_verifier_create(self._cb, None, sample_rate, queue_cap, seed, ctypes.byref(h)), "tt_verifier_create")
        self._h = h

    def submit(self, text, ids) -> int:
        a = np.frombuffer(bytes(text), dtype=np.uint8) if isinstance(text, (bytes, bytearray)) else np.ascontiguousarray(text, dtype=np.uint8)
        i = np.ascontiguousarray(ids, dtype=np.int32)
        return int(lib().tt_verifier_submit(self._h, a.ctypes.data if a.size else None, a.size, i.ctypes.data if i.size else None, i.size))

    def drain(self):
        lib().tt_verifier_drain(self._h)

    def stats(self) -> dict:
        st = VerifierStats()
        lib().tt_verifier_get_stats(self._h, ctypes.byref(st))
        return {k: int(getattr(st, k)) for k, _ in VerifierStats._fields_}

    def quarantined(self, index: int):
        h, n, d = ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_int64()
        _check(lib().tt_verifier_quarantined(self._h, index, ctypes.byref(h), ctypes.byref(n), ctypes.byref(d)), "tt_verifier_quarantined")
        return h.value, n.value, d.value

    def close(self):
        if getattr(self, "_h", None):
            lib().tt_verifier_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
