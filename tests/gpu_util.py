"""Helpers for the GPU parity tests: run the C-ABI entry points on device tensors, and the one comparison
every parity test applies to what comes back."""
import functools

import numpy as np

import workloads as wl


def same(got, want) -> bool:
    """Bit-exact equality of two integer sequences (token ids, piece offsets, token offsets): same length,
    same dtype kind, same value at every index.  This is the whole tolerance of the parity tests; the
    planted-fault test (test_harness_faults.py) feeds it mutated GPU output and expects False every time."""
    got, want = np.asarray(got), np.asarray(want)
    if got.ndim != 1 or want.ndim != 1 or got.dtype.kind not in "iu" or want.dtype.kind not in "iu":
        return False
    return got.shape == want.shape and bool(np.array_equal(got, want))


def first_difference(got, want) -> str:
    """Where two sequences part, for assertion messages."""
    got, want = np.asarray(got), np.asarray(want)
    n = min(got.size, want.size)
    d = np.flatnonzero(got[:n] != want[:n])
    k = int(d[0]) if d.size else n
    return (f"sizes {got.size} / {want.size}, first difference at index {k}: "
            f"got {got[k:k + 4].tolist()} want {want[k:k + 4].tolist()}")


@functools.lru_cache(maxsize=None)
def gpu_vocab(name: str, n_merges: int | None = None, pattern: int | None = None):
    import paper_2607_29678_b200 as tt
    cfg = wl.CONFIGS[name]
    merges, byte_map = wl.load_vocab(cfg)
    if n_merges is not None:
        merges = merges[:n_merges]
    return tt.Vocab(merges, byte_map, cfg.pattern_id if pattern is None else pattern)


@functools.lru_cache(maxsize=None)
def cpu_vocab(name: str, n_merges: int | None = None):
    import oracle
    cfg = wl.CONFIGS[name]
    merges, byte_map = wl.load_vocab(cfg)
    if n_merges is not None:
        merges = merges[:n_merges]
    return oracle.Vocab(merges, byte_map)


def to_dev(a: np.ndarray, offset: int = 0):
    """Copies a uint8 array to the device; `offset` > 0 places it at a misaligned address."""
    import torch
    buf = torch.zeros(a.size + offset + 64, dtype=torch.uint8, device="cuda")
    t = buf[offset:offset + a.size]
    t.copy_(torch.from_numpy(np.array(a, dtype=np.uint8, copy=True)))
    return t


def gpu_encode(v, text: np.ndarray, offset: int = 0, ids_cap: int | None = None):
    """tt_encode; returns (ids, status)."""
    import torch
    d = to_dev(text, offset)
    bufs = v.alloc(max(text.size, 1))
    if ids_cap is not None:
        bufs["ids"] = torch.empty(max(ids_cap, 1), dtype=torch.int32, device="cuda")
    v.encode(d, bufs, length=text.size)
    torch.cuda.synchronize()
    n = int(bufs["count"].item())
    return bufs["ids"][:n].cpu().numpy(), int(bufs["status"].item())


def gpu_encode_batch(v, text: np.ndarray, doc_off: np.ndarray):
    """tt_encode_batch; returns (ids, ids_off, status)."""
    import torch
    d = to_dev(text)
    off = torch.from_numpy(np.ascontiguousarray(doc_off, dtype=np.int64)).cuda()
    bufs = v.alloc(max(text.size, 1), max_docs=doc_off.size - 1)
    v.encode_batch(d, off, bufs)
    torch.cuda.synchronize()
    ioff = bufs["ids_off"].cpu().numpy()
    return bufs["ids"][:int(ioff[-1])].cpu().numpy(), ioff, int(bufs["status"].item())


def gpu_pretok(v, text: np.ndarray, doc_off: np.ndarray | None = None, offset: int = 0):
    """tt_pretokenize; returns (piece_off, status)."""
    import torch
    d = to_dev(text, offset)
    n_docs = 1 if doc_off is None else doc_off.size - 1
    bufs = v.alloc(max(text.size, 1), max_docs=n_docs)
    po = torch.empty(text.size + 2, dtype=torch.int32, device="cuda")
    npc = torch.zeros(1, dtype=torch.int64, device="cuda")
    off = None if doc_off is None else torch.from_numpy(np.ascontiguousarray(doc_off, dtype=np.int64)).cuda()
    v.pretokenize(d, po, npc, bufs, doc_off=off)
    torch.cuda.synchronize()
    return po[:int(npc.item())].cpu().numpy().astype(np.int64), int(bufs["status"].item())
