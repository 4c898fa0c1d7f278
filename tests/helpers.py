"""Shared test helpers: rank-counting brute force and the GPU-vs-oracle row comparison."""
import struct

import numpy as np


def py_key(x):
    """Monotone key of one fp32 value, from its packed bytes (pure Python)."""
    (u,) = struct.unpack("<I", struct.pack("<f", x))
    return (~u & 0xFFFFFFFF) if (u >> 31) else (u | 0x80000000)


def rank_count_topk(row, K):
    """Indices whose rank is < K, where rank(i) counts the elements that precede i:
    a strictly larger key, or an equal key at a lower index.  O(L^2); tiny rows only."""
    keys = [py_key(float(v)) for v in row]
    chosen = []
    for i, ki in enumerate(keys):
        rank = sum(1 for j, kj in enumerate(keys) if kj > ki or (kj == ki and j < i))
        if rank < K:
            chosen.append(i)
    return chosen


def assert_rows_match(scores, row_starts, row_lengths, K, got_idx, got_val, want_idx, rows=None):
    """Set-wise, bit-exact comparison of a selector's output with the oracle's.

    got_idx/got_val: [M, K] from the selector under test (slot order free, valid
    slots first); want_idx: [M, K] oracle indices.  Values must be bit copies of
    the inputs, padding must be (-1, -inf).
    """
    sbits = np.ascontiguousarray(scores, dtype=np.float32).view(np.uint32)
    gbits = None if got_val is None else np.ascontiguousarray(got_val, dtype=np.float32).view(np.uint32)
    for r in (range(len(row_lengths)) if rows is None else rows):
        L = max(int(row_lengths[r]), 0)
        m = min(K, L)
        g = got_idx[r]
        assert (g[m:] == -1).all(), f"row {r}: padding slots must hold -1"
        assert (g[:m] >= 0).all() and (g[:m] < L).all(), f"row {r}: index out of range"
        order = np.argsort(g[:m], kind="stable")
        gs = g[:m][order]
        ws = np.sort(want_idx[r, :m])
        if not np.array_equal(gs, ws):
            missing = np.setdiff1d(ws, gs)[:5]
            extra = np.setdiff1d(gs, ws)[:5]
            raise AssertionError(f"row {r} (L={L}): index set differs; missing {missing}, extra {extra}")
        if gbits is not None:
            s0 = int(row_starts[r])
            assert np.array_equal(gbits[r, :m][order], sbits[s0:s0 + L][gs]), f"row {r}: value bits differ"
            assert (gbits[r, m:] == 0xFF800000).all(), f"row {r}: padding values must be -inf"
