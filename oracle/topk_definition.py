"""Plain definition of the operator: per row, the K largest FP32 scores.

Operator contract (Section 2.1, "Operator contract"), with the three choices the
contract leaves open fixed as follows:

* order of scores: the monotone float-to-uint key on the raw bit pattern, so
  -0.0 sorts directly below +0.0, +-inf and subnormals sort numerically and a
  NaN bit pattern has a defined place (positive NaN above +inf, negative NaN
  below -inf);
* ties at rank K: the lower index wins, which makes the selected set unique;
* a row with L <= K returns every valid index followed by -1 sentinels; the
  returned values are bit copies of the inputs and padding values are -inf.

The sampled method of the paper reaches exactly this result (Theorem
"End-to-End Exactness", Section 4.4), so the oracle is the definition itself:
a stable sort of the row's indices by descending key.  Nothing is blocked,
fused or reordered.
"""
import numpy as np

NEG_INF_BITS = np.uint32(0xFF800000)


def float_bits(x):
    """Raw 32-bit patterns of an fp32 array (no numeric conversion)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return x.view(np.uint32)


def key_ascending(bits):
    """Monotone float-to-uint key: larger score <=> larger key.

    Sign bit clear: set it.  Sign bit set: invert all bits.  (The "sortable
    key" used in Sections 4.2 and 4.3; the paper's kappa_32-descending key is
    the bitwise complement of this one.)
    """
    bits = np.asarray(bits, dtype=np.uint32)
    negative = (bits >> np.uint32(31)).astype(bool)
    return np.where(negative, ~bits, bits | np.uint32(0x80000000)).astype(np.uint32)


def topk_row(row, K):
    """Indices (int32, best first) of the min(K, L) largest entries of one row."""
    key = key_ascending(float_bits(row))
    # descending key == ascending complement; a stable sort keeps the lower
    # index first among equal keys.
    order = np.argsort(~key, kind="stable")
    return order[: min(K, len(order))].astype(np.int32)


def topk_rows(scores, row_starts, row_lengths, K):
    """Apply the definition to every row of a packed ragged batch.

    scores      : 1-D fp32 array holding all rows back to back
    row_starts  : element offset of each row inside ``scores``
    row_lengths : valid length of each row (a negative length counts as 0)
    returns (out_idx [M, K] int32, out_val [M, K] fp32): best first, then
    (-1, -inf) padding.
    """
    scores = np.ascontiguousarray(scores, dtype=np.float32)
    M = len(row_lengths)
    out_idx = np.full((M, K), -1, dtype=np.int32)
    out_val_bits = np.full((M, K), NEG_INF_BITS, dtype=np.uint32)
    sbits = scores.view(np.uint32)
    for r in range(M):
        L = max(int(row_lengths[r]), 0)
        s = int(row_starts[r])
        sel = topk_row(scores[s:s + L], K)
        out_idx[r, : len(sel)] = sel
        out_val_bits[r, : len(sel)] = sbits[s:s + L][sel]
    return out_idx, out_val_bits.view(np.float32)
