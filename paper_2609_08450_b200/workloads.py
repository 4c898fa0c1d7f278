"""Seeded synthetic score batches (shared by the tests, the oracle runs and the bench).

This module only *produces inputs*: packed ragged FP32 score rows with int32
``row_starts`` / ``row_lengths``.  It contains none of the selector's arithmetic
and imports neither the CUDA binding nor the oracle.

The five recipes stand in for the indexer-score captures the paper evaluates on
(FP32 scores, K = 2048, causal ragged lengths, widths 16K-1M; Section 6.1):

  config 1  small ragged batch, i.i.d. N(0,1), lengths U[1, 32768], two rows < K
  config 2  decode batch: one row per sequence, lengths U[16384, 131072],
            scores s_j = sum_h w_h ReLU(q_h . k_j)  (the indexer of Eq. 1)
  config 3  prefill chunk: causal rows L_i = offset + 1 + i over one key matrix
            whose keys carry a slow positional drift
  config 4  long context: few rows of 0.5M-1M heavy-tailed (Student-t, nu = 3)
  config 5  adversarial structure: constant, 16-level, sorted, block, periodic
            at the sampling stride, signed zeros, -inf padding

Every size is a parameter so that CPU tests can run reduced copies of the same
recipes.  Lengths come from numpy's PCG64 on the host; scores come from a
``torch.Generator`` on the target device.
"""
from dataclasses import dataclass, field

import numpy as np
import torch

BASE_SEED = 20260908


@dataclass
class Batch:
    name: str
    scores: torch.Tensor        # 1-D fp32, rows packed back to back
    row_starts: torch.Tensor    # int32 [M]
    row_lengths: torch.Tensor   # int32 [M]
    kinds: list = field(default_factory=list)   # per-row label (config 5)

    @property
    def num_rows(self):
        return int(self.row_lengths.numel())

    @property
    def total_elements(self):
        return int(self.row_lengths.clamp(min=0).sum().item())

    def host(self):
        """(scores, row_starts, row_lengths) as numpy arrays."""
        return (self.scores.detach().cpu().numpy(), self.row_starts.cpu().numpy(),
                self.row_lengths.cpu().numpy())


def _starts(lengths):
    lengths = np.asarray(lengths, dtype=np.int64)
    starts = np.zeros(len(lengths), dtype=np.int64)
    if len(lengths) > 1:
        starts[1:] = np.cumsum(lengths[:-1])
    total = int(lengths.sum())
    assert total < 2 ** 31, "packed batch must be addressable with int32 offsets"
    return starts.astype(np.int32), total


def _finish(name, scores, lengths, device, kinds=None):
    starts, total = _starts(lengths)
    assert scores.numel() == total
    return Batch(name, scores.contiguous(), torch.from_numpy(starts).to(device),
                 torch.from_numpy(np.asarray(lengths, dtype=np.int32)).to(device), kinds or [])


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def config1(device="cpu", seed=BASE_SEED + 1, num_rows=8, max_len=32768, K=2048):
    rng = np.random.default_rng(seed)
    lengths = rng.integers(1, max_len + 1, size=num_rows)
    if K > 1:
        lengths[:2] = rng.integers(1, K, size=2)      # at least two rows shorter than K
    g = _gen(device, seed)
    scores = torch.randn(int(lengths.sum()), generator=g, device=device, dtype=torch.float32)
    return _finish("config1_ragged_normal", scores, lengths, device)


def _indexer_scores(q, k, w):
    """s_j = sum_h w_h ReLU(q_h . k_j): bf16 logits, FP32 weighted sum (Eq. 1).

    q [R, H, D] bf16, k [N, D] bf16, w [R, H] fp32  ->  [R, N] fp32
    """
    R, H, D = q.shape
    logits = torch.matmul(q.reshape(R * H, D), k.t())            # [R*H, N] bf16
    act = torch.relu(logits).reshape(R, H, -1).float()
    return torch.einsum("rh,rhn->rn", w, act).contiguous()


def config2(device="cpu", seed=BASE_SEED + 2, num_rows=64, len_lo=16384, len_hi=131072,
            heads=64, dim=128):
    rng = np.random.default_rng(seed)
    lengths = rng.integers(len_lo, len_hi + 1, size=num_rows)
    g = _gen(device, seed)
    std = float(dim) ** -0.25            # variance 1/sqrt(dim): q.k ~ N(0, 1)
    parts = []
    for L in lengths.tolist():
        q = (torch.randn(1, heads, dim, generator=g, device=device) * std).bfloat16()
        k = (torch.randn(L, dim, generator=g, device=device) * std).bfloat16()
        w = torch.randn(1, heads, generator=g, device=device) / 8.0
        parts.append(_indexer_scores(q, k, w).reshape(-1))
    return _finish("config2_decode_indexer", torch.cat(parts), lengths, device)


def config3(device="cpu", seed=BASE_SEED + 3, num_rows=4096, seq_len=131072, offset=126976,
            heads=64, dim=128, slab=32):
    assert offset + num_rows <= seq_len
    lengths = offset + 1 + np.arange(num_rows, dtype=np.int64)    # causal: L_i = offset + 1 + i
    starts, total = _starts(lengths)
    g = _gen(device, seed)
    std = float(dim) ** -0.25
    pos = torch.arange(seq_len, device=device, dtype=torch.float32)
    drift = 0.3 * torch.sin(pos / 4096.0)
    k = (torch.randn(seq_len, dim, generator=g, device=device) * std + drift[:, None]).bfloat16()
    scores = torch.empty(total, device=device, dtype=torch.float32)
    for r0 in range(0, num_rows, slab):
        r1 = min(r0 + slab, num_rows)
        q = (torch.randn(r1 - r0, heads, dim, generator=g, device=device) * std).bfloat16()
        w = torch.randn(r1 - r0, heads, generator=g, device=device) / 8.0
        s = _indexer_scores(q, k[: int(lengths[r1 - 1])], w)
        for r in range(r0, r1):
            L = int(lengths[r])
            scores[int(starts[r]): int(starts[r]) + L] = s[r - r0, :L]
    return _finish("config3_prefill_causal", scores, lengths, device)


def config4(device="cpu", seed=BASE_SEED + 4, num_rows=16, len_lo=524288, len_hi=1048576):
    rng = np.random.default_rng(seed)
    lengths = rng.integers(len_lo, len_hi + 1, size=num_rows)
    g = _gen(device, seed)
    n = int(lengths.sum())
    z = torch.randn(n, generator=g, device=device)
    chi2 = torch.zeros(n, device=device)
    for _ in range(3):
        chi2 += torch.randn(n, generator=g, device=device) ** 2
    scores = (z / torch.sqrt(chi2 / 3.0)).float()                 # Student-t, nu = 3
    return _finish("config4_long_student_t", scores, lengths, device)


ADVERSARIAL_KINDS = ("constant", "levels16", "ascending", "descending", "block", "periodic",
                     "signed_zeros", "neg_inf_pad")


def adversarial_row(kind, L, K, stride, rng):
    """One structured row (numpy fp32) of the named kind."""
    if kind == "constant":
        return np.full(L, np.float32(rng.normal()), dtype=np.float32)
    if kind == "levels16":
        levels = np.sort(rng.normal(size=16)).astype(np.float32)
        return levels[rng.integers(0, 16, size=L)]
    if kind == "ascending":
        return (np.arange(L, dtype=np.float64) * 0.25 - 1000.0).astype(np.float32)
    if kind == "descending":
        return (np.arange(L, dtype=np.float64)[::-1] * 0.25 - 1000.0).astype(np.float32)
    if kind == "block":
        x = rng.normal(size=L).astype(np.float32)
        width = min(K, L)
        o = int(rng.integers(0, L - width + 1))
        x[o:o + width] += np.float32(100.0)
        return x
    if kind == "periodic":
        v = rng.normal(size=stride).astype(np.float32)
        return v[np.arange(L) % stride]
    if kind == "signed_zeros":
        x = np.where(rng.random(L) < 0.5, np.float32(0.0), np.float32(-0.0)).astype(np.float32)
        few = rng.random(L) < 0.01
        x[few] = rng.normal(size=int(few.sum())).astype(np.float32)
        return x
    if kind == "neg_inf_pad":
        x = rng.normal(size=L).astype(np.float32)
        finite = int(rng.integers(0, L + 1)) if rng.random() < 0.5 else int(rng.integers(0, min(K, L) + 1))
        x[finite:] = -np.inf                                       # padded suffix
        x[rng.random(L) < 0.05] = -np.inf                          # scattered
        return x
    raise ValueError(kind)


def config5(K, stride, device="cpu", seed=BASE_SEED + 5, num_rows=256, long_len=65536):
    """Adversarial batch for one K; ``stride`` is the sampling stride the selector
    uses at this K (period of the "periodic" rows)."""
    rng = np.random.default_rng(seed + K)
    choices = [1, K - 1, K, K + 1, 4 * K, long_len]
    rows, lengths, kinds = [], [], []
    for r in range(num_rows):
        kind = ADVERSARIAL_KINDS[r % len(ADVERSARIAL_KINDS)]
        L = max(1, int(choices[(r // len(ADVERSARIAL_KINDS)) % len(choices)]))
        rows.append(adversarial_row(kind, L, K, stride, rng))
        lengths.append(L)
        kinds.append(kind)
    scores = torch.from_numpy(np.concatenate(rows)).to(device)
    return _finish(f"config5_adversarial_K{K}", scores, np.asarray(lengths), device, kinds)
