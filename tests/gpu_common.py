"""Helpers for the GPU parity tests: run the CUDA library through its C ABI and compare
with the CPU oracle on the same materialised FP32 bits."""
import numpy as np
import torch

from oracle import native, sampled_steps as S
from paper_2609_08450_b200 import binding as B, build
from tests.helpers import assert_rows_match

build.build()


def run_gpu(batch, K, want_values=True, workspace=None):
    out_idx, out_val, ws = B.hpctopk_select(batch.scores, batch.row_starts, batch.row_lengths, K,
                                            want_values=want_values, workspace=workspace)
    torch.cuda.synchronize()
    return out_idx.cpu().numpy(), (out_val.cpu().numpy() if out_val is not None else None), ws


def check_batch(batch, K, rows=None, check_trace=False, want_values=True):
    """Bit-exact comparison of every (or the listed) row(s) with the stable-sort oracle."""
    got_idx, got_val, ws = run_gpu(batch, K, want_values)
    scores, starts, lengths = batch.host()
    M = len(lengths)
    if rows is None:
        want_idx, _, _ = native.topk_stable_sort(scores, starts, lengths, K)
        assert_rows_match(scores, starts, lengths, K, got_idx, got_val, want_idx)
    else:
        rows = np.asarray(rows)
        want_sub, _, _ = native.topk_stable_sort(scores, starts[rows], lengths[rows], K)
        want_idx = np.full((M, K), -2, dtype=np.int32)
        want_idx[rows] = want_sub
        assert_rows_match(scores, starts, lengths, K, got_idx, got_val, want_idx, rows=rows.tolist())
    stats = B.hpctopk_read_stats(ws)
    info = B.hpctopk_read_row_info(ws, M)
    assert stats["error_flags"] == 0
    assert sum(stats[f"rows_{n}"] for n in B.ROUTE_NAMES) + stats["rows_band2"] == M
    assert stats["elements_valid"] == int(np.clip(lengths, 0, None).sum())
    if check_trace:
        for r in (range(M) if rows is None else rows):
            L = max(int(lengths[r]), 0)
            _, t = S.select_row(scores[int(starts[r]):int(starts[r]) + L], int(r), K)
            cap = S.capacity_for(K)
            # candidates are stored per scanner warp; a row whose admitted tail is close to the
            # capacity and unevenly spread may take the overflow route although the total fits
            uneven = (info["route"][r] == S.ROUTE_OVERFLOW and t.route in (S.ROUTE_PRIMARY, S.ROUTE_BAND)
                      and max(t.C0, t.C1) > cap // 2)
            # the library's complete-row pass admits the nested tail A(tau_1) at once: the route is the
            # paper's unless that larger tail exceeds the capacity, and an underfilled row first tries a
            # wider band (route 6) where the paper's steps go straight to the recovery
            x = scores[int(starts[r]):int(starts[r]) + L]
            early_overflow = (info["route"][r] == S.ROUTE_OVERFLOW and t.route == S.ROUTE_PRIMARY
                              and int(np.count_nonzero(S.coarse_bin(x) <= t.tau1)) > cap)
            band2 = info["route"][r] == 6 and t.route == S.ROUTE_RECOVERY and t.tau0 >= 0
            assert info["route"][r] == t.route or uneven or early_overflow or band2, \
                (r, L, info[r], S.ROUTE_NAMES[t.route])
            if t.tau0 >= 0:
                assert info["tau"][r] == (t.tau0 | (t.tau1 << 16)), (r, info[r], t.tau0, t.tau1)
                if info["route"][r] == S.ROUTE_OVERFLOW:      # counted over the stored part of the tail only
                    assert info["c_tau0"][r] <= t.C0, (r, info[r], t.C0)
                else:
                    assert info["c_tau0"][r] == t.C0, (r, info[r], t.C0)
    return stats, info, got_idx, got_val
