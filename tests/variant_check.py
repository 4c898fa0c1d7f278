"""Runs a few batches through the selector in a fresh process and compares them with the CPU
oracle; used by test_gpu_variants.py to exercise the kernel variants that are selected per
process by the HPCTOPK_VARIANT environment variable."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from oracle import native  # noqa: E402
from paper_2609_08450_b200 import binding as B, workloads as W  # noqa: E402
from tests.helpers import assert_rows_match  # noqa: E402


def main():
    dev = "cuda"
    cases = [(W.config1(dev), 2048), (W.config1(dev, seed=5, num_rows=600, max_len=30000, K=512), 512),
             (W.config5(1024, B.hpctopk_query_policy(1024, 65536)[0], dev, num_rows=96), 1024),
             (W.config4(dev, seed=9, num_rows=3, len_lo=200000, len_hi=300000), 4096)]
    for batch, K in cases:
        oi, ov, ws = B.hpctopk_select(batch.scores, batch.row_starts, batch.row_lengths, K)
        torch.cuda.synchronize()
        s, st, ln = batch.host()
        want, _, _ = native.topk_stable_sort(s, st, ln, K)
        assert_rows_match(s, st, ln, K, oi.cpu().numpy(), ov.cpu().numpy(), want)
        stats = B.hpctopk_read_stats(ws)
        assert stats["error_flags"] == 0
        assert sum(stats[f"rows_{n}"] for n in B.ROUTE_NAMES) + stats["rows_band2"] == batch.num_rows
    print("variant ok", os.environ.get("HPCTOPK_VARIANT", "default"))


if __name__ == "__main__":
    main()
