"""Host-side parts of bench.py that need no GPU: the work counts the roofline figures rest on and the reference arm."""
import json
import math
import os
import subprocess
import sys

import bench

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_compare_exchange_count_of_the_sorting_network():
    # 32 keys per lane by odd-even merge sort (Batcher: (p^2 - p + 4) 2^(p-2) - 1 compare-exchanges for 2^p keys),
    # then bitonic merges of width 64 .. n: n/2 compare-exchanges per stage, log2(width) stages per merge
    assert bench.odd_even_merge_sort_size(32) == (25 - 5 + 4) * 8 - 1 == 191
    assert bench.odd_even_merge_sort_size(4) == 5 and bench.odd_even_merge_sort_size(8) == 19
    for n in (32, 64, 256, 1024, 4096):
        e = min(32, n // 32)                      # keys per lane: a row is spread over at least 32 lanes
        want, w = (n // e) * bench.odd_even_merge_sort_size(e), 2 * e
        while w <= n:
            want += (n // 2) * int(math.log2(w))
            w *= 2
        assert bench.compare_exchanges(n) == want
    assert bench.compare_exchanges(32) == 16 * (1 + 2 + 3 + 4 + 5)           # one key per lane: a plain bitonic sort
    assert bench.compare_exchanges(1024) == 32 * 191 + 512 * (6 + 7 + 8 + 9 + 10) == 26592
    assert bench.compare_exchanges(4096) == 128 * 191 + 2048 * (6 + 7 + 8 + 9 + 10 + 11 + 12)


def test_stage_work_counts():
    from paper_1803_04209_b200 import inputs
    wl = inputs.WORKLOADS["n1024"]
    work = bench.stage_work(wl, wl.S)
    assert work["emission"] == ("tensor", 2 * wl.S * wl.H * 2 * wl.N)          # [mean | logvar] = W4 v: 2N x H per sample
    assert work["sort"] == ("alu", wl.S * 2 * 26592)                            # a compare-exchange is a min and a max
    assert work["chain"][0] == "alu" and work["chain"][1] == wl.S * (wl.window * (2 * 16 * 256 + 256) + 4 * 16 * 256)
    fp32 = bench.stage_work(inputs.WORKLOADS["n128"], 16384)
    assert fp32["emission"][0] == "alu"                                         # no tensor cores on the fp32 precision


def test_reference_arm_prints_the_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "1", "--warmup", "0", "--reference-samples", "128"], capture_output=True, text=True,
                         cwd=ROOT, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    assert line["impl"] == "reference" and line["higher_is_better"] is True and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["config"]["workload"] == "tiny" and line["metric"] == "predicted_worker_times_per_sec"
