"""Pins for the oracle's footprint report against the sizes the paper prints."""
import os

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_accumulate_sizes.txt")


def _golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = [t.strip() for t in line.split("=")]
            out[k] = float(v)
    return out


def test_paper_accumulate_sizes():
    g = _golden()
    R = int(g["processes"])
    n = int(g["tokens_per_process"] * g["lookups_per_process"])
    rep = oracle.bytes_report([n] * R, int(g["d"]), int(g["vocab"]))
    # dense accumulate: printed 139 MB
    assert abs(rep["dense_bytes"] / 1e6 - g["dense_accumulate_MB"]) / g["dense_accumulate_MB"] < 0.01
    # sparse accumulate: printed 11.4 GB ("exceeding 11GB")
    assert abs(rep["gather_all_value_bytes"] / 1e9 - g["sparse_accumulate_GB"]) / g["sparse_accumulate_GB"] < 0.01
    assert rep["gather_all_value_bytes"] / 1e9 > 11.0
    # "82x" / "more than 82x"
    assert int(rep["gather_all_over_dense"]) == int(g["reduction_factor"])


def test_plain_arithmetic():
    rep = oracle.bytes_report([10240] * 64, 1024, 33708)
    assert rep["n_rows_total"] == 655360
    assert rep["sparse_value_bytes"] == 655360 * 1024 * 4 == 2684354560
    assert rep["sparse_index_bytes"] == 655360 * 8
    assert rep["dense_bytes"] == 33708 * 1024 * 4 == 138067968
    assert abs(rep["sparse_over_dense"] - (2684354560 + 5242880) / 138067968) < 1e-12
    rep = oracle.bytes_report([1048576], 1024, 65536, index_dtype="i32", value_dtype="bf16", out_dtype="bf16")
    assert rep["sparse_value_bytes"] == 1048576 * 1024 * 2
    assert rep["sparse_index_bytes"] == 1048576 * 4
    assert rep["dense_bytes"] == 65536 * 1024 * 2
    rep = oracle.bytes_report([], 8, 0)
    assert rep["sparse_bytes"] == 0 and rep["dense_bytes"] == 0 and rep["sparse_over_dense"] == 0.0


def test_growth_with_ranks():
    # Section 3: the gathered buffer grows with the number of processes, the dense one does not.
    a = oracle.bytes_report([10000] * 32, 1024, 33708)
    b = oracle.bytes_report([10000] * 64, 1024, 33708)
    assert b["gather_all_value_bytes"] == 2 * a["gather_all_value_bytes"]
    assert b["sparse_bytes"] == 2 * a["sparse_bytes"]
    assert b["dense_bytes"] == a["dense_bytes"]
