"""The speed-up model and bit-width calculators against numbers the paper prints."""
import json
import os

import pytest

from oracle import roofline_model as rm


@pytest.fixture(scope="module")
def printed(golden_dir):
    with open(os.path.join(golden_dir, "paper_printed_values.json")) as f:
        return json.load(f)


def test_speedup_thresholds_l40s(printed):
    hw, sm = printed["l40s"], printed["speedup_model"]
    nu = hw["r_compute_flops"] / hw["r_transfer_bytes_per_s"]
    assert round(nu) == 419
    assert int(rm.memory_bound_batch_limit(4.25, nu)) == sm["memory_bound_m_4p25"]
    assert int(rm.memory_bound_batch_limit(1.25, nu)) == sm["memory_bound_m_1p25"]
    assert int(rm.memory_bound_batch_limit(16.0, nu)) == sm["no_speedup_beyond_m"]
    assert round(rm.speedup(16, 4.25, 1, nu), 1) == sm["peak_speedup_4p25"]
    assert round(rm.speedup(16, 1.25, 1, nu), 1) == sm["peak_speedup_1p25"]
    # regimes: flat up to the limit, ~1/m between, 1 beyond
    assert rm.speedup(16, 4.25, 111, nu) == pytest.approx(16 / 4.25)
    assert rm.speedup(16, 4.25, 112, nu) < 16 / 4.25
    assert rm.speedup(16, 1.25, 33, nu) < 16 / 1.25
    assert rm.speedup(16, 4.25, 419, nu) == 1.0 and rm.speedup(16, 1.25, 1000, nu) == 1.0
    mid = rm.speedup(16, 4.25, 200, nu) / rm.speedup(16, 4.25, 400, nu)
    assert mid == pytest.approx(2.0)


def test_speedup_is_ratio_of_kernel_times(printed):
    hw = printed["l40s"]
    rc, rt = hw["r_compute_flops"], hw["r_transfer_bytes_per_s"]
    for m in (1, 16, 64, 200, 512):
        for p1, p2 in ((16, 4.25), (16, 1.25), (4.25, 1.25)):
            t1 = rm.kernel_time(m, 8192, p1, rc, rt)
            t2 = rm.kernel_time(m, 8192, p2, rc, rt)
            assert t1 / t2 == pytest.approx(rm.speedup(p1, p2, m, rc / rt))


def test_bit_width_tables(printed):
    for n, pw in printed["integer_format_bit_width"].items():
        if n == "cite":
            continue
        # n = 5 is printed as 5.22 while log2(31) + 0.25 = 5.204: the table is
        # at odds with its own formula there, every other entry agrees to 0.01.
        slack = 0.02 if n == "5" else 0.005
        assert abs(rm.integer_format_bit_width(int(n)) - pw) <= slack
    ex = printed["block_format_example"]
    assert rm.block_bit_width(ex["n"], ex["scale_bits"], ex["block"]) == ex["p_w"]
    assert rm.per_row_codebook_bit_width(4, 4096) == 4 + 16 * 16 / 4096


def test_printed_effective_bandwidth_is_operand_bytes_over_time(printed):
    t = printed["table_microbench_h8192_m1"]
    h = t["h"]
    for row in t["rows"]:
        gbs = row["p_w"] * h * h / 8 / (row["time_us"] * 1e-6) / 1e9
        assert abs(gbs - row["eff_gbs"]) <= 1.5
