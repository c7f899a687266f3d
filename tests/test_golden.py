"""The numbers the paper prints that the path depends on (tests/golden/), against the constants
of the oracle-side generators, the C header and the library's own arithmetic."""
import math
import os
import re

from paper_2609_37626_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def golden():
    vals = {}
    for line in open(os.path.join(ROOT, "tests", "golden", "model_dimensions.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            vals[k] = int(v)
    return vals


def test_row_widths_head_count_and_scale_follow_the_printed_dimensions():
    g = golden()
    assert W.D_QK == g["d_c"] + g["d_r"] == 576 and W.D_V == g["d_c"] == 512
    assert W.SOFTMAX_SCALE == 1.0 / math.sqrt(g["d_n"] + g["d_r"])
    header = open(os.path.join(ROOT, "include", "splash_mla.h")).read()
    assert re.search(r"d_qk;\s*/\* 576", header) and re.search(r"d_v;\s*/\* 512", header)
    assert re.search(r"num_heads;\s*/\* H, 1\.\.%d" % g["H"], header)


def test_printed_weight_sizes_follow_from_the_dimensions():
    # the same paragraph derives bf16 projection sizes from the tuple; re-deriving them pins the reading of the
    # tuple's order (a swapped d_n / d_r or d_c / d_v would miss these integers)
    g = golden()
    mib = 1 << 20
    q_b = g["r_q"] * g["H"] * (g["d_n"] + g["d_r"]) * 2 / mib
    kv_b = g["d_c"] * g["H"] * (g["d_n"] + g["d_v"]) * 2 / mib
    o = g["H"] * g["d_v"] * g["d"] * 2 / mib
    assert (q_b, kv_b, o) == (g["q_b_mib"], g["kv_b_mib"], g["o_mib"])
    assert q_b + kv_b + o == g["total_mib"]
