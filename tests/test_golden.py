"""The numbers the paper prints that the path depends on (tests/golden/), against the constants
of the oracle-side generators, the C header and the library's own arithmetic."""
import math
import os
import re

from paper_2609_37626_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def golden(name="model_dimensions.txt"):
    vals = {}
    for line in open(os.path.join(ROOT, "tests", "golden", name)):
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


def test_the_656_byte_row_fits_the_printed_kv_payloads():
    # per token and layer the printed payloads come to 788 bytes on both machines; the attention row read by sparse
    # decode (512 e4m3 codes + 4 fp32 block scales + 64 bf16 rope values) leaves 132 = 128 + 4 bytes, an fp8 indexer
    # key with one fp32 scale
    g = golden("kv_payload.txt")
    per_layer = g["payload_bytes_61_layers"] / g["layers_h200_model"]
    assert per_layer == 788
    tokens_per_card = g["dp_attention_distinct_tokens"] / g["group_size"]
    b200 = g["dp_attention_gib_per_card_x100"] / 100 * 2 ** 30 / tokens_per_card / g["layers_b200_model"]
    assert abs(b200 - 788) < 0.2                       # the table rounds GiB to two decimals
    row = W.D_LATENT + 4 * (W.D_LATENT // W.SPARSE_BLOCK) + 2 * W.D_ROPE
    assert row == W.SPARSE_ROW_BYTES == 656 and per_layer - row == 128 + 4
    header = open(os.path.join(ROOT, "include", "splash_mla.h")).read()
    assert re.search(r"#define SPLASH_SPARSE_ROW_BYTES 656", header)
