"""lpdt_message_bytes (host arithmetic of the C library) against hand cases and against the Data (GB)
column of the paper's CIFAR-10 table (tests/golden/cifar_data_column.txt).

What the table fixes, and what it does not:
  - uncompressed full-precision rows = 4 bytes x parameters x iterations (iterations = 200 epochs x
    ceil(50 000 / (nodes x 32))); the printed parameter counts have 2-3 digits, so the match is to 2 %;
  - every low-precision entry is the full-precision entry divided by four (to the printed digits): the
    table counts 8-bit values and scales whatever else the message holds by the same factor;
  - the compressed ResNet rows are 1.5 x (kept fraction) of the uncompressed rows: a kept entry costs one
    and a half values, i.e. a 32-bit value plus a 16-bit position;
  - the compressed VGG-11 row is 1.09 x the kept fraction: it fits neither 0, 16 nor 32 index bits; it lies
    between "values only" and "16-bit positions", which is all this test asserts for it.
"""
import math
import os

import pytest

from paper_2111_09389_b200 import api

HERE = os.path.dirname(os.path.abspath(__file__))


def rows():
    out = []
    for line in open(os.path.join(HERE, "golden", "cifar_data_column.txt")):
        if line.startswith("#") or not line.strip():
            continue
        m, p, n, c, fp, lp = line.split()
        out.append((m, float(p) * 1e6, int(n), int(c), float(fp), float(lp)))
    return out


def iterations(nodes, batch=32, samples=50000, epochs=200):
    return epochs * math.ceil(samples / (nodes * batch))


def test_hand_cases():
    mb = api.lpdt_message_bytes
    assert mb(1000, [0, 1000], [1000], 32, 32) == 4000            # dense: no positions
    assert mb(1000, [0, 1000], [5000], 32, 32) == 4000            # k beyond the segment = dense
    assert mb(1000, [0, 1000], [10], 32, 32) == 80                # 10 values + 10 positions
    assert mb(1000, [0, 1000], [10], 32, 0) == 40                 # values only
    assert mb(1000, [0, 1000], [10], 8, 32) == 10 + 40 + 4        # codes + positions + one fp32 step
    assert mb(1000, [0, 1000], [1000], 8, 32) == 1000 + 4
    assert mb(1000, [0, 400, 1000], [4, 600], 32, 16) == 4 * 6 + 600 * 4       # one compressed, one dense segment
    assert mb(1000, [0, 400, 1000], [0, 0], 8, 16) == 0           # nothing kept: nothing sent, no step either
    assert mb(10, [0, 10], [3], 8, 12) == (3 * 8 + 3 * 12 + 32 + 7) // 8       # rounded up to whole bytes
    assert mb(1000, [0, 999], [10], 32, 32) == -1                 # segments must tile [0, d)
    assert mb(1000, [0, 1000], [10], 12, 32) == -1                # value width not offered


@pytest.mark.parametrize("row", rows(), ids=lambda r: f"{r[0]}-n{r[2]}-c{r[3]}")
def test_data_column(row):
    model, d, nodes, comp, fp_gb, lp_gb = row
    d = int(d)
    it = iterations(nodes)
    k = d if comp == 0 else max(1, round(d * (100 - comp) / 100))
    gb = lambda value_bits, index_bits, kk=k: api.lpdt_message_bytes(d, [0, d], [kk], value_bits, index_bits) * it / 1e9
    assert lp_gb == pytest.approx(fp_gb / 4, rel=2e-3)            # the table's own factor of four
    if comp == 0:
        assert gb(32, 32) == pytest.approx(fp_gb, rel=0.02)       # the parameter count is printed to 2-3 digits
        assert gb(8, 32) == pytest.approx(lp_gb, rel=0.02)        # d codes + one 4-byte step per message
        assert gb(8, 32) / gb(32, 32) == pytest.approx(0.25, abs=1e-4)
        return
    # compressed rows relative to the uncompressed row of the same model and graph (the parameter count cancels)
    dense_fp = [r[4] for r in rows() if r[0] == model and r[2] == nodes and r[3] == 0][0]
    table_ratio = fp_gb / dense_fp
    ours = lambda value_bits, index_bits: gb(value_bits, index_bits) / gb(32, 32, d)
    if model != "vgg11":
        assert ours(32, 16) == pytest.approx(table_ratio, rel=0.02)     # a 32-bit value + a 16-bit position per kept entry
        assert ours(32, 0) < 0.7 * table_ratio and ours(32, 32) > 1.25 * table_ratio
        # 8-bit values with the same positions shrink the message by 2 (6 -> 3 bytes per entry), not by 4;
        # the table's low-precision figure is the values-only factor applied to the whole message
        assert gb(8, 16) / gb(32, 16) == pytest.approx(0.5, abs=1e-3)
        assert gb(8, 0) / gb(32, 0) == pytest.approx(0.25, abs=1e-3)
    else:
        assert ours(32, 0) < table_ratio < ours(32, 16)
