"""The byte model of Sec. 6 (Eq. 4 static, Eq. 5 dynamic) against the paper's Table 5."""
import os

import pytest

from paper_2105_04246_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table5_memory_movement.txt")


def _rows():
    with open(GOLDEN) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                yield [int(v) for v in line.split()]


@pytest.mark.parametrize("row", list(_rows()))
def test_table5(row):
    k, cin, cout, w, h, dw, static_kb, dynamic_kb = row
    s = wl.ConvShape("t5", 1, h, w, cin, cout, k, k, 1, k // 2, groups=cin if dw else 1)
    tol = 2.0 if (dw and cin == 144) else 0.51
    assert wl.layer_static_bytes(s) / 1024 == pytest.approx(static_kb, abs=tol)
    assert wl.layer_dynamic_bytes(s) / 1024 == pytest.approx(dynamic_kb, abs=tol)


def test_overhead_statements():
    # "in most cases about 4x", up to "8x" for point-wise convolutions (Sec. 6)
    r = [wl.layer_dynamic_bytes(s) / wl.layer_static_bytes(s) for s in (wl.CFG2_CONV.with_batch(1), wl.CFG4_EXPAND.with_batch(1))]
    assert 4.0 < r[0] < 5.1 and 7.5 < r[1] < 8.0


def test_resnet18_inventory():
    convs, fc = wl.resnet18_layers(128)
    assert len(convs) == 20 and fc.N == 1000 and fc.K == 512
    assert sum(c.ops for c in convs) + fc.ops == pytest.approx(464.4e9, rel=2e-3)
    assert convs[0].Ho == 112 and convs[-1].Ho == 7
