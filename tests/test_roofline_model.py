"""The ops/bytes model used for roofline figures reproduces the intensities the paper prints."""
import os

from paper_2606_14598_b200 import roofline

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "arithmetic_intensity.txt")


def test_arithmetic_intensity_end_points():
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) == 2
    for M, N, K, want in rows:
        got = roofline.arithmetic_intensity(int(M), int(N), int(K))
        assert round(got) == int(want), (M, N, K, got)
