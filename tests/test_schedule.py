"""Host-side schedule and cost-model helpers of the library against the oracle (no GPU needed)."""
import os

from paper_2601_17818_b200 import binding as vb
from paper_2601_17818_b200.build import build_library

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def test_schedule_helpers_match_the_oracle_and_the_printed_counts():
    build_library()
    rows = [list(map(float, l.split())) for l in open(os.path.join(GOLDEN, "retention_ratios.txt"))
            if l.strip() and not l.startswith("#")]
    printed = {66.7: (288, 253, 50), 77.8: (230, 165, 33), 88.9: (172, 77, 15), 94.4: (144, 33, 6)}
    for rate, p1, p2, p3 in rows:
        assert tuple(vb.vitcop_stage_count(576, p) for p in (p1, p2, p3)) == printed[rate]
        assert abs(vb.vitcop_cr_int(p1, p2, p3) - oracle.cr_int(p1, p2, p3)) < 1e-12
        for n_text, d in ((64, 4096), (128, 5120)):
            a = vb.vitcop_flops_total(576, n_text, d, p1, p2, p3)
            b = oracle.flops_vitcop(576, n_text, d, p1, p2, p3)
            assert abs(a - b) <= 1e-12 * b
        for l in (1, 2, 21, 22, 32):
            assert vb.vitcop_visual_tokens_at_layer(l, 576, p1, p2, p3) == oracle.visual_tokens_at_layer(l, 576, p1, p2, p3)
    for N, d in ((1, 1), (640, 4096), (2944.5, 5120)):
        assert vb.vitcop_flops_layer(N, d) == oracle.flops_layer(N, d)
    assert vb.vitcop_stage_count(2880, 0.05) == 144 and vb.vitcop_stage_count(0, 0.5) == 0
