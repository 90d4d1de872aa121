"""The byte / operation model behind bench.py's roofline figures (host logic, no GPU): totals that the paper's
tables and simple counting fix."""
from __future__ import annotations

import bench
from paper_2011_10680_b200 import inputs


def test_resnet50_operation_count_matches_the_papers_bops_column():
    # Table 1b: ResNet-50 at W8A8 has 247 G BOPS = 64 x MACs, i.e. 3.86 G MACs per image (stride on the first 1x1)
    rows = bench.layer_work(bench.workload_table("resnet50_int8_b256"), 1)
    macs = sum(r["ops"] for r in rows) // 2
    assert abs(macs * 64 / 1e9 - 247) < 1.0


def test_bytes_count_every_operand_once_at_its_own_width():
    t = bench.workload_table("inception_modules_int4_b256")
    rows = bench.layer_work(t, 2)
    shapes, bits = t["shapes"], t["bits"]
    size = lambda i: 2 * shapes[i][0] * shapes[i][1] * shapes[i][2] * bits[i] // 8
    for r in rows:
        l = t["layers"][r["layer"]]
        if l["op"] == "concat":           # every branch (the INT32 pooling branch at four bytes a value) + the output
            assert r["bytes"] == sum(size(i) for i in l["ins"]) + size(r["layer"])
        elif l["op"] == "sumpool":        # 8-bit module input, INT32 sums
            assert r["bytes"] == size(l["in0"]) + size(r["layer"])
    # the INT32 residual stream moves several times the bytes of the fused 8-bit stream (Fig. 2 against the fused form)
    wide = sum(r["bytes"] for r in bench.layer_work(bench.workload_table("resnet50_int8_int32stream_b256"), 256))
    fused = sum(r["bytes"] for r in bench.layer_work(bench.workload_table("resnet50_int8_b256"), 256))
    assert 4.5 < wide / fused < 6.5
