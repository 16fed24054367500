"""Shape bookkeeping pins: the counting rules reproduce the totals the paper prints."""
import os

from paper_2010_00704_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_table2_counts.txt")


def _golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


def test_paper_table2_totals():
    g = _golden()
    p1, m1 = wl.paper_table1_binary_counts(1)
    p2, m2 = wl.paper_table1_binary_counts(2)
    assert (p1, m1) == (9042944, 2414870528)
    # the paper prints three significant digits
    assert abs(p1 - g["binary_parameters_P1"]) < 0.005e6
    assert abs(m1 - g["binary_macs_P1"]) < 0.005e9
    assert abs(p2 - g["binary_parameters_P2"]) < 0.005e6
    assert abs(m2 - g["binary_macs_P2"]) < 0.005e9


def test_workload_shapes():
    l = wl.SINGLE_3X3
    assert (l.M(1), l.C_out, l.K) == (1024, 128, 1152) and l.ops(1) == 2 * 1024 * 128 * 1152
    a, b = wl.STEM_DOWN
    assert (a.OH, a.M(64), a.K) == (56, 200704, 288)
    assert (b.OH, b.M(64), b.K) == (28, 50176, 576)
    assert [l.K for l in wl.BLOCK_STACK] == [256, 1152, 128, 4608]
    assert [l.M(128) for l in wl.BLOCK_STACK] == [100352, 100352, 100352, 25088]
    assert len(wl.BACKBONE18) == 18
    assert wl.chain_macs(wl.BACKBONE18) == 1374420992
    # every layer's input is the previous layer's output
    for prev, nxt in zip(wl.BACKBONE18[:-1], wl.BACKBONE18[1:]):
        assert (prev.OH, prev.OW, prev.C_out) == (nxt.H, nxt.W, nxt.C_in)
    for prev, nxt in zip(wl.BLOCK_STACK[:-1], wl.BLOCK_STACK[1:]):
        assert (prev.OH, prev.OW, prev.C_out) == (nxt.H, nxt.W, nxt.C_in)
    assert wl.BACKBONE18[2] == wl.STEM_DOWN[0].__class__(wl.BACKBONE18[2].name, 112, 112, 32, 64, 3, 2, 1)
    assert wl.BACKBONE18[-1].OH == 7 and wl.BACKBONE18[-1].C_out == 512


def test_paper_1x1_conv_list_reproduces_table2():
    # the per-layer list used as a workload must add up to the totals the paper prints
    for P in (1, 2):
        convs = wl.paper_binary_1x1_convs(P)
        params = sum(n * l.C_in * l.C_out for l, n in convs)
        macs = sum(n * l.macs(1) for l, n in convs)
        assert (params, macs) == wl.paper_table1_binary_counts(P)
    convs = wl.paper_binary_1x1_convs(1)
    assert sum(n for _, n in convs) == 32
    assert all(l.k == 1 and l.C_in == l.C_out for l, _ in convs)
    assert {l.C_in for l, _ in convs} == {32, 64, 128, 256, 512, 1024}
    assert {l.H for l, _ in convs} == {224, 112, 56, 28, 14, 7}
