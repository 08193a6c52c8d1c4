"""The seeded input generator: shapes, reproducibility, target statistics."""
import numpy as np

import synthgen as sg


def test_resnet_shapes_and_totals():
    r18, r50 = sg.resnet18_conv_shapes(), sg.resnet50_conv_shapes()
    assert len(r18) == 20 and sum(int(np.prod(s)) for _, s in r18) == 11_166_912
    assert len(r50) == 53 and sum(int(np.prod(s)) for _, s in r50) == 23_454_912
    assert min(int(np.prod(s)) for _, s in r50) == 4096
    assert max(int(np.prod(s)) for _, s in r50) == 2_359_296


def test_c_helper_equals_numpy_statement():
    for spec in sg.workload_conv3x3() + sg.workload_resnet50()[:3]:
        assert (sg.draw_symbols(spec) == sg.draw_symbols_numpy(spec)).all()


def test_generator_is_seeded():
    a, b = sg.workload_conv3x3(0)[0], sg.workload_conv3x3(1)[0]
    assert (sg.draw_symbols(a) == sg.draw_symbols(a)).all()
    assert (sg.draw_symbols(a) != sg.draw_symbols(b)).any()
    assert sg.splitmix64_at(0, 0) == 0xE220A8397B1DCDAF      # SplitMix64, first output for seed 0


def test_target_statistics():
    c1 = sg.workload_conv3x3()[0]
    x = sg.draw_symbols(c1)
    assert c1.alphabet == 15 and c1.zero_point == 7 and c1.n == 36864
    assert abs((x == 7).mean() - 0.6) < 0.01
    r18 = sg.workload_resnet18()
    assert {l.bitwidth for l in r18} <= {2, 3, 4, 6}
    assert all(0.75 <= sg.entropy_bits(l.pmf()) <= 1.55 for l in r18)
    r50 = sg.workload_resnet50()
    assert {l.bitwidth for l in r50} <= set(range(1, 9))
    assert all(0.849 <= l.pmf()[l.zero_point] <= 0.951 for l in r50)
    tot = sum(l.n * sg.entropy_bits(l.pmf()) for l in r50) / sum(l.n for l in r50)
    assert tot < 1.0
    big = sg.workload_large()[0]
    assert big.alphabet == 7 and abs(big.pmf()[3] - 0.7) < 1e-4
    sw = sg.workload_sweep(n=1 << 16)[0]
    assert abs(sg.entropy_bits(sw.pmf()) - 2.5) < 1e-3
