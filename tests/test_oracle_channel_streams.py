"""Stream grouping by input channel, at the level of the oracle (paper Section III-B, Table III).

The paper codes a ResNet-50 once as a single stream per layer and once with the weights of each
layer "grouped by input channel and separately encoded", for tables of 256, 128 and 64 states, and
reports (i) that the parallel streams cost less than 1 % more than the single stream and (ii) the
gap to the entropy bound: under 3 % with 256 states, under 15 % with 64.  Its sizes need the
trained network; the two statements can be checked on synthetic layers of the same shapes and a
similar statistic (31 bins early, fewer later, about 0.85 bit per weight): every input channel of
every conv layer is coded as its own lane by the plain coder, and a lane costs its bits plus the
R bits of its initial state."""
import math

import numpy as np
import pytest

import oracle
import synthgen as sg


def _study_layers():
    """All 53 ResNet-50 convs (23.5 M weights): 31 bins in the first half of the network, 15 then
    7 bins later (the paper's training ends between 31 and 13 bins), entropy 0.85 bit per weight."""
    shapes = sg.resnet50_conv_shapes()
    layers = []
    for li, (name, shape) in enumerate(shapes):
        b = 5 if li < len(shapes) // 2 else 4 if li < 3 * len(shapes) // 4 else 3
        A, zp = sg.alphabet_for_bits(b)
        spec = sg.LayerSpec(name, shape, b, A, zp, sg.theta_for_entropy(A, zp, 0.85), 1.0, 8, 1 << 20, "u8",
                            sg.stream_key(77, li))
        layers.append((spec, sg.draw_symbols(spec).reshape(shape)))
    return layers


def _entropy_bits(sym):
    c = np.bincount(sym.ravel(), minlength=256).astype(np.float64)
    p = c[c > 0] / sym.size
    return float(-(p * np.log2(p)).sum()) * sym.size


@pytest.fixture(scope="module")
def study():
    layers = _study_layers()
    rows = {}
    container = {}
    for R in (8, 7, 6):
        single = parallel = packed = 0
        for spec, w in layers:
            T = oracle.Table(oracle.normalize_freqs(oracle.histogram(w.ravel()), spec.alphabet, R), R)
            single += oracle.encode_plain(T, w.ravel())[2] + R
            per_channel = np.ascontiguousarray(np.moveaxis(w, 1, 0)).reshape(w.shape[1], -1)
            here = 0
            for c in range(per_channel.shape[0]):
                here += oracle.encode_plain(T, per_channel[c])[2] + R
            parallel += here
            # the same streams in the channels container (one chunk per layer, a lane per input
            # channel, pieces of H*W symbols over the O x I x H x W tensor as stored); the first
            # conv has 3 input channels and stays outside, as the paper leaves it uncompressed
            if w.shape[1] % 32 == 0:
                P = oracle.pack(T, w.ravel(), w.size, w.shape[1] // 32, oracle.CHANNELS, piece=w.shape[2] * w.shape[3])
                lanes_bits = here + 16 * w.shape[1]        # every lane adds a 16-bit length
                assert lanes_bits <= P.stream.size * 8 < lanes_bits + (w.shape[1] // 32) * (128 + 32)
                packed += P.total_bytes() * 8
            else:
                packed += here
        rows[R] = (single, parallel)
        container[R] = packed
    bound = sum(_entropy_bits(w) for _, w in layers)
    return rows, bound, sum(w.size for _, w in layers), container


def test_parallel_streams_cost_under_one_percent(study):
    rows, bound, n, _ = study
    for R, (single, parallel) in rows.items():
        assert single < parallel < 1.01 * single, (R, single, parallel)


def test_size_against_the_entropy_bound_by_table_size(study):
    rows, bound, n, container = study
    gap = {R: rows[R][0] / bound - 1.0 for R in rows}
    print("\nstates  single-stream MB  parallel MB  overhead  gap to entropy bound (%.3f MB, %.3f bit/weight)"
          % (bound / 8e6, bound / n))
    for R in (8, 7, 6):
        s, p = rows[R]
        print("%6d  %16.3f  %11.3f  %7.2f%%  %5.1f%%   channels container: %.3f MB (%.2f%% over the single stream)"
              % (1 << R, s / 8e6, p / 8e6, 100 * (p / s - 1), 100 * gap[R], container[R] / 8e6,
                 100 * (container[R] / s - 1)))
        assert container[R] < 1.04 * s                    # 16-bit lengths, padding and offsets included
    assert 0 < gap[8] < gap[7] < gap[6]
    assert gap[8] < 0.05 and gap[6] < 0.20          # the paper: under 3 % and under 15 %
    assert math.isclose(bound / n, 0.85, abs_tol=0.02)
