"""The handful of numbers the paper prints, as a fixture (tests/golden/paper_values.txt), against
the oracle."""
from pathlib import Path

import numpy as np

import oracle

GOLD = {}
for line in (Path(__file__).parent / "golden" / "paper_values.txt").read_text().splitlines():
    if line.strip() and not line.startswith("#"):
        key, value, _where = [p.strip() for p in line.split("|")]
        GOLD[key] = value


def test_dense_ternary_costs_what_the_paper_counts():
    bits = float(GOLD["reference_round_bits"]) / float(GOLD["reference_round_as_ternary_iterations"])
    assert bits == 2.0
    d = 128 * 50
    assert oracle.words_per_worker(d, oracle.CODEC_TERN2) * 32 / d == bits
    # on top of the symbols: one fp32 scale per block and the K coefficients of the fusion
    assert oracle.bits_per_coord(d, 4, oracle.CODEC_TERN2, 128) == bits + 32 / 128 + 64 * 4 / d


def test_rosenbrock_minimum():
    point = np.array([float(t) for t in GOLD["rosenbrock_minimum_point"].split()], dtype=np.float32)
    x = np.tile(point, 8)
    assert oracle.rosenbrock_value(x) == float(GOLD["rosenbrock_minimum_value"])
    assert not oracle.rosenbrock_grad(x).any()


def test_ternary_alphabet_and_initial_state():
    alphabet = sorted(float(t) for t in GOLD["ternary_alphabet"].split())
    rng = np.random.default_rng(0)
    g = rng.standard_normal((1, 1280)).astype(np.float32)
    st = oracle.State(1280, 1, 2, oracle.CODEC_TERN2, oracle.NORM_DIFF, seed_lo=1)
    out = st.step(g)
    assert GOLD["initial_reference"] == "zeros" and not st.ref().any()
    scales = np.repeat(st.scales()[0], 128)
    symbols = np.unique(np.round(out / scales, 6))
    assert set(symbols.tolist()) <= set(alphabet)
    # zero reference: the normalised gradient is the gradient, C_nz = 1
    assert oracle.cnz(g, st.ref()) == float(GOLD["degenerate_cnz"])
