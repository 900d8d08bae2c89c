"""Operation head-count (Appendix H) and the budget of a sparse expansion (Sec. 3.1 / 4.3): host-side
helpers of the C ABI against the oracle's closed forms, and the closed forms against what the paper
prints and what the formulas imply."""
import math
import os

import numpy as np
import pytest

from oracle import pipe_oracle as O
from paper_2311_15806_b200 import binding as B
from paper_2311_15806_b200 import build as pipe_build

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")

SHAPES = [  # d, D, n_i, n_o, s
    (3, 56, 256, 256, 1),     # the 3x3 convolution of the ConvNet configuration
    (1, 1, 768, 3072, 1),     # fully connected: d = D = s = 1
    (1, 1, 11008, 4096, 1),
    (3, 112, 32, 64, 2),
    (7, 224, 3, 64, 2),
    (1, 14, 960, 160, 1),
]


@pytest.fixture(scope="module")
def lib():
    pipe_build.build()
    return B.lib()


def _budget_rows():
    with open(os.path.join(GOLDEN, "budgets.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if line:
                yield int(line[0]), float(line[1]), float(line[2])


# ---- the oracle's closed forms against the appendix ------------------------------------------
def test_fully_connected_layer_counts_its_products():
    """Appendix H: for a fully connected layer D = s = d = 1, so the fp32 layer costs n_i n_o products of
    32 * log 32 = 160 bit operations, and one int-b order costs n_i n_o * b log b plus the two rescalings."""
    n_i, n_o = 768, 3072
    assert O.bit_ops_original(1, 1, n_i, n_o, 1) == n_i * n_o * 160.0
    assert O.bit_ops_expanded(1, 1, n_i, n_o, 1, 4, 1.0) == (n_i + n_o) * 160.0 + n_i * n_o * 8.0
    assert O.bit_ops_expanded(1, 1, n_i, n_o, 1, 8, 3.0) == (n_i + n_o) * 160.0 + 3 * n_i * n_o * 24.0


@pytest.mark.parametrize("shape", SHAPES)
def test_each_order_adds_one_integer_convolution(shape):
    """The k-th order adds exactly D^2 d^2 n_i n_o / s^2 products of b log b bit operations, and with
    32-bit "codes" one order is the fp32 layer plus the rescalings."""
    d, D, n_i, n_o, s = shape
    products = D * D * d * d * n_i * n_o / (s * s)
    for bits in (2, 3, 4, 8):
        for k in (1, 2, 5):
            step = O.bit_ops_expanded(*shape, bits, k) - O.bit_ops_expanded(*shape, bits, k - 1)
            assert math.isclose(step, products * bits * math.log2(bits), rel_tol=1e-12)
    extra = O.bit_ops_expanded(*shape, 32, 1.0) - O.bit_ops_original(*shape)
    assert math.isclose(extra, D * D * (n_i + n_o / (s * s)) * 160.0, rel_tol=1e-12)


def test_printed_budgets():
    """The budgets the paper prints (tests/golden/budgets.txt): beta = 1 + (K - 1) gamma; and Sec. 4.3's
    equal-cost argument "150 % of 4 bits ~ 6 bits"."""
    for K, gamma, beta in _budget_rows():
        assert math.isclose(O.budget_of(K, gamma), beta, rel_tol=1e-12)
    assert O.budget_of(2, 0.5) * 4 == 6.0


# ---- the library against the oracle ----------------------------------------------------------
@pytest.mark.parametrize("shape", SHAPES)
def test_library_counts_match_the_oracle(lib, shape):
    assert math.isclose(B.pipe_bit_ops_original(*shape), O.bit_ops_original(*shape), rel_tol=1e-13)
    for bits in (2, 3, 4, 6, 8, 32):
        for orders in (0.0, 1.0, 1.5, 2.75, 7.0):
            assert math.isclose(B.pipe_bit_ops_expanded(*shape, bits, orders), O.bit_ops_expanded(*shape, bits, orders),
                                rel_tol=1e-13)


@pytest.mark.parametrize("shape", SHAPES)
def test_max_orders_is_the_last_one_within_the_fp32_count(lib, shape):
    """Brute force over k with the oracle's formulas."""
    for bits in (2, 4, 8, 16):
        k = B.pipe_max_orders_within_original(*shape, bits)
        base = O.bit_ops_original(*shape)
        expect = 0
        while O.bit_ops_expanded(*shape, bits, expect + 1) <= base:
            expect += 1
        assert k == expect
        if k > 0:
            assert O.bit_ops_expanded(*shape, bits, k) <= base < O.bit_ops_expanded(*shape, bits, k + 1)
    # 32-bit codes never fit: one order already costs the fp32 layer plus the rescalings
    assert B.pipe_max_orders_within_original(*shape, 32) == 0


def test_gamma_from_budget(lib):
    for K, gamma, beta in _budget_rows():
        g = B.pipe_gamma_from_budget(beta, K)
        assert math.isclose(g, gamma, rel_tol=1e-12)
        assert math.isclose(O.budget_of(K, g), beta, rel_tol=1e-12)
        # and the kept groups of a layer follow from it
        assert B.pipe_keep_groups_from_gamma(56, g) == O.keep_groups(56, gamma)
    assert B.pipe_gamma_from_budget(1.0, 1) == 1.0 and B.pipe_gamma_from_budget(1.0, 4) == 0.0
    assert B.pipe_gamma_from_budget(4.0, 4) == 1.0
    for beta, K in ((0.5, 2), (3.5, 3), (2.0, 1), (float("nan"), 2), (1.5, 0), (1.5, 17)):
        with pytest.raises(B.PipeError):
            B.pipe_gamma_from_budget(beta, K)


def test_invalid_shapes_are_refused(lib):
    assert B.pipe_bit_ops_original(0, 1, 1, 1, 1) < 0
    assert B.pipe_bit_ops_expanded(1, 1, 1, 1, 1, 1, 1.0) < 0
    assert B.pipe_bit_ops_expanded(1, 1, 1, 1, 1, 4, -1.0) < 0
    assert B.pipe_max_orders_within_original(1, 1, 1, 0, 1, 4) == -1
