"""Layers that keep their codes as int8 in the tensor-core operand layout as well (pipe_layer_desc.int8_copy): the
convolution, inner-layer and chained cases of the other modules once more with such layers.  Results must be the same
bits as the oracle's, as they are from the packed codes."""
import pytest

from paper_2311_15806_b200 import binding as B
from tests import gpu_harness as H
from tests import test_gpu_inner_layer as TI
from tests import test_gpu_parity_small as TP

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def layers_keep_an_int8_copy(monkeypatch):
    monkeypatch.setattr(H, "INT8_COPY_DEFAULT", True)


def test_the_switch_reaches_the_descriptor():
    assert H.desc_of(64, 128, 4, 2, 8, 4).int8_copy == 1
    assert H.desc_of(64, 128, 4, 2, 4, 4).int8_copy == 0     # groups of 4 rows cannot keep one


@pytest.mark.parametrize("kernel", [B.KERNEL_AUTO, B.KERNEL_TCGEN05_PAIR])
@pytest.mark.parametrize("case", TP.CONV_CASES)
def test_implicit_convolution(oracle, kernel, case):
    TP.test_implicit_convolution_matches_oracle(oracle, kernel, *case)


@pytest.mark.parametrize("case", TP.ENSEMBLE_CONV_CASES)
def test_ensemble_convolution(oracle, case):
    TP.test_ensemble_convolution_matches_oracle(oracle, *case)


def test_ensemble_convolution_inner_layer(oracle):
    TP.test_ensemble_convolution_inner_layer_matches_oracle(oracle)


def test_two_layer_convolutional_chain(oracle):
    TP.test_two_layer_convolutional_ensemble_chain(oracle)


@pytest.mark.parametrize("kernel", [B.KERNEL_AUTO, B.KERNEL_TCGEN05_PAIR])
@pytest.mark.parametrize("case", TI.INNER_CASES)
def test_requantized_inner_layer(oracle, kernel, case):
    TI.test_requantized_inner_layer_matches_oracle(oracle, kernel, *case)


@pytest.mark.parametrize("case", TI.CONV_INNER_CASES)
def test_requantized_convolution(oracle, case):
    TI.test_requantized_convolution_matches_oracle(oracle, *case)


@pytest.mark.parametrize("T", [5, 300])
def test_two_layer_chain_of_predictors(oracle, T):
    TI.test_two_layer_chain_of_predictors(oracle, T)
