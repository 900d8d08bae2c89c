"""Seeded random layer shapes through the forward parity check (expanded layer on one input, grouped ensemble, summed
ensemble; partial sums and outputs bit-equal to the oracle) with the automatic kernel choice and with the SM-pair kernel
forced: shapes nobody picked by hand -- odd block counts, single and ragged token tiles, clusters of one to eight orders,
every storage width."""
import numpy as np
import pytest

from paper_2311_15806_b200 import binding as B
from tests import test_gpu_parity_small as TP

pytestmark = pytest.mark.gpu


def _cases(n, seed, tokens=(17, 31, 64, 100, 128, 129, 255, 256, 257, 300, 511, 640, 1000)):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        bits = int(rng.choice([8, 4, 4, 2, 2]))
        g = int(rng.choice([8, 8, 16, 32]))
        G = int(rng.integers(1, 60))
        K = int(rng.integers(1, 9))
        M = int(rng.integers(1, min(K, 4) + 1))
        n_keep = int(rng.integers(1, G + 1))
        I = int(rng.integers(1, 40)) * int(rng.choice([8, 16, 56, 128]))
        T = int(rng.choice(tokens))
        out.append((G * g, I, T, bits, K, g, n_keep, M))
    return out


@pytest.mark.parametrize("kernel", [B.KERNEL_AUTO, B.KERNEL_TCGEN05_PAIR])
@pytest.mark.parametrize("O,I,T,bits,K,g,n_keep,M", _cases(24, 20231115))
def test_random_shapes_match_oracle(oracle, kernel, O, I, T, bits, K, g, n_keep, M):
    TP.test_forward_matches_oracle(oracle, kernel, O, I, T, bits, K, g, n_keep, M)
    assert B.pipe_poll_status() == B.PIPE_OK


@pytest.mark.parametrize("O,I,T,bits,K,g,n_keep,M", _cases(24, 20231116))
def test_random_shapes_with_int8_copy_match_oracle(oracle, O, I, T, bits, K, g, n_keep, M):
    TP.test_forward_matches_oracle(oracle, B.KERNEL_TCGEN05_PAIR, O, I, T, bits, K, g, n_keep, M, int8_copy=True)
    assert B.pipe_poll_status() == B.PIPE_OK


@pytest.mark.parametrize("O,I,T,bits,K,g,n_keep,M", _cases(16, 20231117, tokens=(1, 2, 5, 8, 9, 16)))
def test_random_shapes_on_few_tokens_match_oracle(oracle, O, I, T, bits, K, g, n_keep, M):
    """Up to 16 tokens: the weight-streaming kernel (and whatever the automatic choice falls back to), the summed
    ensemble on a shared input as one launch included."""
    TP.test_forward_matches_oracle(oracle, B.KERNEL_AUTO, O, I, T, bits, K, g, n_keep, M)
    assert B.pipe_poll_status() == B.PIPE_OK
