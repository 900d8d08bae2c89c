"""The room pipe_layout leaves for block records is a BOUND on the blocks the cut of a channel-block table can make
(include/pipe.h: rec_cap).  Checked here on the host against the table definition evaluated on kept-group lists of
every kind the mask can produce: random, all at one end, alternating, and the adversarial ones that close a block as
early as the rule allows."""
import numpy as np
import pytest

from paper_2311_15806_b200 import binding as B
from tests import gpu_harness as H


def _kept_lists(rng, G, n_keep, K, kind):
    lists = [np.arange(G)]
    for k in range(1, K):
        if kind == "random":
            kept = np.sort(rng.choice(G, n_keep, replace=False))
        elif kind == "front":
            kept = np.arange(n_keep)
        elif kind == "back":
            kept = np.arange(G - n_keep, G)
        elif kind == "stride":
            kept = np.unique((np.arange(n_keep) * G) // n_keep)
            kept = np.sort(np.concatenate([kept, np.setdiff1d(np.arange(G), kept)[:n_keep - len(kept)]]))
        else:   # "shifted": every order keeps a different stretch
            start = (k * G) // K
            kept = np.sort((start + np.arange(n_keep)) % G)
        lists.append(kept)
    return lists


CASES = [
    # O, g, K, n_keep, M
    (256, 8, 3, 8, 1), (256, 8, 4, 16, 2), (3072, 8, 4, 192, 2), (11008, 8, 4, 688, 2), (4096, 8, 4, 256, 2),
    (8192, 16, 8, 128, 4), (1024, 32, 8, 8, 4), (1024, 32, 8, 32, 1), (520, 8, 2, 1, 1), (64, 8, 8, 8, 8),
    (2048, 16, 5, 17, 2), (4096, 64, 4, 3, 2), (768, 8, 6, 96, 3), (8, 8, 2, 1, 1),
]


@pytest.mark.parametrize("O,g,K,n_keep,M", CASES)
@pytest.mark.parametrize("kind", ["random", "front", "back", "stride", "shifted"])
def test_record_capacity_bounds_the_block_count(O, g, K, n_keep, M, kind):
    rng = np.random.default_rng(O + 7 * K + n_keep)
    G = O // g
    desc = B.make_desc(O, 256, 4, K, g, n_keep, M)
    lay = B.pipe_layout(desc)
    kept = _kept_lists(rng, G, n_keep, K, kind)
    split = [lay.branch_orders[m] for m in range(M)]
    begin = np.concatenate([[0], np.cumsum(split)]).astype(int)
    for m in range(M + 1):
        k0, k1 = (begin[m], begin[m + 1]) if m < M else (0, K)
        if lay.blk_off[m] == 0:
            assert lay.rec_off[m] == 0 and ((k1 - k0) > 8 or (k1 - k0) * g > 256)
            continue
        table = H.expected_block_table([kept[k] for k in range(k0, k1)], G, g)
        assert 1 <= table[0] <= lay.rec_cap[m] <= lay.blk_cap[m], (m, int(table[0]), lay.rec_cap[m])
        assert lay.rec_off[m] % 16 == 0
