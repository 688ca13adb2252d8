"""Pool filter + seeded uniform sampling on the device, bit for bit against the oracle."""
import numpy as np
import pytest
import torch

from oracle import sapo_oracle as orc
from paper_2509_08721_b200 import binding as B
from tests import util as U

pytestmark = pytest.mark.gpu


def pool(seed, n, max_size=8):
    rng = np.random.default_rng(seed)
    sizes = rng.integers(0, max_size + 1, size=n)
    go = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    r = rng.choice([0.0, 0.5, 1.0], p=[0.6, 0.1, 0.3], size=go[-1]).astype(np.float32)
    return r, go


@pytest.mark.parametrize("n,J,seed", [(64, 6, 1), (448, 384, 2), (5000, 37, 3), (5000, 4999, 2**40 + 7),
                                      (3, 10, 4), (70000, 1000, 5)])
def test_select_external_is_bit_exact(n, J, seed):
    r, go = pool(seed, n)
    ref = orc.select_external(r, go, J, seed)
    sel, n_sel, n_cand = B.sapo_select_external(U.to_torch(r), U.to_torch(go), J, seed)
    torch.cuda.synchronize()
    assert n_cand.item() == ref["n_candidates"] and n_sel.item() == ref["n_selected"]
    assert np.array_equal(sel.cpu().numpy()[:ref["n_selected"]], ref["selected"])


def test_select_external_edge_cases():
    r, go = pool(9, 100)
    sel, n_sel, n_cand = B.sapo_select_external(U.to_torch(r), U.to_torch(go), 0, 1)
    assert n_sel.item() == 0 and n_cand.item() == orc.select_external(r, go, 0, 1)["n_candidates"]
    ones = np.ones(40, np.float32)                       # every entry uninformative
    go8 = (np.arange(6) * 8).astype(np.int32)
    sel, n_sel, n_cand = B.sapo_select_external(U.to_torch(ones), U.to_torch(go8), 3, 1)
    assert n_sel.item() == 0 and n_cand.item() == 0
