"""Training labels (Section 3.3) on the GPU against the oracle's definition."""

import numpy as np
import pytest
import torch

import workloads as W
from oracle import locret_oracle as O

pytestmark = pytest.mark.gpu


def draw(shape, seed, scale=1.0):
    g = np.random.default_rng(9000 + seed)
    return W.to_bf16_grid((g.standard_normal(shape) * scale).astype(np.float32))


@pytest.mark.parametrize("n_a,n_q,h,hk,d", [(40, 300, 4, 2, 64), (257, 1000, 8, 2, 128), (1, 129, 3, 3, 64),
                                            (300, 70, 4, 1, 128), (257, 1000, 6, 3, 96), (33, 129, 32, 32, 96)])
def test_cis_labels_match_the_definition(n_a, n_q, h, hk, d):
    from parity_util import bf16_dev
    from paper_2410_01805_b200 import cis_labels
    q, k = draw((n_a, h, d), 1), draw((n_q, hk, d), 2)
    k[3] = 0.0                                   # a key with all-zero scores (label exactly 0)
    q[:, :, :] -= 0.05                           # and mostly negative scores somewhere
    q, k = W.to_bf16_grid(q), W.to_bf16_grid(k)
    for scale in (1.0, 1.0 / np.sqrt(d)):
        ref = O.cis_labels(q, k, hk, scale)
        got = cis_labels(bf16_dev(q), bf16_dev(k), scale).cpu().numpy().astype(np.float64)
        # bf16 products are exact in fp32; only the order of the fp32 additions differs
        assert np.abs(got - ref).max() <= 1e-4 * max(1.0, np.abs(ref).max()), (n_a, n_q, h, hk, d, scale)
    assert got[0, 3] == 0.0


def test_cis_labels_argument_checks():
    from paper_2410_01805_b200 import LocretError, cis_labels
    q = torch.zeros((4, 2, 80), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((8, 2, 80), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(LocretError):
        cis_labels(q, k)                          # head_dim 64, 96 or 128
    q = torch.zeros((4, 2, 64), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((8, 2, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(LocretError):
        cis_labels(q, k, scale=0.0)
