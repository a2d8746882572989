"""Pins of the oracle's per-token policy entropy: closed forms, a library routine, invariances."""
import math

import torch
from scipy.stats import entropy as scipy_entropy

from oracle import mrl_oracle as O

F64 = torch.float64


def test_uniform_rows_have_entropy_log_V_and_one_entry_rows_zero():
    for V in (1, 2, 7, 1024, 151936):
        H = O.token_entropy(torch.full((3, V), 0.37, dtype=F64))
        assert (H - math.log(V)).abs().max() <= 1e-12 * max(1.0, math.log(V))


def test_two_point_closed_form_and_dominant_logit():
    # softmax of (a, 0): p = sigmoid(a); H = -p log p - (1-p) log(1-p)
    for a in (0.0, 0.5, -3.0, 12.0):
        p = 1 / (1 + math.exp(-a))
        want = -(p * math.log(p) + (1 - p) * math.log(1 - p))
        assert abs(float(O.token_entropy(torch.tensor([[a, 0.0]], dtype=F64))[0]) - want) <= 1e-14
    z = torch.zeros(1, 50, dtype=F64)
    z[0, 3] = 800.0                                   # one-hot limit, no overflow
    assert float(O.token_entropy(z)[0]) == 0.0


def test_matches_scipy_entropy_of_the_softmax_and_is_shift_invariant():
    g = torch.Generator().manual_seed(2)
    z = torch.randn(9, 333, generator=g, dtype=F64) * 3
    H = O.token_entropy(z)
    p = torch.softmax(z, dim=1).numpy()
    for t in range(9):
        assert abs(float(H[t]) - float(scipy_entropy(p[t]))) <= 1e-12
    assert (O.token_entropy(z + 41.5) - H).abs().max() <= 1e-11
    # identity used by a streaming evaluation: H = lse - sum_v p_v z_v
    lse = torch.logsumexp(z, dim=1)
    assert (H - (lse - (torch.softmax(z, 1) * z).sum(1))).abs().max() <= 1e-12


def test_masked_and_bad_id_rows_give_zero():
    z = torch.randn(4, 10, dtype=F64)
    H = O.token_entropy(z, ids=torch.tensor([1, 10, 3, -1]), mask=torch.tensor([1, 1, 0, 1]))
    assert float(H[0]) > 0 and float(H[1]) == 0 and float(H[2]) == 0 and float(H[3]) == 0
