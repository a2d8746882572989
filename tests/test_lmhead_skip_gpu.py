"""Fused LM head: blocks of rows without a gradient are left out of the backward products (always; the results do
not change), and under MRL_FLAG_SKIP_ZERO_ROWS rows whose multiplier is zero beforehand are not produced by the
forward product either (they report logp = 0, as on the logits-in path)."""
import pytest
import torch

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import binding as B
from paper_2605_07244_b200 import build

from helpers import GRAD_REL_L2_BF16, LOGP_ATOL, make_lp, oracle_lp, rel_l2
import test_lmhead_gpu as LM

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    B.lib()


def batch_with_dead_blocks(N, H, V, seq_len, dead_seqs, seed, mask_rows=None):
    """Equal-length sequences; the advantage of `dead_seqs` is zero."""
    S = N // seq_len
    hidden, W, ids, _, _, adv, _, g = LM.toy(N, H, V, S, seed)
    cu = torch.arange(0, N + 1, seq_len, dtype=torch.int32)
    adv = torch.randn(S, generator=g)
    adv[adv.abs() < 0.05] = 0.3
    adv[dead_seqs] = 0.0
    mask = None
    if mask_rows is not None:
        mask = torch.ones(N, dtype=torch.uint8)
        mask[mask_rows] = 0
    logp, _, _ = O.token_logprobs(hidden.double() @ W.double().T, ids, mask)
    old = (logp + 0.1 * torch.randn(N, generator=g, dtype=torch.float64)).float()
    return hidden, W, ids, mask, cu, adv, old


@pytest.mark.parametrize("pair", [False, True])
@pytest.mark.parametrize("N,seq_len,dead", [
    (1024, 64, list(range(4, 12))),            # rows 256..767: two whole blocks of 256 dead, aligned
    (1024, 64, list(range(3, 13))),            # dead rows 192..831: the blocks at both ends are partly live
    (900, 50, list(range(0, 18))),             # every sequence dead: the products run on the stand-in block
    (700, 70, [9]),                            # N not a multiple of 64; the last, short block is dead
    (650, 130, [0, 1, 2, 3]),                  # only the last, short block is live
])
def test_dead_blocks_are_left_out_of_the_backward_products(N, seq_len, dead, pair):
    H, V = 128, 1500
    hidden, W, ids, mask, cu, adv, old = batch_with_dead_blocks(N, H, V, seq_len, dead, seed=N + len(dead))
    lp = make_lp(flags=B.FLAG_PAIR_TILES if pair else 0)
    got = LM.run_gpu_lmhead(hidden, W, ids, mask, cu, adv, old, None, None, lp)
    ref = O.fused_lmhead_loss(hidden, W, ids, mask, cu, adv, old, None, None, oracle_lp(lp))
    if ref["dW"].abs().max() == 0:             # nothing has a gradient: exact zeros, nothing to take a relative error of
        LM.compare(got, ref, check_grads=False)
        assert got["dH"].abs().max() == 0 and got["dW"].abs().max() == 0
    else:
        LM.compare(got, ref)
    assert int(got["stats"][2]) == N           # without the flag every row is still read


@pytest.mark.parametrize("pair", [False, True])
def test_skip_zero_rows_leaves_blocks_out_of_the_forward_product_too(pair):
    N, H, V, seq_len = 1280, 128, 2000, 64
    dead = list(range(4, 13))                  # rows 256..831: two whole blocks and a part of a third
    masked = torch.arange(1024, 1280)          # an all-masked block: never produced, with or without the flag
    hidden, W, ids, mask, cu, adv, old = batch_with_dead_blocks(N, H, V, seq_len, dead, seed=17, mask_rows=masked)
    nllw = torch.zeros(N)
    nllw[5 * 64:6 * 64] = 1.0                  # a zero-advantage sequence that carries the NLL weight stays live
    lp = make_lp(flags=B.FLAG_SKIP_ZERO_ROWS | (B.FLAG_PAIR_TILES if pair else 0), nll_coeff=0.1)
    got = LM.run_gpu_lmhead(hidden, W, ids, mask, cu, adv, old, None, nllw, lp)
    ref = O.fused_lmhead_loss(hidden, W, ids, mask, cu, adv, old, None, nllw, oracle_lp(lp))
    skipped = torch.zeros(N, dtype=torch.bool)
    for s in dead:
        if s != 5:
            skipped[s * 64:(s + 1) * 64] = True
    ref["logp"] = torch.where(skipped, torch.zeros_like(ref["logp"]), ref["logp"])
    LM.compare(got, ref)
    assert int(got["stats"][0]) == N - 256 and int(got["stats"][2]) == N - 256 - int(skipped.sum())
    assert float(got["loss"][1]) > 0
    # the same call without the flag: same gradients, full log-probs
    lp0 = make_lp(flags=B.FLAG_PAIR_TILES if pair else 0, nll_coeff=0.1)
    full = LM.run_gpu_lmhead(hidden, W, ids, mask, cu, adv, old, None, nllw, lp0)
    assert torch.equal(full["dH"], got["dH"]) and torch.equal(full["dW"], got["dW"])
    assert (full["logp"][skipped] != 0).all() and torch.equal(full["logp"][~skipped], got["logp"][~skipped])


def test_skip_flag_is_ignored_by_the_response_level_ratio():
    N, H, V, seq_len = 512, 128, 1200, 64
    hidden, W, ids, mask, cu, adv, old = batch_with_dead_blocks(N, H, V, seq_len, [0, 1, 2, 3], seed=23)
    old = (old.double() + 0.0).float()
    lp = make_lp(flags=B.FLAG_SKIP_ZERO_ROWS, ratio_level=B.RATIO_SEQUENCE)
    got = LM.run_gpu_lmhead(hidden, W, ids, mask, cu, adv, old, None, None, lp)
    z = hidden.double() @ W.double().T
    ref = O.policy_loss_sequence_ratio(z, ids, mask, cu, adv, old, None, oracle_lp(lp))
    assert (got["logp"].double() - ref["logp"]).abs().max() <= LOGP_ATOL      # every row, the dead ones too
    assert int(got["stats"][2]) == N
    assert rel_l2(got["dH"], ref["dlogits"] @ W.double()) <= GRAD_REL_L2_BF16
    assert rel_l2(got["dW"], ref["dlogits"].T @ hidden.double()) <= GRAD_REL_L2_BF16
    assert got["dH"][:256].abs().max() == 0
