"""Large float32 logits take the streaming kernels too (256- and 128-bit accesses, rows split over a CTA pair): parity
with the oracle at the float32 tolerances, for the fused pass, the forward-only call, the response-level ratio's
separate backward launch, the entropy and KL outputs, and in place."""
import pytest
import torch

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import binding as B
from paper_2605_07244_b200 import build

from helpers import (GRAD_REL_L2_F32, LOGP_ATOL, KlTerm, compare_policy_loss, dev, loss_close, make_lp, oracle_lp, rel_l2,
                     run_gpu_policy_loss)
import test_seqratio_gpu as SR

pytestmark = pytest.mark.gpu
F32 = torch.float32
# V, pad: 4096 -> 256-bit vectors; 40004 -> 128-bit (not a multiple of 8 elements); 8200 in 8208-wide rows;
# 151,936 float32 = 608 KB per row -> split over a pair of CTAs
SHAPES = [(60, 4096, 0), (40, 40004, 0), (36, 8200, 8), (14, 151936, 0)]


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    B.lib()


@pytest.mark.parametrize("agg", [B.AGG_TOKEN_MEAN, B.AGG_SEQ_MEAN_TOKEN_MEAN])
@pytest.mark.parametrize("N,V,pad", SHAPES)
def test_fused_pass_float32_streaming(N, V, pad, agg):
    z, ids, mask, cu, adv, old, nllw = SR.toy(N, V, 5, F32, seed=V % 97, mask_p=0.85, pad=pad)
    g = torch.Generator().manual_seed(3)
    tw = torch.rand(N, generator=g) + 0.5
    lp = make_lp(agg=agg, nll_coeff=0.05)
    got = run_gpu_policy_loss(z, ids, mask, cu, adv, old, tw, nllw, lp, V=V)
    ref = O.policy_loss(z[:, :V], ids, mask, cu, adv, old, tw, nllw, oracle_lp(lp))
    assert got["status"] == 0
    compare_policy_loss(got, ref, V, F32, cancelling=True)
    if pad:
        assert torch.isnan(got["dlogits"][:, V:]).all()
    # in place gives the same bits
    again = run_gpu_policy_loss(z, ids, mask, cu, adv, old, tw, nllw, lp, V=V, inplace=True)
    assert torch.equal(again["dlogits"][:, :V], got["dlogits"][:, :V]) and torch.equal(again["logp"], got["logp"])


@pytest.mark.parametrize("N,V,pad", SHAPES)
def test_forward_only_and_entropy_float32_streaming(N, V, pad):
    z, ids, mask, cu, adv, old, _ = SR.toy(N, V, 4, F32, seed=11, mask_p=0.9, pad=pad)
    z[0, :V // 2] = float("-inf")
    ids[0] = V - 1
    logp = torch.full((N,), float("nan"), device="cuda")
    lse = torch.full((N,), float("nan"), device="cuda")
    B.mrl_token_logprobs(dev(z), dev(ids), dev(mask), logp, lse, V=V)
    torch.cuda.synchronize()
    ref_logp, ref_lse, valid = O.token_logprobs(z[:, :V], ids, mask)
    assert (logp.cpu().double() - ref_logp).abs().max() <= LOGP_ATOL
    assert (lse.cpu().double() - torch.where(valid, ref_lse, torch.zeros_like(ref_lse))).abs().max() <= LOGP_ATOL
    ent = torch.full((N,), float("nan"), device="cuda")
    lp = make_lp()
    lp.entropy = ent.data_ptr()
    logp_old, _, _ = O.token_logprobs(z[:, :V], ids, mask)
    got = run_gpu_policy_loss(z, ids, mask, cu, adv, logp_old.float(), None, None, lp, V=V)
    assert (ent.cpu().double() - O.token_entropy(z[:, :V], ids, mask)).abs().max() <= 1e-4
    assert got["status"] == 0


@pytest.mark.parametrize("N,V,pad", SHAPES[:3])
def test_response_level_ratio_and_kl_float32_streaming(N, V, pad):
    z, ids, mask, cu, adv, old, nllw = SR.toy(N, V, 5, F32, seed=23, mask_p=0.9, pad=pad, noise=0.02)
    g = torch.Generator().manual_seed(9)
    logp, _, _ = O.token_logprobs(z[:, :V], ids, mask)
    ref_trace = (logp + 0.3 * torch.randn(N, generator=g, dtype=torch.float64)).float()
    lp = make_lp(ratio_level=B.RATIO_SEQUENCE, nll_coeff=0.05)
    kl = KlTerm(lp, ref_trace, 0.02, B.KL_K3)
    got = run_gpu_policy_loss(z, ids, mask, cu, adv, old, None, nllw, lp, V=V)
    ref = O.policy_loss_sequence_ratio(z[:, :V], ids, mask, cu, adv, old, nllw, oracle_lp(lp), logp_ref=ref_trace)
    SR.compare(got, ref, got["dlogits"][:, :V].double(), ref["dlogits"], GRAD_REL_L2_F32)
    assert loss_close(kl.value(), ref["loss_kl"])          # k3 terms share one sign: the strict form
