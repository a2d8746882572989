"""GPU parity of the policy-entropy diagnostic (mrl_loss_params.entropy) against the oracle, on every row kernel."""
import pytest
import torch

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import binding as B
from paper_2605_07244_b200 import build

from helpers import dev, make_lp

pytestmark = pytest.mark.gpu
ENT_ATOL = 1e-4     # float32 sums like the log-probs': lse and sum_v p_v z_v are each good to ~1e-6 relative of ~10


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    B.lib()


def run(z, ids, mask, cu, adv, V, ratio_level=0, want_grad=True):
    zl = dev(z)
    N = zl.shape[0]
    S = cu.numel() - 1
    ent = torch.full((N,), float("nan"), device="cuda")
    lp = make_lp(ratio_level=ratio_level)
    lp.entropy = ent.data_ptr()
    ws = torch.empty(max(B.workspace_bytes(B.WS_POLICY_LOSS, N, V, 0, B.BF16, S), 256), dtype=torch.uint8, device="cuda")
    dl = torch.empty_like(zl) if want_grad else None
    logp = torch.empty(N, device="cuda")
    loss = torch.empty(2, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.mrl_policy_loss_fwd_bwd(zl, dev(ids, torch.int32), dev(mask, torch.uint8), dev(cu, torch.int32),
                              dev(adv, torch.float32), None, None, None, lp, dl, logp, loss, None, status, ws, V=V)
    torch.cuda.synchronize()
    return ent.cpu(), logp.cpu()


@pytest.mark.parametrize("N,V,dtype,pad,mask_p", [
    (33, 1000, torch.float32, 0, 0.8), (9, 1, torch.float32, 0, None), (21, 999, torch.bfloat16, 5, None),
    (40, 4096, torch.bfloat16, 0, 0.8), (17, 40008, torch.bfloat16, 0, None), (12, 151936, torch.bfloat16, 0, 0.9),
    (3, 262160, torch.bfloat16, 0, None),       # long rows: the whole-row variant carries the entropy
])
@pytest.mark.parametrize("ratio_level", [B.RATIO_TOKEN, B.RATIO_SEQUENCE])
def test_entropy_matches_oracle(N, V, dtype, pad, mask_p, ratio_level):
    g = torch.Generator().manual_seed(N + V)
    z = (torch.randn(N, V + pad, generator=g) * 2.0).to(dtype)
    if V > 8:
        z[0, :V // 2] = float("-inf")            # a row with half of the vocabulary masked out
        z[1, 5] = 30.0                           # a nearly one-hot row
    ids = torch.randint(V // 2 if V > 8 else 0, V, (N,), generator=g, dtype=torch.int32)
    mask = None if mask_p is None else (torch.rand(N, generator=g) < mask_p).to(torch.uint8)
    cu = torch.tensor([0, N // 2, N], dtype=torch.int32)
    adv = torch.tensor([0.7, -1.1])
    ent, logp = run(z, ids, mask, cu, adv, V, ratio_level)
    ref = O.token_entropy(z[:, :V], ids, mask)
    assert torch.isfinite(ent).all()
    assert (ent.double() - ref).abs().max() <= ENT_ATOL
    ref_logp, _, _ = O.token_logprobs(z[:, :V], ids, mask)
    assert (logp.double() - ref_logp).abs().max() <= 1e-4      # the log-probs are unchanged by asking for the entropy


def test_entropy_is_refused_on_the_hidden_in_path():
    h = torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(8, 64, dtype=torch.bfloat16, device="cuda")
    ent = torch.zeros(4, device="cuda")
    lp = make_lp()
    lp.entropy = ent.data_ptr()
    with pytest.raises(B.MrlError):
        B.mrl_fused_lmhead_loss_fwd_bwd(h, W, torch.zeros(4, dtype=torch.int32, device="cuda"), None,
                                        torch.tensor([0, 4], dtype=torch.int32, device="cuda"),
                                        torch.ones(1, device="cuda"), None, None, None, lp, None, None,
                                        torch.zeros(4, device="cuda"), torch.zeros(2, device="cuda"), None, None,
                                        torch.zeros(1 << 20, dtype=torch.uint8, device="cuda"))
