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


@pytest.mark.parametrize("pair", [False, True])
@pytest.mark.parametrize("N,H,V,S,mask_p", [
    (300, 128, 1000, 5, None),       # ragged tiles, one chunk
    (260, 192, 40000, 7, 0.8),       # many column tiles to merge, masked rows
    (1, 64, 37, 1, None),
])
def test_entropy_on_the_hidden_in_path(N, H, V, S, mask_p, pair):
    import test_lmhead_gpu as LM
    hidden, W, ids, mask, cu, adv, old, g = LM.toy(N, H, V, S, seed=N + V, mask_p=mask_p)
    lp = make_lp(flags=B.FLAG_PAIR_TILES if pair else 0)
    ent = torch.full((N,), float("nan"), device="cuda")
    lp.entropy = ent.data_ptr()
    got = LM.run_gpu_lmhead(hidden, W, ids, mask, cu, adv, old, None, None, lp)
    z = hidden.double() @ W.double().T
    ref = O.token_entropy(z, ids, mask)
    assert torch.isfinite(ent).all()
    assert (ent.cpu().double() - ref).abs().max() <= ENT_ATOL
    lp0 = make_lp(flags=B.FLAG_PAIR_TILES if pair else 0)
    plain = LM.run_gpu_lmhead(hidden, W, ids, mask, cu, adv, old, None, None, lp0)
    assert torch.equal(plain["logp"], got["logp"]) and torch.equal(plain["dW"], got["dW"])   # nothing else changes
