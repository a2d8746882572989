"""mrl_policy_loss_fwd_bwd_host: the logits-in pass on host tensors, pipelined in micro-batches of whole sequences.
Per-row outputs must equal, bit for bit, those of one device call on the whole batch (same kernels, rows are
independent once the step's denominators are fixed); the loss may differ by the order of its float sums; both are also
compared with the oracle."""
import ctypes as C

import pytest
import torch

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import binding as B
from paper_2605_07244_b200 import build

from helpers import KlTerm, LOSS_RTOL, compare_policy_loss, make_lp, oracle_lp, run_gpu_policy_loss
import test_seqratio_gpu as SR

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    B.lib()


def pin(t, dtype=None):
    if t is None:
        return None
    t = torch.as_tensor(t)
    if dtype is not None:
        t = t.to(dtype)
    return t.contiguous().pin_memory()


def run_host(z, ids, mask, cu, adv, old, tw, nw, lp, slab_rows, V=None, want_dlogits=True, inplace=False, out_pad=0,
             logp_ref=None, want_entropy=False):
    N = z.shape[0]
    Vv = z.shape[1] if V is None else V
    S = cu.numel() - 1
    hz = pin(z)
    hd = None
    if want_dlogits:
        hd = hz if inplace else torch.full((N, z.shape[1] + out_pad), float("nan"), dtype=z.dtype).pin_memory()
    h_logp = torch.full((N,), float("nan")).pin_memory()
    h_loss = torch.full((2,), float("nan")).pin_memory()
    h_stats = torch.full((4,), -1, dtype=torch.int64).pin_memory()
    h_status = torch.full((1,), -1, dtype=torch.int32).pin_memory()
    keep = []
    h_kl = h_ent = None
    if logp_ref is not None:
        h_ref, h_kl = pin(logp_ref, torch.float32), torch.full((1,), float("nan")).pin_memory()
        lp.logp_ref, lp.kl_loss = h_ref.data_ptr(), h_kl.data_ptr()
        keep.append(h_ref)
    if want_entropy:
        h_ent = torch.full((N,), float("nan")).pin_memory()
        lp.entropy = h_ent.data_ptr()
    ld = z.shape[1]
    ws = torch.empty(max(B.host_pipeline_workspace_bytes(N, ld, B.BF16 if z.dtype == torch.bfloat16 else B.F32, S, slab_rows), 256),
                     dtype=torch.uint8, device="cuda")
    B.mrl_policy_loss_fwd_bwd_host(hz, pin(ids, torch.int32), pin(mask, torch.uint8), pin(cu, torch.int32),
                                   pin(adv, torch.float32), pin(old, torch.float32), pin(tw, torch.float32),
                                   pin(nw, torch.float32), lp, hd, h_logp, h_loss, h_stats, h_status, slab_rows, ws, V=Vv)
    torch.cuda.synchronize()
    return dict(logp=h_logp.clone(), loss=h_loss.clone(), stats=h_stats.clone(), status=int(h_status),
                dlogits=None if hd is None else hd.clone(), kl=None if h_kl is None else float(h_kl),
                entropy=None if h_ent is None else h_ent.clone())


@pytest.mark.parametrize("agg", [B.AGG_TOKEN_MEAN, B.AGG_SEQ_MEAN_TOKEN_MEAN])
@pytest.mark.parametrize("N,V,S,dtype,pad,mask_p,slab_rows", [
    (200, 4096, 9, torch.bfloat16, 0, 0.9, 64),       # streaming kernel; several slabs, the last one short
    (200, 4096, 9, torch.bfloat16, 0, None, 1000),    # everything in one slab
    (150, 40000, 7, torch.bfloat16, 0, 0.8, 40),      # 128-bit path (ld not a multiple of 16 elements is refused: 40000 is)
    (90, 1000, 6, torch.float32, 0, 0.8, 32),         # general kernel, float32
    (70, 151936, 5, torch.bfloat16, 0, None, 24),     # full vocabulary
])
def test_host_pipeline_equals_one_device_call_and_the_oracle(N, V, S, dtype, pad, mask_p, slab_rows, agg):
    z, ids, mask, cu, adv, old, nllw = SR.toy(N, V, S, dtype, seed=3 + S, mask_p=mask_p, pad=pad)
    slab_rows = max(slab_rows, int((cu[1:] - cu[:-1]).max()))
    g = torch.Generator().manual_seed(5)
    tw = torch.rand(N, generator=g) + 0.5
    lp = make_lp(agg=agg, nll_coeff=0.05)
    dev_run = run_gpu_policy_loss(z, ids, mask, cu, adv, old, tw, nllw, lp, V=V)
    got = run_host(z, ids, mask, cu, adv, old, tw, nllw, make_lp(agg=agg, nll_coeff=0.05), slab_rows, V=V)
    assert got["status"] == 0
    assert torch.equal(got["logp"], dev_run["logp"])
    assert torch.equal(got["dlogits"][:, :V].view(torch.int16 if dtype == torch.bfloat16 else torch.int32),
                       dev_run["dlogits"][:, :V].view(torch.int16 if dtype == torch.bfloat16 else torch.int32))
    assert torch.equal(got["stats"], dev_run["stats"])
    ref = O.policy_loss(z[:, :V], ids, mask, cu, adv, old, tw, nllw, oracle_lp(lp))
    compare_policy_loss(got, ref, V, dtype, cancelling=True)


def test_host_pipeline_with_kl_entropy_and_padded_output():
    N, V, S = 180, 8192, 8
    z, ids, mask, cu, adv, old, nllw = SR.toy(N, V, S, torch.bfloat16, seed=12, mask_p=0.9)
    g = torch.Generator().manual_seed(6)
    logp, _, _ = O.token_logprobs(z, ids, mask)
    ref_trace = (logp + 0.3 * torch.randn(N, generator=g, dtype=torch.float64)).float()
    slab = max(48, int((cu[1:] - cu[:-1]).max()))
    lp = make_lp()
    lp.kl_coeff, lp.kl_estimator = 0.02, B.KL_K3
    got = run_host(z, ids, mask, cu, adv, old, None, None, lp, slab, out_pad=16, logp_ref=ref_trace, want_entropy=True)
    olp = O.LossParams(kl_coeff=float(lp.kl_coeff), kl_estimator=O.KL_K3)
    ref = O.policy_loss(z, ids, mask, cu, adv, old, None, None, olp, logp_ref=ref_trace)
    compare_policy_loss(got, ref, V, torch.bfloat16, cancelling=True)
    assert abs(got["kl"] - ref["loss_kl"]) <= LOSS_RTOL * ref["loss_kl"]
    ent = O.token_entropy(z, ids, mask)
    assert (got["entropy"].double() - ent).abs().max() <= 1e-4
    assert torch.isnan(got["dlogits"][:, V:].float()).all()          # the padding columns of the output are not touched


def test_host_pipeline_in_place_forward_only_and_sequence_ratio():
    N, V, S = 160, 4096, 7
    z, ids, mask, cu, adv, old, nllw = SR.toy(N, V, S, torch.bfloat16, seed=8, noise=0.02)
    slab = max(50, int((cu[1:] - cu[:-1]).max()))
    ref = O.policy_loss(z, ids, mask, cu, adv, old, None, None, O.LossParams())
    got = run_host(z, ids, mask, cu, adv, old, None, None, make_lp(), slab, inplace=True)
    compare_policy_loss(got, ref, V, torch.bfloat16, cancelling=True)
    fwd = run_host(z, ids, mask, cu, adv, old, None, None, make_lp(), slab, want_dlogits=False)
    assert torch.equal(fwd["logp"], got["logp"]) and torch.equal(fwd["loss"], got["loss"])
    lp = make_lp(ratio_level=B.RATIO_SEQUENCE, nll_coeff=0.05)
    sq = run_host(z, ids, mask, cu, adv, old, None, nllw, lp, slab)
    dev_run = run_gpu_policy_loss(z, ids, mask, cu, adv, old, None, nllw, make_lp(ratio_level=B.RATIO_SEQUENCE, nll_coeff=0.05))
    assert torch.equal(sq["logp"], dev_run["logp"]) and torch.equal(sq["stats"], dev_run["stats"])
    assert torch.equal(sq["dlogits"].view(torch.int16), dev_run["dlogits"].view(torch.int16))
    rs = O.policy_loss_sequence_ratio(z, ids, mask, cu, adv, old, nllw, oracle_lp(lp))
    SR.compare(sq, rs, sq["dlogits"].double(), rs["dlogits"], 1e-2)


def test_host_pipeline_edge_cases_and_refusals():
    z, ids, mask, cu, adv, old, nllw = SR.toy(60, 4096, 4, torch.bfloat16, seed=2)
    longest = int((cu[1:] - cu[:-1]).max())
    with pytest.raises(B.MrlError) as e:
        run_host(z, ids, mask, cu, adv, old, None, None, make_lp(), longest - 1)
    assert e.value.code == 7                                           # a sequence longer than a staging buffer
    with pytest.raises(B.MrlError) as e:
        run_host(z, ids, mask, cu, adv, old, None, None, make_lp(flags=B.FLAG_ACCUMULATE_LOSS), 64)
    assert e.value.code == 1
    with pytest.raises(B.MrlError) as e:                               # device tensors are refused by the binding
        B.mrl_policy_loss_fwd_bwd_host(z.cuda(), ids, None, cu, adv, None, None, None, make_lp(), None, None,
                                       torch.zeros(2), None, None, 64, torch.empty(256, dtype=torch.uint8, device="cuda"))
    # empty sequences inside the batch, and a batch without any sequence
    cu2 = torch.tensor([0, 0, 20, 20, 60], dtype=torch.int32)
    adv2 = torch.tensor([1.0, -0.7, 0.3, 0.9])
    got = run_host(z, ids, None, cu2, adv2, old, None, None, make_lp(), 40)
    ref = O.policy_loss(z, ids, None, cu2, adv2, old, None, None, O.LossParams())
    compare_policy_loss(got, ref, 4096, torch.bfloat16, cancelling=True)
    h_loss = torch.ones(2).pin_memory()
    h_stats = torch.ones(4, dtype=torch.int64).pin_memory()
    B.mrl_policy_loss_fwd_bwd_host(torch.empty(0, 4096, dtype=torch.bfloat16).pin_memory(), torch.empty(0, dtype=torch.int32),
                                   None, torch.zeros(1, dtype=torch.int32), torch.empty(0), None, None, None, make_lp(),
                                   None, None, h_loss, h_stats, None, 16, torch.empty(1 << 20, dtype=torch.uint8, device="cuda"),
                                   V=4096)
    torch.cuda.synchronize()
    assert float(h_loss.sum()) == 0 and int(h_stats.sum()) == 0
