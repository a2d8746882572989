"""The entry points only enqueue work on the caller's stream (no allocation, no synchronisation), so a step can be
captured into a CUDA graph and replayed: the replay on new input values in the same buffers must give what a direct
call gives."""
import pytest
import torch

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import binding as B
from paper_2605_07244_b200 import build, synth

from helpers import compare_policy_loss, dev, make_lp, oracle_lp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    B.lib()


@pytest.mark.parametrize("V,dtype", [(1024, torch.float32), (8192, torch.bfloat16)])
def test_advantages_and_loss_pass_replay_from_a_cuda_graph(V, dtype):
    w = synth.scaled(synth.C1, V=V, dtype=dtype)
    meta = synth.make_meta(w, seed=5)
    batch = synth.make_batch(meta)
    N, S = batch.N, batch.S
    z = batch.logits_rows(0, N, device="cuda")
    ids, cu = dev(batch.ids), dev(batch.cu_seqlens)
    rewards, seq_len = dev(meta.rewards), dev(meta.seq_len)
    adv = torch.empty(w.P, w.M, w.G, device="cuda")
    logp0, _, _ = O.token_logprobs(z.cpu(), batch.ids, None)
    old = dev((logp0 + batch.noise.double()).float())
    dz = torch.empty_like(z)
    logp = torch.empty(N, device="cuda")
    loss = torch.zeros(2, device="cuda")
    stats = torch.zeros(4, dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(B.workspace_bytes(B.WS_POLICY_LOSS, N, V, 0, B.BF16, S), dtype=torch.uint8, device="cuda")
    ap = B.AdvParams(B.ADV_GROUP_ZNORM, 0, 1e-6, 0.8, 0.2, B.PICK_NONE, 0)
    lp = make_lp()

    def step(stream):
        B.mrl_group_advantages(rewards, seq_len, 0, ap, adv, None, None, None, None, None, stream=stream)
        B.mrl_policy_loss_fwd_bwd(z, ids, None, cu, adv, old, None, None, lp, dz, logp, loss, stats, status, ws,
                                  stream=stream)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step(side)                      # warm-up outside capture (function attributes, module load)
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        step(side)
    # new values in the same buffers, then replay
    meta2 = synth.make_meta(w, seed=6)
    rewards.copy_(meta2.rewards)
    batch2 = synth.make_batch(meta2)
    z2 = batch2.logits_rows(0, N, device="cuda")
    z.copy_(z2)
    ids.copy_(batch2.ids)
    logp2, _, _ = O.token_logprobs(z2.cpu(), batch2.ids, None)
    old.copy_((logp2 + batch2.noise.double()).float())
    dz.fill_(float("nan"))
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    adv_ref, _ = O.group_advantages(meta2.rewards)
    adv_seq = adv_ref[batch2.seq_p.long(), batch2.seq_m.long(), batch2.seq_g.long()].float()
    assert (adv.cpu().reshape(-1).double() - adv_seq.double()).abs().max() <= 2e-6
    ref = O.policy_loss(z2.cpu(), batch2.ids, None, batch2.cu_seqlens, adv.cpu().reshape(-1), old.cpu(), None, None, oracle_lp(lp))
    got = dict(logp=logp.cpu(), loss=loss.cpu(), stats=stats.cpu(), status=int(status.cpu()), dlogits=dz.cpu())
    assert got["status"] == 0
    compare_policy_loss(got, ref, V, dtype, cancelling=True)


def test_fused_lm_head_replays_from_a_cuda_graph():
    """The hidden-in pass too: tensor maps are built on the host at capture time from the same pointers, the live-block
    counts are read on the device, so a replay on new values gives what a direct call gives, bit for bit."""
    import test_lmhead_gpu as LM
    N, H, V, S = 700, 128, 20000, 6
    hidden, W, ids, mask, cu, adv, old, g = LM.toy(N, H, V, S, seed=5, mask_p=0.9)
    d = dict(h=dev(hidden), W=dev(W), ids=dev(ids), mask=dev(mask), cu=dev(cu), adv=dev(adv), old=dev(old))
    dH = torch.empty(N, H, dtype=torch.bfloat16, device="cuda")
    dW = torch.empty(V, H, dtype=torch.bfloat16, device="cuda")
    logp = torch.empty(N, device="cuda")
    loss = torch.zeros(2, device="cuda")
    stats = torch.zeros(4, dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(B.workspace_bytes(B.WS_FUSED_LMHEAD, N, V, H, B.BF16, S), dtype=torch.uint8, device="cuda")
    lp = make_lp()

    def step(stream):
        B.mrl_fused_lmhead_loss_fwd_bwd(d["h"], d["W"], d["ids"], d["mask"], d["cu"], d["adv"], d["old"], None, None, lp,
                                        dH, dW, logp, loss, stats, status, ws, stream=stream)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step(side)
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        step(side)
    # new values (another batch with a block of zero-advantage sequences), same buffers
    hidden2, W2, ids2, mask2, _, adv2, old2, _ = LM.toy(N, H, V, S, seed=6, mask_p=0.8)
    adv2 = adv2.clone()
    adv2[:2] = 0.0
    for k, t in (("h", hidden2), ("W", W2), ("ids", ids2), ("mask", mask2), ("adv", adv2), ("old", old2)):
        d[k].copy_(t)
    dH.fill_(float("nan"))
    dW.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    replayed = dict(logp=logp.cpu(), loss=loss.cpu(), stats=stats.cpu(), dH=dH.cpu(), dW=dW.cpu(), status=int(status.cpu()))
    direct = LM.run_gpu_lmhead(hidden2, W2, ids2, mask2, cu, adv2, old2, None, None, make_lp())
    assert replayed["status"] == 0
    for k in ("logp", "loss", "stats"):
        assert torch.equal(replayed[k], direct[k]), k
    for k in ("dH", "dW"):
        assert torch.equal(replayed[k].view(torch.int16), direct[k].view(torch.int16)), k
    ref = O.fused_lmhead_loss(hidden2, W2, ids2, mask2, cu, adv2, old2, None, None, oracle_lp(lp))
    LM.compare(replayed, ref)
