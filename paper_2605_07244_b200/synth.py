"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random inputs (rewards, lengths, token ids, logits,
noise, weights) and lays sequences out in packed order.  It holds none of the
method's arithmetic: no log-sum-exp, no advantage, no gate, no loss.  Both the
CUDA path and the CPU oracle are fed from here.

Shapes follow the paper: vocabulary sizes of its model families (151,936 and
128,256), K-rollout groups with binary verifier rewards (App. B), response
lengths of hundreds to a few thousand tokens (App. A), ratio noise of the size
of the reported ratio statistics (App. E, Tab. 5).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    P: int                    # prompts
    M: int                    # policies (index 0 is the learner)
    G: int                    # rollouts per policy per prompt
    V: int                    # vocabulary
    dtype: torch.dtype        # logits / hidden dtype
    own_len: tuple            # (lo, hi) inclusive range of own response lengths
    peer_len_scale: tuple | None = None   # peer length = round(own_hi * U(lo, hi))
    logit_std: float = 2.0
    spike: float = 0.0        # added to one column per row
    spike_on_target: float = 0.7
    reward_beta: bool = True  # per-(prompt, policy) p ~ Beta(0.5, 0.5); else p = 0.5
    noise_std: float = 0.1    # logp_old = logp + N(0, noise_std)
    density_std: float = 0.0  # peer log density ratio ~ N(0, std) clipped to [-3, 3]
    H: int = 0                # hidden size (hidden-in path only)
    hidden_std: float = 1.0
    w_std: float = 0.02
    rows_per_block: int = 1024


C1 = Workload("C1-tiny-grpo", P=4, M=1, G=4, V=1024, dtype=torch.float32, own_len=(64, 64),
              logit_std=1.0, reward_beta=False, noise_std=0.05)
C2 = Workload("C2-qwen-vocab", P=8, M=1, G=8, V=151936, dtype=torch.bfloat16, own_len=(128, 1024),
              spike=12.0)
C3 = Workload("C3-prp-pool", P=16, M=2, G=8, V=128256, dtype=torch.bfloat16, own_len=(2048, 2048),
              peer_len_scale=(0.8, 1.25), density_std=0.5)
C4 = Workload("C4-xgrpo-sgt", P=64, M=2, G=16, V=151936, dtype=torch.bfloat16, own_len=(512, 512))
C5 = Workload("C5-fused-lmhead", P=64, M=1, G=16, V=151936, dtype=torch.bfloat16, own_len=(64, 64),
              reward_beta=False, H=4096)
# App. A's training setup as a shape: groups of 5, responses up to 3,072 tokens, a learner with the 128,256-token
# vocabulary and one peer whose rollouts arrive re-tokenised (lengths a third to all of 3,072), spiked logits
C6 = Workload("C6-appA-pool-3072", P=4, M=2, G=5, V=128256, dtype=torch.bfloat16, own_len=(1024, 3072),
              peer_len_scale=(1.0 / 3.0, 1.0), spike=12.0, density_std=0.5)
# config 2 with a quarter of the prompts: still far larger than L2, small enough for a profiler capture
C2_SMALL = replace(C2, name="C2-qwen-vocab-2-prompts", P=2)
# config 5 with an eighth of the rows and two vocabulary chunks: operands and scratch still exceed L2
C5_SMALL = replace(C5, name="C5-fused-lmhead-8k-rows-32k-vocab", P=8, V=32768)
# config 5 with per-prompt success rates drawn like the logits-in configs: many groups are all-success or all-failure
C5_BETA = replace(C5, name="C5-fused-lmhead-beta-success-rates", reward_beta=True)
CONFIGS = {"C1": C1, "C2": C2, "C3": C3, "C4": C4, "C5": C5, "C6": C6, "C2s": C2_SMALL, "C5s": C5_SMALL, "C5b": C5_BETA}


def scaled(w: Workload, **kw) -> Workload:
    """A reduced twin of a workload (same recipe, smaller sizes)."""
    return replace(w, **kw)


def _seed(seed: int, tag: int, idx: int = 0) -> int:
    return (seed * 1000003 + tag * 7919 + idx * 104729 + 12345) % (2 ** 62)


def _gen(seed: int, tag: int, idx: int = 0, device="cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_seed(seed, tag, idx))
    return g


@dataclass
class Meta:
    """Per-sequence inputs of one step: rewards and lengths, [P, M, G] each (CPU)."""
    w: Workload
    seed: int
    rewards: torch.Tensor     # f32 [P, M, G], binary
    seq_len: torch.Tensor     # i32 [P, M, G]


def make_meta(w: Workload, seed: int) -> Meta:
    g = _gen(seed, 1)
    if w.reward_beta:
        # Beta(1/2, 1/2) is the arcsine law: sin^2(pi U / 2) has exactly that distribution
        p = torch.sin(torch.rand(w.P, w.M, generator=g) * torch.pi / 2) ** 2
    else:
        p = torch.full((w.P, w.M), 0.5)
    rewards = (torch.rand(w.P, w.M, w.G, generator=g) < p[:, :, None]).float()
    lo, hi = w.own_len
    seq_len = torch.randint(lo, hi + 1, (w.P, w.M, w.G), generator=g, dtype=torch.int32)
    if w.peer_len_scale is not None and w.M > 1:
        a, b = w.peer_len_scale
        s = a + (b - a) * torch.rand(w.P, w.M - 1, w.G, generator=g)
        seq_len[:, 1:, :] = torch.round(hi * s).to(torch.int32)
    return Meta(w, seed, rewards, seq_len)


@dataclass
class Batch:
    """A packed batch: selected sequences laid end to end, one logits row per response token."""
    w: Workload
    seed: int
    seq_p: torch.Tensor       # i32 [S] prompt of each sequence
    seq_m: torch.Tensor       # i32 [S] policy
    seq_g: torch.Tensor       # i32 [S] rollout
    cu_seqlens: torch.Tensor  # i32 [S+1]
    ids: torch.Tensor         # i32 [N]
    noise: torch.Tensor       # f32 [N]  logp_old = logp + noise
    tok_weight: torch.Tensor | None   # f32 [N] or None
    is_peer: torch.Tensor     # bool [N]
    spike_col: torch.Tensor | None = None   # i32 [N]
    extra: dict = field(default_factory=dict)

    @property
    def S(self) -> int:
        return int(self.seq_p.numel())

    @property
    def N(self) -> int:
        return int(self.cu_seqlens[-1])

    def logits_rows(self, a: int, b: int, device="cpu") -> torch.Tensor:
        """Logits rows [a, b) as [b-a, V]; reproducible for any split into ranges."""
        w = self.w
        R = w.rows_per_block
        out = torch.empty(b - a, w.V, dtype=w.dtype, device=device)
        blk = a // R
        while blk * R < b:
            lo, hi = max(a, blk * R), min(b, (blk + 1) * R)
            g = _gen(self.seed, 7, blk, device)
            block = torch.empty(R, w.V, dtype=w.dtype, device=device)
            block.normal_(0.0, w.logit_std, generator=g)
            out[lo - a:hi - a] = block[lo - blk * R:hi - blk * R]
            blk += 1
        if w.spike != 0.0:
            cols = self.spike_col[a:b].to(device).long()
            r = torch.arange(b - a, device=device)
            out[r, cols] = (out[r, cols].float() + w.spike).to(w.dtype)
        return out

    def hidden_rows(self, a: int, b: int, device="cpu") -> torch.Tensor:
        w = self.w
        R = w.rows_per_block
        out = torch.empty(b - a, w.H, dtype=w.dtype, device=device)
        blk = a // R
        while blk * R < b:
            lo, hi = max(a, blk * R), min(b, (blk + 1) * R)
            g = _gen(self.seed, 8, blk, device)
            block = torch.empty(R, w.H, dtype=w.dtype, device=device)
            block.normal_(0.0, w.hidden_std, generator=g)
            out[lo - a:hi - a] = block[lo - blk * R:hi - blk * R]
            blk += 1
        return out

    def lm_head(self, device="cpu") -> torch.Tensor:
        w = self.w
        R = 4096
        out = torch.empty(w.V, w.H, dtype=w.dtype, device=device)
        for blk in range((w.V + R - 1) // R):
            g = _gen(self.seed, 9, blk, device)
            block = torch.empty(R, w.H, dtype=w.dtype, device=device)
            block.normal_(0.0, w.w_std, generator=g)
            n = min(R, w.V - blk * R)
            out[blk * R:blk * R + n] = block[:n]
        return out


def make_batch(meta: Meta, select: torch.Tensor | None = None) -> Batch:
    """Pack the selected sequences (bool [P, M, G]; default: the learner's own rollouts)."""
    w, seed = meta.w, meta.seed
    if select is None:
        select = torch.zeros(w.P, w.M, w.G, dtype=torch.bool)
        select[:, 0, :] = True
    idx = select.nonzero()                       # lexicographic (p, m, g) order
    seq_p, seq_m, seq_g = (idx[:, k].to(torch.int32) for k in range(3))
    lens = meta.seq_len[select].to(torch.int64)
    cu = torch.zeros(idx.shape[0] + 1, dtype=torch.int64)
    cu[1:] = torch.cumsum(lens, 0)
    N = int(cu[-1])
    g = _gen(seed, 3)
    ids = torch.randint(0, w.V, (N,), generator=g, dtype=torch.int32)
    noise = torch.randn(N, generator=g) * w.noise_std
    is_peer = torch.repeat_interleave(seq_m != 0, lens)
    tok_weight = None
    if w.density_std > 0:
        d = (torch.randn(N, generator=g) * w.density_std).clamp_(-3.0, 3.0)
        tok_weight = torch.where(is_peer, torch.exp(d), torch.ones(N))
    spike_col = None
    if w.spike != 0.0:
        other = torch.randint(0, w.V, (N,), generator=g, dtype=torch.int32)
        on_target = torch.rand(N, generator=g) < w.spike_on_target
        spike_col = torch.where(on_target, ids, other)
    return Batch(w, seed, seq_p, seq_m, seq_g, cu.to(torch.int32), ids, noise, tok_weight, is_peer,
                 spike_col)


@dataclass
class WordMaps:
    """Token-to-word maps of one batch under two tokenizers (what Alg. 1 of App. D would return), packed."""
    src_word: torch.Tensor   # i32 [N_src], -1 = no word
    src_cu: torch.Tensor     # i32 [B+1]
    tgt_word: torch.Tensor   # i32 [N_tgt]
    tgt_cu: torch.Tensor     # i32 [B+1]
    word_cu: torch.Tensor    # i32 [B+1]: sequence i uses word ids [0, word_cu[i+1] - word_cu[i])
    src_logp: torch.Tensor   # f32 [N_src]


def make_word_maps(B: int, words: tuple, seed: int, p_uncovered: float = 0.03, p_leading_none: float = 0.3,
                   p_source_gap: float = 0.02, max_pieces: int = 4) -> WordMaps:
    """Sequences of `words` = (lo, hi) whitespace-delimited words; every word is cut into 1..max_pieces tokens by
    the source tokenizer and, independently, by the target tokenizer (maps are non-decreasing, as a span-by-span
    tokenisation produces them).  With small probabilities a word has no target token (a source-covered word
    without a target slot), a word has no source token, and a sequence starts with delimiter tokens mapped to no
    word.  Source log-probs are -Exp(1)-like draws of the size of per-token NLLs (App. F reports 0.2 .. 1.1)."""
    g = _gen(seed, 21)
    sw, tw, scu, tcu, wcu = [], [], [0], [0], [0]
    for _ in range(B):
        nw = int(torch.randint(words[0], words[1] + 1, (1,), generator=g))
        s_cnt = torch.randint(1, max_pieces + 1, (nw,), generator=g)
        t_cnt = torch.randint(1, max_pieces + 1, (nw,), generator=g)
        t_cnt[torch.rand(nw, generator=g) < p_uncovered] = 0
        s_cnt[torch.rand(nw, generator=g) < p_source_gap] = 0
        ids = torch.arange(nw, dtype=torch.int32)
        s_map, t_map = torch.repeat_interleave(ids, s_cnt), torch.repeat_interleave(ids, t_cnt)
        if float(torch.rand(1, generator=g)) < p_leading_none:
            s_map = torch.cat([torch.full((int(torch.randint(1, 3, (1,), generator=g)),), -1, dtype=torch.int32), s_map])
            t_map = torch.cat([torch.full((int(torch.randint(1, 3, (1,), generator=g)),), -1, dtype=torch.int32), t_map])
        sw.append(s_map)
        tw.append(t_map)
        scu.append(scu[-1] + s_map.numel())
        tcu.append(tcu[-1] + t_map.numel())
        wcu.append(wcu[-1] + nw)
    src_word = torch.cat(sw) if sw else torch.zeros(0, dtype=torch.int32)
    tgt_word = torch.cat(tw) if tw else torch.zeros(0, dtype=torch.int32)
    src_logp = torch.log(torch.rand(src_word.numel(), generator=g).clamp_min(1e-6)) * 0.7
    i32 = lambda x: torch.tensor(x, dtype=torch.int32)
    return WordMaps(src_word.to(torch.int32), i32(scu), tgt_word.to(torch.int32), i32(tcu), i32(wcu), src_logp.float())
