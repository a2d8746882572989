#!/usr/bin/env python
"""Benchmark of the policy-loss hot path on B200 (one process per GPU).

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--workload C2|C2s|C3|C4|C5|C5s|C5b]

A step is one pass of the whole hot path over one batch of synthetic input: group advantages and
SGT gate (mrl_group_advantages), then log-probs, ratio, clipped surrogate, aggregation and dlogits
(mrl_policy_loss_fwd_bwd).  The workload at N = 1 is the Qwen-size-vocabulary configuration (151,936 columns,
logits in, bf16, packed ragged sequences; `C2` in synth.py); each rank of an N-GPU run processes its own batch of the
same shape (independent replicas, no data-path collective), so scaling is weak.

Beside the headline the default run times, as sub-objects of the same line, the same batch with every row live (KL
penalty on), one slab of the PRP-pool shape and one of the XGRPO + SGT shape, and the fused LM head.  Started without a
launcher, `--gpus N` starts the N ranks itself.

Rank 0 prints ONE JSON line.  `--impl reference` times the CPU float64 oracle on a bounded sample
of the same workload instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_07244_b200 import synth  # noqa: E402

METRIC = "policy_loss_fwd_bwd_tokens_per_s"
UNIT = "tokens/s"
ORACLE_ROWS = 2048          # rows of the workload the CPU baseline is timed on
REFERENCE_ROWS = 1024       # rows per step of the --impl reference arm
LMHEAD_ORACLE_ROWS = 128    # rows of config 5 the CPU baseline is timed on (full V and H)
LMHEAD_SUB_STEPS = 5        # timed steps of the config-5 leg inside the default (config 2) run


# ------------------------------------------------------------------------------------------ helpers

def measured_peaks():
    """Measured roofline denominators; the stated fallback when the file is absent."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# DRAM bytes per token (dram__bytes_read.sum + dram__bytes_write.sum over the rows of one ncu capture of the small
# case) of the dominant kernel, keyed by the kernel the library reports it launched, the vocabulary and whether every
# row had a gradient; traffic grows in proportion to the rows.  A launch of any other kernel, shape or batch kind
# prints `traffic: null`, and so does an entry set to None because its kernel changed after the counters were taken.
DRAM_BYTES_PER_TOKEN = {
    ("row_stream_kernel", 151936, "half-live"): 637544,
    ("row_stream_kernel", 151936, "all-live"): 668781,
    ("row_stream_kernel", 128256, "prp-pool"): 535630,      # config-3 slab of 12,288 rows (pooled advantages, density weights)
}
NOMINAL_HBM_GBS = 8000.0        # B200 data sheet (7.7 TB/s on HGX boards): context beside the measured copy rate
NOMINAL_BF16_TFLOPS = 2250.0    # dense bf16


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, device_index: int, period_s: float = 0.005):
        self.period = period_s
        self.samples = []
        self.timed = []          # (host time, SM MHz, board power in W) of every sample
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                self._h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid) if not uuid.startswith("GPU-") else uuid)
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _loop(self):
        nv = self._nv
        names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
                 0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                self.samples.append(mhz)
                try:
                    watts = nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0
                except Exception:
                    watts = None
                self.timed.append((time.perf_counter(), mhz, watts))
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def median_between(self, t0: float, t1: float):
        """(median SM MHz, median W, samples) over the samples taken in [t0, t1] of the host clock."""
        mhz = sorted(m for t, m, _ in self.timed if t0 <= t <= t1)
        w = sorted(p for t, _, p in self.timed if t0 <= t <= t1 and p is not None)
        return (mhz[len(mhz) // 2] if mhz else None, w[len(w) // 2] if w else None, len(mhz))

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


def aggregate_over_ranks(local_ms: float, local_units: float, world: int):
    """Max time over ranks and total units (the whole-job view); a no-op for one rank."""
    if world == 1:
        return local_ms, local_units
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([local_units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def launch_ranks(n: int, argv, script=None, extra_env=None) -> int:
    """Starts one process per GPU on this node (ranks 0 .. n-1, rendezvous on 127.0.0.1) running `script` with
    `argv`, waits for all of them and returns 0 only if every rank exited 0.  As soon as one rank fails the others
    are terminated (they would otherwise wait for it in a collective)."""
    import socket
    import subprocess
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    script = script or os.path.abspath(__file__)
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        env.update(extra_env or {})
        procs.append(subprocess.Popen([sys.executable, script] + list(argv), env=env))
    worst = 0
    pending = set(range(n))
    while pending:
        for r in sorted(pending):
            rc = procs[r].poll()
            if rc is None:
                continue
            pending.discard(r)
            if rc != 0:
                worst = worst or (rc if rc > 0 else 1)
                for q in sorted(pending):        # exact children of this process, nothing else
                    procs[q].terminate()
        time.sleep(0.05)
    return worst


def resolve_world(gpus: int):
    """(rank, world, local_rank) from the launcher's environment; None when this process has to start the ranks
    itself (`--gpus N` > 1 given to a plain `python bench.py`).  A world size that contradicts --gpus is an error:
    a number labelled N GPUs must come from N ranks."""
    if "WORLD_SIZE" not in os.environ:
        if gpus > 1:
            return None
        return 0, 1, 0
    world = int(os.environ["WORLD_SIZE"])
    if world != gpus:
        raise SystemExit(f"bench.py: --gpus {gpus} but the launcher started WORLD_SIZE={world} ranks")
    return int(os.environ.get("RANK", "0")), world, int(os.environ.get("LOCAL_RANK", "0"))


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


# ------------------------------------------------------------------------------------------ workloads

class LogitsInWorkload:
    """Config 2: 8 prompts x G = 8, ragged lengths in [128, 1024] packed, V = 151,936, bf16 logits."""

    def __init__(self, w: synth.Workload, seed: int, device, ratio_level: int = 0, with_entropy: bool = False,
                 with_kl: bool = False):
        from paper_2605_07244_b200 import binding as B
        self.B = B
        self.w = w
        self.ratio_level = ratio_level
        self.meta = synth.make_meta(w, seed)
        self.batch = synth.make_batch(self.meta)
        b = self.batch
        self.N, self.V, self.S = b.N, w.V, b.S
        P, M, G = w.P, w.M, w.G
        dev = device
        self.z = torch.empty(self.N, self.V, dtype=w.dtype, device=dev)
        for a in range(0, self.N, w.rows_per_block):
            e = min(self.N, a + w.rows_per_block)
            self.z[a:e] = b.logits_rows(a, e, device=dev)
        self.dz = torch.empty_like(self.z)
        self.ids = b.ids.to(dev)
        self.cu = b.cu_seqlens.to(dev)
        self.rewards = self.meta.rewards.to(dev)
        self.seq_len = self.meta.seq_len.to(dev)
        self.adv_own = torch.empty(P, M, G, device=dev)
        self.adv_pool = torch.empty(P, M, G, device=dev)
        self.rescue = torch.empty(P, dtype=torch.uint8, device=dev)
        self.pick = torch.empty(P, dtype=torch.int32, device=dev)
        self.nllw_seq = torch.empty(P, M, G, device=dev)
        self.n_gated = torch.empty(1, dtype=torch.int32, device=dev)
        self.logp = torch.empty(self.N, device=dev)
        self.loss = torch.zeros(2, device=dev)
        self.stats = torch.zeros(4, dtype=torch.int64, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.ws = torch.empty(B.workspace_bytes(B.WS_POLICY_LOSS, self.N, self.V, 0, B.BF16, self.S),
                              dtype=torch.uint8, device=dev)
        self.ap = B.AdvParams(B.ADV_GROUP_ZNORM, 0, 1e-6, 0.8, 0.2, B.PICK_SHORTEST, 0)
        self.lp = B.LossParams(0.2, 0.2, B.AGG_TOKEN_MEAN, 0, 0.0, 0.0, 0.0, ratio_level)
        # behaviour trace: logp_old = logp + N(0, 0.1); logp from the library's forward (input preparation).
        # For the response-level ratio the noise is scaled by 1 / sqrt(mean length) so that w stays of order one.
        B.mrl_token_logprobs(self.z, self.ids, None, self.logp)
        if with_entropy:     # the policy-entropy diagnostic from the same pass
            self.entropy = torch.empty(self.N, device=dev)
            self.lp.entropy = self.entropy.data_ptr()
        scale = 1.0 if ratio_level == 0 else (self.S / max(self.N, 1)) ** 0.5
        self.logp_old = self.logp + b.noise.to(dev) * scale
        if with_kl:          # Eq. (1)'s beta R(theta): k3 estimate against a reference trace, beta = 1e-3 (App. A)
            self.logp_ref = self.logp + b.noise.to(dev).flip(0) * 2.0
            self.kl_loss = torch.zeros(1, device=dev)
            self.lp.logp_ref, self.lp.kl_loss = self.logp_ref.data_ptr(), self.kl_loss.data_ptr()
            self.lp.kl_coeff, self.lp.kl_estimator = 1e-3, B.KL_K3
        torch.cuda.synchronize()
        # adv_prompt, seq_prepare, row_stream, row_terms (which also finalises); the response-level ratio has a forward
        # launch, the per-response kernel, the partial sums and a backward launch instead of one fused row kernel
        self.kernels_per_step = 4 if ratio_level == 0 else 6
        self.dominant_per_step = 1 if ratio_level == 0 else 2
        # read V + write V elements; the response-level ratio reads the row a second time from HBM
        self.bytes_per_token = (2 if ratio_level == 0 else 3) * self.V * self.z.element_size()

    def step(self, z=None, dz=None):
        B = self.B
        B.mrl_group_advantages(self.rewards, self.seq_len, 0, self.ap, self.adv_own, self.adv_pool, self.rescue,
                               self.pick, self.nllw_seq, self.n_gated)
        # M = 1: adv_own laid out [P, 1, G] is the per-sequence advantage in packed (p, g) order
        B.mrl_policy_loss_fwd_bwd(self.z if z is None else z, self.ids, None, self.cu, self.adv_own, self.logp_old,
                                  None, None, self.lp, self.dz if dz is None else dz, self.logp, self.loss,
                                  self.stats, self.status, self.ws)

    def measure_forward_only(self, peaks, steps=20):
        """mrl_token_logprobs alone on the same logits: one read of every row, nothing written but N floats."""
        B = self.B
        f = lambda: B.mrl_token_logprobs(self.z, self.ids, None, self.logp)
        for _ in range(3):
            f()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            f()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        alg = self.N * self.V * self.z.element_size()
        gbs = alg / (ms * 1e-3) / 1e9
        return {"metric": "token_logprobs_tokens_per_s", "value": self.N / (ms * 1e-3), "unit": UNIT, "ms_per_call": ms,
                "steps": steps, "gpu_launches": steps,
                "roofline": {"bound": "hbm", "kernel": "row_stream_kernel (forward only)", "achieved": gbs,
                             "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                             "frac_nominal": gbs / NOMINAL_HBM_GBS,
                             "peak_source": peaks["source"] + " (copy, burst)", "algorithmic_bytes_per_launch": alg,
                             "traffic": None}}

    def measure_in_place(self, peaks, steps=20):
        """The same step with dlogits written over the logits (the buffer a trainer would reuse for the gradient):
        pass 2's stores then land on lines L2 already holds, so they take no capacity from the rows waiting for their
        second read.  Runs on a copy of the logits; after the first step that copy holds gradients, which changes no
        access pattern (rows keep their live / dead kind: it depends on the advantages, and on the KL term when on)."""
        zc = self.z.clone()
        for _ in range(3):
            self.step(zc, zc)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            self.step(zc, zc)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        gbs = self.bytes_per_token * self.N / (ms * 1e-3) / 1e9
        return {"value": self.N / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "steps": steps,
                "algorithmic_gbs_whole_step": gbs, "frac_whole_step": gbs / peaks["hbm_gbs"],
                "note": "dlogits aliases logits (ld_out = ld); whole step by CUDA events, not the kernel alone"}

    def measure_skip_zero_rows(self, steps=10):
        """The same step with MRL_FLAG_SKIP_ZERO_ROWS: rows of zero-advantage groups are not read (their gradient
        rows are still written, as zeros).  Reported beside the headline, which streams every row."""
        B = self.B
        self.lp.flags |= B.FLAG_SKIP_ZERO_ROWS
        try:
            for _ in range(3):
                self.step()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(steps):
                self.step()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / steps
            st = self.stats.cpu()
        finally:
            self.lp.flags &= ~B.FLAG_SKIP_ZERO_ROWS
        streamed = int(st[2])
        V2 = self.V * self.z.element_size()
        return {"value": self.N / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "steps": steps, "rows": self.N,
                "streamed_rows": streamed, "algorithmic_bytes_per_step": streamed * 2 * V2 + (self.N - streamed) * V2,
                "note": "tokens/s over all valid tokens; rows with A = 0 are not read, their dlogits rows are zero-filled"}

    def tokens(self):
        return self.N

    def describe(self):
        return {"workload": f"{self.w.name}: Qwen-scale vocab, logits-in: {self.w.P} prompts x G={self.w.G}, packed "
                            "ragged T in [128,1024], V=151936, bf16 logits N(0,2^2) + one +12 spike per row, "
                            "GRPO group z-norm, eps 0.2",
                "rows": self.N, "sequences": self.S, "V": self.V, "logits_dtype": "bf16",
                "ratio_level": "token" if self.ratio_level == 0 else "response (App. H)",
                "entropy_output": bool(self.lp.entropy), "kl_term": bool(self.lp.logp_ref),
                "l2": "inputs (%.1f GB logits) exceed the 126 MB L2; no flush needed" % (self.z.numel() * 2 / 1e9)}

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region
    def e2e_setup(self):
        """Host buffers in, host buffers out through mrl_policy_loss_fwd_bwd_host: the batch goes through the device
        in micro-batches of whole sequences with the copies of both directions overlapping the kernels."""
        B = self.B
        self.h_z = torch.empty(self.z.shape, dtype=self.z.dtype, pin_memory=True)
        self.h_z.copy_(self.z)
        self.h_dz = torch.empty(self.z.shape, dtype=self.z.dtype, pin_memory=True)
        self.h_ids, self.h_cu, self.h_rewards, self.h_seq_len, self.h_logp_old = (
            t.cpu().pin_memory() for t in (self.ids, self.cu, self.rewards, self.seq_len, self.logp_old))
        self.h_adv = torch.empty(self.S, pin_memory=True)
        self.h_logp = torch.empty(self.N, pin_memory=True)
        self.h_loss = torch.empty(2, pin_memory=True)
        self.h_stats = torch.empty(4, dtype=torch.int64, pin_memory=True)
        self.h_status = torch.empty(1, dtype=torch.int32, pin_memory=True)
        self.slab_rows = max(getattr(self, "e2e_slab_rows", 1024), int((self.h_cu[1:] - self.h_cu[:-1]).max()))
        self.host_ws = torch.empty(B.host_pipeline_workspace_bytes(self.N, self.V, B.BF16, self.S, self.slab_rows),
                                   dtype=torch.uint8, device=self.z.device)
        self.host_lp = B.LossParams(0.2, 0.2, B.AGG_TOKEN_MEAN, 0, 0.0, 0.0, 0.0, self.ratio_level)
        self.e2e_note = ("mrl_policy_loss_fwd_bwd_host on pinned host buffers: every input (logits included) crosses "
                         "to the device and dlogits, logp, loss come back inside the timed region, in micro-batches of "
                         f"<= {self.slab_rows} rows over three staging buffers so that both copy directions overlap "
                         "the kernels")
        small = (self.h_ids, self.h_cu, self.h_rewards, self.h_seq_len, self.h_logp_old)
        h2d = self.h_z.numel() * 2 + sum(t.numel() * t.element_size() for t in small) + self.S * 4
        d2h = self.h_dz.numel() * 2 + self.N * 4 + 8 + 32 + 4 + self.S * 4
        return h2d, d2h

    def e2e_step(self):
        B = self.B
        self.rewards.copy_(self.h_rewards, non_blocking=True)
        self.seq_len.copy_(self.h_seq_len, non_blocking=True)
        B.mrl_group_advantages(self.rewards, self.seq_len, 0, self.ap, self.adv_own, self.adv_pool, self.rescue,
                               self.pick, self.nllw_seq, self.n_gated)
        self.h_adv.copy_(self.adv_own.reshape(-1), non_blocking=True)
        torch.cuda.current_stream().synchronize()     # S advantages are on the host; the pass takes host arrays
        B.mrl_policy_loss_fwd_bwd_host(self.h_z, self.h_ids, None, self.h_cu, self.h_adv, self.h_logp_old, None, None,
                                       self.host_lp, self.h_dz, self.h_logp, self.h_loss, self.h_stats, self.h_status,
                                       self.slab_rows, self.host_ws)

    def roofline(self, kernel_ms, peaks):
        k_avg_ms = sum(kernel_ms) / (len(kernel_ms) / self.dominant_per_step)
        alg_bytes = self.bytes_per_token * self.tokens()
        if self.ratio_level != 0:
            # forward reads every row, backward writes every row but reads only rows with a gradient: those of
            # responses with A != 0 that are not clipped (stats[1] = valid rows of clipped responses)
            lens = (self.cu[1:] - self.cu[:-1]).cpu()
            live_rows = int(lens[(self.adv_own.reshape(-1) != 0).cpu()].sum()) - int(self.stats.cpu()[1])
            alg_bytes = (2 * self.tokens() + live_rows) * self.V * self.z.element_size()
        achieved = alg_bytes / (k_avg_ms * 1e-3) / 1e9
        launched = getattr(self, "last_kernel", "")
        kind = "all-live" if self.lp.logp_ref else "half-live"
        per_token = None if (self.ratio_level != 0 or self.lp.entropy) else DRAM_BYTES_PER_TOKEN.get((launched, self.V, kind))
        kernel = launched if self.ratio_level == 0 else "row_stream_kernel (forward) + row_backward_stream_kernel"
        return {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peaks["hbm_gbs"],
                "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "frac_nominal": achieved / NOMINAL_HBM_GBS,
                "peak_source": peaks["source"] + " (copy, burst)", "algorithmic_bytes_per_launch": alg_bytes,
                "kernel_ms": k_avg_ms, "traffic": None if per_token is None else per_token * self.tokens()}

    def time_oracle(self, scale=1):
        O, oargs, n = self.oracle_sample(ORACLE_ROWS // scale)
        dt = time_oracle(O, oargs)
        return n, dt, f"first {n} rows of the same batch, full V, fwd+bwd, float64, {dt:.1f} s"

    # ---- CPU baseline: the oracle on the first ORACLE_ROWS rows of the same batch
    def oracle_sample(self, rows):
        from oracle import mrl_oracle as O
        b = self.batch
        rows = min(rows, self.N)
        s_end = int(torch.searchsorted(b.cu_seqlens.long(), torch.tensor(rows), right=True)) - 1
        s_end = max(s_end, 1)
        n = int(b.cu_seqlens[s_end])
        z = self.z[:n].cpu()
        adv, _ = O.group_advantages(self.meta.rewards)
        adv_seq = adv[b.seq_p.long(), b.seq_m.long(), b.seq_g.long()][:s_end]
        args = (z, b.ids[:n], None, b.cu_seqlens[:s_end + 1], adv_seq, self.logp_old[:n].cpu())
        return O, args, n


class PoolSlabWorkload:
    """One seeded micro-batch (a slab of whole sequences, at most `slab_rows` rows) of a step that is too large to
    exist at once, timed as the step's calls on that slab with the whole step's denominators:

    C3 (PRP pool, Sec. 5.1): own and peer rollouts of the 16-candidate pool, V = 128,256, ragged peer lengths,
        pooled advantages, stop-gradient density weights on peer rows.
    C4 (XGRPO + SGT, Sec. 5.2-5.3): the learner's own rollouts with the pooled cross-policy baseline plus the peer
        rollouts the rescue gate selected, which carry only the NLL weight; MRL_FLAG_SKIP_ZERO_ROWS on (rows of
        zero-advantage groups are not read).
    Slab generation and the behaviour trace are input preparation, outside the timed region."""

    def __init__(self, name: str, seed: int, device, slab_rows: int):
        from paper_2605_07244_b200 import binding as B
        self.B = B
        w = synth.CONFIGS[name]
        self.w, self.name = w, name
        self.ratio_level = 0
        meta = synth.make_meta(w, seed)
        P, M, G = w.P, w.M, w.G
        dev = device
        self.rewards = meta.rewards.to(dev)
        self.seq_len = meta.seq_len.to(dev)
        # per-prompt outputs of the advantage / gate call; adv_pool gets one more slot that stays zero, so that a
        # sequence without a policy-gradient term (a selected peer rollout of config 4) can point at it
        self.adv_own = torch.empty(P, M, G, device=dev)
        self.adv_ext = torch.zeros(P * M * G + 1, device=dev)
        self.adv_pool = self.adv_ext[:P * M * G].view(P, M, G)
        self.rescue = torch.empty(P, dtype=torch.uint8, device=dev)
        self.pick = torch.empty(P, dtype=torch.int32, device=dev)
        self.nllw_seq = torch.empty(P, M, G, device=dev)
        self.n_gated_dev = torch.empty(1, dtype=torch.int32, device=dev)
        sgt = name == "C4"
        self.ap = B.AdvParams(B.ADV_GROUP_ZNORM, 0, 1e-6, 0.8, 0.2, B.PICK_SHORTEST if sgt else B.PICK_NONE, 0)
        B.mrl_group_advantages(self.rewards, self.seq_len, 0, self.ap, self.adv_own, self.adv_pool, self.rescue,
                               self.pick, self.nllw_seq, self.n_gated_dev)
        torch.cuda.synchronize()
        select = torch.ones(P, M, G, dtype=torch.bool)
        n_gated = 0
        if sgt:      # the step's batch: own rollouts and the peer rollouts the gate selected (input preparation)
            picked = self.nllw_seq.cpu() > 0
            n_gated = int(self.n_gated_dev.cpu())
            select = torch.zeros(P, M, G, dtype=torch.bool)
            select[:, 0, :] = True
            select |= picked
        batch = synth.make_batch(meta, select)
        self.step_rows, self.step_seqs = batch.N, batch.S
        s1 = 1
        while s1 < batch.S and int(batch.cu_seqlens[s1 + 1]) <= slab_rows:
            s1 += 1
        n = int(batch.cu_seqlens[s1])
        self.N, self.V, self.S = n, w.V, s1
        self.z = torch.empty(n, w.V, dtype=w.dtype, device=dev)
        for a in range(0, n, 4096):
            e = min(n, a + 4096)
            self.z[a:e] = batch.logits_rows(a, e, device=dev)
        self.dz = torch.empty_like(self.z)
        self.ids = batch.ids[:n].to(dev)
        self.cu = batch.cu_seqlens[:s1 + 1].to(dev)
        flat = (batch.seq_p.long() * M + batch.seq_m.long()) * G + batch.seq_g.long()
        lens = (batch.cu_seqlens[1:] - batch.cu_seqlens[:-1]).long()
        self.tok_weight = self.nll_weight = None
        if sgt:      # selected peer rollouts: no policy-gradient term (the zero slot), NLL weight 1 on their rows
            peer = batch.seq_m != 0
            flat = torch.where(peer, torch.full_like(flat, P * M * G), flat)
            self.nll_weight = torch.repeat_interleave(peer.float(), lens)[:n].to(dev)
            self.peer_rows = int(self.nll_weight.sum())
        else:
            self.tok_weight = batch.tok_weight[:n].to(dev)
        self.adv_index = flat[:s1].to(dev)
        self.adv_seq = torch.empty(s1, device=dev)
        self.logp = torch.empty(n, device=dev)
        self.loss = torch.zeros(2, device=dev)
        self.stats = torch.zeros(4, dtype=torch.int64, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.ws = torch.empty(B.workspace_bytes(B.WS_POLICY_LOSS, n, w.V, 0, B.BF16, s1), dtype=torch.uint8, device=dev)
        flags = B.FLAG_SKIP_ZERO_ROWS if sgt else 0
        nll_coeff = 0.1 / n_gated if n_gated > 0 else 0.0        # lambda_SGT / n_gated (Eq. (2))
        self.lp = B.LossParams(0.2, 0.2, B.AGG_TOKEN_MEAN, flags, float(batch.N), float(batch.S), nll_coeff, 0)
        B.mrl_token_logprobs(self.z, self.ids, None, self.logp)
        self.logp_old = self.logp + batch.noise[:n].to(dev)
        torch.cuda.synchronize()
        self.kernels_per_step = 4        # adv_prompt, seq_prepare, row_stream, row_terms (+ one torch gather)
        self.dominant_per_step = 1
        self.n_gated = n_gated

    def step(self):
        B = self.B
        B.mrl_group_advantages(self.rewards, self.seq_len, 0, self.ap, self.adv_own, self.adv_pool, self.rescue,
                               self.pick, self.nllw_seq, self.n_gated_dev)
        # the slab's sequences pick their advantage out of the [P, M, G] array (one small gather between the two calls)
        torch.index_select(self.adv_ext, 0, self.adv_index, out=self.adv_seq)
        B.mrl_policy_loss_fwd_bwd(self.z, self.ids, None, self.cu, self.adv_seq, self.logp_old, self.tok_weight,
                                  self.nll_weight, self.lp, self.dz, self.logp, self.loss, self.stats, self.status,
                                  self.ws)

    def tokens(self):
        return self.N

    def describe(self):
        what = {"C3": "PRP pool (Sec. 5.1): own + peer rollouts of the 16-candidate pool, ragged peer lengths, pooled "
                      "advantages, per-token density weights on peer rows",
                "C4": "XGRPO + SGT (Sec. 5.2-5.3): own rollouts with the pooled baseline, rescue-selected peer rollouts "
                      "with NLL weight 1, MRL_FLAG_SKIP_ZERO_ROWS"}[self.name]
        d = {"workload": f"{self.w.name}: one slab of {self.S} whole sequences ({self.N} rows, "
                         f"{self.z.numel() * 2 / 1e9:.1f} GB of bf16 logits) of a step of {self.step_rows} rows / "
                         f"{self.step_seqs} sequences; {what}",
             "rows": self.N, "sequences": self.S, "V": self.V, "logits_dtype": "bf16", "step_rows": self.step_rows,
             "l2": "the slab exceeds the 126 MB L2 by two orders of magnitude; no flush needed"}
        if self.name == "C4":
            d.update(selected_peer_rollouts_in_step=self.n_gated, nll_rows_in_slab=self.peer_rows)
        return d

    def roofline(self, kernel_ms, peaks):
        k_avg_ms = sum(kernel_ms) / len(kernel_ms)
        streamed = int(self.stats.cpu()[2])
        row_bytes = self.V * self.z.element_size()
        alg_bytes = streamed * 2 * row_bytes + (self.N - streamed) * row_bytes      # unread rows are still zero-filled
        achieved = alg_bytes / (k_avg_ms * 1e-3) / 1e9
        # DRAM traffic from the small-slab captures, scaled by the rows: config 3 by its own figure; config 4's read rows
        # all carry a gradient (the others are not read), so they take the every-row-live figure of the same vocabulary
        # (a 10,240-row slab of config 4 measured 669,884 B per token against that figure's 668,781) and its unread
        # rows one row of zeros each
        launched = getattr(self, "last_kernel", "")
        per_token = DRAM_BYTES_PER_TOKEN.get((launched, self.V, "prp-pool" if self.name == "C3" else "all-live"))
        traffic = None if per_token is None else per_token * streamed + (self.N - streamed) * row_bytes
        return {"bound": "hbm", "kernel": launched, "achieved": achieved, "peak": peaks["hbm_gbs"],
                "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "frac_nominal": achieved / NOMINAL_HBM_GBS,
                "peak_source": peaks["source"] + " (copy, burst)", "algorithmic_bytes_per_launch": alg_bytes,
                "rows_read": streamed, "kernel_ms": k_avg_ms, "traffic": traffic}


class LmheadWorkload:
    """Config 5: N = 65,536 response tokens, H = 4,096, V = 151,936, bf16 hidden and LM-head weight; the logits
    are never stored; outputs logp, loss, dHidden, dW."""

    def __init__(self, w: synth.Workload, seed: int, device, pair_tiles: bool = False, skip_zero_rows: bool = False):
        from paper_2605_07244_b200 import binding as B
        self.B = B
        self.pair_tiles = pair_tiles
        self.skip_zero_rows = skip_zero_rows
        self.w = w
        self.meta = synth.make_meta(w, seed)
        self.batch = synth.make_batch(self.meta)
        b = self.batch
        self.N, self.V, self.H, self.S = b.N, w.V, w.H, b.S
        P, M, G = w.P, w.M, w.G
        dev = device
        self.hidden = torch.empty(self.N, self.H, dtype=w.dtype, device=dev)
        for a in range(0, self.N, w.rows_per_block):
            e = min(self.N, a + w.rows_per_block)
            self.hidden[a:e] = b.hidden_rows(a, e, device=dev)
        self.W = b.lm_head(device=dev)
        self.dH = torch.empty_like(self.hidden)
        self.dW = torch.empty_like(self.W)
        self.ids = b.ids.to(dev)
        self.cu = b.cu_seqlens.to(dev)
        self.rewards = self.meta.rewards.to(dev)
        self.seq_len = self.meta.seq_len.to(dev)
        self.adv_own = torch.empty(P, M, G, device=dev)
        self.adv_pool = torch.empty(P, M, G, device=dev)
        self.rescue = torch.empty(P, dtype=torch.uint8, device=dev)
        self.pick = torch.empty(P, dtype=torch.int32, device=dev)
        self.nllw_seq = torch.empty(P, M, G, device=dev)
        self.n_gated = torch.empty(1, dtype=torch.int32, device=dev)
        self.logp = torch.empty(self.N, device=dev)
        self.loss = torch.zeros(2, device=dev)
        self.stats = torch.zeros(4, dtype=torch.int64, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.ws = torch.empty(B.workspace_bytes(B.WS_FUSED_LMHEAD, self.N, self.V, self.H, B.BF16, self.S),
                              dtype=torch.uint8, device=dev)
        self.ap = B.AdvParams(B.ADV_GROUP_ZNORM, 0, 1e-6, 0.8, 0.2, B.PICK_SHORTEST, 0)
        self.lp = B.LossParams(0.2, 0.2, B.AGG_TOKEN_MEAN, (B.FLAG_PAIR_TILES if pair_tiles else 0) |
                               (B.FLAG_SKIP_ZERO_ROWS if skip_zero_rows else 0), 0.0, 0.0, 0.0, 0)
        # behaviour trace: logp_old = logp + N(0, 0.1); logp from a forward-only call (input preparation)
        B.mrl_group_advantages(self.rewards, self.seq_len, 0, self.ap, self.adv_own, self.adv_pool, self.rescue,
                               self.pick, self.nllw_seq, self.n_gated)
        B.mrl_fused_lmhead_loss_fwd_bwd(self.hidden, self.W, self.ids, None, self.cu, self.adv_own, None, None, None,
                                        self.lp, None, None, self.logp, self.loss, self.stats, self.status, self.ws)
        self.logp_old = self.logp + b.noise.to(dev)
        torch.cuda.synchronize()
        chunks = -(-self.V // 16384)
        self.dominant_per_step = 1 + 3 * chunks          # forward GEMM, then (dZ, dHidden, dW) per vocabulary chunk
        # adv, seq_prepare, forward GEMM, rows, row_terms, two live-block list builds of two kernels each (forward,
        # backward), then 3 GEMMs per chunk
        self.kernels_per_step = 9 + 3 * chunks
        # Blocks of 256 rows without any gradient are left out of the three backward products, and of the forward one
        # too under MRL_FLAG_SKIP_ZERO_ROWS: count the rows of the blocks that are worked on (a block whose rows are
        # all clipped is not expected and not counted as skipped).
        lens = (self.cu[1:] - self.cu[:-1]).long()
        row_live = torch.repeat_interleave(self.adv_own.reshape(-1) != 0, lens)
        pad = (-self.N) % 256
        blocks = torch.nn.functional.pad(row_live, (0, pad)).view(-1, 256).any(dim=1)
        rows_bwd = min(int(blocks.sum()) * 256, self.N) if bool(blocks.any()) else min(256, self.N)
        rows_fwd = rows_bwd if skip_zero_rows else self.N
        self.rows_worked = {"forward": rows_fwd, "backward": rows_bwd}
        hv = float(self.H) * self.V
        self.flops_executed = 2.0 * hv * rows_fwd + 6.0 * hv * rows_bwd   # forward; recompute, dHidden, dW
        self.flops_algorithmic = 2.0 * hv * rows_fwd + 4.0 * hv * rows_bwd   # without the recompute

    def step(self):
        B = self.B
        B.mrl_group_advantages(self.rewards, self.seq_len, 0, self.ap, self.adv_own, self.adv_pool, self.rescue,
                               self.pick, self.nllw_seq, self.n_gated)
        B.mrl_fused_lmhead_loss_fwd_bwd(self.hidden, self.W, self.ids, None, self.cu, self.adv_own, self.logp_old,
                                        None, None, self.lp, self.dH, self.dW, self.logp, self.loss, self.stats,
                                        self.status, self.ws)

    def product_kinds(self, steps):
        """Kind of every tensor-core launch of `steps` steps, in launch order, and the flops of one launch of each kind
        (all rows worked on, as in config 5; the last, ragged vocabulary chunk is kept apart)."""
        vchunk = 16384
        chunks = -(-self.V // vchunk)
        last = self.V - (chunks - 1) * vchunk
        one = ["forward"]
        for c in range(chunks):
            tag = "" if (c < chunks - 1 or last == vchunk) else " (last chunk)"
            one += ["dZ" + tag, "dHidden" + tag, "dW" + tag]
        nh = 2.0 * self.rows_worked["backward"] * self.H
        flops = {"forward": 2.0 * self.rows_worked["forward"] * self.H * self.V}
        for k in ("dZ", "dHidden", "dW"):
            flops[k] = nh * min(vchunk, self.V)
            flops[k + " (last chunk)"] = nh * last
        return one * steps, flops

    def tokens(self):
        return self.N

    def describe(self):
        return {"workload": f"{self.w.name}: fused LM-head, hidden-in: N={self.N} response tokens ({self.w.P} prompts x "
                            f"G=16 x T=64), H={self.H} bf16 hidden N(0,1), W[V={self.V},H] bf16 N(0,0.02^2), logits never "
                            "materialised, GRPO clipped surrogate, binary rewards, fwd+bwd -> dHidden, dW",
                "rows": self.N, "sequences": self.S, "V": self.V, "H": self.H, "pair_tiles": self.pair_tiles,
                "skip_zero_rows": self.skip_zero_rows,
                "sequences_with_nonzero_advantage": int((self.adv_own != 0).sum()),
                "rows_worked_on": self.rows_worked,
                "l2": "operands (1.8 GB) and scratch exceed the 126 MB L2; no flush needed"}

    def roofline(self, kernel_ms, peaks):
        """All tensor-core launches of a step against the bf16 rate cuBLAS sustains inside a long step."""
        per_step_ms = sum(kernel_ms) / (len(kernel_ms) / self.dominant_per_step)
        achieved = self.flops_executed / (per_step_ms * 1e-3) / 1e12
        peak = peaks["bf16_tflops_sustained"]
        alg = self.flops_algorithmic / (per_step_ms * 1e-3) / 1e12
        return {"bound": "tensor", "kernel": "lmhead_gemm_kernel (forward, dZ recompute, dHidden, dW launches)",
                "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "peak_source": peaks["source"] + " (cuBLAS bf16, sustained)",
                # the same rate against the other denominators: the burst cuBLAS rate and the data-sheet dense peak;
                # and the rate on algorithmic flops (the dZ recompute not counted) against all three
                "frac_burst": achieved / peaks["bf16_tflops"], "frac_nominal": achieved / NOMINAL_BF16_TFLOPS,
                "flops_per_step_executed": self.flops_executed, "flops_per_step_algorithmic": self.flops_algorithmic,
                "achieved_algorithmic": alg, "frac_algorithmic": alg / peak,
                "frac_algorithmic_burst": alg / peaks["bf16_tflops"], "frac_algorithmic_nominal": alg / NOMINAL_BF16_TFLOPS,
                "kernel_ms": per_step_ms, "launches_per_step": self.dominant_per_step, "traffic": None}

    def e2e_setup(self):
        self.h_hidden = self.hidden.cpu().pin_memory()
        self.h_W = self.W.cpu().pin_memory()
        self.h_dH = torch.empty(self.hidden.shape, dtype=self.hidden.dtype, pin_memory=True)
        self.h_dW = torch.empty(self.W.shape, dtype=self.W.dtype, pin_memory=True)
        self.h_small_in = [t.cpu().pin_memory() for t in (self.ids, self.cu, self.rewards, self.seq_len, self.logp_old)]
        self.d_small_in = [self.ids, self.cu, self.rewards, self.seq_len, self.logp_old]
        self.h_logp = torch.empty(self.N, pin_memory=True)
        self.h_loss = torch.empty(2, pin_memory=True)
        h2d = (self.h_hidden.numel() + self.h_W.numel()) * 2 + sum(t.numel() * t.element_size() for t in self.h_small_in)
        d2h = (self.h_dH.numel() + self.h_dW.numel()) * 2 + self.N * 4 + 8
        return h2d, d2h

    def e2e_step(self):
        for h, d in zip(self.h_small_in, self.d_small_in):
            d.copy_(h, non_blocking=True)
        self.hidden.copy_(self.h_hidden, non_blocking=True)
        self.W.copy_(self.h_W, non_blocking=True)
        self.step()
        self.h_dH.copy_(self.dH, non_blocking=True)
        self.h_dW.copy_(self.dW, non_blocking=True)
        self.h_logp.copy_(self.logp, non_blocking=True)
        self.h_loss.copy_(self.loss, non_blocking=True)

    def time_oracle(self, scale=1):
        from oracle import mrl_oracle as O
        b = self.batch
        n_seq = max(1, LMHEAD_ORACLE_ROWS // scale // int(b.cu_seqlens[1]))
        n = int(b.cu_seqlens[n_seq])
        adv, _ = O.group_advantages(self.meta.rewards)
        adv_seq = adv[b.seq_p.long(), b.seq_m.long(), b.seq_g.long()][:n_seq]
        args = (self.hidden[:n].cpu(), self.W.cpu(), b.ids[:n], None, b.cu_seqlens[:n_seq + 1], adv_seq,
                self.logp_old[:n].cpu())
        t0 = time.perf_counter()
        O.fused_lmhead_loss(*args, None, None, O.LossParams())
        dt = time.perf_counter() - t0
        return n, dt, f"first {n} rows of the same batch, full V and H, fwd+bwd incl. dW, float64, {dt:.1f} s"


def measure_tiny_latency(seed):
    """Config 1 (P = 4, G = 4, T = 64: 1,024 rows of 1,024 float32 logits, 4 MiB, L2-resident): a step is launch-bound,
    so it is reported as time per step, launched call by call and replayed from a CUDA graph."""
    wl = LogitsInWorkload(synth.CONFIGS["C1"], seed, torch.device("cuda", torch.cuda.current_device()))
    reps = 200
    side = torch.cuda.Stream()
    B = wl.B

    def step(stream):
        B.mrl_group_advantages(wl.rewards, wl.seq_len, 0, wl.ap, wl.adv_own, wl.adv_pool, wl.rescue, wl.pick,
                               wl.nllw_seq, wl.n_gated, stream=stream)
        B.mrl_policy_loss_fwd_bwd(wl.z, wl.ids, None, wl.cu, wl.adv_own, wl.logp_old, None, None, wl.lp, wl.dz, wl.logp,
                                  wl.loss, wl.stats, wl.status, wl.ws, stream=stream)

    def timed(f):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(side):
            for _ in range(10):
                f()
            side.synchronize()
            e0.record(side)
            for _ in range(reps):
                f()
            e1.record(side)
        side.synchronize()
        return e0.elapsed_time(e1) * 1e3 / reps

    direct = timed(lambda: step(side))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        step(side)
    replay = timed(graph.replay)
    return {"workload": wl.w.name, "rows": wl.N, "V": wl.V, "us_per_step_direct": direct, "us_per_step_graph": replay,
            "kernels_per_step": wl.kernels_per_step, "steps": reps, "status": int(wl.status.cpu())}


def measure_float32_rows(seed, peaks):
    """The same pass on float32 logits at the 151,936-column vocabulary (608 KB per row: each row is shared by a pair of
    CTAs): 8,192 rows, 5 GB in and 5 GB out per step."""
    from paper_2605_07244_b200 import binding as B
    N, V, S = 8192, 151936, 16
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    z = torch.empty(N, V, device="cuda")
    z.normal_(0.0, 2.0, generator=g)
    ids = torch.randint(0, V, (N,), dtype=torch.int32, device="cuda", generator=g)
    cu = torch.arange(0, N + 1, N // S, dtype=torch.int32, device="cuda")
    adv = torch.randn(S, device="cuda", generator=g)
    logp = torch.empty(N, device="cuda")
    B.mrl_token_logprobs(z, ids, None, logp)
    old = logp + 0.1 * torch.randn(N, device="cuda", generator=g)
    dz = torch.empty_like(z)
    loss = torch.zeros(2, device="cuda")
    stats = torch.zeros(4, dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(B.workspace_bytes(B.WS_POLICY_LOSS, N, V, 0, B.F32, S), dtype=torch.uint8, device="cuda")
    lp = B.LossParams(0.2, 0.2, B.AGG_TOKEN_MEAN, 0, 0.0, 0.0, 0.0, 0)
    f = lambda: B.mrl_policy_loss_fwd_bwd(z, ids, None, cu, adv, old, None, None, lp, dz, logp, loss, stats, status, ws)
    for _ in range(3):
        f()
    steps = 20
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        f()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    alg = 2 * N * V * 4
    gbs = alg / (ms * 1e-3) / 1e9
    return {"metric": METRIC, "value": N / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "steps": steps, "rows": N, "V": V,
            "logits_dtype": "f32", "status": int(status.cpu()),
            "roofline": {"bound": "hbm", "kernel": "row_stream_kernel (float32, row split over two CTAs)", "achieved": gbs,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                         "frac_nominal": gbs / NOMINAL_HBM_GBS,
                         "peak_source": peaks["source"] + " (copy, burst)", "algorithmic_bytes_per_launch": alg,
                         "traffic": None}}


def measure_thl_align(seed, with_cpu):
    """THL word alignment on a batch shaped like one PRP step of App. G.1: 256 prompts x 5 peer rollouts of
    ~630 response tokens, words cut into 1..4 tokens by each tokenizer.  It is tiny next to the loss pass (a few
    tens of MB, L2-resident), so it is reported as time per call and tokens/s, not against a roofline."""
    from paper_2605_07244_b200 import binding as B
    wm = synth.make_word_maps(1280, (150, 350), seed)
    total_words = int(wm.word_cu[-1])
    d = {k: getattr(wm, k).cuda() for k in ("src_logp", "src_word", "src_cu", "tgt_word", "tgt_cu", "word_cu")}
    n_src, n_tgt = int(wm.src_cu[-1]), int(wm.tgt_cu[-1])
    out = torch.empty(n_tgt, device="cuda")
    tot = torch.empty(2, 1280, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(B.workspace_bytes(B.WS_THL_WORD_ALIGN, total_words, 0), dtype=torch.uint8, device="cuda")
    call = lambda: B.mrl_thl_word_align_logprobs(d["src_logp"], d["src_word"], d["src_cu"], d["tgt_word"], d["tgt_cu"],
                                                 d["word_cu"], total_words, 0.0, out, tot[0], tot[1], status, ws)
    for _ in range(3):
        call()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 50
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        call()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / reps
    alg_bytes = 8 * n_src + 8 * n_tgt      # log-prob + word id per source token, word id + output per target token
    res = {"metric": "thl_word_align_target_tokens_per_s", "value": n_tgt / (us * 1e-6), "unit": "tokens/s",
           "us_per_call": us, "sequences": 1280, "source_tokens": n_src, "target_tokens": n_tgt, "words": total_words,
           "algorithmic_bytes": alg_bytes, "achieved_gbs": alg_bytes / (us * 1e-6) / 1e9, "gpu_launches": reps,
           "status": int(status.cpu())}
    if with_cpu:
        from oracle import mrl_oracle as O
        k = 32
        t0 = time.perf_counter()
        O.thl_word_align_logprobs(wm.src_logp[:int(wm.src_cu[k])], wm.src_word[:int(wm.src_cu[k])], wm.src_cu[:k + 1],
                                  wm.tgt_word[:int(wm.tgt_cu[k])], wm.tgt_cu[:k + 1], 0.0)
        dt = time.perf_counter() - t0
        res["cpu_baseline"] = {"value": int(wm.tgt_cu[k]) / dt, "unit": "tokens/s", "cores": 1, "kind": "oracle",
                               "sample": f"first {k} sequences, {dt:.1f} s"}
    return res


def per_product_table(kinds, flops, offsets_ms, durations_ms, t_start, clocks: ClockSampler, sms: int):
    """Time x SM clock of every kind of tensor-core launch: mean duration, the median SM clock and board power sampled
    while launches of that kind ran (their start offsets are CUDA-event times after `t_start`, the host time at which
    the device was idle and the first launch was queued), and from them flop per clock per SM."""
    out = {}
    for kind in sorted(set(kinds)):
        idx = [i for i, k in enumerate(kinds) if k == kind]
        ms = sum(durations_ms[i] for i in idx) / len(idx)
        mhz, watts = [], []
        for i in idx:
            a = t_start + offsets_ms[i] * 1e-3
            m, w, _ = clocks.median_between(a, a + durations_ms[i] * 1e-3)
            if m is not None:
                mhz.append(m)
            if w is not None:
                watts.append(w)
        mhz.sort()
        watts.sort()
        med = mhz[len(mhz) // 2] if mhz else None
        out[kind] = {"launches": len(idx), "ms": ms, "sm_mhz": med, "watts": watts[len(watts) // 2] if watts else None,
                     "tflops": flops[kind] / (ms * 1e-3) / 1e12,
                     "flop_per_clk_per_sm": None if not med else flops[kind] / (ms * 1e-3 * med * 1e6 * sms)}
    return out


def library_loop_per_product(N, H, V, vchunk, steps, device_index):
    """The same five product shapes as torch.matmul calls (the vendor library), in the step's order: the forward product
    with its [N, V] store, then per full vocabulary chunk the dZ-, dHidden- and dW-shaped products.  A comparison leg
    only: nothing of the library is on the product path."""
    dev = torch.device("cuda", device_index)
    g = torch.Generator(device=dev)
    g.manual_seed(1)
    hid = torch.randn(N, H, device=dev, dtype=torch.bfloat16, generator=g)
    W = torch.randn(V, H, device=dev, dtype=torch.bfloat16, generator=g) * 0.02
    Z = torch.empty(N, V, device=dev, dtype=torch.bfloat16)
    D = torch.randn(N, vchunk, device=dev, dtype=torch.bfloat16, generator=g) * 0.01
    Dz = torch.empty(N, vchunk, device=dev, dtype=torch.bfloat16)
    dH = torch.empty(N, H, device=dev, dtype=torch.bfloat16)
    dW = torch.empty(vchunk, H, device=dev, dtype=torch.bfloat16)
    Wc = W[:vchunk]
    chunks = V // vchunk
    names = ["forward"] + ["dZ", "dHidden", "dW"] * chunks

    def run(events):
        calls = [lambda: torch.matmul(hid, W.t(), out=Z)]
        for _ in range(chunks):
            calls += [lambda: torch.matmul(hid, Wc.t(), out=Dz), lambda: torch.matmul(D, Wc, out=dH),
                      lambda: torch.matmul(D.t(), hid, out=dW)]
        for j, call in enumerate(calls):
            if events is not None:
                events[2 * j].record()
            call()
            if events is not None:
                events[2 * j + 1].record()

    run(None)
    run(None)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(2 * len(names))] for _ in range(steps)]
    with ClockSampler(device_index, 0.002) as clocks:
        torch.cuda.synchronize()
        t_start = time.perf_counter()
        for ev in evs:
            run(ev)
        torch.cuda.synchronize()
    kinds, offs, durs = [], [], []
    for ev in evs:
        for j, nm in enumerate(names):
            kinds.append(nm)
            offs.append(evs[0][0].elapsed_time(ev[2 * j]))
            durs.append(ev[2 * j].elapsed_time(ev[2 * j + 1]))
    fl = {"forward": 2.0 * N * H * V, "dZ": 2.0 * N * H * vchunk, "dHidden": 2.0 * N * H * vchunk, "dW": 2.0 * N * H * vchunk}
    sms = torch.cuda.get_device_properties(device_index).multi_processor_count
    table = per_product_table(kinds, fl, offs, durs, t_start, clocks, sms)
    return {"what": "torch.matmul (vendor library) on the step's product shapes, full chunks only, plain bf16 stores",
            "ms_per_pass": (offs[-1] + durs[-1]) / steps, "per_product": table}


def time_oracle(O, args, repeats=1):
    best = None
    for _ in range(repeats):
        t0 = time.perf_counter()
        O.policy_loss(*args, None, None, O.LossParams())
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return best


# ------------------------------------------------------------------------------------------ arms

def run_reference(args, rank, world):
    """The oracle as it stands on the host cores; each step is a bounded sample of the workload."""
    if rank != 0:
        return
    from oracle import mrl_oracle as O
    w = synth.CONFIGS[args.workload]
    meta = synth.make_meta(w, args.seed)
    batch = synth.make_batch(meta)
    adv, _ = O.group_advantages(meta.rewards)
    if w.H > 0:      # hidden-in workloads: the oracle's float64 LM head on a few sequences, full V and H
        n_seq = max(1, LMHEAD_ORACLE_ROWS // int(batch.cu_seqlens[1]))
        n = int(batch.cu_seqlens[n_seq])
        hidden, W = batch.hidden_rows(0, n), batch.lm_head()
        adv_seq = adv[batch.seq_p.long(), batch.seq_m.long(), batch.seq_g.long()][:n_seq]
        logp, _, _ = O.token_logprobs(hidden.double() @ W.double().T, batch.ids[:n])
        logp_old = (logp + batch.noise[:n].double()).float()
        call = (hidden, W, batch.ids[:n], None, batch.cu_seqlens[:n_seq + 1], adv_seq, logp_old)
        run_once = lambda: O.fused_lmhead_loss(*call, None, None, O.LossParams())
    else:
        n_seq = 1
        while int(batch.cu_seqlens[n_seq]) < REFERENCE_ROWS and n_seq < batch.S:
            n_seq += 1
        n = int(batch.cu_seqlens[n_seq])
        z = batch.logits_rows(0, n)
        adv_seq = adv[batch.seq_p.long(), batch.seq_m.long(), batch.seq_g.long()][:n_seq]
        logp, _, _ = O.token_logprobs(z, batch.ids[:n])
        logp_old = (logp + batch.noise[:n].double()).float()
        call = (z, batch.ids[:n], None, batch.cu_seqlens[:n_seq + 1], adv_seq, logp_old)
        run_once = lambda: O.policy_loss(*call, None, None, O.LossParams())
    for _ in range(min(args.warmup, 1)):
        run_once()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        O.group_advantages(meta.rewards)
        run_once()
    dt = time.perf_counter() - t0
    value = n * args.steps / dt
    cores = torch.get_num_threads()
    sample = f"first {n} rows ({n_seq} sequences) of the workload per step, full V, fwd+bwd"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "rows_per_step": n, "V": w.V, "H": w.H},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_e2e(args, wl, world):
    e2e_steps = max(1, min(args.steps, 3))
    wl.e2e_slab_rows = args.e2e_slab_rows
    h2d, d2h = wl.e2e_setup()
    wl.e2e_step()
    torch.cuda.synchronize()
    barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        wl.e2e_step()
    e1.record()
    torch.cuda.synchronize()
    barrier(world)
    e2e_ms, e2e_tokens = aggregate_over_ranks(e0.elapsed_time(e1), wl.tokens() * e2e_steps, world)
    return {"value": e2e_tokens / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "steps": e2e_steps,
            "note": wl.e2e_note if hasattr(wl, "e2e_note") else
            "C-ABI calls on device buffers bracketed by pinned-host copies of every input and of the gradients, "
            "logp and loss"}


def measure(wl, steps, warmup, world, local_rank, rank, peaks, with_e2e, with_cpu, args, single_thread=True):
    """Warm up, time `steps` steps with CUDA events (max over ranks), and build the result fields."""
    B = wl.B
    for _ in range(max(warmup, 3)):
        wl.step()
    torch.cuda.synchronize()
    timer = B.DominantKernelTimer(steps * wl.dominant_per_step)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(world)
    torch.cuda.synchronize()
    with ClockSampler(local_rank, 0.002 if hasattr(wl, "product_kinds") else 0.005) as clocks, timer:
        t_start = time.perf_counter()        # the device is idle: the first launch starts about now
        ev0.record()
        for _ in range(steps):
            wl.step()
        ev1.record()
        torch.cuda.synchronize()
    barrier(world)
    local_ms = ev0.elapsed_time(ev1)
    kernel_ms = timer.elapsed_ms(steps * wl.dominant_per_step)
    wl.last_kernel = timer.last_kernel
    per_product = None
    if hasattr(wl, "product_kinds"):       # time x clock of every kind of tensor-core launch
        n = steps * wl.dominant_per_step
        kinds, flops = wl.product_kinds(steps)
        offsets = [ev0.elapsed_time(timer.start[i]) for i in range(n)]
        per_product = per_product_table(kinds, flops, offsets, kernel_ms[:n], t_start, clocks,
                                        torch.cuda.get_device_properties(local_rank).multi_processor_count)
    status = int(wl.status.cpu())
    if status != 0:
        raise SystemExit(f"device status word is {status} after the timed region")
    total_ms, total_tokens = aggregate_over_ranks(local_ms, wl.tokens() * steps, world)
    out = {"value": total_tokens / (total_ms * 1e-3), "ms_per_step": total_ms / steps, "steps": steps,
           "config": dict(wl.describe(), parallelism=f"replicas x{world}"), "clocks": clocks.summary(),
           "gpu_launches": wl.kernels_per_step * steps, "roofline": wl.roofline(kernel_ms, peaks)}
    if per_product is not None:
        out["roofline"]["per_product"] = per_product
    # end to end: pinned host buffers -> device -> kernels -> pinned host buffers
    out["e2e"] = run_e2e(args, wl, world) if with_e2e else None
    if world == 1 and with_e2e and hasattr(wl, "measure_skip_zero_rows") and wl.ratio_level == 0 and not wl.lp.logp_ref:
        out["skip_zero_rows"] = wl.measure_skip_zero_rows()
        out["token_logprobs"] = wl.measure_forward_only(peaks)
    if world == 1 and hasattr(wl, "measure_in_place") and wl.ratio_level == 0 and getattr(args, "in_place_leg", True):
        out["in_place"] = wl.measure_in_place(peaks)
    out["cpu_baseline"] = None
    if with_cpu and rank == 0 and world == 1:
        n, dt, sample = wl.time_oracle()
        out["cpu_baseline"] = {"value": n / dt, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
                               "sample": sample}
        if not single_thread:
            return out
        # the same oracle on one thread, on a sample an eighth the size
        threads = torch.get_num_threads()
        torch.set_num_threads(1)
        try:
            n1, dt1, sample1 = wl.time_oracle(scale=8)
        finally:
            torch.set_num_threads(threads)
        out["cpu_baseline"]["single_thread"] = {"value": n1 / dt1, "unit": UNIT, "cores": 1, "kind": "oracle",
                                                "sample": sample1}
    return out


def run_ours(args, rank, world, local_rank):
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    if torch.cuda.device_count() <= local_rank:
        raise SystemExit(f"bench.py: rank {rank} wants cuda:{local_rank} but {torch.cuda.device_count()} device(s) are visible")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    from paper_2605_07244_b200 import binding as B
    from paper_2605_07244_b200 import build
    build.build()
    B.lib()
    if args.workload not in ("C2", "C2s", "C5", "C5s", "C5b", "C3", "C4"):
        raise SystemExit("bench.py times config 2 (logits-in; C2s is its small profiling case), config 5 (fused LM "
                         "head) and one slab of config 3 or 4; configs 1 and 6 are parity-test cases")
    peaks = measured_peaks()
    lmhead_main = args.workload in ("C5", "C5s", "C5b")
    slab_main = args.workload in ("C3", "C4")
    cls = LmheadWorkload if lmhead_main else LogitsInWorkload
    wl = (PoolSlabWorkload(args.workload, args.seed + rank, device, args.slab_rows) if slab_main else
          cls(synth.CONFIGS[args.workload], args.seed + rank, device, args.pair_tiles, args.skip_zero_rows)
          if lmhead_main else
          cls(synth.CONFIGS[args.workload], args.seed + rank, device, 1 if args.ratio_level == "sequence" else 0,
              args.with_entropy, args.with_kl))
    res = measure(wl, args.steps, args.warmup, world, local_rank, rank, peaks, not args.no_e2e and not slab_main,
                  not args.no_cpu_baseline and not slab_main, args)
    if lmhead_main and args.library_loop and world == 1:
        N_, H_, V_ = wl.N, wl.H, wl.V
        del wl
        torch.cuda.empty_cache()
        res["roofline"]["library_loop"] = library_loop_per_product(N_, H_, V_, min(16384, V_), max(2, min(args.steps, 4)),
                                                                    local_rank)
        wl = None
    del wl
    torch.cuda.empty_cache()

    # beside the headline: the shapes the paper's setup runs, one sub-object each with its own roofline and clocks
    sub_keys = ("value", "ms_per_step", "steps", "config", "clocks", "gpu_launches", "roofline")
    shapes = {}
    if args.workload == "C2" and not args.no_lmhead:
        sub_steps = min(args.steps, 20)
        # every row with a gradient: the KL penalty of Eq. (1) on (App. A: beta = 1e-3), same batch as the headline
        wl_kl = LogitsInWorkload(synth.CONFIGS["C2"], args.seed + rank, device, 0, False, True)
        r = measure(wl_kl, sub_steps, 3, world, local_rank, rank, peaks, False, False, args)
        shapes["all_rows_live"] = {"metric": METRIC, "unit": UNIT, **{k: r[k] for k in sub_keys}, "in_place": r.get("in_place")}
        del wl_kl
        torch.cuda.empty_cache()
        for key, name in (("prp_pool_slab", "C3"), ("xgrpo_sgt_slab", "C4")):
            wls = PoolSlabWorkload(name, args.seed + rank, device, args.slab_rows)
            r = measure(wls, sub_steps, 3, world, local_rank, rank, peaks, False, False, args)
            shapes[key] = {"metric": METRIC, "unit": UNIT, **{k: r[k] for k in sub_keys}}
            del wls
            torch.cuda.empty_cache()

    # the tensor-core family: a short config-5 leg in the default run
    lmhead = None
    if args.workload == "C2" and not args.no_lmhead:
        wl5 = LmheadWorkload(synth.CONFIGS["C5"], args.seed + rank, device)
        r5 = measure(wl5, min(args.steps, LMHEAD_SUB_STEPS), 3, world, local_rank, rank, peaks, False,
                     not args.no_cpu_baseline, args, single_thread=False)
        lmhead = {"metric": METRIC, "unit": UNIT, **{k: r5[k] for k in sub_keys + ("cpu_baseline",)}}
        del wl5
        # the same shape with success rates drawn per prompt (many all-success / all-failure groups), zero rows skipped
        wl5b = LmheadWorkload(synth.CONFIGS["C5b"], args.seed + rank, device, False, True)
        r5b = measure(wl5b, min(args.steps, LMHEAD_SUB_STEPS), 3, world, local_rank, rank, peaks, False, False, args)
        lmhead["skip_zero_rows"] = {k: r5b[k] for k in ("value", "ms_per_step", "steps", "config", "clocks", "roofline")}
        del wl5b

    thl = tiny = f32 = None
    if args.workload == "C2" and not args.no_lmhead and rank == 0 and world == 1:
        thl = measure_thl_align(args.seed, not args.no_cpu_baseline)
        tiny = measure_tiny_latency(args.seed)
        f32 = measure_float32_rows(args.seed, peaks)

    if rank == 0:
        line = {
            "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": res["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if lmhead_main else "f32", "data": "synthetic",
            "config": res["config"], "clocks": res["clocks"], "e2e": res["e2e"], "gpu_launches": res["gpu_launches"],
            "roofline": res["roofline"], "cpu_baseline": res["cpu_baseline"],
        }
        if res.get("skip_zero_rows") is not None:
            line["skip_zero_rows"] = res["skip_zero_rows"]
            line["token_logprobs"] = res["token_logprobs"]
        if res.get("in_place") is not None:
            line["in_place"] = res["in_place"]
        line.update(shapes)
        if lmhead is not None:
            line["lmhead"] = lmhead
        if thl is not None:
            line["thl_align"] = thl
        if tiny is not None:
            line["tiny_step_latency"] = tiny
        if f32 is not None:
            line["float32_logits"] = f32
        print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C2")
    ap.add_argument("--seed", type=int, default=2)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="profiling runs only: skip the host-buffer leg")
    ap.add_argument("--ratio-level", default="token", choices=["token", "sequence"],
                    help="logits-in workloads: importance ratio per token (Eq. (1), default) or per response (App. H)")
    ap.add_argument("--with-kl", action="store_true",
                    help="logits-in workloads: add the KL penalty to a reference trace (k3 estimate, beta = 1e-3)")
    ap.add_argument("--with-entropy", action="store_true", help="logits-in workloads: also emit the per-row policy entropy")
    ap.add_argument("--e2e-slab-rows", type=int, default=1024,
                    help="logits-in end-to-end leg: rows per micro-batch of the host pipeline")
    ap.add_argument("--skip-zero-rows", action="store_true",
                    help="fused LM-head workloads: MRL_FLAG_SKIP_ZERO_ROWS (zero-multiplier rows are not produced)")
    ap.add_argument("--library-loop", action="store_true",
                    help="fused LM-head workloads: also time torch.matmul (the vendor library) on the same product shapes, "
                         "per product with the SM clock, beside the step's own per-product table (a comparison leg)")
    ap.add_argument("--pair-tiles", action="store_true",
                    help="fused LM-head workloads: 256-row tiles worked by CTA pairs (MRL_FLAG_PAIR_TILES)")
    ap.add_argument("--no-lmhead", action="store_true",
                    help="skip the legs beside the headline (all-rows-live, config-3 / config-4 slabs, config 5, ...)")
    ap.add_argument("--slab-rows", type=int, default=40960,
                    help="config-3 / config-4 legs: largest slab (whole sequences) in rows; 40,960 rows are 10.5 / 12.4 GB of logits")
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be at least 1")
    placed = resolve_world(args.gpus)
    if placed is None:          # plain `python bench.py --gpus N`: start the N ranks here
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))
    rank, world, local_rank = placed
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    try:
        run_ours(args, rank, world, local_rank)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
