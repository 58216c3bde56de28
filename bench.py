#!/usr/bin/env python
"""Benchmark of the T-PPO token-selective update path on B200.

One "step" is one pass of the whole hot path over one synthetic batch shaped like the paper's
Qwen2.5-32B long-CoT step: EGAE + Monte-Carlo returns over the full batch of 512 ragged responses,
policy / value token selection, the fused log-prob + clipped-surrogate loss forward/backward over a
[16384, 152064] bf16 logits micro-batch (gradient written to a second buffer), and the value loss
on 16384 value tokens.  The metric is selected (policy) tokens per second.

  python bench.py [--gpus N] [--steps K] [--warmup W]            CUDA path (this repo)
  python bench.py --impl reference ...                           float64 CPU oracle on host cores
  python bench.py --workload lmhead ...                          the LM-head variant as the bench line
  python bench.py --workload cfg4 ...                            EGAE + compaction sweep (config 4)

The default line also carries an "lmhead_variant" object: the tensor-core variant that forms the
logits from hidden states [16384, 5120] and the LM-head weight [5120, 152064] without storing them,
timed on its own after the main measurement (a few calls) against the bf16 tensor roofline.

Prints one JSON line.  With N > 1 (torchrun) every rank runs the same per-GPU workload (the path
shards by sequence with no data-path collective); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2506_15050_b200 import synth  # noqa: E402

METRIC = "selected tokens/s, fused logprob+PPO loss fwd+bwd, V=152064 bf16; % HBM peak"
UNIT = "selected tokens/s"
ALGO_BYTES_PER_TOKEN = 2 * 2 * synth.V_QWEN       # bf16 row read once + bf16 gradient row written once
# dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture at 2048 rows (the full workload is too
# large to capture) of the two kernels that share the rows of a policy-loss call: policy_cluster_kernel
# 569.41 + 517.59 MB on 1872 rows, policy_two_pass_kernel (side launch) 53.58 + 12.89 MB on 176 rows;
# per row, scaled by rows.  (Reads are exactly one pass over the logits; of the writes about 90 MB were
# still in L2 when the capture ended, at any row count, so the scaled figure understates full-size
# writes by about 7 %.)  The summary of that capture under profiles/ has the command.
NCU_TRAFFIC_BYTES_PER_TOKEN = (569.413376e6 + 517.587200e6 + 53.582080e6 + 12.886528e6) / 2048


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def measured_tensor_peaks():
    """(burst, sustained) dense bf16 TFLOP/s of this machine's B200s and where the figures come from."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            j = json.load(f)
            return float(j["bf16_tflops"]), float(j["bf16_tflops_sustained"]), "measured"
    except Exception:
        return 1590.0, 1400.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons while the timed region runs: NVML from a thread every
    2 ms (read-only queries), or `nvidia-smi -lms` when the NVML binding is not importable.  A timed
    region of a few tens of milliseconds still gets its samples this way."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None
        self.sm, self.reasons, self.sm_max = [], set(), None
        self.stop_flag, self.thread, self.nvml = threading.Event(), None, None

    def _nvml_loop(self):
        n, h = self.nvml
        bits = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                "sw_power_cap": 0x4}
        get_reasons = getattr(n, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(n, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self.stop_flag.is_set():
            try:
                self.sm.append(float(n.nvmlDeviceGetClockInfo(h, n.NVML_CLOCK_SM)))
                r = int(get_reasons(h))
                for name, bit in bits.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        try:
            import pynvml as n
            n.nvmlInit()
            # torch's device index is an index into CUDA_VISIBLE_DEVICES
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = self.index
            if vis:
                ent = vis.split(",")[self.index].strip()
                phys = int(ent) if ent.isdigit() else None
            h = n.nvmlDeviceGetHandleByIndex(phys) if phys is not None else \
                n.nvmlDeviceGetHandleByUUID(ent.encode())
            self.sm_max = float(n.nvmlDeviceGetMaxClockInfo(h, n.NVML_CLOCK_SM))
            self.nvml = (n, h)
            self.thread = threading.Thread(target=self._nvml_loop, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.nvml is not None:
            self.stop_flag.set()
            self.thread.join(timeout=1.0)
            return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.sm_max,
                    "reasons": sorted(self.reasons), "samples": len(self.sm), "source": "nvml, every 2 ms"}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(self.NAMES, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm), "source": "nvidia-smi -lms 100"}


def spawn_ranks(n_gpus: int) -> int:
    """`python bench.py --gpus N` outside torchrun: start the N ranks of one node ourselves (the same
    launcher and rendezvous a torchrun command line would use) and return their exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def dist_setup(n_gpus: int, need_cuda: bool = True):
    """Rank, world size and local rank from the launcher's environment; NCCL between GPUs (gloo when
    there is no GPU, which only the launcher's own test uses).  The world that came up must be the
    one that was asked for."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != n_gpus:
        raise SystemExit(f"bench.py: --gpus {n_gpus} but the launcher started {world} rank(s)")
    if world > 1:
        import torch.distributed as dist
        if need_cuda and torch.cuda.is_available():
            if torch.cuda.device_count() < world:
                raise SystemExit(f"bench.py: {world} ranks but {torch.cuda.device_count()} GPU(s)")
            os.environ.setdefault("NCCL_DEBUG", "INFO")          # the init log shows the ranks of the communicator
            os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
            torch.cuda.set_device(local)
            dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
        else:
            dist.init_process_group("gloo")
        if dist.get_world_size() != n_gpus:
            raise SystemExit(f"bench.py: process group has {dist.get_world_size()} ranks, wanted {n_gpus}")
    return rank, world, local


def time_stats(ms_list):
    """mean / median / min of per-step device times (ms)."""
    a = np.asarray(ms_list, np.float64)
    return {"mean": float(a.mean()), "median": float(np.median(a)), "min": float(a.min())}


class Step:
    """Device-resident state of the workload and the four C-ABI calls of one step."""

    def __init__(self, dev, seed=2, rows=16384):
        from paper_2506_15050_b200 import binding as b
        self.b, self.dev = b, dev
        c = synth.config3(dev, seed=seed, n_tokens=rows)
        self.c = c
        t = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).to(dev)
        self.N, self.B, self.V, self.n = c["N"], c["B"], c["V"], c["n_tokens"]
        self.host = {k: c[k] for k in ("rewards", "values", "old_values", "seg_begin", "seg_end",
                                       "truncated", "seq_begin", "prompt_len", "prev_len", "new_len",
                                       "extra_policy_mask", "extra_value_mask", "targets")}
        self.rewards, self.values = t(c["rewards"], torch.float32), t(c["values"], torch.float32)
        self.old_values = t(c["old_values"], torch.float32)
        self.seg_b, self.seg_e = t(c["seg_begin"], torch.int32), t(c["seg_end"], torch.int32)
        self.trunc = t(c["truncated"], torch.uint8)
        self.seq_begin = t(c["seq_begin"], torch.int32)
        self.prompt, self.prev, self.new = (t(c[k], torch.int32) for k in ("prompt_len", "prev_len", "new_len"))
        self.pmask, self.vmask = t(c["extra_policy_mask"], torch.uint8), t(c["extra_value_mask"], torch.uint8)
        self.targets = t(c["targets"], torch.int32)
        self.logits = c["logits"]
        N, n = self.N, self.n
        self.adv, self.ret = torch.zeros(N, device=dev), torch.zeros(N, device=dev)
        self.pol = torch.zeros(N, dtype=torch.int32, device=dev)
        self.val = torch.zeros(N, dtype=torch.int32, device=dev)
        self.counts = torch.zeros(4, dtype=torch.int32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.logp, self.tok_loss = torch.zeros(n, device=dev), torch.zeros(n, device=dev)
        self.loss, self.vloss = torch.zeros(1, device=dev), torch.zeros(1, device=dev)
        self.stats = torch.zeros(4, dtype=torch.int32, device=dev)
        self.vstats = torch.zeros(2, dtype=torch.int32, device=dev)
        self.dlogits = torch.empty_like(self.logits)
        self.dvalues = torch.zeros(N, device=dev)
        self.old_logp = torch.zeros(N, device=dev)
        self.ws_egae = b.workspace(b.OP_EGAE, N, self.B, 0, 0, dev)
        self.ws_sel = b.workspace(b.OP_SELECT_TOKENS, N, self.B, 0, 0, dev)
        self.ws_pol = b.workspace(b.OP_POLICY_LOSS, n, 0, n, self.V, dev)
        self.ws_val = b.workspace(b.OP_VALUE_LOSS, N, 0, N, 0, dev)
        self.ev = None
        self.hint = 0
        # EGAE and the token selection read the same inputs and write disjoint outputs: the selection
        # runs on a second stream beside the scan (both are chains of latencies, not bandwidth)
        self.side = torch.cuda.Stream(device=dev)
        self.overlap = True
        self.denom_pol = 0.0      # > 0: selected-token counts of the whole job (several GPUs)
        self.denom_val = 0.0
        # old-policy log-probs (the old-policy snapshot of Algorithm 1): forward-only pass of the same kernel, plus noise
        self.egae()
        self.select()
        self.policy(forward_only=True)
        torch.cuda.synchronize()
        idx = self.pol[:n].long()
        self.old_logp[idx] = self.logp + t(c["old_logp_noise"], torch.float32)[idx]

    def egae(self):
        c = self.c
        self.b.tppo_egae(self.rewards, self.values, self.seg_b, self.seg_e, self.trunc, None,
                         c["gamma"], c["lam"], self.adv, self.ret, self.status, self.ws_egae)

    def select(self):
        self.b.tppo_select_tokens(self.seq_begin, self.prompt, self.prev, self.new, self.trunc, 0,
                                  self.pmask, self.vmask, self.N, self.pol, self.val, self.counts,
                                  self.ws_sel)

    def policy(self, forward_only=False):
        c, b = self.c, self.b
        b.tppo_policy_loss_fwd_bwd(
            self.logits, self.targets, None, self.counts[0:1], self.n, self.pol, self.old_logp,
            self.adv, c["eps_low"], c["eps_high"], self.denom_pol, self.logp, self.tok_loss, self.loss,
            self.stats, None if forward_only else self.dlogits,
            b.DLOGITS_NONE if forward_only else b.DLOGITS_COMPACT, self.ws_pol, kernel_hint=self.hint)

    def value(self):
        c = self.c
        self.b.tppo_value_loss(self.values, self.old_values, self.ret, self.val, self.counts[1:2],
                               self.N, c["xi_low"], c["xi_high"], self.denom_val, self.vloss, self.dvalues,
                               self.vstats, self.ws_val)

    def run(self, events=None):
        """One step.  With `events` (a list), five CUDA events are recorded around the four calls and
        appended as one tuple: the calls' device times come out of the same run that is timed."""
        timed = events is not None
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(5)] if timed else None
        if timed:
            ev[0].record()
        if self.overlap:
            main = torch.cuda.current_stream()
            fork, join = torch.cuda.Event(), torch.cuda.Event()
            fork.record(main)
            self.side.wait_event(fork)
            with torch.cuda.stream(self.side):
                self.select()
                join.record(self.side)
            self.egae()
            if timed:
                ev[1].record()
            main.wait_event(join)       # ev[1] -> ev[2]: what of the selection is left after the scan
        else:
            self.egae()
            if timed:
                ev[1].record()
            self.select()
        if not timed:
            self.policy()
            self.value()
            return
        ev[2].record()
        self.policy()
        ev[3].record()
        self.value()
        ev[4].record()
        events.append(tuple(ev))

    # EGAE clear + scan, selection clear + kernel, policy prepare + cluster sweep + side sweep + finish,
    # value clear + kernel (a policy call below 2048 rows has no side sweep)
    KERNELS_PER_STEP = 10


class LmHeadStep:
    """Device-resident state of the LM-head workload (config 5) and its one C-ABI call."""
    KERNELS_FIXED = 4      # prepare, statistics GEMM, row merge, finish

    def __init__(self, dev, M=16384, K=5120, V=synth.V_QWEN):
        from paper_2506_15050_b200 import binding as b
        self.b, self.dev = b, dev
        c = synth.config5(dev, M=M, K=K, V=V)
        self.c, self.M, self.K, self.V = c, M, K, V
        t = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).to(dev)
        self.hidden, self.weight = c["hidden"], c["weight"]
        self.targets, self.adv = t(c["targets"], torch.int32), t(c["adv"], torch.float32)
        self.old_logp = torch.zeros(M, device=dev)
        self.logp, self.tok_loss = torch.zeros(M, device=dev), torch.zeros(M, device=dev)
        self.loss = torch.zeros(1, device=dev)
        self.stats = torch.zeros(4, dtype=torch.int32, device=dev)
        self.dhidden = torch.empty_like(self.hidden)
        self.dweight = torch.empty_like(self.weight)
        self.ws = b.workspace(b.OP_LMHEAD, M, K, 0, V, dev)
        # old-policy log-probs: forward-only call of the same entry point, plus noise
        self.run(forward_only=True)
        torch.cuda.synchronize()
        self.old_logp.copy_(self.logp + t(c["old_logp_noise"], torch.float32))

    def run(self, forward_only=False):
        c = self.c
        self.b.tppo_lmhead_logprob_fwd_bwd(
            self.hidden, self.weight, self.targets, None, self.old_logp, self.adv, c["eps_low"],
            c["eps_high"], 0.0, self.logp, self.tok_loss, self.loss, self.stats,
            None if forward_only else self.dhidden, None if forward_only else self.dweight, self.ws)

    def gemm_flops(self):
        return 2.0 * self.M * self.K * self.V

    def roofline(self, ms):
        """Tensor roofline: three GEMM-sized contractions are what the result needs (logits, dhidden,
        dweight); the kernels execute a fourth (the logits are recomputed instead of stored)."""
        burst, sustained, kind = measured_tensor_peaks()
        achieved = 3.0 * self.gemm_flops() / (ms * 1e-3) / 1e12
        return {"bound": "tensor", "achieved": achieved, "peak": sustained, "unit": "TFLOP/s",
                "frac": achieved / sustained, "peak_kind": kind + ", sustained (calls run back to back)",
                "frac_of_burst_peak": achieved / burst, "traffic": None,
                "executed_tflops": 4.0 * self.gemm_flops() / (ms * 1e-3) / 1e12,
                "executed_frac": 4.0 * self.gemm_flops() / (ms * 1e-3) / 1e12 / sustained,
                "kernel": "umma_gemm_kernel (statistics, dX, dhidden, dweight epilogues)",
                "call_ms": ms, "algorithmic_flops_per_call": 3.0 * self.gemm_flops()}


def time_lmhead(lm, calls, warmup):
    for _ in range(warmup):
        lm.run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(calls):
        lm.run()
    e1.record()
    torch.cuda.synchronize()
    assert int(lm.stats[3].item()) == 0 and int(lm.stats[0].item()) == lm.M
    return e0.elapsed_time(e1) / calls


def time_lmhead_rank_of_shards(lm, shards, calls, warmup):
    """What ONE rank of a vocabulary-parallel LM-head executes per step (its statistics call, the
    rescale between the two all-reduces, its loss + gradient call), with the other ranks' statistics
    produced beforehand on the same GPU.  The collectives themselves are not part of the number."""
    b, dev, M, K, V = lm.b, lm.dev, lm.M, lm.K, lm.V
    width = (V // shards + 7) // 8 * 8
    bounds = [min(i * width, V) for i in range(shards)] + [V]
    stats = []
    for lo, hi in zip(bounds[:-1], bounds[1:]):
        w = lm.weight[:, lo:hi].contiguous()
        m_, s_, xy_ = (torch.empty(M, device=dev) for _ in range(3))
        st = torch.zeros(4, dtype=torch.int32, device=dev)
        ws = b.workspace(b.OP_LMHEAD, M, K, 0, hi - lo, dev)
        b.tppo_lmhead_shard_stats(lm.hidden, w, lo, V, lm.targets, m_, s_, xy_, st, ws)
        stats.append((m_, s_, xy_))
        del w, ws
    m_all = torch.stack([x[0] for x in stats]).max(dim=0).values
    for m_, s_, _ in stats:
        b.tppo_lmhead_shard_rescale(m_, m_all, s_)
    s_all = torch.stack([x[1] for x in stats]).sum(dim=0)
    xy_all = torch.stack([x[2] for x in stats]).sum(dim=0)
    w0 = lm.weight[:, bounds[0]:bounds[1]].contiguous()
    dw0 = torch.empty_like(w0)
    ws = b.workspace(b.OP_LMHEAD, M, K, 0, bounds[1] - bounds[0], dev)
    m0, s0, xy0 = (torch.empty(M, device=dev) for _ in range(3))
    st = torch.zeros(4, dtype=torch.int32, device=dev)
    c = lm.c

    def rank_step():
        b.tppo_lmhead_shard_stats(lm.hidden, w0, 0, V, lm.targets, m0, s0, xy0, st, ws)
        b.tppo_lmhead_shard_rescale(m0, m_all, s0)
        b.tppo_lmhead_shard_fwd_bwd(lm.hidden, w0, 0, V, lm.targets, None, lm.old_logp, lm.adv,
                                    c["eps_low"], c["eps_high"], 0.0, m_all, s_all, xy_all, lm.logp,
                                    lm.tok_loss, lm.loss, lm.stats, lm.dhidden, dw0, ws)

    for _ in range(warmup):
        rank_step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(calls):
        rank_step()
    e1.record()
    torch.cuda.synchronize()
    assert int(lm.stats[3].item()) == 0
    return {"shards": shards, "per_rank_ms": e0.elapsed_time(e1) / calls,
            "exchange_bytes_per_rank": {"row_statistics_allreduce": 12 * M, "dhidden_allreduce": 2 * M * K},
            "note": "one rank's three calls timed on one GPU; the other ranks' statistics were "
                    "produced beforehand; the two small all-reduces and the dhidden all-reduce are "
                    "not timed"}


def cpu_oracle_lmhead_seconds(lm, sample_rows):
    """The oracle on `sample_rows` rows of the LM-head workload: float64 logits, Eq. 1, dhidden rows
    and those rows' share of dweight; scaled by rows to the whole call."""
    import oracle
    f32 = lambda x: float(np.float32(x))
    c = lm.c
    rows = np.arange(sample_rows, dtype=np.int32)
    hb = synth.bf16_bits(lm.hidden[:sample_rows])
    wb = synth.bf16_bits(lm.weight)
    old = lm.old_logp[:sample_rows].cpu().numpy()
    t0 = time.perf_counter()
    x = oracle.lmhead_logits_rows(hb, wb, rows)
    ref = oracle.policy_loss(x, c["targets"][:sample_rows], None, None, old, c["adv"][:sample_rows],
                             f32(c["eps_low"]), f32(c["eps_high"]), denom=float(lm.M))
    oracle.lmhead_dhidden_rows(ref["dlogits"], wb)
    oracle.lmhead_dweight_cols(hb, ref["dlogits"])
    t = time.perf_counter() - t0
    return t * (lm.M / sample_rows), oracle.num_threads()


def cpu_oracle_step_seconds(c, n_tokens, sample_rows):
    """Times the oracle, as it stands, on host cores: EGAE and selection on the full batch, policy
    loss forward+backward on `sample_rows` rows of the micro-batch (scaled to n_tokens), value loss."""
    import oracle
    f32 = lambda x: float(np.float32(x))
    t0 = time.perf_counter()
    adv, ret = oracle.egae(c["rewards"], c["values"], c["seg_begin"], c["seg_end"], c["truncated"],
                           None, f32(c["gamma"]), f32(c["lam"]))
    t1 = time.perf_counter()
    pol, val = oracle.select_tokens(c["seq_begin"], c["prompt_len"], c["prev_len"], c["new_len"],
                                    c["truncated"], 0, c["extra_policy_mask"], c["extra_value_mask"])
    t2 = time.perf_counter()
    logits = c["logits_sample"]
    rows = np.arange(sample_rows, dtype=np.int32)
    old = np.zeros(c["N"], np.float32)
    out = oracle.policy_loss(logits, c["targets"], rows, pol[:sample_rows], old,
                             adv.astype(np.float32), f32(c["eps_low"]), f32(c["eps_high"]),
                             float(n_tokens))
    t3 = time.perf_counter()
    oracle.value_loss(c["values"], c["old_values"], ret.astype(np.float32), val, f32(c["xi_low"]),
                      f32(c["xi_high"]))
    t4 = time.perf_counter()
    del out
    t_policy = (t3 - t2) * (n_tokens / sample_rows)
    return (t1 - t0) + (t2 - t1) + t_policy + (t4 - t3), oracle.num_threads(), \
        {"egae_s": t1 - t0, "select_s": t2 - t1, "policy_sample_s": t3 - t2, "value_s": t4 - t3}


def workload_config(N, n_tok, n_val, hint=0):
    """The `config` object of the bench line: the same for this repo's arm and the reference arm."""
    return {"workload": "cfg3: EGAE over 512 ragged responses (N=%d tokens), selection, [%d,152064] bf16 "
                        "fused log-prob+PPO loss fwd+bwd, value loss on %d tokens" % (N, n_tok, n_val),
            "l2": "inputs larger than L2 (%.2f GB logits per step)" % (n_tok * synth.V_QWEN * 2 / 1e9),
            "dlogits": "compact, separate buffer", "kernel_hint": hint}


def run_reference(args, rank):
    """The oracle on the host cores, as it stands: same metric, a bounded sample per step.  A step is
    EGAE, selection and the value loss on the full batch plus the policy loss forward+backward on
    `--ref-rows` rows of the micro-batch; the reported time is the measured time of that step and the
    value counts the rows that went through the policy loss in it."""
    if rank != 0:
        return
    c = synth.config3("cpu", with_logits=False)
    sample_rows = args.ref_rows
    c["logits_sample"] = synth.bf16_bits(synth.randn_bf16((sample_rows, synth.V_QWEN), 2.0, 2, "cpu"))
    times = []
    cores = 1
    for i in range(args.warmup + args.steps):
        w0 = time.perf_counter()
        _, cores, parts = cpu_oracle_step_seconds(c, c["n_tokens"], sample_rows)
        if i >= args.warmup:
            times.append(time.perf_counter() - w0)
    t = float(np.mean(times))
    value = sample_rows / t
    sample = (f"per step: EGAE+selection+value loss on the full batch, policy loss fwd+bwd on {sample_rows} "
              f"of {c['n_tokens']} rows (V=152064); value = those {sample_rows} rows / measured step time")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(c["N"], c["n_tokens"], int(c["extra_value_mask"].sum()), args.hint),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def run_stub(args, rank, world):
    """A step that needs no GPU, for the launcher's own test: every rank does a fixed piece of host
    work, the ranks meet at a barrier, and rank 0 prints the line with the world size that came up."""
    import torch.distributed as dist
    x = torch.arange(1 << 16, dtype=torch.float64)
    w0 = time.perf_counter()
    for _ in range(args.warmup + args.steps):
        x = (x * 1.0000001).cumsum(0) % 7.0
    t = torch.tensor([time.perf_counter() - w0], dtype=torch.float64)
    if world > 1:
        dist.barrier()
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        print(json.dumps({"metric": "stub steps/s (launcher test)", "value": world * args.steps / float(t),
                          "unit": "steps/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                          "ms_per_step": float(t) * 1e3 / max(args.steps, 1), "higher_is_better": True,
                          "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                          "config": {"workload": "stub"}, "gpu_launches": 0}))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ref-rows", type=int, default=512, help="oracle sample rows per step")
    ap.add_argument("--cpu-rows", type=int, default=1024, help="rows of the cpu_baseline sample")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--hint", type=int, default=0, help="kernel_hint passed to the policy loss")
    ap.add_argument("--rows", type=int, default=16384,
                    help="rows of the loss micro-batch (smaller only for profiler captures)")
    ap.add_argument("--workload", default="cfg3", choices=["cfg3", "lmhead", "cfg4", "configs", "stub"])
    ap.add_argument("--lmhead-calls", type=int, default=5)
    ap.add_argument("--lm-shards", type=int, default=1,
                    help="with --workload lmhead: also time one rank of this many vocabulary shards")
    ap.add_argument("--lm-rows", type=int, default=16384,
                    help="rows of the LM-head workload (smaller only for profiler captures)")
    ap.add_argument("--cfg4-steps", type=int, default=30, help="steps of the small-kernel measurement")
    ap.add_argument("--serial", action="store_true",
                    help="run the token selection after EGAE on the same stream instead of beside it")
    ap.add_argument("--no-lmhead", action="store_true")
    ap.add_argument("--no-small", action="store_true", help="skip the config-4 small-kernel measurement")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--graph-steps", type=int, default=50,
                    help="steps of the extra measurement that replays the step as one CUDA graph (0: skip)")
    args = ap.parse_args()

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus))           # one process per GPU, started here
    rank, world, local = dist_setup(args.gpus, need_cuda=args.workload != "stub" and args.impl == "ours")
    if args.workload == "stub":
        run_stub(args, rank, world)
        return
    if args.impl == "reference":
        run_reference(args, rank)
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA path has no CPU fallback")
    warmup = max(args.warmup, 3)
    dev = f"cuda:{local}"
    torch.cuda.set_device(local)
    if args.workload == "lmhead":
        run_lmhead_workload(args, rank, world, local, dev, warmup)
        return
    if args.workload == "cfg4":
        run_cfg4_workload(args, rank, world, local, dev, warmup)
        return
    if args.workload == "configs":
        run_config_table(args, dev)
        return
    st = Step(dev, seed=2 + rank, rows=args.rows)      # every rank holds its own batch
    st.overlap = not args.serial
    st.hint = args.hint
    if world > 1:
        # token-level mean over the whole job: each rank divides by the global selected-token counts
        from paper_2506_15050_b200 import shard
        torch.cuda.synchronize()
        n_pol, n_val = shard.global_token_counts(int(st.counts[0].item()), int(st.counts[1].item()),
                                                 device=dev)
        st.denom_pol, st.denom_val = float(n_pol), float(n_val)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        st.run()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    events, marks = [], [torch.cuda.Event(enable_timing=True)]
    marks[0].record()
    for _ in range(args.steps):
        st.run(events)
        marks.append(torch.cuda.Event(enable_timing=True))
        marks[-1].record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms_total = marks[0].elapsed_time(marks[-1])
    if world > 1:
        import torch.distributed as dist
        tt = torch.tensor([ms_total], device=dev)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        ms_total = float(tt.item())
    ms_step = ms_total / args.steps
    step_ms = time_stats([a.elapsed_time(b) for a, b in zip(marks[:-1], marks[1:])])
    n_tok = int(st.counts[0].item())
    n_val = int(st.counts[1].item())
    assert n_tok == st.n and int(st.stats[3].item()) == 0 and int(st.status.item()) == 0
    value = world * n_tok / (ms_step * 1e-3)
    pol = time_stats([e[2].elapsed_time(e[3]) for e in events])
    sel_name = "select_after_egae (the selection runs beside the scan on a second stream)" if st.overlap else "select"
    calls_us = {name: time_stats([e[k].elapsed_time(e[k + 1]) * 1e3 for e in events])
                for k, name in enumerate(("egae", sel_name, "policy", "value"))}
    pol_ms = pol["mean"]
    peak, peak_kind = measured_peaks()
    algo_bytes = n_tok * ALGO_BYTES_PER_TOKEN
    achieved = algo_bytes / (pol_ms * 1e-3) / 1e9
    traffic = n_tok * NCU_TRAFFIC_BYTES_PER_TOKEN if (st.V == synth.V_QWEN and NCU_TRAFFIC_BYTES_PER_TOKEN) else None

    # ---- the same step captured once into a CUDA graph and replayed: what the launch gaps between
    #      the step's fourteen stream operations cost (reported beside the headline, not as it) ------
    graph = None
    if args.graph_steps > 0:
        try:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                st.run()
            for _ in range(3):
                g.replay()
            barrier()
            gm = [torch.cuda.Event(enable_timing=True)]
            gm[0].record()
            for _ in range(args.graph_steps):
                g.replay()
                gm.append(torch.cuda.Event(enable_timing=True))
                gm[-1].record()
            barrier()
            gs = time_stats([a.elapsed_time(b) for a, b in zip(gm[:-1], gm[1:])])
            assert int(st.counts[0].item()) == n_tok and int(st.stats[3].item()) == 0
            graph = {"ms_per_step": gs, "value_at_mean": world * n_tok / (gs["mean"] * 1e-3),
                     "steps": args.graph_steps}
            del g
        except Exception as e:      # capture is an extra: the headline above does not depend on it
            graph = {"error": repr(e)[:200]}
            torch.cuda.synchronize()

    # ---- end to end: host buffers in, losses out, copies inside the timed region ---------------
    e2e = None
    if not args.no_e2e:
        pin = lambda x: x.cpu().pin_memory()
        h_logits = pin(st.logits)
        small = [st.rewards, st.values, st.old_values, st.seg_b, st.seg_e, st.trunc, st.seq_begin,
                 st.prompt, st.prev, st.new, st.pmask, st.vmask, st.targets, st.old_logp]
        h_small = [pin(x) for x in small]
        h_out = torch.empty(2, dtype=torch.float32).pin_memory()
        h_cnt = torch.empty(4, dtype=torch.int32).pin_memory()
        h2d = h_logits.numel() * 2 + sum(x.numel() * x.element_size() for x in h_small)
        d2h = 2 * 4 + 4 * 4

        def e2e_step():
            st.logits.copy_(h_logits, non_blocking=True)
            for d, h in zip(small, h_small):
                d.copy_(h, non_blocking=True)
            st.run()
            h_out[0:1].copy_(st.loss, non_blocking=True)
            h_out[1:2].copy_(st.vloss, non_blocking=True)
            h_cnt.copy_(st.counts, non_blocking=True)
            torch.cuda.synchronize()

        e2e_step()
        barrier()
        w0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            e2e_step()
        barrier()
        e2e_s = (time.perf_counter() - w0) / args.e2e_steps
        if world > 1:
            import torch.distributed as dist
            tt = torch.tensor([e2e_s], device=dev)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            e2e_s = float(tt.item())
        e2e = {"value": world * n_tok / e2e_s, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "ms_per_step": e2e_s * 1e3, "steps": args.e2e_steps}
        del h_logits

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        c = dict(st.c)
        c["logits_sample"] = synth.bf16_bits(st.logits[:args.cpu_rows])
        t, cores, parts = cpu_oracle_step_seconds(c, n_tok, args.cpu_rows)
        cpu = {"value": n_tok / t, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": (f"EGAE+selection+value loss on the full batch, policy loss fwd+bwd on "
                          f"{args.cpu_rows} of {n_tok} rows scaled to the micro-batch"),
               "seconds": {k: round(v, 4) for k, v in parts.items()}}

    small_kernels = None
    lmhead = None
    if rank == 0 and not (args.no_small and args.no_lmhead):
        del st.logits, st.dlogits, st.c["logits"]
        torch.cuda.empty_cache()
    if rank == 0 and not args.no_small:
        # the four small calls, against their own algorithmic bytes, on the bandwidth-sized config 4
        small_kernels = measure_cfg4(dev, args.cfg4_steps, 3)
        small_kernels.pop("clocks", None)
        torch.cuda.empty_cache()
    if rank == 0 and not args.no_lmhead:
        lm = LmHeadStep(dev, M=args.lm_rows)
        ms = time_lmhead(lm, args.lmhead_calls, 3)
        lmhead = {"workload": "cfg5: hidden [%d,%d] x LM-head weight [%d,%d] bf16, loss + dhidden + "
                              "dweight, logits never stored" % (lm.M, lm.K, lm.K, lm.V),
                  "value": lm.M / (ms * 1e-3), "unit": UNIT, "ms_per_call": ms,
                  "calls": args.lmhead_calls, "roofline": lm.roofline(ms)}
        del lm
    if world > 1:
        import torch.distributed as dist
        dist.barrier()

    if rank == 0:
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "peak_kind": peak_kind,
                    "frac_of_nominal_8TBs": achieved / 8000.0,
                    "traffic": traffic,
                    "traffic_note": "ncu dram__bytes_read.sum + dram__bytes_write.sum of a 2048-row capture "
                                    "of the same kernel, scaled by rows",
                    # the same launch time against the bytes ncu saw cross the DRAM interface (less than the
                    # algorithmic bytes: the last gradient rows are still in L2 when the kernel ends)
                    "achieved_measured_traffic": None if traffic is None else traffic / (pol_ms * 1e-3) / 1e9,
                    "frac_measured_traffic": None if traffic is None else traffic / (pol_ms * 1e-3) / 1e9 / peak,
                    "kernel": "policy_cluster_kernel (+ policy_prepare / policy_finish)",
                    "kernel_ms": pol_ms, "kernel_ms_median": pol["median"], "kernel_ms_min": pol["min"],
                    "algorithmic_bytes_per_launch": algo_bytes,
                    "small_kernels": None if small_kernels is None else small_kernels["kernels"],
                    "lmhead_variant": None if lmhead is None else lmhead["roofline"]}
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": ms_step, "ms_per_step_median": step_ms["median"],
            "ms_per_step_min": step_ms["min"],
            "value_at_median_step": world * n_tok / (step_ms["median"] * 1e-3),
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16 in, f32 accumulate", "data": "synthetic",
            "config": workload_config(st.N, st.n, n_val, args.hint),
            "step_calls_us": calls_us, "cuda_graph_replay": graph,
            "roofline": roofline,
            "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": (Step.KERNELS_PER_STEP - (st.n < 2048)) * args.steps,
            "clocks": clocks, "small_kernels": small_kernels, "lmhead_variant": lmhead}))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


class LmHeadShardStep:
    """One rank of the vocabulary-parallel LM-head (the weight split by columns over the ranks, rows and
    per-token scalars replicated): its two shard calls with the exchange between them and the dhidden
    all-reduce after them, all through `shard.vocab_parallel_step` (NCCL collectives; no rank reads
    another rank's memory)."""

    def __init__(self, dev, rank, world, M=16384, K=5120, V=synth.V_QWEN):
        from paper_2506_15050_b200 import binding as b
        from paper_2506_15050_b200 import shard
        self.b, self.shard, self.dev, self.M, self.K, self.V = b, shard, dev, M, K, V
        c = synth.config5(dev, M=M, K=K, V=V)                 # same seed on every rank: replicated inputs
        self.c = c
        self.lo, self.hi = shard.vocab_shard_bounds(V, world)[rank]
        self.weight = c["weight"][:, self.lo:self.hi].contiguous()
        del c["weight"]
        torch.cuda.empty_cache()
        t = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).to(dev)
        self.hidden = c["hidden"]
        self.targets, self.adv = t(c["targets"], torch.int32), t(c["adv"], torch.float32)
        self.old_logp = torch.full((M,), -12.0, device=dev)
        self.m_, self.s_, self.xy_ = (torch.empty(M, device=dev) for _ in range(3))
        self.logp, self.tok_loss = torch.zeros(M, device=dev), torch.zeros(M, device=dev)
        self.loss = torch.zeros(1, device=dev)
        self.stats = torch.zeros(4, dtype=torch.int32, device=dev)
        self.sstats = torch.zeros(4, dtype=torch.int32, device=dev)
        self.dhidden = torch.empty_like(self.hidden)
        self.dweight = torch.empty_like(self.weight)
        self.ws = b.workspace(b.OP_LMHEAD, M, K, 0, self.hi - self.lo, dev)
        # old-policy log-probs: the merged statistics of a first pass give the current ones; add the noise
        self.run(grads=False)
        torch.cuda.synchronize()
        self.old_logp.copy_(self.logp + t(c["old_logp_noise"], torch.float32))

    def run(self, grads=True):
        b, c = self.b, self.c

        def stats_fn():
            b.tppo_lmhead_shard_stats(self.hidden, self.weight, self.lo, self.V, self.targets, self.m_,
                                      self.s_, self.xy_, self.sstats, self.ws)
            return self.m_, self.s_, self.xy_

        def grads_fn(m, s_, xy):
            b.tppo_lmhead_shard_fwd_bwd(self.hidden, self.weight, self.lo, self.V, self.targets, None,
                                        self.old_logp, self.adv, c["eps_low"], c["eps_high"], 0.0, m, s_, xy,
                                        self.logp, self.tok_loss, self.loss, self.stats,
                                        self.dhidden if grads else None, self.dweight if grads else None,
                                        self.ws)
            return self.dhidden if grads else None

        self.shard.vocab_parallel_step(stats_fn, b.tppo_lmhead_shard_rescale, grads_fn)


def run_lmhead_vocab_parallel(args, rank, world, local, dev, warmup):
    """`--workload lmhead --gpus N`: config 5 with the vocabulary split over N ranks.  One step = the
    whole exchange (statistics GEMM, two small all-reduces, gradient GEMMs, dhidden all-reduce), timed on
    the device with the collectives inside; total work is fixed as N grows ("strong")."""
    import torch.distributed as dist
    lm = LmHeadShardStep(dev, rank, world, M=args.lm_rows)
    steps = args.steps if args.steps != 200 else 20
    for _ in range(warmup):
        lm.run()
    dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        lm.run()
    t1.record()
    dist.barrier()
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    tt = torch.tensor([t0.elapsed_time(t1) / steps], device=dev)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    ms = float(tt.item())
    bits = torch.tensor([int(lm.stats[3].item()) | int(lm.sstats[3].item())], device=dev)
    dist.all_reduce(bits, op=dist.ReduceOp.MAX)
    assert int(bits.item()) == 0
    burst, sustained, kind = measured_tensor_peaks()
    flops = 2.0 * lm.M * lm.K * lm.V
    achieved = 3.0 * flops / (ms * 1e-3) / 1e12 / world           # per GPU
    if rank == 0:
        print(json.dumps({
            "metric": "selected tokens/s, LM-head variant, vocabulary split over the ranks; % tensor peak",
            "value": lm.M / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
            "dtype": "bf16 in, f32 accumulate", "data": "synthetic",
            "config": {"workload": "cfg5 vocabulary-parallel: hidden [%d,%d] replicated, LM-head weight "
                                   "[%d,%d] bf16 in %d column shards" % (lm.M, lm.K, lm.K, lm.V, world),
                       "exchange_bytes_per_rank": {"row_statistics": 12 * lm.M, "dhidden_allreduce": 2 * lm.M * lm.K}},
            "roofline": {"bound": "tensor", "achieved": achieved, "peak": sustained, "unit": "TFLOP/s per GPU",
                         "frac": achieved / sustained, "peak_kind": kind + ", sustained", "traffic": None,
                         "kernel": "umma_gemm_kernel, one column shard per rank, collectives inside the step"},
            "cpu_baseline": None, "e2e": None, "clocks": clocks,
            "gpu_launches": (6 + 3 * (((lm.hi - lm.lo + 255) // 256 + 61) // 62)) * steps}))
    dist.destroy_process_group()


def run_lmhead_workload(args, rank, world, local, dev, warmup):
    """The LM-head variant as the bench line: one step = one call (loss, dhidden, dweight).  With
    several ranks the vocabulary is split over them (see run_lmhead_vocab_parallel)."""
    if world > 1:
        run_lmhead_vocab_parallel(args, rank, world, local, dev, warmup)
        return
    lm = LmHeadStep(dev, M=args.lm_rows)
    steps = args.steps if args.steps != 200 else 20

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        lm.run()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        lm.run()
    t1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms = t0.elapsed_time(t1) / steps
    if world > 1:
        import torch.distributed as dist
        tt = torch.tensor([ms], device=dev)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        ms = float(tt.item())
    assert int(lm.stats[3].item()) == 0
    e2e = None
    if not args.no_e2e:
        h_h, h_w = lm.hidden.cpu().pin_memory(), lm.weight.cpu().pin_memory()
        h_loss = torch.empty(1, dtype=torch.float32).pin_memory()

        def e2e_step():
            lm.hidden.copy_(h_h, non_blocking=True)
            lm.weight.copy_(h_w, non_blocking=True)
            lm.run()
            h_loss.copy_(lm.loss, non_blocking=True)
            torch.cuda.synchronize()

        e2e_step()
        barrier()
        w0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            e2e_step()
        barrier()
        e2e_s = (time.perf_counter() - w0) / args.e2e_steps
        e2e = {"value": world * lm.M / e2e_s, "unit": UNIT,
               "h2d_bytes_per_step": int((h_h.numel() + h_w.numel()) * 2), "d2h_bytes_per_step": 4,
               "ms_per_step": e2e_s * 1e3, "steps": args.e2e_steps}
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        t, cores = cpu_oracle_lmhead_seconds(lm, 8)
        cpu = {"value": lm.M / t, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": "8 of %d rows (float64 logits, Eq. 1, dhidden rows, dweight share), scaled by rows" % lm.M}
    n_chunk_launches = 3 * ((lm.V + 255) // 256 + 61) // 62
    shard_info = None
    if args.lm_shards > 1 and world == 1:
        shard_info = time_lmhead_rank_of_shards(lm, args.lm_shards, max(3, steps // 4), warmup)
        shard_info["unsharded_ms"] = ms
    if rank == 0:
        print(json.dumps({
            "vocab_shards": shard_info,
            "metric": "selected tokens/s, LM-head variant: fused hidden x vocab contraction + PPO loss "
                      "fwd+bwd, V=152064 bf16; % tensor peak",
            "value": world * lm.M / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16 in, f32 accumulate", "data": "synthetic",
            "config": {"workload": "cfg5: hidden [%d,%d] x LM-head weight [%d,%d] bf16, loss + dhidden + "
                                   "dweight, logits never stored" % (lm.M, lm.K, lm.K, lm.V),
                       "l2": "inputs larger than L2 (%.2f GB of weights per sweep)" % (lm.K * lm.V * 2 / 1e9)},
            "roofline": lm.roofline(ms), "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": (LmHeadStep.KERNELS_FIXED + n_chunk_launches) * steps, "clocks": clocks}))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()




# dram__bytes_read.sum + dram__bytes_write.sum of one launch of each call's kernels on this very
# workload (ncu capture of `python bench.py --workload cfg4 --steps 1 --warmup 3`, summarised under
# profiles/): the scan kernel, the selection kernel, the value kernel plus the kernel that zero-fills
# dvalues, the slot walk plus the copy kernel.  None once a kernel has changed since.
NCU_CFG4_TRAFFIC = {"egae": 140728064 + 94136576, "select": 35152896 + 814336,
                    "value": 145394688 + 21827072 + 7424 + 7879168, "advance": 43362048 + 1535232 + 80896}


def measure_cfg4(dev, steps, warmup):
    """Config 4, the bandwidth test of the small kernels: EGAE, token selection, value loss and the
    batch advance over 4096 ragged segments (17.5 M tokens).  One step = the four calls back to back;
    every call is also timed on its own (CUDA events around the C-ABI call, memsets included) against
    its algorithmic bytes.  Also times the scan on dense (process) rewards with gamma < 1."""
    from paper_2506_15050_b200 import binding as b
    c = synth.config4()
    N, B = c["N"], c["B"]
    t = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).to(dev)
    rng = np.random.default_rng(8)
    rewards, values = t(c["rewards"], torch.float32), t(c["values"], torch.float32)
    gen = torch.Generator(dev).manual_seed(3)
    old_values = values + 0.2 * torch.randn(N, device=dev, generator=gen)
    dense_rewards = torch.randn(N, device=dev, generator=gen)
    sb, se, tr = t(c["seg_begin"], torch.int32), t(c["seg_end"], torch.int32), t(c["truncated"], torch.uint8)
    boot = t(c["bootstrap"], torch.float32)
    seqb = t(c["seq_begin"], torch.int32)
    pl, pv, nl = (t(c[k], torch.int32) for k in ("prompt_len", "prev_len", "new_len"))
    pm, vm = t(c["extra_policy_mask"], torch.uint8), t(c["extra_value_mask"], torch.uint8)
    tokens = t(rng.integers(0, synth.V_QWEN, N).astype(np.int32), torch.int32)
    n_fin = int((c["truncated"] == 0).sum())
    qlens = rng.integers(16, 2048, n_fin)
    qb = t(np.concatenate([[0], np.cumsum(qlens)]).astype(np.int32), torch.int32)
    qt = t(rng.integers(0, synth.V_QWEN, int(qlens.sum())).astype(np.int32), torch.int32)
    adv, ret = torch.empty(N, device=dev), torch.empty(N, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    pol = torch.empty(N, dtype=torch.int32, device=dev)
    val = torch.empty(N, dtype=torch.int32, device=dev)
    counts = torch.zeros(4, dtype=torch.int32, device=dev)
    loss, dv = torch.zeros(1, device=dev), torch.empty(N, device=dev)
    vst = torch.zeros(2, dtype=torch.int32, device=dev)
    npl, npv = torch.empty(B, dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.int32, device=dev)
    nsb = torch.empty(B + 1, dtype=torch.int32, device=dev)
    ntk = torch.empty(N + qt.numel(), dtype=torch.int32, device=dev)
    fs, src = torch.empty(B, dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.int32, device=dev)
    acn = torch.zeros(4, dtype=torch.int32, device=dev)
    ws1 = b.workspace(b.OP_EGAE, N, B, 0, 0, dev)
    ws2 = b.workspace(b.OP_SELECT_TOKENS, N, B, 0, 0, dev)
    ws3 = b.workspace(b.OP_VALUE_LOSS, N, 0, N, 0, dev)
    calls = {
        "egae": lambda: b.tppo_egae(rewards, values, sb, se, tr, boot, 1.0, 0.95, adv, ret, status, ws1),
        "select": lambda: b.tppo_select_tokens(seqb, pl, pv, nl, tr, 0, pm, vm, N, pol, val, counts, ws2),
        "value": lambda: b.tppo_value_loss(values, old_values, ret, val, counts[1:2], N, 0.5, 0.6, 0.0,
                                           loss, dv, vst, ws3),
        "advance": lambda: b.tppo_advance_batch(seqb, pl, pv, nl, tr, tokens, qb, qt, npl, npv, nsb, ntk,
                                                fs, src, acn),
    }

    def timed(f, events):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); f(); e1.record()
        events.append((e0, e1))

    def step(events=None):
        for name, f in calls.items():
            if events is None:
                f()
            else:
                timed(f, events[name])

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    events = {k: [] for k in calls}
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        step(events)
    t1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = t0.elapsed_time(t1) / steps
    cn, an = counts.cpu().numpy(), acn.cpu().numpy()
    assert int(status) == 0 and cn[2] == 0 and an[3] == 0 and int(vst[1]) == 0
    # the scan on dense rewards with discounting (process rewards; the paper trains on gamma = 1)
    dense = {}
    for gamma in (0.99, 0.999):
        ev = []
        for i in range(3 + max(steps // 3, 5)):
            timed(lambda: b.tppo_egae(dense_rewards, values, sb, se, tr, boot, gamma, 0.95, adv, ret, status, ws1), ev)
        torch.cuda.synchronize()
        assert int(status) == 0
        dense["gamma_%g" % gamma] = time_stats([a.elapsed_time(b_) * 1e3 for a, b_ in ev[3:]])
    peak, kind = measured_peaks()
    algo = {"egae": 16 * N, "select": 2 * N + 4 * (int(cn[0]) + int(cn[1])),
            "value": 20 * int(cn[1]) + 4 * N, "advance": 8 * int(an[2])}
    per_unit = {"egae": "16 B/token (rewards, values in; advantages, returns out)",
                "select": "1 B/token per byte mask read (two masks) + 4 B per selected index written",
                "value": "20 B/value token (index, value, old value, return, gradient) + 4 B/token of dvalues written",
                "advance": "8 B/context token (read + write)"}
    kernels = {}
    for k, ev in events.items():
        st = time_stats([a.elapsed_time(b_) * 1e3 for a, b_ in ev])
        gbs = algo[k] / st["mean"] / 1e3
        kernels[k] = {"bound": "hbm", "us": st["mean"], "us_median": st["median"], "us_min": st["min"],
                      "algorithmic_bytes": algo[k], "per_unit": per_unit[k], "achieved": gbs,
                      "unit": "GB/s", "peak": peak, "peak_kind": kind, "frac": gbs / peak,
                      "frac_at_median": algo[k] / st["median"] / 1e3 / peak,
                      "traffic": NCU_CFG4_TRAFFIC[k] if N == 17506416 else None}
    kernels["egae"]["dense_rewards_us"] = dense
    return {"workload": "cfg4: %d ragged segments, %d tokens, lengths log-uniform in [16, 32768], half "
                        "truncated with a bootstrap value, Bernoulli(0.5) byte masks" % (B, N),
            "steps": steps, "ms_per_step": ms, "tokens_per_s": N / (ms * 1e-3),
            "selected": {"policy": int(cn[0]), "value": int(cn[1])},
            "advance": {"freed": int(an[0]), "context_tokens": int(an[2])},
            "timing": "CUDA events around each C-ABI call (its memset and kernels)",
            "kernels": kernels, "clocks": clocks}


def _time_call(f, reps, warm=3):
    """Mean / median / min device time of one call (ms), CUDA events around every repetition."""
    for _ in range(warm):
        f()
    torch.cuda.synchronize()
    ev = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); f(); e1.record()
        ev.append((e0, e1))
    torch.cuda.synchronize()
    return time_stats([a.elapsed_time(b_) for a, b_ in ev])


def run_config_table(args, dev):
    """The benchmark configurations that are not the bench line, one after another (configs 1, 2 and
    4; config 3 is the default workload, config 5 `--workload lmhead`): GPU time of the hot path on
    each, and the oracle on the host cores on the whole of the small ones and a bounded sample of
    the large one.  Prints one JSON object; one entry per config."""
    import oracle
    from paper_2506_15050_b200 import binding as b
    f32 = lambda x: float(np.float32(x))
    t = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).to(dev)
    out = {"cores": oracle.num_threads()}

    def path(c, logits, rows_sel, mode):
        """Device buffers and one closure that runs EGAE, selection, policy loss, value loss."""
        N, B, V = c["N"], c["B"], c["V"]
        r, v, ov = t(c["rewards"], torch.float32), t(c["values"], torch.float32), t(c["old_values"], torch.float32)
        sb, se, tr = t(c["seg_begin"], torch.int32), t(c["seg_end"], torch.int32), t(c["truncated"], torch.uint8)
        sq = t(c["seq_begin"], torch.int32)
        pl, pv, nl = (t(c[k], torch.int32) for k in ("prompt_len", "prev_len", "new_len"))
        tg = t(c["targets"], torch.int32)
        adv, ret = torch.zeros(N, device=dev), torch.zeros(N, device=dev)
        pol, val = torch.zeros(N, dtype=torch.int32, device=dev), torch.zeros(N, dtype=torch.int32, device=dev)
        cnt, st = torch.zeros(4, dtype=torch.int32, device=dev), torch.zeros(1, dtype=torch.int32, device=dev)
        logp, loss, vloss = torch.zeros(N, device=dev), torch.zeros(1, device=dev), torch.zeros(1, device=dev)
        stats, vstats = torch.zeros(4, dtype=torch.int32, device=dev), torch.zeros(2, dtype=torch.int32, device=dev)
        old = torch.zeros(N, device=dev)
        dl = torch.empty_like(logits) if mode == b.DLOGITS_FULL else torch.empty((rows_sel, V), dtype=logits.dtype, device=dev)
        dv = torch.zeros(N, device=dev)
        w1, w2 = b.workspace(b.OP_EGAE, N, B, 0, 0, dev), b.workspace(b.OP_SELECT_TOKENS, N, B, 0, 0, dev)
        w3, w4 = b.workspace(b.OP_POLICY_LOSS, N, 0, N, V, dev), b.workspace(b.OP_VALUE_LOSS, N, 0, N, 0, dev)

        def small():
            b.tppo_egae(r, v, sb, se, tr, None, c["gamma"], c["lam"], adv, ret, st, w1)
            b.tppo_select_tokens(sq, pl, pv, nl, tr, 0, None, None, N, pol, val, cnt, w2)

        def policy():
            b.tppo_policy_loss_fwd_bwd(logits, tg, pol[:rows_sel], cnt[0:1], rows_sel, None, old, adv,
                                       c["eps_low"], c["eps_high"], 0.0, logp, None, loss, stats, dl, mode, w3)

        def value():
            b.tppo_value_loss(v, ov, ret, val, cnt[1:2], N, c["xi_low"], c["xi_high"], 0.0, vloss, dv, vstats, w4)

        small()
        b.tppo_policy_loss_fwd_bwd(logits, tg, pol, cnt[0:1], N, None, old, adv, 0.2, 0.2, 0.0, logp, None, loss,
                                   stats, None, b.DLOGITS_NONE, w3)       # old-policy log-probs
        torch.cuda.synchronize()
        idx = pol[:int(cnt[0])].long()
        old[idx] = logp[:len(idx)] + t(c["old_logp_noise"], torch.float32)[idx]
        return small, policy, value, cnt, stats

    # ---- config 1 -----------------------------------------------------------------------------------
    c1 = synth.config1()
    small, policy, value, cnt, stats = path(c1, t(c1["logits"], torch.float32), 170, b.DLOGITS_COMPACT)
    step = lambda: (small(), policy(), value())
    g = _time_call(step, 200)
    w0 = time.perf_counter()
    for _ in range(20):
        a_, r_ = oracle.egae(c1["rewards"], c1["values"], c1["seg_begin"], c1["seg_end"], c1["truncated"], None, 1.0, f32(0.95))
        p_, v_ = oracle.select_tokens(c1["seq_begin"], c1["prompt_len"], c1["prev_len"], c1["new_len"], c1["truncated"])
        oracle.policy_loss(c1["logits"], c1["targets"], p_, None, np.zeros(c1["N"], np.float32), a_.astype(np.float32), f32(0.2), f32(0.2))
        oracle.value_loss(c1["values"], c1["old_values"], r_.astype(np.float32), v_, f32(0.5), f32(0.6))
    o = (time.perf_counter() - w0) / 20
    out["cfg1"] = {"n_selected": int(cnt[0]), "gpu_step_us": {k: v * 1e3 for k, v in g.items()},
                   "oracle_step_ms": o * 1e3, "note": "whole path, V=1000 fp32; latency-bound (9 kernel launches, no memsets)"}
    # ---- config 2 -----------------------------------------------------------------------------------
    c2 = synth.config2(dev)
    res2 = {}
    for name, mode in (("compact", b.DLOGITS_COMPACT), ("full_zero_filled", b.DLOGITS_FULL)):
        small, policy, value, cnt, stats = path(c2, c2["logits"], 4096, mode)
        g = _time_call(policy, 30)
        n = int(cnt[0])
        algo = n * ALGO_BYTES_PER_TOKEN + (0 if mode == b.DLOGITS_COMPACT else (c2["N"] - n) * 2 * c2["V"])
        res2[name] = {"policy_call_ms": g, "algorithmic_bytes": algo, "GB/s": algo / (g["mean"] * 1e-3) / 1e9,
                      "selected_tokens_per_s": n / (g["mean"] * 1e-3)}
        assert n == 4096 and int(stats[3]) == 0
        del small, policy, value
        torch.cuda.empty_cache()
    rows = 256
    host = synth.bf16_bits(c2["logits"][:rows])
    w0 = time.perf_counter()
    oracle.policy_loss(host, c2["targets"], np.arange(rows, dtype=np.int32), None, np.zeros(c2["N"], np.float32),
                       np.ones(c2["N"], np.float32), f32(0.2), f32(0.2), 4096.0)
    o = time.perf_counter() - w0
    out["cfg2"] = {"n_selected": 4096, "gpu": res2,
                   "oracle": {"sample_rows": rows, "seconds": o, "selected_tokens_per_s": rows / o,
                              "scaled_to_4096_rows_s": o * 4096 / rows}}
    del c2
    torch.cuda.empty_cache()
    # ---- config 4 -----------------------------------------------------------------------------------
    m = measure_cfg4(dev, 30, 3)
    c4 = synth.config4()
    w0 = time.perf_counter()
    oracle.egae(c4["rewards"], c4["values"], c4["seg_begin"], c4["seg_end"], c4["truncated"], c4["bootstrap"], 1.0, f32(0.95))
    w1 = time.perf_counter()
    oracle.select_tokens(c4["seq_begin"], c4["prompt_len"], c4["prev_len"], c4["new_len"], c4["truncated"], 0,
                         c4["extra_policy_mask"], c4["extra_value_mask"])
    w2 = time.perf_counter()
    out["cfg4"] = {"tokens": c4["N"], "gpu_us": {k: v["us"] for k, v in m["kernels"].items()},
                   "gpu_frac_of_measured_hbm": {k: v["frac"] for k, v in m["kernels"].items()},
                   "oracle_egae_s": w1 - w0, "oracle_select_s": w2 - w1,
                   "oracle_egae_tokens_per_s": c4["N"] / (w1 - w0), "oracle_select_tokens_per_s": c4["N"] / (w2 - w1)}
    print(json.dumps(out))


def run_cfg4_workload(args, rank, world, local, dev, warmup):
    """Config 4 as the bench line (the scan is the roofline kernel of this workload)."""
    steps = args.steps if args.steps != 200 else 50
    m = measure_cfg4(dev, steps, warmup)
    k = m["kernels"]
    if rank == 0:
        print(json.dumps({
            "metric": "tokens/s, EGAE + token compaction + value loss + batch advance, config 4",
            "value": m["tokens_per_s"], "unit": "tokens/s", "n_gpus": 1, "steps": steps, "warmup": warmup,
            "ms_per_step": m["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32 (f64 scan carries), int32 indices", "data": "synthetic",
            "config": {"workload": m["workload"], "l2": "inputs larger than L2 (70 MB per array)",
                       "selected": m["selected"], "advance": m["advance"]},
            "roofline": {"bound": "hbm", "achieved": k["egae"]["achieved"], "peak": k["egae"]["peak"],
                         "unit": "GB/s", "frac": k["egae"]["frac"], "peak_kind": k["egae"]["peak_kind"],
                         "traffic": k["egae"]["traffic"], "kernel": "egae_scan_kernel",
                         "kernel_ms": k["egae"]["us"] / 1e3,
                         "algorithmic_bytes_per_launch": k["egae"]["algorithmic_bytes"]},
            "kernels": k, "gpu_launches": 8 * steps, "clocks": m["clocks"]}))


if __name__ == "__main__":
    main()
