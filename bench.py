#!/usr/bin/env python
"""Benchmark of the DSpark hot path on B200: one step = schedule -> ragged offsets ->
fused verification of one synthetic batch, through the C ABI.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3] [--impl ours|reference]

Prints ONE JSON line.  `value` is verified target rows per second over all GPUs with the
inputs resident in HBM; `e2e` is the same metric with the step's inputs copied from pinned
host memory and its results copied back inside the timed region; `roofline` is the dominant
kernel against the measured HBM peak; `cpu_baseline` times the CPU oracle on the same batch.
Multi-GPU runs are independent replicas (requests are independent and the scheduler is per
engine), one process per GPU under torchrun; time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

METRIC = "verified rows/sec and achieved HBM GB/s (% of B200 peak) at V=129280, 1 GPU"
UNIT = "rows/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126 * 1024 * 1024

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# captures summarised under profiles/: cfg2 and cfg3 were captured as they are; cfg4 and cfg5 are too large
# for a multi-pass capture, so their figure is the algorithmic bytes times the traffic / algorithmic ratio of
# the smaller capture of the same kernel (traffic is proportional to the rows streamed).
NCU_TRAFFIC_BYTES = {"cfg3": 198612480 + 3035136, "cfg2": 152069376 + 3132160}
NCU_TRAFFIC_RATIO = {"cfg4": 1.0135, "cfg5": 1.0165}


# ----------------------------------------------------------------------------- workloads ----
REQUESTS_OVERRIDE = 0
ASYNC_TOPK = False
CUDA_GRAPH = False
OVERLAP = False
PER_REQUEST_T = False
TRUNCATE = None          # (top_k, top_p) for every request: dspark_verify_truncated


def make_workload(name: str, device, rank: int, n_sets=None, oracle_schedule=False):
    """Returns a dict describing the step: schedule input (or None) and a list of batches that
    differ only in their logits (rotated so consecutive steps never touch the same bytes).
    n_sets None: as many batches as it takes to exceed four times the L2 capacity."""
    from paper_2607_05147_b200 import workloads as W
    sched = None
    greedy = False
    if name == "cfg3":
        sched = W.config_3_schedule(device)
        desc = "Confidence-scheduled, high concurrency: 256 requests, V=129280, blocks of 16, budget 1024, bf16 sampling"
    elif name == "cfg5":
        sched = W.config_5_schedule(device)
        desc = "Long-block stress: 512 requests, V=129280, blocks of 32, budget 4096, bf16 sampling T=0.7"
    elif name == "cfg2":
        desc = "Sampling, moderate batch: 64 requests, V=129280, ragged k~U{1..8}, bf16, T=1"
    elif name == "cfg2_fp32":
        desc = "cfg2 with fp32 logits (fp32 sampling path): 64 requests, V=129280, ragged k~U{1..8}, T=1"
    elif name == "cfg4":
        greedy = True
        desc = "Large batch greedy: 1024 requests, V=129280, ragged k~U{0..8}, fp32"
    elif name == "cfg4_bf16":
        greedy = True
        desc = "cfg4 with bf16 logits (bf16 greedy path): 1024 requests, V=129280, ragged k~U{0..8}"
    else:
        raise SystemExit(f"unknown workload {name}")

    lengths = None
    prof = None
    steady_K = 0
    if sched is not None:
        # the schedule is fixed by the confidences: run it once to size the logits
        if oracle_schedule:
            import oracle
            tab = oracle.sps_table(sched.bp_tokens, sched.bp_sps, sched.max_tokens)
            lengths = torch.from_numpy(oracle.schedule(sched.conf.cpu().numpy(), tab, sched.budget_tokens,
                                                       oracle.MODE_EARLY_STOP).lengths)
        else:
            from paper_2607_05147_b200 import binding as B
            prof = B.Profile(sched.bp_tokens, sched.bp_sps, sched.max_tokens)
            R, gamma = sched.conf.shape
            out_len = torch.zeros(R, dtype=torch.int32, device=device)
            ws = B.workspace(B.dspark_schedule_workspace_bytes(R, gamma))
            # asynchronous scheduling with constant confidences settles on the global optimum as its capacity
            mode = B.DSPARK_SCHED_GLOBAL if ASYNC_TOPK else B.DSPARK_SCHED_EARLY_STOP
            info = torch.zeros(32, dtype=torch.uint8, device=device)
            B.dspark_schedule(prof, sched.conf, sched.budget_tokens, mode, out_len=out_len, out_info=info,
                              workspace=ws)
            torch.cuda.synchronize()
            lengths = out_len.cpu()
            steady_K = B.read_sched_info(info).n_admitted

    def one(k):
        from paper_2607_05147_b200.replicas import rank_seed
        seed = rank_seed(5000, rank, k)
        if name == "cfg3":
            return W.sampling_batch(lengths, W.V_FULL, seed, device, temperature=1.0, draft_noise=1.0, verify_seed=2)
        if name == "cfg5":
            return W.sampling_batch(lengths, W.V_FULL, seed, device, temperature=0.7, draft_noise=2.0, verify_seed=4)
        if name in ("cfg2", "cfg2_fp32"):
            g = torch.Generator(device="cpu"); g.manual_seed(1)
            ln = torch.randint(1, 9, (REQUESTS_OVERRIDE or 64,), generator=g)
            return W.sampling_batch(ln, W.V_FULL, seed, device, temperature=1.0, draft_noise=1.0, verify_seed=1,
                                    dtype=torch.float32 if name == "cfg2_fp32" else torch.bfloat16)
        g = torch.Generator(device="cpu"); g.manual_seed(3)
        ln = torch.randint(0, 9, (REQUESTS_OVERRIDE or 1024,), generator=g)
        return W.greedy_batch(ln, W.V_FULL, seed, device, sigma=4.0, tie_frac=0.01,
                              match_prob=[0.85 ** (j + 1) for j in range(8)],
                              dtype=torch.bfloat16 if name == "cfg4_bf16" else torch.float32)

    batches = [one(0)]
    if n_sets is None:
        stream_b = algorithmic_bytes(batches[0], greedy, 0)[0]
        n_sets = max(2, min(8, -(-4 * L2_BYTES // stream_b)))
    for k in range(1, n_sets):
        batches.append(one(k))
    return dict(name=name, desc=desc, sched=sched, prof=prof, batches=batches, greedy=greedy, steady_K=steady_K)


class Step:
    """Device buffers + the calls of one step (all through the C ABI binding)."""

    def __init__(self, wl, device):
        from paper_2607_05147_b200 import binding as B
        self.B = B
        self.wl = wl
        b0 = wl["batches"][0]
        self.R, self.n_rows, self.V = b0.R, b0.n_rows, b0.V
        self.acc = torch.zeros(self.R, dtype=torch.int32, device=device)
        self.out = torch.zeros(self.n_rows, dtype=torch.int32, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.ws = B.workspace(B.dspark_verify_workspace_bytes(self.R, self.n_rows, self.V))
        self.sched = wl["sched"]
        if self.sched is not None:
            R, gamma = self.sched.conf.shape
            self.out_len = torch.zeros(R, dtype=torch.int32, device=device)
            self.offsets = torch.zeros(R + 1, dtype=torch.int32, device=device)
            self.sws = B.workspace(B.dspark_schedule_workspace_bytes(R, gamma))
            if ASYNC_TOPK:
                self.state = torch.zeros(4, dtype=torch.int32, device=device)
                B.dspark_async_state_init(self.state, wl["steady_K"])
        self.graphs = {}
        if OVERLAP and self.sched is not None:
            # two sets of scheduler outputs: step t+1 is scheduled while step t is still being verified
            self.side = torch.cuda.Stream(device=device)
            self.off2 = [self.offsets, torch.zeros_like(self.offsets)]
            self.len2 = [self.out_len, torch.zeros_like(self.out_len)]
            self.sched_done = [torch.cuda.Event(), torch.cuda.Event()]
            self.verify_done = [torch.cuda.Event(), torch.cuda.Event()]
            self.tick = 0
            self.primed = False
        # kernels of the library per step: scheduler (prep, rank + final stage; a selection kernel when the
        # candidates are many and the budget admits fewer than half)
        n_sched = 0
        if self.sched is not None:
            gamma = self.sched.conf.shape[1]
            gpad = 1 << max(0, (gamma - 1).bit_length()) if gamma <= 32 else (gamma + 31) // 32 * 32
            entries = self.R * gpad
            n_sched = 2 + (1 if entries >= 8192 and 2 * (self.sched.budget_tokens - self.R) <= entries else 0)
        # verifier: statistics pass, accept tests, residual pass, draws (greedy: argmax pass + accept tests); one more
        # for per-request temperatures on large batches; for a truncated target the window preparation, the histogram pass and the
        # threshold scan, both a second time for the rows of the second look, the restricted sums of the bonus rows
        # and the per-row fallback (fp32 rows: the per-row descent alone)
        if wl["greedy"]:
            n_verify = 2
        else:
            n_verify = 4
            if PER_REQUEST_T:
                # the kernel that expands the temperatures to rows runs only when the requests' scales do not fit in
                # the statistics pass's shared memory beside its request table (the library's rule, restated)
                R, nd = self.R, self.n_rows - self.R
                fits = R <= 2048 and ((R + 4) // 4) * 16 + ((nd + 7) // 8) * 16 + ((R + 3) // 4) * 16 <= 9 * 1024
                n_verify += 0 if (fits and TRUNCATE is None) else 1
            if TRUNCATE is not None:
                n_verify += 1 if b0.target.dtype == torch.float32 else 7
        self.launches_per_step = n_sched + n_verify

    def run(self, batch, conf=None):
        """One step; with --cuda-graph the step of every resident batch is captured once and replayed."""
        if CUDA_GRAPH and conf is None:
            g = self.graphs.get(id(batch))
            if g is None:
                self._launch(batch, None)                      # eager warm-up outside the capture
                torch.cuda.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    self._launch(batch, None)
                self.graphs[id(batch)] = g
            g.replay()
            return
        self._launch(batch, conf)

    def _schedule_on_side_stream(self, k):
        B = self.B
        with torch.cuda.stream(self.side):
            self.side.wait_event(self.verify_done[k])          # the verifier that last read this slot is done
            B.dspark_schedule_async(self.wl["prof"], self.sched.conf, self.sched.budget_tokens, self.state,
                                    out_len=self.len2[k], out_row_offsets=self.off2[k], workspace=self.sws)
            self.sched_done[k].record(self.side)

    def _launch_overlapped(self, batch):
        B = self.B
        main = torch.cuda.current_stream()
        if not self.primed:
            self.verify_done[0].record(main); self.verify_done[1].record(main)
            self._schedule_on_side_stream(0)
            self.primed = True
        k = self.tick & 1
        self._schedule_on_side_stream(k ^ 1)                    # next step's schedule runs beside this verify
        main.wait_event(self.sched_done[k])
        B.dspark_verify(batch.target, batch.draft, self.off2[k], batch.draft_tokens, batch.temperature, batch.seed,
                        draft_row_start=batch.draft_row_start, accepted_len=self.acc, out_tokens=self.out,
                        dev_status=self.status, workspace=self.ws, n_rows=self.n_rows)
        self.verify_done[k].record(main)
        self.tick += 1

    def _launch(self, batch, conf):
        B = self.B
        if OVERLAP and self.sched is not None and conf is None:
            return self._launch_overlapped(batch)
        offsets = batch.row_offsets
        if self.sched is not None:
            c = self.sched.conf if conf is None else conf
            if ASYNC_TOPK:
                B.dspark_schedule_async(self.wl["prof"], c, self.sched.budget_tokens, self.state,
                                        out_len=self.out_len, out_row_offsets=self.offsets, workspace=self.sws)
            else:
                B.dspark_schedule(self.wl["prof"], c, self.sched.budget_tokens, B.DSPARK_SCHED_EARLY_STOP,
                                  out_len=self.out_len, out_row_offsets=self.offsets, workspace=self.sws)
            offsets = self.offsets            # the verifier reads the schedule's offsets from device memory
        self._verify(batch, offsets)

    def verify(self, batch):
        """The verifier call alone, on the offsets the last schedule left on the device."""
        self._verify(batch, self.offsets if self.sched is not None else batch.row_offsets)

    def _verify(self, batch, offsets):
        B = self.B
        if self.wl["greedy"]:
            B.dspark_verify_greedy(batch.target, offsets, batch.draft_tokens, accepted_len=self.acc,
                                   out_tokens=self.out, dev_status=self.status, workspace=self.ws, n_rows=self.n_rows)
        elif TRUNCATE is not None:
            if not hasattr(self, "top_k"):
                self.top_k = torch.full((self.R,), int(TRUNCATE[0]), dtype=torch.int32, device=self.acc.device)
                self.top_p = torch.full((self.R,), float(TRUNCATE[1]), dtype=torch.float32, device=self.acc.device)
            B.dspark_verify_truncated(batch.target, batch.draft, offsets, batch.draft_tokens, batch.seed,
                                      temperature=batch.temperature, top_k=self.top_k, top_p=self.top_p,
                                      draft_row_start=batch.draft_row_start, accepted_len=self.acc, out_tokens=self.out,
                                      dev_status=self.status, workspace=self.ws, n_rows=self.n_rows)
        elif PER_REQUEST_T:
            if not hasattr(self, "temps"):
                self.temps = torch.full((self.R,), float(batch.temperature), device=self.acc.device)
            B.dspark_verify_per_request(batch.target, batch.draft, offsets, batch.draft_tokens, self.temps, batch.seed,
                                        draft_row_start=batch.draft_row_start, accepted_len=self.acc,
                                        out_tokens=self.out, dev_status=self.status, workspace=self.ws,
                                        n_rows=self.n_rows)
        else:
            B.dspark_verify(batch.target, batch.draft, offsets, batch.draft_tokens, batch.temperature, batch.seed,
                            draft_row_start=batch.draft_row_start, accepted_len=self.acc, out_tokens=self.out,
                            dev_status=self.status, workspace=self.ws, n_rows=self.n_rows)


def algorithmic_bytes(batch, greedy, n_rejected):
    """(bytes the dominant launch streams, bytes the whole call streams, the call's bytes by the formula that counts
    every row once plus a re-read of each rejected pair).  The sampling verifier streams the target and draft row of
    every draft position in its statistics pass and, in its second pass, the rejected pairs and the bonus rows of the
    requests that accepted everything: one row per rejected request fewer than the formula (with a truncated target
    all bonus rows go through the first pass and the two figures coincide)."""
    elem = batch.target.element_size()
    row = elem * batch.V
    n_draft = batch.n_rows - batch.R
    if greedy:
        return row * batch.n_rows, row * batch.n_rows, row * batch.n_rows
    formula = row * (batch.n_rows + n_draft + 2 * n_rejected)
    if TRUNCATE is not None or batch.R > 2048:
        return row * (batch.n_rows + n_draft), formula, formula
    return row * 2 * n_draft, row * (2 * n_draft + 2 * n_rejected + (batch.R - n_rejected)), formula


# -------------------------------------------------------------------------------- clocks ----
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the GPU is busy."""

    def __init__(self, index: int, period=0.02):
        super().__init__(daemon=True)
        self.period = period
        self.samples, self.reasons = [], set()
        self.stop_flag = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.max_mhz = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown",
        }
        while not self.stop_flag.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, nm in names.items():
                    if mask & bit:
                        self.reasons.add(nm)
            except Exception:
                pass
            time.sleep(self.period)

    def finish(self):
        self.stop_flag.set()
        if self.is_alive():
            self.join(timeout=2)
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


# -------------------------------------------------------------------------- reference arm ----
def oracle_step(wl, batch, n_requests, threads):
    """The CPU oracle over the first n_requests requests of the batch (schedule on all of them:
    it is cheap and not separable)."""
    import numpy as np
    import oracle
    from paper_2607_05147_b200 import workloads as W
    host = wl["host"]
    if wl["sched"] is not None:
        oracle.schedule(host["conf"], host["table"], wl["sched"].budget_tokens, oracle.MODE_EARLY_STOP)
    off = host["offsets"][: n_requests + 1]
    if wl["greedy"]:
        oracle.verify_greedy_mt(host["target"], off, host["tokens"], threads)
    else:
        oracle.verify(host["target"], host["draft"], off, host["tokens"], batch.temperature, batch.seed,
                      eval_all=False, n_threads=threads)
    return int(off[-1])


def host_copy(wl):
    import oracle
    from paper_2607_05147_b200 import workloads as W
    b = wl["batches"][0]
    host = dict(target=W.bf16_bits(b.target), draft=None if b.draft is None else W.bf16_bits(b.draft),
                offsets=b.row_offsets.cpu().numpy(), tokens=b.draft_tokens.cpu().numpy())
    if wl["sched"] is not None:
        host["conf"] = wl["sched"].conf.cpu().numpy()
        host["table"] = oracle.sps_table(wl["sched"].bp_tokens, wl["sched"].bp_sps, wl["sched"].max_tokens)
    wl["host"] = host


def workload_config(wl, b0, n_rows, n_rejected, n_sets, stream_bytes):
    """The `config` object of the JSON line: what the workload is, the same for both arms."""
    return {"workload": wl["desc"], "name": wl["name"], "requests": b0.R, "rows_per_step": n_rows,
            "draft_rows_per_step": b0.n_rows - b0.R, "rejected_requests": n_rejected,
            "logit_dtype": str(b0.target.dtype).replace("torch.", ""),
            "l2": f"inputs larger than L2: {n_sets} distinct batches rotated "
                  f"({n_sets * stream_bytes / 1e6:.0f} MB of logits)",
            "scheduler": ("async top-K, capacity from two steps earlier" if ASYNC_TOPK else "early stop")
            if wl["sched"] is not None else None,
            "temperature": "per request (device array)" if PER_REQUEST_T else "one per batch",
            "truncation": None if TRUNCATE is None else f"top_k={TRUNCATE[0]}, top_p={TRUNCATE[1]} (dspark_verify_truncated)",
            "launch": "CUDA graph replay" if CUDA_GRAPH else
            ("stream launches, scheduler of step t+1 overlapped on a second stream" if OVERLAP else "stream launches"),
            "parallelism": "replicas only (one engine per GPU, no collective)"}


def oracle_rejected(wl, batch):
    """Requests whose first rejection comes before the end of their block, by the oracle."""
    import oracle
    host = wl["host"]
    if wl["greedy"]:
        return 0
    o = oracle.verify(host["target"], host["draft"], host["offsets"], host["tokens"], batch.temperature, batch.seed,
                      eval_all=False, n_threads=os.cpu_count() or 1)
    lens = host["offsets"][1:] - host["offsets"][:-1] - 1
    return int((o.accepted_len < lens).sum())


def run_reference(args, rank):
    """--impl reference: the CPU oracle, as it stands, on the machine's host cores."""
    from paper_2607_05147_b200 import replicas
    if not replicas.is_reporting_rank(rank):
        return                      # under torchrun only rank 0 runs and prints the reference arm
    import oracle
    oracle.build()
    device = "cuda" if torch.cuda.is_available() else "cpu"     # only to draw the synthetic batches faster
    wl = make_workload(args.workload, device, 0, None, oracle_schedule=True)
    n_sets = len(wl["batches"])
    hosts = []
    for b in wl["batches"]:                                      # the same rotation of batches as the CUDA arm
        wl["batches"] = [b]
        host_copy(wl)
        hosts.append(wl["host"])
    b = b0 = wl["batches"][0]
    wl["host"] = hosts[0]
    threads = os.cpu_count() or 1
    n_rejected = oracle_rejected(wl, b0)
    t0 = time.perf_counter()
    oracle_step(wl, b, b.R, threads)
    t1 = time.perf_counter() - t0
    budget_s = 150.0
    frac = min(1.0, budget_s / max(1e-9, (args.steps + args.warmup) * t1))
    n_req = max(1, int(b.R * frac))
    for i in range(args.warmup):
        wl["host"] = hosts[i % n_sets]
        oracle_step(wl, b, n_req, threads)
    t0 = time.perf_counter()
    rows = 0
    for i in range(args.steps):
        wl["host"] = hosts[i % n_sets]
        rows += oracle_step(wl, b, n_req, threads)
    dt = time.perf_counter() - t0
    value = rows / dt
    stream_bytes = algorithmic_bytes(b0, wl["greedy"], 0)[0]
    sample = f"first {n_req} of {b.R} requests per step ({rows // max(1, args.steps)} rows), schedule over all requests"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(wl, b0, b0.n_rows, n_rejected, n_sets, stream_bytes),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------- main ----
def bench_markov(args, device, rank, world, dist, barrier):
    """One Markov-head draft position for R requests: logits = U + W1[x_prev] W2 on the tensor cores, the
    confidence head, one draw per request.  Reported beside the verification step, not instead of it."""
    from paper_2607_05147_b200 import binding as B, replicas, workloads as W
    R = args.requests or 256
    V = W.V_FULL
    B.dspark_markov_set_epilogue_path(args.markov_epilogue)
    n_sets = 3                                   # rotate base logits and outputs: 2 x 66 MB x 3 > L2
    m = W.markov_input(R, V, 4242 + rank, device)
    Us = [m.U] + [m.U.roll(i, 0).contiguous() for i in range(1, n_sets)]
    outs = [torch.empty_like(m.U) for _ in range(n_sets)]
    packed = torch.empty(B.dspark_markov_w2_packed_bytes(V), dtype=torch.uint8, device=device)
    B.dspark_markov_pack_w2(m.W2, packed)
    conf = torch.empty(R, dtype=torch.float32, device=device)
    toks = torch.empty(R, dtype=torch.int32, device=device)
    st = torch.zeros(1, dtype=torch.int32, device=device)
    ws = B.workspace(B.dspark_markov_workspace_bytes(R, V))

    # sequential drafting: the tokens drawn at one position are the previous tokens of the next one
    tok2 = [m.x_prev.clone(), toks]

    def step(i):
        B.dspark_markov_draft_step(Us[i % n_sets], m.W1, packed, tok2[i & 1], 1.0, 77 + i, H=m.H, w_conf=m.w_conf,
                                   out_logits=outs[i % n_sets], out_tokens=tok2[(i + 1) & 1], out_conf=conf, dev_status=st,
                                   workspace=ws)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    sampler = ClockSampler(device.index or 0)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for i in range(args.steps):
        step(i)
    ev1.record()
    barrier()
    ms = ev0.elapsed_time(ev1)
    t_end = time.perf_counter() + 1.0
    i = 0
    while time.perf_counter() < t_end:
        step(i); i += 1
        if i % 64 == 0:
            torch.cuda.synchronize()
    torch.cuda.synchronize()
    clocks = sampler.finish()
    timer = B.KernelTimer(args.steps * 8)
    timer.attach()
    for i in range(args.steps):
        step(i)
    torch.cuda.synchronize()
    timer.detach()
    kernels = timer.read()
    timer.close()

    # the contraction kernel alone, launched back to back (no events between launches: an event pair around
    # one launch adds several microseconds of launch latency that the stream normally hides)
    def logits_only(i):
        B.dspark_markov_logits(Us[i % n_sets], m.W1, packed, m.x_prev, out_logits=outs[i % n_sets], dev_status=st, workspace=ws)
    for i in range(args.warmup):
        logits_only(i)
    torch.cuda.synchronize()
    ev0.record()
    for i in range(args.steps):
        logits_only(i)
    ev1.record()
    torch.cuda.synchronize()
    gemm_call_ms = ev0.elapsed_time(ev1) / args.steps
    (ms,) = replicas.max_over_ranks([ms], dist, device)
    if rank != 0:
        return None
    peaks_file = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peaks = json.load(open(peaks_file)) if os.path.exists(peaks_file) else {}
    peak = float(peaks.get("hbm_gbs", FALLBACK_HBM_GBS))
    gemm_bytes = 2 * R * V * 2 + 256 * V * 2 + R * 512       # base logits in, draft logits out, W2 once, embeddings
    k = kernels.get("markov_gemm", {"ms": float("nan"), "launches": 1})
    gemm_ms = k["ms"] / args.steps              # one launch per group of 1024 rows
    achieved = gemm_bytes / (gemm_call_ms * 1e-3) / 1e9
    flops = 2.0 * ((R + 127) // 128 * 128) * 256 * ((V + 127) // 128 * 128)
    return {
        "metric": "markov_draft_rows_per_s", "value": replicas.whole_job_rate(R, args.steps, ms, world), "unit": "rows/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16 x bf16 -> f32", "data": "synthetic",
        "config": {"workload": f"Markov-head draft position, R={R}, V={V}, rank 256, T=1, confidence head d=1024",
                   "l2": f"{n_sets} base-logit / output buffer pairs rotated ({n_sets * 4 * R * V / 1e6:.0f} MB)"},
        "roofline": {"bound": "hbm", "kernel": "markov_gemm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak,
                     # dram__bytes_read + write of one launch from the ncu capture summarised under profiles/ (R = 256;
                     # part of the written tile is still in L2 when the kernel ends)
                     "traffic": 132_567_040 + 32_054_784 if R == 256 else None,
                     "algorithmic_bytes_per_launch": gemm_bytes,
                     "us_per_launch": gemm_call_ms * 1e3,
                     "timing": "logits-only calls back to back (statistics off), CUDA events around the whole loop",
                     "us_per_launch_inside_step_with_events": gemm_ms * 1e3,
                     "launches_per_step": k["launches"] // max(1, args.steps),
                     "tensor_tflops": flops / (gemm_call_ms * 1e-3) / 1e12,
                     "tensor_frac_of_measured_bf16": flops / (gemm_call_ms * 1e-3) / 1e12 / float(peaks.get("bf16_tflops", 1590.0))},
        "step_frac_of_peak": gemm_bytes / (ms / args.steps * 1e-3) / 1e9 / peak,
        "kernels_us_per_launch": {n: 1e3 * v["ms"] / v["launches"] for n, v in kernels.items()},
        "clocks": clocks, "dev_status": int(st.item())}


def launch_replicas(argv, n):
    """`bench.py --gpus N` started as one plain process: start N ranks of itself, one per GPU, the way the
    driver's launcher does (rank 0 prints the line)."""
    import socket
    import subprocess
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + argv
    raise SystemExit(subprocess.call(cmd))


def measure_workload(name, args, device, rank, local_rank, world, dist, barrier, with_e2e, with_cpu):
    """Times one workload: the step (schedule -> verify) as the median over repeats of the --steps loop, the
    verifier call alone, the kernels one by one, and (main workload only) the end-to-end and CPU legs."""
    from paper_2607_05147_b200 import binding as B, replicas
    steps, warmup = args.steps, args.warmup
    # enough distinct batches that consecutive steps cannot be served from the 126 MB L2
    wl = make_workload(name, device, rank)
    step = Step(wl, device)
    batches = wl["batches"]
    n_sets = len(batches)
    for i in range(warmup):
        step.run(batches[i % n_sets])
    torch.cuda.synchronize()
    dev_status = int(step.status.item())
    n_rows = batches[0].n_rows
    lens = batches[0].meta["lengths"].to(device)
    n_rejected = int((step.acc < lens).sum().item()) if not wl["greedy"] else 0
    if wl["sched"] is not None:
        assert torch.equal(step.offsets, batches[0].row_offsets), "scheduled offsets differ from the generated batch"

    sampler = ClockSampler(local_rank)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed_loop(fn, k):
        barrier()
        ev0.record()
        for i in range(k):
            fn(i)
        ev1.record()
        barrier()
        return ev0.elapsed_time(ev1)

    # EXACTLY `steps` steps between a barrier + synchronize on both sides, repeated: one repeat is a millisecond
    # or two for the small workloads, too short to attribute a few per cent; the line reports the median repeat
    first = timed_loop(lambda i: step.run(batches[i % n_sets]), steps)
    if args.quick:
        sampler.finish()
        return dict(wl=wl, step=step, ms=first, n_rows=n_rows, n_rejected=n_rejected, quick=True)
    repeats = max(args.repeats, int(50.0 / max(first, 1e-3)) + 1)
    repeats = min(repeats, 400)
    times = [first] + [timed_loop(lambda i: step.run(batches[i % n_sets]), steps) for _ in range(repeats - 1)]
    times = replicas.max_over_ranks(times, dist, device)                # every repeat: the slowest rank
    ts = sorted(times)
    ms, ms_min = ts[len(ts) // 2], ts[0]

    # the verifier call alone (the schedule's offsets stay where the last step left them), un-instrumented
    def verify_only(i):
        step.verify(batches[i % n_sets])
    vt = sorted(timed_loop(verify_only, steps) for _ in range(max(5, repeats // 5)))
    verify_ms = replicas.max_over_ranks([vt[len(vt) // 2]], dist, device)[0]

    # keep the same load running until the clock sampler has seen enough of it (not timed)
    t_end = time.perf_counter() + 1.0
    i = 0
    while time.perf_counter() < t_end and len(sampler.samples) < 40:
        step.run(batches[i % n_sets]); i += 1
        if i % 64 == 0:
            torch.cuda.synchronize()
    torch.cuda.synchronize()
    clocks = sampler.finish()

    # per-kernel timing of the same steps (events around every launch of the library)
    n_inst = max(steps, 200)                                 # averages per launch: a short --steps run still sees 200 launches
    timer = B.KernelTimer(n_inst * 12)
    timer.attach()
    for i in range(n_inst):
        step.run(batches[i % n_sets])
    torch.cuda.synchronize()
    timer.detach()
    kernels = timer.read()
    timer.close()

    # the same call when the drafter hands over the statistics of its rows (dspark_verify_draft_stats): the pairs are
    # computed once, outside the timed region, the way a draft step leaves them behind
    draft_stats_ms = None
    if not wl["greedy"] and TRUNCATE is None and not PER_REQUEST_T:
        row_stats = []
        for b in batches:
            st_b = torch.empty(b.draft.shape[0], 2, device=device)
            B.dspark_row_stats(b.draft, b.temperature, out_row_stats=st_b)
            row_stats.append(st_b)
        torch.cuda.synchronize()
        off_now = step.offsets if step.sched is not None else None

        def verify_stats(i):
            b = batches[i % n_sets]
            B.dspark_verify_draft_stats(b.target, b.draft, off_now if off_now is not None else b.row_offsets, b.draft_tokens,
                                        row_stats[i % n_sets], b.seed, temperature=b.temperature,
                                        draft_row_start=b.draft_row_start, accepted_len=step.acc, out_tokens=step.out,
                                        dev_status=step.status, workspace=step.ws, n_rows=step.n_rows)
        for i in range(min(warmup, 5)):
            verify_stats(i)
        dt = sorted(timed_loop(verify_stats, steps) for _ in range(max(5, repeats // 5)))
        draft_stats_ms = replicas.max_over_ranks([dt[len(dt) // 2]], dist, device)[0]
        assert int(step.status.item()) == dev_status

    res = dict(wl=wl, step=step, ms=ms, ms_min=ms_min, repeats=repeats, timed_ms=sum(times), verify_ms=verify_ms,
               draft_stats_ms=draft_stats_ms,
               n_rows=n_rows, n_rejected=n_rejected, kernels=kernels, clocks=clocks, dev_status=dev_status, n_sets=n_sets)

    if with_e2e:
        # end to end: inputs start in pinned host memory, results end in host memory, every step
        b = batches[0]
        host_in = [t.cpu().pin_memory() for t in (b.target, b.draft, b.draft_tokens) if t is not None]
        conf_h = wl["sched"].conf.cpu().pin_memory() if wl["sched"] is not None else None
        off_h = None if wl["sched"] is not None else b.row_offsets.cpu().pin_memory()
        dev_in = [torch.empty_like(t, device=device) for t in host_in]
        conf_d = torch.empty_like(wl["sched"].conf) if conf_h is not None else None
        off_d = torch.empty_like(b.row_offsets) if off_h is not None else None
        acc_h = torch.empty(step.R, dtype=torch.int32).pin_memory()
        out_h = torch.empty(step.n_rows, dtype=torch.int32).pin_memory()
        from paper_2607_05147_b200 import workloads as W
        h2d = sum(t.numel() * t.element_size() for t in host_in)
        h2d += conf_h.numel() * 4 if conf_h is not None else off_h.numel() * 4
        d2h = acc_h.numel() * 4 + out_h.numel() * 4

        def e2e_step(_):
            for h, d in zip(host_in, dev_in):
                d.copy_(h, non_blocking=True)
            if conf_h is not None:
                conf_d.copy_(conf_h, non_blocking=True)
            else:
                off_d.copy_(off_h, non_blocking=True)
            if wl["greedy"]:
                eb = W.VerifyBatch(dev_in[0], None, off_d if off_d is not None else b.row_offsets, dev_in[1],
                                   None, b.temperature, b.seed)
            else:
                eb = W.VerifyBatch(dev_in[0], dev_in[1], off_d if off_d is not None else b.row_offsets,
                                   dev_in[2], None, b.temperature, b.seed)
            step.run(eb, conf=conf_d)
            acc_h.copy_(step.acc, non_blocking=True)
            out_h.copy_(step.out, non_blocking=True)

        e2e_steps = max(3, min(steps, 20))
        for k in range(3):
            e2e_step(k)
        e2e_ms = replicas.max_over_ranks([timed_loop(e2e_step, e2e_steps)], dist, device)[0]
        res["e2e"] = dict(ms=e2e_ms, steps=e2e_steps, h2d=h2d, d2h=d2h)

    if with_cpu and rank == 0:
        import oracle
        oracle.build()
        host_copy(wl)
        threads = os.cpu_count() or 1
        oracle_step(wl, batches[0], batches[0].R, threads)          # first touch of the host copies
        t0 = time.perf_counter()
        rows, reps = 0, 0
        while reps < 3 or (time.perf_counter() - t0 < 2.0 and reps < 200):
            rows += oracle_step(wl, batches[0], batches[0].R, threads)
            reps += 1
        dt = time.perf_counter() - t0
        res["cpu"] = {"value": rows / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
                      "sample": f"whole batch ({batches[0].R} requests, {rows // reps} rows) x {reps} passes in "
                                f"{dt:.2f} s, pthreads over requests, stops at each first rejection"}
        # the same oracle on one core: a bounded number of requests (about ten seconds at most)
        t0 = time.perf_counter()
        probe = max(1, batches[0].R // 16)
        r1 = oracle_step(wl, batches[0], probe, 1)
        t_probe = time.perf_counter() - t0
        n_req = max(probe, min(batches[0].R, int(probe * 8.0 / max(t_probe, 1e-6))))
        t0 = time.perf_counter()
        r1 = oracle_step(wl, batches[0], n_req, 1)
        dt1 = time.perf_counter() - t0
        res["cpu"]["single_thread"] = {"value": r1 / dt1, "unit": UNIT, "cores": 1,
                                       "sample": f"first {n_req} of {batches[0].R} requests ({r1} rows), one pass in {dt1:.2f} s"}
    return res


def roofline_of(res, peak, peak_src):
    """Dominant kernel of the step against the measured HBM peak (bytes the method must move / its time)."""
    wl = res["wl"]
    b0 = wl["batches"][0]
    stream_bytes, all_bytes, _ = algorithmic_bytes(b0, wl["greedy"], res["n_rejected"])
    dom = "greedy_stream" if wl["greedy"] else "stream_stats"
    k = res["kernels"].get(dom, {"ms": float("nan"), "launches": 1})
    dom_ms = k["ms"] / max(1, k["launches"])
    achieved = stream_bytes / (dom_ms * 1e-3) / 1e9
    traffic = NCU_TRAFFIC_BYTES.get(wl["name"]) if not REQUESTS_OVERRIDE else None
    if traffic is None and wl["name"] in NCU_TRAFFIC_RATIO and not REQUESTS_OVERRIDE:
        traffic = int(NCU_TRAFFIC_RATIO[wl["name"]] * stream_bytes)
    if wl["greedy"]:
        rows = "every target row once"
    elif TRUNCATE is not None or b0.R > 2048:
        rows = "every target row and every draft row once"
    else:
        rows = ("the target and the draft row of every draft position (the bonus rows are left to the second pass, which "
                "streams them only for requests that accepted every draft token)")
    return {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS, "traffic": traffic,
            "peak_source": peak_src, "algorithmic_bytes_per_launch": stream_bytes, "us_per_launch": dom_ms * 1e3,
            "rows_per_launch": stream_bytes // (b0.target.element_size() * b0.V), "launch_streams": rows}


def verify_call_of(res, steps, peak):
    """The verifier call as a whole (every kernel of dspark_verify / dspark_verify_greedy, no scheduler): the
    bytes the method must move, re-reads of rejected pairs included, over its un-instrumented time."""
    wl = res["wl"]
    _, all_bytes, formula = algorithmic_bytes(wl["batches"][0], wl["greedy"], res["n_rejected"])
    us = 1e3 * res["verify_ms"] / steps
    gbs = all_bytes / (us * 1e-6) / 1e9
    return {"us_per_call": us, "algorithmic_bytes": all_bytes, "gbs": gbs, "frac": gbs / peak,
            "bytes_every_row_once_plus_rejected_pairs": formula, "frac_of_that": formula / (us * 1e-6) / 1e9 / peak,
            "timing": "CUDA events around `steps` back-to-back calls, median over repeats, batches rotated"}


def draft_stats_call_of(res, steps, peak):
    """The verifier call with the draft rows' statistics supplied by the drafter: the statistics pass streams the
    target rows alone, so the bytes the method must move shrink by the draft rows."""
    if res.get("draft_stats_ms") is None:
        return None
    wl = res["wl"]
    b0 = wl["batches"][0]
    elem = b0.target.element_size()
    # statistics pass: the target rows of the draft positions; second pass: rejected pairs and the bonus rows of the rest
    all_bytes = elem * b0.V * ((b0.n_rows - b0.R) + 2 * res["n_rejected"] + (b0.R - res["n_rejected"]))
    us = 1e3 * res["draft_stats_ms"] / steps
    gbs = all_bytes / (us * 1e-6) / 1e9
    return {"us_per_call": us, "algorithmic_bytes": all_bytes, "gbs": gbs, "frac": gbs / peak,
            "rows_per_s": b0.n_rows / (us * 1e-6),
            "what": "dspark_verify_draft_stats: (reference, sum) of every draft row handed over by the drafter "
                    "(computed outside the timed region, as a draft step leaves them); same timing rule as verify_call"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--repeats", type=int, default=25,
                    help="how often the timed --steps loop is repeated (the line reports the median and the minimum)")
    ap.add_argument("--workload", default="cfg3",
                    choices=["cfg2", "cfg3", "cfg4", "cfg5", "cfg2_fp32", "cfg4_bf16"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--all-workloads", action="store_true",
                    help="besides cfg2 / cfg4 / cfg5 and the Markov step also time the fp32 sampling and bf16 greedy variants")
    ap.add_argument("--only", action="store_true", help="time --workload alone (no other workloads, no Markov step)")
    ap.add_argument("--async-topk", action="store_true",
                    help="schedule with dspark_schedule_async (capacity from two steps earlier, Section 5.2)")
    ap.add_argument("--per-request-temperature", action="store_true",
                    help="verify with dspark_verify_per_request (a device array of R temperatures)")
    ap.add_argument("--top-k", type=int, default=0, help="verify against the top-k truncated target (every request)")
    ap.add_argument("--top-p", type=float, default=1.0, help="verify against the top-p truncated target (every request)")
    ap.add_argument("--overlap-schedule", action="store_true",
                    help="with --async-topk: schedule step t+1 on a second stream while step t is verified "
                         "(the asynchronous scheduler is off the critical path, Section 5.2)")
    ap.add_argument("--cuda-graph", action="store_true",
                    help="capture the step (schedule -> verify) in CUDA graphs and time their replay")
    ap.add_argument("--requests", type=int, default=0,
                    help="override the request count of cfg2 / cfg4 (smaller cases for profiler captures)")
    ap.add_argument("--markov-draft", action="store_true",
                    help="time the Markov-head draft step (Section 3.1) for --requests rows (default 256) instead of "
                         "the verification step; prints its own JSON line")
    ap.add_argument("--markov-epilogue", type=int, default=0, help="epilogue path of the Markov GEMM (diagnostic)")
    ap.add_argument("--quick", action="store_true",
                    help="timed steps only (no clock probe, per-kernel timing, e2e or CPU legs): for profiler captures")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    global REQUESTS_OVERRIDE, ASYNC_TOPK, CUDA_GRAPH, OVERLAP, PER_REQUEST_T, TRUNCATE
    if args.top_k > 0 or args.top_p < 1.0:
        TRUNCATE = (args.top_k, args.top_p)
    PER_REQUEST_T = args.per_request_temperature
    REQUESTS_OVERRIDE = args.requests
    ASYNC_TOPK, CUDA_GRAPH = args.async_topk, args.cuda_graph
    OVERLAP = args.overlap_schedule
    if OVERLAP and (not ASYNC_TOPK or CUDA_GRAPH):
        raise SystemExit("--overlap-schedule needs --async-topk and stream launches")

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        launch_replicas(sys.argv[1:], args.gpus)

    from paper_2607_05147_b200 import replicas
    rank, local_rank, world = replicas.env_ranks()
    if args.impl == "reference":
        run_reference(args, rank)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=device)

    from paper_2607_05147_b200 import binding as B
    B.lib()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    if args.markov_draft:
        line = bench_markov(args, device, rank, world, dist, barrier)
        if line is not None:
            print(json.dumps(line), flush=True)
        if dist is not None:
            dist.destroy_process_group()
        return

    res = measure_workload(args.workload, args, device, rank, local_rank, world, dist, barrier, True, world == 1 or rank == 0)
    wl = res["wl"]
    if res.get("quick"):
        print(json.dumps({"quick": True, "workload": wl["name"], "ms_per_step": res["ms"] / args.steps,
                          "rows_per_s": res["n_rows"] * args.steps / (res["ms"] * 1e-3)}), flush=True)
        return

    b0 = wl["batches"][0]
    stream_bytes, all_bytes, _ = algorithmic_bytes(b0, wl["greedy"], res["n_rejected"])
    ms, e2e_ms = res["ms"], res["e2e"]["ms"]
    value = replicas.whole_job_rate(res["n_rows"], args.steps, ms, world)
    e2e_value = replicas.whole_job_rate(res["n_rows"], res["e2e"]["steps"], e2e_ms, world)

    peaks_file = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_file):
        peak, peak_src = float(json.load(open(peaks_file))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    else:
        peak, peak_src = FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"

    line = None
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(wl, b0, res["n_rows"], res["n_rejected"], res["n_sets"], stream_bytes),
            "timing": {"repeats": res["repeats"], "ms_per_step_min": res["ms_min"] / args.steps,
                       "timed_region_ms": res["timed_ms"],
                       "rule": "ms_per_step is the median over `repeats` repeats of the --steps loop, each between a "
                               "barrier + synchronize on both sides (max over ranks per repeat)"},
            "step_algorithmic_bytes": all_bytes,
            "step_effective_gbs": all_bytes / (ms / args.steps * 1e-3) / 1e9,
            "step_frac_of_peak": all_bytes / (ms / args.steps * 1e-3) / 1e9 / peak,
            "roofline": roofline_of(res, peak, peak_src),
            "verify_call": verify_call_of(res, args.steps, peak),
            "verify_call_draft_stats": draft_stats_call_of(res, args.steps, peak),
            "kernels_us_per_launch": {n: 1e3 * v["ms"] / v["launches"] for n, v in res["kernels"].items()},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": res["e2e"]["h2d"],
                    "d2h_bytes_per_step": res["e2e"]["d2h"], "ms_per_step": e2e_ms / res["e2e"]["steps"],
                    "steps": res["e2e"]["steps"]},
            "gpu_launches": res["step"].launches_per_step * args.steps,
            "clocks": res["clocks"], "dev_status": res["dev_status"],
            "cpu_baseline": res.get("cpu"),
        }
    if not args.only and world == 1:
        # the other V = 129 280 configurations and the Markov-head draft step, each with its own clocks
        names = ["cfg2", "cfg3", "cfg4", "cfg5"] + (["cfg2_fp32", "cfg4_bf16"] if args.all_workloads else [])
        others = {}
        for name in names:
            if name == args.workload:
                continue
            del res, wl
            torch.cuda.empty_cache()
            res = measure_workload(name, args, device, rank, local_rank, world, dist, barrier, False, False)
            wl = res["wl"]
            _, ab, _ = algorithmic_bytes(wl["batches"][0], wl["greedy"], res["n_rejected"])
            roof = roofline_of(res, peak, peak_src)
            step_ms = res["ms"] / args.steps
            others[name] = {"value": res["n_rows"] * args.steps / (res["ms"] * 1e-3), "unit": UNIT,
                            "ms_per_step": step_ms, "ms_per_step_min": res["ms_min"] / args.steps, "repeats": res["repeats"],
                            "rows_per_step": res["n_rows"], "rejected_requests": res["n_rejected"],
                            "step_algorithmic_bytes": ab, "step_frac_of_peak": ab / (step_ms * 1e-3) / 1e9 / peak,
                            "dominant_kernel": roof["kernel"], "dominant_kernel_gbs": roof["achieved"],
                            "dominant_kernel_frac": roof["frac"], "dominant_kernel_us": roof["us_per_launch"],
                            "verify_call": verify_call_of(res, args.steps, peak),
            "verify_call_draft_stats": draft_stats_call_of(res, args.steps, peak),
                            "kernels_us_per_launch": {n: 1e3 * v["ms"] / v["launches"] for n, v in res["kernels"].items()},
                            "clocks": res["clocks"], "dev_status": res["dev_status"]}
        del res, wl
        torch.cuda.empty_cache()
        line["other_workloads"] = others
        # the option rows on cfg3 (each is what `bench.py --only <flags>` prints as its own line): the step with
        # top-k / top-p truncation inside the verifier, with one temperature per request, with the asynchronous
        # top-K scheduler
        if args.workload == "cfg3" and TRUNCATE is None and not (PER_REQUEST_T or ASYNC_TOPK or CUDA_GRAPH or OVERLAP):
            variants = {}
            for label, setting in (("top_k50_top_p0.9", {"TRUNCATE": (50, 0.9)}), ("top_p0.9", {"TRUNCATE": (0, 0.9)}),
                                   ("top_k50", {"TRUNCATE": (50, 1.0)}), ("per_request_temperature", {"PER_REQUEST_T": True}),
                                   ("async_topk", {"ASYNC_TOPK": True})):
                saved = {k: globals()[k] for k in setting}
                globals().update(setting)
                try:
                    res = measure_workload("cfg3", args, device, rank, local_rank, world, dist, barrier, False, False)
                finally:
                    globals().update(saved)
                variants[label] = {"ms_per_step": res["ms"] / args.steps, "ms_per_step_min": res["ms_min"] / args.steps,
                                   "verify_call_us": verify_call_of(res, args.steps, peak)["us_per_call"],
                                   "kernels_us_per_launch": {n: 1e3 * v["ms"] / v["launches"] for n, v in res["kernels"].items()},
                                   "gpu_launches_per_step": res["step"].launches_per_step,
                                   "clocks": res["clocks"], "dev_status": res["dev_status"]}
                del res
                torch.cuda.empty_cache()
            line["variants_cfg3"] = variants
        margs = argparse.Namespace(**vars(args))
        margs.requests = 256
        m = bench_markov(margs, device, rank, world, dist, barrier)
        line["markov_draft"] = {"requests": 256, "us_per_launch": m["roofline"]["us_per_launch"], "frac": m["roofline"]["frac"],
                                "gbs": m["roofline"]["achieved"], "tensor_tflops": m["roofline"]["tensor_tflops"],
                                "step_us": 1e3 * m["ms_per_step"], "algorithmic_bytes_per_launch": m["roofline"]["algorithmic_bytes_per_launch"],
                                "kernels_us_per_launch": m["kernels_us_per_launch"], "clocks": m["clocks"], "dev_status": m["dev_status"]}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
