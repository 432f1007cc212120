#!/usr/bin/env python
"""Benchmark of the Carryover drafting round (one step = one whole round: verify-accept,
K/V projection with E_carry, scatter, block attention in every drafter layer, LM head + argmax).

    python bench.py --gpus 1 --steps 20 --warmup 5            # default: batch 32 on the line, batch 1 under "batch1"
    python bench.py --workload cfg2                           # one configuration only (cfg2: batch 1, cfg3: batch 32)
    python bench.py --workload cfg2f                          # batch 1, complete drafter layer (MLP, q/k norm)
    python bench.py --impl reference                          # the CPU oracle on the host cores
    python bench.py --workload cfg3 --micro gemm --shape qkv  # one-layer round, one contraction class timed

Prints ONE JSON line.  Inputs are seeded and synthetic (the recipe is in the docstrings of
paper_2609_14717_b200/synth.py: weights ~ N(0, 0.02), hidden states with a per-layer RMS ramp,
randomly permuted page tables, geometric acceptance lengths); the weights (about 2 GB) are re-read from HBM every round, so no L2 flush is needed between steps.
With N > 1 (torchrun) every rank runs an independent replica: the round has no exchange step.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_14717_b200 import synth  # noqa: E402

METRIC = "drafting rounds/s"
UNIT = "rounds/s"
HBM_NOMINAL_GBS = 7700.0     # the data-sheet figure, quoted beside fractions that exceed the copy-measured peak
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.txt")
CSRC = os.path.join(ROOT, "paper_2609_14717_b200", "csrc")
# source files whose change invalidates a recorded DRAM-traffic figure of a kernel class
KERNEL_SOURCES = {"lmhead": ("k_gemm_tc.cu", "k_gemm_tc2.cu", "tc_common.cuh"),
                  "attn": ("k_attn_tc.cu", "tc_common.cuh")}


def source_hash(klass: str) -> str:
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES.get(klass, ()):
        with open(os.path.join(CSRC, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload: str, klass: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of a kernel class, from the ncu capture recorded
    in profiles/dram_traffic.txt ("workload class source-hash bytes" per line, rewritten by --record-traffic).
    None when there is no record or the kernel's sources changed since the capture."""
    try:
        with open(TRAFFIC_FILE) as f:
            for line in f:
                part = line.split()
                if len(part) >= 4 and not line.startswith("#") and part[0] == workload and part[1] == klass:
                    return int(part[3]) if part[2] == source_hash(klass) else None
    except OSError:
        pass
    return None


def record_traffic(args):
    """--record-traffic FILE: FILE is the CSV ncu wrote for ONE launch of the workload's dominant kernel with
    --metrics dram__bytes_read.sum,dram__bytes_write.sum; its sum replaces the workload's line in the table."""
    import csv
    total = 0.0
    with open(args.record_traffic) as f:
        rows = [r for r in csv.reader(f) if len(r) > 3]
    head = next(r for r in rows if "Metric Name" in r)
    i_name, i_unit, i_val = head.index("Metric Name"), head.index("Metric Unit"), head.index("Metric Value")
    for r in rows[rows.index(head) + 1:]:
        if r[i_name] in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
            total += float(r[i_val].replace(",", "")) * {"byte": 1, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}[r[i_unit]]
    klass = args.shape or "lmhead"
    keep = []
    if os.path.exists(TRAFFIC_FILE):
        keep = [l for l in open(TRAFFIC_FILE) if l.startswith("#") or l.split()[:2] != [args.workload, klass]]
    if not keep:
        keep = ["# workload class source-hash dram-bytes-per-launch (ncu: dram__bytes_read.sum + dram__bytes_write.sum)\n"]
    keep.append(f"{args.workload} {klass} {source_hash(klass)} {int(total)}\n")
    open(TRAFFIC_FILE, "w").writelines(keep)
    print(json.dumps({"recorded": args.workload, "class": klass, "bytes": int(total)}))


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "tflops": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "tflops_burst": float(p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops": 1400.0, "tflops_burst": 1590.0, "source": "fallback"}


# --------------------------------------------------------------------------- replicas
def replica_seed(seed: int, rank: int) -> int:
    """Every rank runs its own replica of the workload on its own inputs."""
    return seed + rank


def max_over_ranks(ms: float, world: int, device="cuda") -> float:
    """The timed region of the job is that of its slowest replica."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(ms: float, steps: int, world: int) -> float:
    """Rounds per second of the whole job: all replicas' rounds over the slowest replica's time."""
    return world * steps / (ms * 1e-3)


# --------------------------------------------------------------------------- byte / flop model
def round_model(wl, L_after, carry, kept_rows, es=2):
    """Algorithmic bytes and flops of one round, per kernel class (weights read once per round,
    committed KV read once per layer per sequence)."""
    sh = wl.shape
    D, Din, Ld = sh.d_model, sh.d_in, sh.n_layers
    kvw, qw, R, V = sh.n_kv * sh.hd, sh.n_q * sh.hd, wl.R, sh.vocab
    keys = float(np.sum(L_after + carry))
    out = {
        "fc": (D * Din * es + kept_rows * Din * es + kept_rows * D * es, 2.0 * kept_rows * Din * D),
        "kv": (2 * Ld * kvw * D * es + kept_rows * Ld * 2 * kvw * es, 2.0 * kept_rows * D * 2 * Ld * kvw),
        "qkv": (Ld * ((qw + 2 * kvw) * D * es + R * (D + qw + 2 * kvw) * es), 2.0 * R * D * (qw + 2 * kvw) * Ld),
        "oproj": (Ld * (D * qw * es + R * (qw * es + D * 4)), 2.0 * R * qw * D * Ld),
        "attn": (Ld * (keys * 2 * kvw * es + 2 * R * qw * es),
                 Ld * 4.0 * sh.W * sh.n_q * sh.hd * float(np.sum(L_after + carry + sh.W))),
        "lmhead": (V * D * es + R * D * es, 2.0 * R * D * V),
    }
    if sh.d_ff > 0:      # complete layer: gate, up and down matrices once per layer
        out["mlp"] = (Ld * (3 * D * sh.d_ff * es + R * (D + 2 * sh.d_ff) * es), 2.0 * R * 3 * D * sh.d_ff * Ld)
    return out


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Polls NVML (read-only) for SM clock, power and throttle reasons while the timed region runs."""

    def __init__(self, device_index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self._nv = pynvml
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._h = None

    def _loop(self):
        nv = self._nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20,
                 "hw_thermal_slowdown": 0x40, "hw_power_brake": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    bits = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                except Exception:
                    bits = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for k, b in names.items():
                    if bits & b:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.004)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------- workload set-up
def bench_workload(name: str, n_rounds: int):
    wl = synth.workload(name)
    return synth.scaled(wl, n_rounds=n_rounds)


def host_rounds(wl, seed, n, ring):
    """Tokens for n rounds and a ring of H tensors (open loop: inputs never depend on outputs)."""
    toks, Hs = [], []
    for r in range(n):
        rng = np.random.default_rng([seed, 4, r])
        m = synth.draw_accept(wl, rng)
        draft, target = synth.make_tokens(wl, rng, m)
        toks.append((draft, target, m))
        if r < ring:
            Hs.append(synth.make_hidden(wl, rng))
    return toks, Hs


# --------------------------------------------------------------------------- the CPU oracle leg
def oracle_objects(wl, seed, weights, S_sample):
    from oracle import cod_oracle as orc
    sh = wl.shape
    sub = synth.scaled(wl, S=S_sample)
    lay = synth.make_layout(sub, seed)
    cfg = orc.OracleConfig(d_target=sh.d_target, n_cap=sh.n_cap, d_model=sh.d_model, n_layers=sh.n_layers,
                           n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, vocab=sh.vocab, mask_token_id=sh.mask_token_id,
                           W=sh.W, page=sh.page, rope_theta=sh.rope_theta, rms_eps=sh.rms_eps,
                           hidden_norm=sh.hidden_norm)
    # compact page table: only the pages this sample can touch
    L = lay["committed_len"]
    per = (int(L.max()) + (sub.n_rounds + 2) * sh.W) // sh.page + 2
    bt = np.arange(S_sample * per, dtype=np.int64).reshape(S_sample, per)
    st = orc.OracleState(cfg, S_sample, S_sample * per, bt, L)
    rng = np.random.default_rng([seed, 3])
    for s in range(S_sample):
        used = (int(L[s]) + sh.page - 1) // sh.page
        st.pool[:, bt[s, :used]] = synth.to_storage(
            rng.standard_normal((sh.n_layers, used, sh.n_kv, 2, sh.page, sh.hd), dtype=np.float32), sh.dtype)
    return orc, sub, st, orc.prepare_weights(weights)


def time_oracle(wl, seed, weights, n_rounds, S_sample, budget_s=None):
    """Runs the oracle, as it stands, for n_rounds rounds of the first S_sample sequences."""
    orc, sub, st, w64 = oracle_objects(wl, seed, weights, S_sample)
    times = []
    for r in range(n_rounds):
        rd = synth.make_round(sub, seed, r)
        t0 = time.perf_counter()
        orc.draft_round(rd["draft"], rd["target"], rd["H"], st, w64, sub.n_forced, orc.MODE_CARRY)
        times.append(time.perf_counter() - t0)
        if budget_s is not None and sum(times) > budget_s and len(times) >= 3:
            break
    return times


def cores_used():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def config_of(wl, n_gpus: int) -> dict:
    """The workload description both arms print (identical keys and values for the same flags)."""
    sh = wl.shape
    return {"workload": wl.name, "batch": wl.S, "block": sh.W, "context": list(wl.ctx),
            "drafter_layers": sh.n_layers, "vocab": sh.vocab, "parallelism": f"replicas x{n_gpus}",
            "l2": "inputs larger than L2 (weights re-read every round)"}


def default_workloads(args):
    """Without --workload the line carries the batch-32 configuration and, under "batch1", the batch-1 one:
    the metric is quoted at both, and the roofline target is stated at batch 32."""
    return [args.workload] if args.workload else ["cfg3", "cfg2"]


def reference_record(name, args, budget_s):
    """The CPU oracle, as it stands, on a bounded sample of workload `name`."""
    wl = bench_workload(name, args.steps + args.warmup + 1)
    weights = synth.make_weights(wl.shape, args.seed)
    S_sample = 1 if wl.S == 1 else 2
    orc, sub, st, w64 = oracle_objects(wl, args.seed, weights, S_sample)
    per_step = []
    t_start = time.perf_counter()
    for r in range(args.warmup + args.steps):
        rd = synth.make_round(sub, args.seed, r)
        t0 = time.perf_counter()
        orc.draft_round(rd["draft"], rd["target"], rd["H"], st, w64, sub.n_forced, orc.MODE_CARRY)
        dt = time.perf_counter() - t0
        if r >= args.warmup:
            per_step.append(dt)
        if time.perf_counter() - t_start > budget_s and per_step:
            break
    mean = sum(per_step) / len(per_step)
    # a step of the sample covers S_sample of the S sequences of a round
    value = (S_sample / wl.S) / mean
    sample = (f"{len(per_step)} whole rounds of {S_sample} of {wl.S} sequences at full shapes, float64 numpy; "
              f"rounds/s scaled by {S_sample}/{wl.S}")
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": len(per_step), "steps_requested": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * mean * wl.S / S_sample, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config_of(wl, args.gpus),
        "us_per_round": 1e6 * mean * wl.S / S_sample,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores_used(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


def run_reference(args):
    """--impl reference: the CPU oracle timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    names = default_workloads(args)
    line = reference_record(names[0], args, 150.0 if len(names) > 1 else 240.0)
    if len(names) > 1:
        sub = reference_record(names[1], args, 90.0)
        line["batch1"] = {k: sub[k] for k in ("value", "unit", "ms_per_step", "us_per_round", "steps", "config",
                                              "cpu_baseline", "e2e", "dtype")}
    print(json.dumps(line))


# --------------------------------------------------------------------------- the GPU arm
def measure_workload(name, args, rank, world, local, peaks, with_cpu):
    """All numbers of one workload on this rank's GPU; returns the record (rank 0) or None."""
    import torch
    import torch.distributed as dist

    from paper_2609_14717_b200 import binding as B

    K, Wm = args.steps, args.warmup
    n_rounds = K + Wm
    wl = bench_workload(name, n_rounds + 1)
    sh = wl.shape
    seed = replica_seed(args.seed, rank)
    es = 2 if sh.dtype == "bf16" else 4

    # ---- inputs: weights (host, seeded) -> device; layout; pool filled on the device
    weights = synth.make_weights(sh, seed)
    lay = synth.make_layout(wl, seed)
    n_pages, mp = int(lay["n_pages"]), int(lay["max_pages_per_seq"])
    cfg = B.make_config(sh, wl.S, mp, n_pages, attn_split_len=args.attn_split, extra_flags=args.flags)
    ctx = B.Context(cfg)
    w_dev = B.weights_to_device(weights, sh.dtype)
    ctx.set_weights(w_dev)
    state = B.State(cfg, sh.dtype, wl.S, lay["block_table"], lay["committed_len"])
    gen = torch.Generator(device="cuda").manual_seed(seed)
    for l in range(sh.n_layers):
        state.kv_pool[l].copy_(torch.randn(state.kv_pool[l].shape, generator=gen, device="cuda",
                                           dtype=torch.float32).to(state.kv_pool.dtype))
    ring = 8
    toks, Hs = host_rounds(wl, seed, ring, ring)           # inputs repeat with period 8 (open loop)
    H_pin = [torch.from_numpy(h).to(B.torch_dtype(sh.dtype)).pin_memory() for h in Hs]
    d_pin = [torch.from_numpy(t[0]).pin_memory() for t in toks]
    t_pin = [torch.from_numpy(t[1]).pin_memory() for t in toks]
    H_dev = [h.cuda() for h in H_pin]
    d_dev = [d.cuda() for d in d_pin]
    t_dev = [t.cuda() for t in t_pin]
    # end-to-end staging: a round's three inputs sit in ONE pinned host buffer (256-byte aligned parts), so a
    # step pays for one host-to-device copy; stage_H / stage_d / stage_t are views of its device twin
    def _packed(parts, device, pin):
        offs, n = [], 0
        for t in parts:
            offs.append(n)
            n += (t.numel() * t.element_size() + 255) // 256 * 256
        buf = torch.empty(n, dtype=torch.uint8, device=device, pin_memory=pin)
        views = [buf[o:o + t.numel() * t.element_size()].view(t.dtype).view(t.shape) for o, t in zip(offs, parts)]
        return buf, views
    stage_buf, (stage_H, stage_d, stage_t) = _packed((H_pin[0], d_pin[0], t_pin[0]), "cuda", False)
    pin_bufs = []
    for i in range(ring):
        buf, (vh, vd, vt) = _packed((H_pin[i], d_pin[i], t_pin[i]), "cpu", True)
        vh.copy_(H_pin[i]); vd.copy_(d_pin[i]); vt.copy_(t_pin[i])
        pin_bufs.append(buf)
    stage_buf.copy_(pin_bufs[0])                            # the staged graph's warm-up launch reads it
    next_draft = torch.zeros((wl.S, sh.W), dtype=torch.int32, device="cuda")
    out_pin = torch.zeros((wl.S, sh.W), dtype=torch.int32).pin_memory()
    L0 = state.committed_len.clone()

    def reset():
        """Every pass starts from the same state (lengths; the pool's contents are inputs and stay)."""
        state.committed_len.copy_(L0)
        state.carry_len.zero_()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def launch_round(i, mode, staged=False):
        if staged:
            ctx.draft_round(stage_d, stage_t, stage_H, wl.S, wl.n_forced, mode, state, None, next_draft, None)
        else:
            ctx.draft_round(d_dev[i], t_dev[i], H_dev[i], wl.S, wl.n_forced, mode, state, None, next_draft, None)

    # One CUDA graph per input slot (and one bound to the staging buffers for the end-to-end
    # pass): a replay enqueues the round's ~40 kernels with a single launch.
    graphs = {}

    def graph_for(i, mode, staged=False):
        key = (i, mode, staged)
        if key not in graphs:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):                   # warm-up outside capture
                launch_round(i, mode, staged)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                launch_round(i, mode, staged)
            graphs[key] = g
        return graphs[key]

    def timed_pass(mode, e2e=False, profile=(), K=K, use_graph=True):
        """One pass: restore the state, Wm untimed rounds, then K rounds between CUDA events."""
        reset()
        if use_graph:
            for i in range(1 if e2e else ring):
                graph_for(0 if e2e else i, mode, staged=e2e)
        reset()
        ctx.profile_enable(())

        def step(r):
            i = r % ring
            if e2e:
                stage_buf.copy_(pin_bufs[i], non_blocking=True)
                if use_graph:
                    graphs[(0, mode, True)].replay()
                else:
                    launch_round(i, mode, staged=True)
                out_pin.copy_(next_draft, non_blocking=True)  # the step's result, read on the host
                torch.cuda.current_stream().synchronize()
                return out_pin
            if use_graph:
                graphs[(i, mode, False)].replay()
            else:
                launch_round(i, mode)
            return None

        for r in range(Wm):
            step(r)
        barrier()
        ctx.profile_enable(profile)
        n0 = ctx.launch_count()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for r in range(Wm, Wm + K):
            step(r)
        ev1.record()
        barrier()
        ms = ev0.elapsed_time(ev1)
        launches = ctx.launch_count() - n0
        return max_over_ranks(ms, world), launches

    # ---- the byte / flop model of the timed rounds, per kernel class
    L_run = lay["committed_len"].astype(np.int64).copy()
    models = []
    for r in range(n_rounds):
        m = toks[r % ring][2].astype(np.int64)
        L_run = L_run + m
        if r >= Wm:
            models.append(round_model(wl, L_run, sh.W - m, wl.R, es))
    mean_model = {k: (float(np.mean([mm[k][0] for mm in models])), float(np.mean([mm[k][1] for mm in models])))
                  for k in models[0]}
    t_class = {k: max(b / (peaks["hbm_gbs"] * 1e9), f / (peaks["tflops"] * 1e12)) for k, (b, f) in mean_model.items()}
    dominant = max(t_class, key=t_class.get)

    # stream launches first (also counts the kernels of a round and times the dominant one) ...
    ms_stream, launches = timed_pass(B.COD_CARRY, profile=(dominant,), use_graph=False)
    dom_ms, dom_n = ctx.profile_read(dominant)
    K_prof = min(K, 32)                                     # bounded by the library's event slots
    timed_pass(B.COD_CARRY, profile=B.KERNEL_CLASSES, K=K_prof, use_graph=False)
    per_class = {k: ctx.profile_read(k) for k in B.KERNEL_CLASSES}
    # ... then the same rounds replayed as CUDA graphs, every pass from the restored state, carry and
    # baseline passes interleaved (C B C B ...), at least 7 of each and about a second of timed work in all;
    # the medians are the headline numbers
    use_graph = not args.no_graph
    t_carry, t_base, t_e2e = [], [], []
    with ClockSampler(local) as clk:
        first, _ = timed_pass(B.COD_CARRY, use_graph=use_graph)
        reps = int(min(61, max(7, np.ceil(400.0 / max(first, 1e-3)))))
        if world > 1:                                       # every rank must run the same number of passes
            t = torch.tensor([reps], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            reps = int(t.item())
        for _ in range(reps):
            t_carry.append(timed_pass(B.COD_CARRY, use_graph=use_graph)[0])
            t_base.append(timed_pass(B.COD_BASELINE, use_graph=use_graph)[0])
        for _ in range(max(7, reps // 2)):
            t_e2e.append(timed_pass(B.COD_CARRY, e2e=True, use_graph=use_graph)[0])
    ms, ms_base, ms_e2e = (statistics.median(v) for v in (t_carry, t_base, t_e2e))
    # the overhead as the median of the paired differences (pass i of each mode ran back to back)
    overhead = statistics.median(100.0 * (c - b) / b for c, b in zip(t_carry, t_base))
    status = ctx.poll_status()
    ws_bytes = ctx.workspace_bytes()
    h2d = int(stage_buf.numel())                            # the one packed copy (parts padded to 256 bytes)
    d2h = int(next_draft.numel() * 4)
    ctx.close()
    graphs.clear()
    del state, w_dev, H_dev, stage_buf
    torch.cuda.empty_cache()
    if rank != 0:
        return None

    # ---- roofline of the dominant kernel, of every kernel class and of the whole round
    bw, tf_sus, tf_burst = peaks["hbm_gbs"] * 1e9, peaks["tflops"] * 1e12, peaks["tflops_burst"] * 1e12
    b_dom, f_dom = mean_model[dominant]
    launches_per_round = max(dom_n // K, 1)
    dur = dom_ms / max(dom_n, 1) * 1e-3                      # seconds per launch
    b_launch, f_launch = b_dom / launches_per_round, f_dom / launches_per_round
    hbm_bound = b_launch / bw >= f_launch / tf_sus
    if hbm_bound:
        achieved, peak, unit, bound = b_launch / dur / 1e9, peaks["hbm_gbs"], "GB/s", "hbm"
    else:
        achieved, peak, unit, bound = f_launch / dur / 1e12, peaks["tflops"], "TFLOP/s", "tensor"
    roofline = {"bound": bound, "kernel": dominant, "achieved": achieved, "peak": peak, "unit": unit,
                "frac": achieved / peak, "traffic": recorded_traffic(wl.name, dominant),
                "peak_source": peaks["source"], "algorithmic_bytes_per_launch": b_launch,
                "algorithmic_flops_per_launch": f_launch, "us_per_launch": dur * 1e6, "launches_timed": dom_n}
    if hbm_bound and roofline["frac"] > 1.0:
        # the denominator is a COPY (read + write); a read-only stream can run above it
        roofline["frac_of_nominal"] = achieved / HBM_NOMINAL_GBS
        roofline["note"] = ("above the copy-measured peak: this kernel only reads; frac_of_nominal is against the "
                            "data-sheet 7700 GB/s")
    kernels_roofline = {}
    for k in B.KERNEL_CLASSES:
        us_k = per_class[k][0] / K_prof * 1e3
        n_k = per_class[k][1] / K_prof
        if us_k <= 0.0:
            continue
        rec = {"us_per_round": us_k, "launches_per_round": n_k}
        if k in mean_model:
            b, f = mean_model[k]
            t_h, t_t = b / bw, f / tf_sus
            rec.update({"bytes": b, "flops": f, "bound": "hbm" if t_h >= t_t else "tensor",
                        "bound_us": max(t_h, t_t) * 1e6, "frac": max(t_h, t_t) * 1e6 / us_k})
        kernels_roofline[k] = rec
    with_model = {k: v for k, v in kernels_roofline.items() if "frac" in v}
    kernels_roofline["worst"] = min(with_model, key=lambda k: with_model[k]["frac"]) if with_model else None
    kernels_roofline["note"] = ("event-bracketed stream launches: each launch carries a few us of bracket, so fractions "
                                "are lower bounds; tensor bounds against the sustained cuBLAS figure; verify and rowops "
                                "have no algorithmic bytes of their own")
    tot_b = sum(v[0] for v in mean_model.values())
    tot_f = sum(v[1] for v in mean_model.values())
    strict_s = max(tot_b / bw, tot_f / tf_burst)
    serial_s = sum(max(b / bw, f / tf_burst) for b, f in mean_model.values())
    us_round = ms / K * 1e3
    round_roofline = {"strict_us": strict_s * 1e6, "serial_us": serial_s * 1e6, "measured_us": us_round,
                      "frac_of_strict": strict_s * 1e6 / us_round, "frac_of_serial": serial_s * 1e6 / us_round,
                      "bytes": tot_b, "flops": tot_f}

    # ---- the CPU oracle on a bounded sample (rank 0, N = 1 only)
    cpu = None
    if with_cpu:
        S_sample = 1 if wl.S == 1 else 2
        # about 12 s of oracle work (at least 3 rounds, at most what the page tables were sized for)
        times = time_oracle(wl, seed, weights, n_rounds=max(3, min(64, wl.n_rounds - 1)), S_sample=S_sample, budget_s=12.0)
        mean = sum(times) / len(times)
        cpu = {"value": (S_sample / wl.S) / mean, "unit": UNIT, "cores": cores_used(), "kind": "oracle",
               "sample": f"{len(times)} whole rounds of {S_sample} of {wl.S} sequences at full shapes "
                         f"(float64 numpy, {mean:.2f} s each); rounds/s scaled by {S_sample}/{wl.S}"}

    spread = lambda v: {"median": statistics.median(v) / K * 1e3, "min": min(v) / K * 1e3, "max": max(v) / K * 1e3,
                        "passes": len(v)}
    return {
        "metric": METRIC, "value": job_throughput(ms, K, world), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": sh.dtype, "data": "synthetic", "config": config_of(wl, world),
        "launch": "cuda_graph" if use_graph else "stream",
        "timing": {"carry_us_per_round": spread(t_carry), "baseline_us_per_round": spread(t_base),
                   "e2e_us_per_round": spread(t_e2e),
                   "protocol": "every pass: state restored, warm-up rounds, K timed rounds between CUDA events; "
                               "carry and baseline passes interleaved; medians reported",
                   "timed_region_s": (sum(t_carry) + sum(t_base) + sum(t_e2e)) * 1e-3},
        "stream_us_per_round": ms_stream / K * 1e3,
        "us_per_round": us_round, "seq_rounds_per_s": world * wl.S * K / (ms * 1e-3),
        "carryover_overhead_pct": overhead,
        "baseline_us_per_round": ms_base / K * 1e3,
        "roofline": roofline, "round_roofline": round_roofline, "kernels_roofline": kernels_roofline,
        "kernels_us_per_round": {k: v[0] / K_prof * 1e3 for k, v in per_class.items()},
        "cpu_baseline": cpu,
        "e2e": {"value": world * K / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h},
        "gpu_launches": launches, "clocks": clk.summary(), "device_status": status,
        "workspace_bytes": ws_bytes,
    }


def run_gpu(args):
    import torch
    import torch.distributed as dist

    import __graft_entry__ as entry

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        entry.build()
    if world > 1:
        dist.barrier()
    peaks = load_peaks()
    with_cpu = world == 1 and not args.no_cpu_baseline
    names = default_workloads(args)
    line = measure_workload(names[0], args, rank, world, local, peaks, with_cpu)
    if len(names) > 1:
        sub = measure_workload(names[1], args, rank, world, local, peaks, with_cpu)
        if rank == 0:
            keep = ("value", "unit", "ms_per_step", "us_per_round", "seq_rounds_per_s", "config", "timing",
                    "carryover_overhead_pct", "baseline_us_per_round", "roofline", "round_roofline",
                    "kernels_roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks", "device_status", "dtype")
            line["batch1"] = {k: sub[k] for k in keep}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_micro_round(args):
    """--micro gemm --shape fc|kv|qkv|oproj|lmhead|attn: whole rounds of a ONE-layer drafter with the workload's
    shapes (small device footprint: meant for profiler captures), plain stream launches, the chosen class timed
    with the library's events. Contractions of one round launch in the order fc, kv, qkv, oproj, lmhead."""
    import torch

    import __graft_entry__ as entry
    from paper_2609_14717_b200 import binding as B

    entry.build()
    torch.cuda.set_device(0)
    peaks = load_peaks()
    K, Wm = args.steps, args.warmup
    wl = bench_workload(args.workload, K + Wm + 2)
    if args.layers > 0:
        wl = synth.scaled(wl, n_layers=args.layers)
    sh = wl.shape
    lay = synth.make_layout(wl, args.seed)
    cfg = B.make_config(sh, wl.S, int(lay["max_pages_per_seq"]), int(lay["n_pages"]), attn_split_len=args.attn_split, extra_flags=args.flags)
    ctx = B.Context(cfg)
    td = B.torch_dtype(sh.dtype)
    gen = torch.Generator(device="cuda").manual_seed(args.seed)
    rnd = lambda *shape, scale=1.0: (torch.randn(*shape, generator=gen, device="cuda") * scale).to(td)
    w = {k: (rnd(*v, scale=0.02) if not k.startswith("g_") else torch.ones(*v, device="cuda", dtype=td))
         for k, v in synth.weight_shapes(sh).items()}
    ctx.set_weights(w)
    state = B.State(cfg, sh.dtype, wl.S, lay["block_table"], lay["committed_len"])
    state.kv_pool.copy_(rnd(*state.kv_pool.shape))
    rd = synth.make_round(wl, args.seed, 0)
    d, t = torch.from_numpy(rd["draft"]).cuda(), torch.from_numpy(rd["target"]).cuda()
    H = B.to_device(rd["H"], sh.dtype)
    nd = torch.zeros((wl.S, sh.W), dtype=torch.int32, device="cuda")
    klass = args.shape or "qkv"
    mode = B.COD_BASELINE if args.baseline else B.COD_CARRY
    for r in range(Wm + K):
        if r == Wm:
            torch.cuda.synchronize()
            ctx.profile_enable((klass,))
        ctx.draft_round(d, t, H, wl.S, wl.n_forced, mode, state, None, nd, None)
    torch.cuda.synchronize()
    ms, n = ctx.profile_read(klass)
    L = lay["committed_len"].astype(np.int64) + K // 2 * 6
    m = rd["m"].astype(np.int64)
    b, f = round_model(wl, L, sh.W - m, wl.R)[klass]
    us = ms / max(n, 1) * 1e3
    per_round = max(n // K, 1)
    print(json.dumps({"micro": "gemm", "class": klass, "workload": wl.name, "rows": wl.R, "us_per_launch": us,
                      "launches_per_round": per_round, "GBps": b / per_round / us / 1e3, "TFLOPs": f / per_round / us / 1e6,
                      "hbm_frac": b / per_round / us / 1e3 / peaks["hbm_gbs"],
                      "tensor_frac": f / per_round / us / 1e6 / peaks["tflops"], "device_status": ctx.poll_status()}))
    ctx.close()


def run_timeline(args):
    """--micro timeline: ONE graph-replayed round of the workload seen through CUPTI activity records
    (torch.profiler): every kernel's start, end and its share of the dependency chain - the time from the later
    of (its start, its predecessor's end) to its own end, which is what the round pays for it when launches
    overlap programmatically. A profiler view for finding where a round's time goes; never a bench value."""
    import torch
    from torch.profiler import ProfilerActivity, profile

    import __graft_entry__ as entry
    from paper_2609_14717_b200 import binding as B

    entry.build()
    torch.cuda.set_device(0)
    wl = bench_workload(args.workload, 40)
    sh = wl.shape
    lay = synth.make_layout(wl, args.seed)
    cfg = B.make_config(sh, wl.S, int(lay["max_pages_per_seq"]), int(lay["n_pages"]), attn_split_len=args.attn_split, extra_flags=args.flags)
    ctx = B.Context(cfg)
    td = B.torch_dtype(sh.dtype)
    gen = torch.Generator(device="cuda").manual_seed(args.seed)
    rnd = lambda *shape, scale=1.0: (torch.randn(*shape, generator=gen, device="cuda") * scale).to(td)
    ctx.set_weights({k: (rnd(*v, scale=0.02) if not k.startswith("g_") else torch.ones(*v, device="cuda", dtype=td))
                     for k, v in synth.weight_shapes(sh).items()})
    state = B.State(cfg, sh.dtype, wl.S, lay["block_table"], lay["committed_len"])
    for l in range(sh.n_layers):
        state.kv_pool[l].copy_(rnd(*state.kv_pool[l].shape))
    rd = synth.make_round(wl, args.seed, 0)
    d, t = torch.from_numpy(rd["draft"]).cuda(), torch.from_numpy(rd["target"]).cuda()
    H = B.to_device(rd["H"], sh.dtype)
    nd = torch.zeros((wl.S, sh.W), dtype=torch.int32, device="cuda")
    mode = B.COD_BASELINE if args.baseline else B.COD_CARRY
    one = lambda: ctx.draft_round(d, t, H, wl.S, wl.n_forced, mode, state, None, nd, None)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        one()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        one()
    for _ in range(max(args.warmup, 3)):
        g.replay()
    torch.cuda.synchronize()
    with profile(activities=[ProfilerActivity.CUDA]) as prof:
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
    ev = sorted((e for e in prof.events() if e.device_type == torch.autograd.DeviceType.CUDA),
                key=lambda e: e.time_range.start)
    rows = [(e.name, e.time_range.start, e.time_range.end) for e in ev]
    first = [i for i, r in enumerate(rows) if "k_verify_accept" in r[0]]
    last = rows[first[-1]:]
    t0, prev_end, out, agg = last[0][1], last[0][1], [], {}
    for name, s0, e0 in last:
        short = name.replace("(anonymous namespace)::", "").replace("void ", "").split("(")[0]
        chain = e0 - max(s0, prev_end)
        out.append({"kernel": short, "start_us": s0 - t0, "end_us": e0 - t0, "chain_us": max(chain, 0.0)})
        a = agg.setdefault(short, [0, 0.0])
        a[0] += 1
        a[1] += max(chain, 0.0)
        prev_end = max(prev_end, e0)
    print(json.dumps({"micro": "timeline", "workload": wl.name, "round_us": prev_end - t0,
                      "chain_us_by_kernel": {k: {"launches": v[0], "chain_us": v[1]} for k, v in
                                             sorted(agg.items(), key=lambda kv: -kv[1][1])},
                      "kernels": out if args.verbose else None}))
    ctx.close()


def run_micro(args):
    """--micro attn|lmhead: one entry point alone on the workload's shapes (one drafter layer, so the
    device footprint stays small enough for a profiler capture). Prints its own JSON line."""
    import torch

    import __graft_entry__ as entry
    from paper_2609_14717_b200 import binding as B

    if args.micro == "gemm":
        return run_micro_round(args)
    if args.micro == "timeline":
        return run_timeline(args)
    entry.build()
    torch.cuda.set_device(0)
    peaks = load_peaks()
    wl = synth.scaled(bench_workload(args.workload, 4), n_layers=1)
    if args.vocab > 0:
        wl = synth.scaled(wl, vocab=args.vocab)
    sh = wl.shape
    lay = synth.make_layout(wl, args.seed)
    n_pages, mp = int(lay["n_pages"]), int(lay["max_pages_per_seq"])
    cfg = B.make_config(sh, wl.S, mp, n_pages, attn_split_len=args.attn_split, extra_flags=args.flags)
    ctx = B.Context(cfg)
    td = B.torch_dtype(sh.dtype)
    gen = torch.Generator(device="cuda").manual_seed(args.seed)
    rnd = lambda *shape, scale=1.0: (torch.randn(*shape, generator=gen, device="cuda") * scale).to(td)
    K, Wm = args.steps, args.warmup
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.micro == "attn":
        state = B.State(cfg, sh.dtype, wl.S, lay["block_table"], lay["committed_len"])
        state.kv_pool.copy_(rnd(*state.kv_pool.shape))
        state.carry_kv.copy_(rnd(*state.carry_kv.shape))
        state.carry_len.fill_(sh.W // 2)
        q, kb, vb = rnd(wl.S, sh.W, sh.n_q, sh.hd), rnd(wl.S, sh.W, sh.n_kv, sh.hd), rnd(wl.S, sh.W, sh.n_kv, sh.hd)
        out = torch.empty_like(q)
        call = lambda: ctx.block_attn(0, q, kb, vb, state, wl.S, 1, out)
        L = lay["committed_len"].astype(np.int64)
        nbytes = float(np.sum(L + sh.W // 2) * 2 * sh.n_kv * sh.hd * 2 + 2 * q.numel() * 2)
        flops = 4.0 * sh.W * sh.n_q * sh.hd * float(np.sum(L + sh.W // 2 + sh.W))
    else:
        w = {k: (rnd(*v, scale=0.02) if k not in ("g_hidden", "g_attn", "g_final") else torch.ones(*v, device="cuda", dtype=td))
             for k, v in synth.weight_shapes(sh).items()}
        ctx.set_weights(w)
        x = torch.randn(wl.R, sh.d_model, generator=gen, device="cuda")
        tok = torch.zeros(wl.R, dtype=torch.int32, device="cuda")
        if args.micro == "lmsample":      # the Gumbel-max draw fused into the same contraction
            qv = torch.zeros(wl.R, dtype=torch.float32, device="cuda")
            step_no = [0]

            def call():
                step_no[0] += 1
                ctx.lm_head_sample(x, wl.R, args.seed, step_no[0], tok, qv, None)
        elif args.micro == "lmrank":      # rank of a reference token, counted in the same contraction
            ref = torch.randint(0, sh.vocab, (wl.R,), generator=gen, device="cuda", dtype=torch.int32)
            call = lambda: ctx.lm_head_rank(x, wl.R, ref, tok)
        else:
            call = lambda: ctx.lm_head_argmax(x, wl.R, tok)
        nbytes = float(sh.vocab * sh.d_model * 2 + wl.R * sh.d_model * 2)
        flops = 2.0 * wl.R * sh.d_model * sh.vocab
    for _ in range(Wm):
        call()
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(K):
        call()
    ev1.record()
    torch.cuda.synchronize()
    us = ev0.elapsed_time(ev1) / K * 1e3
    print(json.dumps({"micro": args.micro, "workload": wl.name, "us_per_call": us, "GBps": nbytes / us / 1e3,
                      "TFLOPs": flops / us / 1e6, "hbm_frac": nbytes / us / 1e3 / peaks["hbm_gbs"],
                      "tensor_frac": flops / us / 1e6 / peaks["tflops"], "device_status": ctx.poll_status()}))
    ctx.close()


def run_sweep(args):
    """--sweep: the carryover-overhead sweep (configuration 5): batch x block x rejected fraction,
    each point timed with carryover and with the baseline drafter on identical inputs (graph replay,
    fixed accepted length m = W - rejected, no forced anchor; plus the anchor corner m = 1)."""
    import torch

    import __graft_entry__ as entry
    from paper_2609_14717_b200 import binding as B

    entry.build()
    torch.cuda.set_device(0)
    base = synth.workload("cfg5")
    weights = B.weights_to_device(synth.make_weights(base.shape, args.seed), "bf16")
    K, Wm = args.steps, args.warmup
    rows = []
    for W in (8, 16):
        for S in (1, 4, 16, 64):
            points = [(W, 0), (W // 2, 0), (0, 0), (1, 1)]            # (accepted rows m, n_forced)
            for m, nf in points:
                wl = synth.sweep_point(S, W, m, n_forced=nf, n_rounds=K + Wm + 2)
                sh = wl.shape
                lay = synth.make_layout(wl, args.seed)
                n_pages, mp = int(lay["n_pages"]), int(lay["max_pages_per_seq"])
                ctx = B.Context(B.make_config(sh, S, mp, n_pages))
                ctx.set_weights(weights)
                state = B.State(ctx.cfg, "bf16", S, lay["block_table"], lay["committed_len"])
                gen = torch.Generator(device="cuda").manual_seed(args.seed)
                for l in range(sh.n_layers):
                    state.kv_pool[l].copy_(torch.randn(state.kv_pool[l].shape, generator=gen, device="cuda").to(torch.bfloat16))
                rd = synth.make_round(wl, args.seed, 0)
                d, t = torch.from_numpy(rd["draft"]).cuda(), torch.from_numpy(rd["target"]).cuda()
                H = B.to_device(rd["H"], "bf16")
                nd = torch.zeros((S, W), dtype=torch.int32, device="cuda")
                L0 = state.committed_len.clone()
                graphs = {}
                for mode, name in ((B.COD_CARRY, "carry"), (B.COD_BASELINE, "baseline")):
                    def one(mode=mode):
                        ctx.draft_round(d, t, H, S, nf, mode, state, None, nd, None)
                    state.committed_len.copy_(L0); state.carry_len.zero_()
                    side = torch.cuda.Stream(); side.wait_stream(torch.cuda.current_stream())
                    with torch.cuda.stream(side):
                        one()
                    torch.cuda.current_stream().wait_stream(side); torch.cuda.synchronize()
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g):
                        one()
                    graphs[name] = g
                # interleaved passes (C B C B ...), each from the restored state; medians reported
                times = {"carry": [], "baseline": []}
                for rep in range(args.sweep_reps):
                    for name in ("carry", "baseline"):
                        state.committed_len.copy_(L0); state.carry_len.zero_()
                        for _ in range(Wm):
                            graphs[name].replay()
                        torch.cuda.synchronize()
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        e0.record()
                        for _ in range(K):
                            graphs[name].replay()
                        e1.record(); torch.cuda.synchronize()
                        times[name].append(e0.elapsed_time(e1) / K * 1e3)
                res = {k: statistics.median(v) for k, v in times.items()}
                paired = [100.0 * (c_ - b_) / b_ for c_, b_ in zip(times["carry"], times["baseline"])]
                status = ctx.poll_status()
                rows.append({"S": S, "W": W, "m": m, "rejected": W - m, "n_forced": nf, "carry_us": res["carry"],
                             "baseline_us": res["baseline"], "overhead_pct": statistics.median(paired),
                             "overhead_pct_min": min(paired), "overhead_pct_max": max(paired),
                             "carry_us_min_max": [min(times["carry"]), max(times["carry"])],
                             "baseline_us_min_max": [min(times["baseline"]), max(times["baseline"])],
                             "passes": args.sweep_reps, "device_status": status})
                ctx.close()
                del state
                torch.cuda.empty_cache()
    print(json.dumps({"sweep": "cfg5", "context": 4096, "steps": K, "points": rows}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5", "cfg2f", "cfg3f", "cfg3p"],
                    help="default: cfg3 (batch 32) on the line and cfg2 (batch 1) under \"batch1\"; cfg2f / cfg3f: the "
                         "same with the complete drafter layer (gated MLP 9728, q/k norms)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time plain stream launches instead of graph replays")
    ap.add_argument("--sweep", action="store_true", help="carryover-overhead sweep over batch, block and rejected fraction")
    ap.add_argument("--sweep-reps", type=int, default=7, help="--sweep: interleaved passes per mode and point")
    ap.add_argument("--attn-split", type=int, default=0, help="keys per attention split (0 = library default)")
    ap.add_argument("--vocab", type=int, default=0, help="--micro lmhead*: override the vocabulary size (0 = the workload's)")
    ap.add_argument("--layers", type=int, default=1,
                    help="--micro gemm: drafter layers of the rounds it runs (default 1; 0 = the workload's own depth)")
    ap.add_argument("--flags", type=int, default=0,
                    help="extra cod_config flags OR-ed in (e.g. 64 = persistent attention, 32 = one-item attention CTAs)")
    ap.add_argument("--micro", default=None, choices=["attn", "lmhead", "lmsample", "lmrank", "gemm", "timeline"],
                    help="time one entry point alone (small footprint; meant for profiler captures)")
    ap.add_argument("--shape", default=None, choices=["fc", "kv", "qkv", "oproj", "lmhead", "attn"],
                    help="--micro gemm: the contraction class to time inside a one-layer round")
    ap.add_argument("--verbose", action="store_true", help="--micro timeline: also list every launch")
    ap.add_argument("--baseline", action="store_true", help="--micro gemm: run the rounds in baseline mode")
    ap.add_argument("--record-traffic", default=None, metavar="NCU_CSV",
                    help="store the DRAM bytes of an ncu capture (one launch) in profiles/dram_traffic.txt")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.record_traffic:
        args.workload = args.workload or "cfg3"
        record_traffic(args)
        return
    if (args.micro or args.sweep) and not args.workload:
        args.workload = "cfg2"
    if args.sweep:
        run_sweep(args)
    elif args.micro:
        run_micro(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
